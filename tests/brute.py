"""Pure-Python brute force used to pin the oracle on tiny inputs.

Nothing here calls the oracle or the CUDA library.  The mask functions are written in the
"relative offset" view (a key that lies o tokens behind the query), which is a different route
to the kept set than the oracle's literal step-by-step replay of Algorithm 1; the attention is
the textbook definition with Python floats and ``math.fsum``.
"""
from __future__ import annotations

import math
from typing import List, Sequence


def kept_offsets_from_trace(t: int, n_r: int, n_att: int, trace: Sequence[int]) -> List[int]:
    """Offsets o (key = t - o) attended at step t when the k-th selection skipped offset trace[k].

    A key chosen at step s with index j is skipped from step s+1 on and moves one index per step,
    so its distance to the query stays s - j forever (Algorithm 1, the "+1" shift).  Selections
    happen at steps N_att-1, N_att, ..., one per step, until N_r - N_att of them exist.
    """
    m = n_r - n_att
    n_active = min(max(t - (n_att - 1), 0), m)
    skipped = set(trace[:n_active])
    window = range(0, min(t, n_r - 1) + 1)
    return [o for o in window if o not in skipped]


def col_dist(o: int, stride: int) -> int:
    r = o % stride
    return min(r, stride - r)


def kept_offsets_grid(t: int, n_r: int, n_att: int, stride: int) -> List[int]:
    """Closed form of the grid-locality selection: dropping the worst attended key at every
    step keeps a running best-(N_att-1) of the offsets seen so far, plus the newest slot."""
    if t < n_att - 1:
        return list(range(t + 1))
    top = min(t, n_r - 1)
    ranked = sorted(range(top), key=lambda o: (col_dist(o, stride), o))
    return sorted(ranked[: n_att - 1] + [top])


def grid_trace(n_r: int, n_att: int, stride: int) -> List[int]:
    """Offset trace of the grid-locality selection, by simulating it in offset space."""
    skipped: List[int] = []
    for s in range(n_att - 1, n_r - 1):
        cand = [o for o in range(s + 1) if o not in skipped]
        skipped.append(max(cand, key=lambda o: (col_dist(o, stride), o)))
    return skipped


def attention(q: Sequence[float], keys: Sequence[Sequence[float]], values: Sequence[Sequence[float]],
              scale: float):
    """Textbook softmax attention of one query: returns (out, lse)."""
    if not keys:
        return [0.0] * len(q), -math.inf
    s = [scale * math.fsum(a * b for a, b in zip(q, k)) for k in keys]
    mx = max(s)
    z = math.fsum(math.exp(x - mx) for x in s)
    lse = mx + math.log(z)
    w = [math.exp(x - lse) for x in s]
    d = len(values[0])
    out = [math.fsum(w[j] * values[j][i] for j in range(len(values))) for i in range(d)]
    return out, lse


def argmin_trace(q_steps: Sequence[Sequence[float]], keys: Sequence[Sequence[float]], n_r: int, n_att: int,
                 scale: float, n_sink: int = 0) -> List[int]:
    """Algorithm 1's own selection simulated in distance space: at steps N_att-1 .. N_r-2 the
    attended decode key (sinks excluded) with the lowest logit is skipped from then on; equal
    logits go to the lowest key index.  Returns the distances in selection order."""
    skipped: List[int] = []
    for s in range(n_att - 1, n_r - 1):
        best = None
        for o in range(s, -1, -1):                     # oldest key first, strict "<" keeps it on ties
            j = s - o
            if o in skipped or j < n_sink:
                continue
            logit = scale * math.fsum(a * b for a, b in zip(q_steps[s], keys[j]))
            if best is None or logit < best[0]:
                best = (logit, o)
        skipped.append(best[1])
    return skipped
