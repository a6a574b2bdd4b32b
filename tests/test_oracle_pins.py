"""Pins for the float64 oracle: each test ties it to something other than itself -- values the
paper prints, closed forms, a second derivation in pure Python, or a library routine on a
special case -- so that a dropped term, an off-by-one or a transposed operand fails here.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import oracle as ora
from paper_2609_19702_b200 import synth
from tests import brute

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_example_nr7_natt4.txt")


def _read_golden():
    g = {"choice": {}, "attended": {}, "skip_after": {}, "skip_shifted": {}, "evicted": {}}
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            tok = line.replace(":", " ").split()
            key = tok[0]
            if key in ("N_r", "N_att", "final_skip_count", "steady_attended_count"):
                g[key] = int(tok[1])
            elif key == "choice":
                g["choice"][int(tok[1])] = int(tok[2])
            else:
                g[key][int(tok[1])] = [int(x) for x in tok[2:]]
    return g


# ---------------------------------------------------------------- Algorithm 1: worked example

def test_worked_example_printed_in_paper():
    g = _read_golden()
    n_r, n_att = g["N_r"], g["N_att"]
    # the paper's two stated choices, as distances behind the query: K_0 at t=3, K_2 at t=4
    trace2 = [t - j for t, j in sorted(g["choice"].items())]
    assert trace2 == [3, 2]
    for third in range(0, 6):          # third choice is not printed: every legal one must agree
        if third in trace2:
            continue
        trace = trace2 + [third]
        for t, want in g["attended"].items():
            idx, _ = ora.replay(t, n_r, n_att, ora.SEL_TRACE, trace)
            assert idx.tolist() == want, (t, third)
        for t, want in g["skip_after"].items():
            _, skip = ora.replay(t, n_r, n_att, ora.SEL_TRACE, trace)
            assert skip.tolist() == want
        for t, want in g["skip_shifted"].items():
            # skip_idx right after the shift of step t = entries of step t-1, each +1
            _, prev = ora.replay(t - 1, n_r, n_att, ora.SEL_TRACE, trace)
            assert (prev + 1).tolist() == want
            idx, _ = ora.replay(t, n_r, n_att, ora.SEL_TRACE, trace)
            assert not set(want) & set(idx.tolist())
        for t in range(5, 40):
            idx, skip = ora.replay(t, n_r, n_att, ora.SEL_TRACE, trace)
            assert len(skip) == g["final_skip_count"]
            if t >= n_att - 1:
                assert len(idx) == g["steady_attended_count"]
        for t, gone in g["evicted"].items():
            idx, _ = ora.replay(t, n_r, n_att, ora.SEL_TRACE, trace)
            assert not set(gone) & set(idx.tolist())
            assert idx.min() >= t - n_r + 1


def test_new_entry_not_skipped_in_its_own_step():
    # Section 4 item 2: the entry appended at step s is still attended at step s
    n_r, n_att = 12, 5
    trace = brute.grid_trace(n_r, n_att, 4)
    for s in range(n_att - 1, n_r - 1):
        idx, skip = ora.replay(s, n_r, n_att, ora.SEL_TRACE, trace)
        assert skip[-1] in idx.tolist()
        assert s - skip[-1] == trace[s - (n_att - 1)]


# ---------------------------------------------------------------- Algorithm 1: closed forms

PARAMS = [(7, 4, 3), (64, 13, 16), (16, 16, 5), (20, 1, 6), (33, 7, 65), (40, 39, 8), (9, 2, 2), (31, 11, 1)]


@pytest.mark.parametrize("n_r,n_att,stride", PARAMS)
def test_attended_count_every_position(n_r, n_att, stride):
    rng = np.random.default_rng(n_r * 1000 + n_att)
    trace = synth.random_valid_trace(rng, n_r, n_att)
    for t in range(0, 3 * n_r + 5):
        want = min(t + 1, n_att)           # phase 1: t+1 keys; phases 2-3: N_att keys
        idx_g, _ = ora.replay(t, n_r, n_att, ora.SEL_GRID, stride=stride)
        idx_l, _ = ora.replay(t, n_r, n_att, ora.SEL_TRACE, trace)
        assert len(idx_g) == want and len(idx_l) == want
        assert idx_g.tolist() == sorted(set(idx_g.tolist()))
        assert idx_g.min() >= max(0, t - n_r + 1) and idx_g.max() <= t
        assert idx_l.min() >= max(0, t - n_r + 1) and idx_l.max() <= t


@pytest.mark.parametrize("n_r,n_att,stride", PARAMS)
def test_steady_state_shift_invariance(n_r, n_att, stride):
    # once selection has stopped the kept set only translates with the query
    rng = np.random.default_rng(7)
    trace = synth.random_valid_trace(rng, n_r, n_att)
    for sel, kw in ((ora.SEL_GRID, {"stride": stride}), (ora.SEL_TRACE, {"trace": trace})):
        base, _ = ora.replay(n_r - 1, n_r, n_att, sel, **kw)
        for t in range(n_r, 2 * n_r + 3):
            idx, _ = ora.replay(t, n_r, n_att, sel, **kw)
            assert (idx - t).tolist() == (base - (n_r - 1)).tolist()


@pytest.mark.parametrize("n_r,n_att,stride", PARAMS)
def test_replay_matches_offset_derivation(n_r, n_att, stride):
    rng = np.random.default_rng(n_r + 17 * n_att)
    for _ in range(3):
        trace = synth.random_valid_trace(rng, n_r, n_att).tolist()
        for t in range(0, 2 * n_r + 4):
            idx, _ = ora.replay(t, n_r, n_att, ora.SEL_TRACE, trace)
            want = sorted(t - o for o in brute.kept_offsets_from_trace(t, n_r, n_att, trace))
            assert idx.tolist() == want


@pytest.mark.parametrize("n_r,n_att,stride", PARAMS)
def test_grid_replay_matches_closed_form(n_r, n_att, stride):
    trace = brute.grid_trace(n_r, n_att, stride)
    for t in range(0, 2 * n_r + 4):
        idx, skip = ora.replay(t, n_r, n_att, ora.SEL_GRID, stride=stride)
        want = sorted(t - o for o in brute.kept_offsets_grid(t, n_r, n_att, stride))
        assert idx.tolist() == want
        n_sel = min(max(t - (n_att - 1) + 1, 0), n_r - n_att)
        assert sorted(t - s for s in skip.tolist()) == sorted(trace[:n_sel])


def test_grid_steady_state_tiny_config():
    # 16-wide grid, N_r 64, N_att 13: own row neighbourhood and the same columns +-1 in the
    # three rows above, plus the oldest window slot that can never be selected
    idx, _ = ora.replay(200, 64, 13, ora.SEL_GRID, stride=16)
    assert sorted(200 - idx) == [0, 1, 2, 15, 16, 17, 31, 32, 33, 47, 48, 49, 63]


def test_invalid_traces_are_rejected():
    with pytest.raises(RuntimeError):
        ora.replay(10, 7, 4, ora.SEL_TRACE, [3, 3, 1])      # repeats an already skipped diagonal
    with pytest.raises(RuntimeError):
        ora.replay(10, 7, 4, ora.SEL_TRACE, [4, 2, 1])      # offset 4 does not exist at t = 3
    with pytest.raises(RuntimeError):
        ora.replay(10, 7, 4, ora.SEL_TRACE, [3, 2])         # too short
    with pytest.raises(RuntimeError):
        ora.replay(3, 4, 5, ora.SEL_GRID, stride=3)         # N_att > N_r


def test_kept_positions_modes():
    l_p, n_r, n_att = 5, 8, 3
    for p in range(0, 30):
        dense = ora.kept(ora.MODE_DENSE, l_p, p)
        assert dense.tolist() == list(range(l_p + p))
        win = ora.kept(ora.MODE_WINDOW, l_p, p, n_r, n_r)
        assert win.tolist() == list(range(l_p)) + list(range(l_p + max(0, p - n_r), l_p + p))
        grid = ora.kept(ora.MODE_GRID, l_p, p, n_r, n_att, 4)
        assert grid[:l_p].tolist() == list(range(l_p))           # prompt always attended in full
        assert len(grid) == l_p + min(p, n_att)
        if p >= 1:
            assert grid[-1] == l_p + p - 1 or n_att == 1         # current token (distance 0)
    # window >= position and nothing skipped is dense attention
    assert ora.kept(ora.MODE_WINDOW, 4, 9, 9, 9).tolist() == list(range(13))


def test_sink_variants_against_set_arithmetic():
    # Section 5.1: StreamingLLM = 4 sinks (first decode tokens) + recent window, prompt always kept;
    # Diagonal + sink4 = the same sinks on top of the diagonal selection
    l_p, n_r, n_att, stride, n_sink = 6, 12, 5, 4, 4
    rng = np.random.default_rng(11)
    trace = synth.random_valid_trace(rng, n_r, n_att).tolist()
    for p in range(0, 40):
        t = p - 1
        sinks = {l_p + j for j in range(min(n_sink, p))}
        prompt = set(range(l_p))
        win = ora.kept(ora.MODE_WINDOW, l_p, p, n_r, n_r, n_sink=n_sink)
        want = prompt | sinks | set(range(l_p + max(0, p - n_r), l_p + p))
        assert win.tolist() == sorted(want)
        grid = ora.kept(ora.MODE_GRID, l_p, p, n_r, n_att, stride, n_sink=n_sink)
        base = {l_p + t - o for o in brute.kept_offsets_grid(t, n_r, n_att, stride)} if p else set()
        assert grid.tolist() == sorted(prompt | sinks | base)
        lst = ora.kept(ora.MODE_LIST, l_p, p, n_r, n_att, trace=trace, n_sink=n_sink)
        base = {l_p + t - o for o in brute.kept_offsets_from_trace(t, n_r, n_att, trace)} if p else set()
        assert lst.tolist() == sorted(prompt | sinks | base)
        if p >= n_r + n_sink:                       # sinks have left the window: budget is exact
            assert len(grid) == l_p + n_att + n_sink and len(lst) == l_p + n_att + n_sink
    assert ora.kept(ora.MODE_GRID, l_p, 9, n_r, n_att, stride, n_sink=0).tolist() == \
        ora.kept(ora.MODE_GRID, l_p, 9, n_r, n_att, stride).tolist()


def test_cost_model_ratio_last_step():
    # Section 4 cost analysis: per-step compute shrinks by (L_dec + L_p) / (N_att + L_p)
    for l_dec, l_p, sparsity in ((576, 50, 0.95), (1024, 50, 0.90)):
        n_att = math.ceil((1 - sparsity) * l_dec)
        n_r = l_dec // 2
        dense = len(ora.kept(ora.MODE_DENSE, l_p, l_dec))
        sparse = len(ora.kept(ora.MODE_GRID, l_p, l_dec, n_r, n_att, int(math.isqrt(l_dec))))
        assert dense * (n_att + l_p) == sparse * (l_dec + l_p)


# ---------------------------------------------------------------- attention

def _rows(n, d):
    return np.arange(n, dtype=np.int64) * d


def test_attend_matches_pure_python_and_torch():
    rng = np.random.default_rng(3)
    for n, d in ((1, 4), (7, 3), (19, 16), (5, 33)):
        q = rng.standard_normal(d)
        k = rng.standard_normal((n, d))
        v = rng.standard_normal((n, d))
        scale = 0.37
        out, lse = ora.attend(q, k.reshape(-1), v.reshape(-1), _rows(n, d), _rows(n, d), d, scale)
        bout, blse = brute.attention(q.tolist(), k.tolist(), v.tolist(), scale)
        np.testing.assert_allclose(out, bout, rtol=1e-12, atol=1e-14)
        assert abs(lse - blse) < 1e-12
        # library route: softmax(q K^T) V in float64
        s = torch.from_numpy(k) @ torch.from_numpy(q) * scale
        tout = torch.softmax(s, 0) @ torch.from_numpy(v)
        np.testing.assert_allclose(out, tout.numpy(), rtol=1e-12, atol=1e-14)
        assert abs(lse - float(torch.logsumexp(s, 0))) < 1e-12


def test_attend_row_gather_and_dtypes():
    # rows are picked by offset, K and V independently; f32 and bf16 inputs widen exactly
    rng = np.random.default_rng(4)
    d, n = 8, 11
    k = rng.standard_normal((n, d)).astype(np.float32)
    v = rng.standard_normal((n, d)).astype(np.float32)
    q = rng.standard_normal(d).astype(np.float32)
    pick = np.array([9, 2, 5])
    out, lse = ora.attend(q, k.reshape(-1), v.reshape(-1), pick * d, pick * d, d, 0.5)
    bout, blse = brute.attention(q.astype(np.float64).tolist(), k[pick].astype(np.float64).tolist(),
                                 v[pick].astype(np.float64).tolist(), 0.5)
    np.testing.assert_allclose(out, bout, rtol=1e-12)
    assert abs(lse - blse) < 1e-12
    qb, kb, vb = (synth.f32_to_bf16_bits(x) for x in (q, k, v))
    out_b, lse_b = ora.attend(qb, kb.reshape(-1), vb.reshape(-1), pick * d, pick * d, d, 0.5)
    qf, kf, vf = (synth.bf16_bits_to_f32(x).astype(np.float64) for x in (qb, kb, vb))
    bout, blse = brute.attention(qf.tolist(), kf[pick].tolist(), vf[pick].tolist(), 0.5)
    np.testing.assert_allclose(out_b, bout, rtol=1e-12)
    assert abs(lse_b - blse) < 1e-12


def test_identical_keys_give_mean_of_values():
    rng = np.random.default_rng(5)
    d, n = 16, 9
    key = rng.standard_normal(d)
    k = np.tile(key, (n, 1))
    v = rng.standard_normal((n, d))
    q = rng.standard_normal(d)
    out, lse = ora.attend(q, k.reshape(-1), v.reshape(-1), _rows(n, d), _rows(n, d), d, 0.25)
    np.testing.assert_allclose(out, v.mean(0), rtol=1e-12)
    assert abs(lse - (0.25 * float(q @ key) + math.log(n))) < 1e-12


def test_one_dominant_key_selects_its_value():
    d, n = 8, 6
    k = np.zeros((n, d))
    k[4] = 100.0
    v = np.arange(n * d, dtype=np.float64).reshape(n, d)
    q = np.ones(d)
    out, lse = ora.attend(q, k.reshape(-1), v.reshape(-1), _rows(n, d), _rows(n, d), d, 1.0)
    np.testing.assert_allclose(out, v[4], rtol=1e-12)
    assert abs(lse - 800.0) < 1e-9
    out0, lse0 = ora.attend(q, k.reshape(-1), v.reshape(-1), _rows(0, d), _rows(0, d), d, 1.0)
    assert lse0 == -math.inf and not out0.any()


def test_combine_is_the_split_identity():
    rng = np.random.default_rng(6)
    d, n = 12, 40
    q = rng.standard_normal(d)
    k = rng.standard_normal((n, d))
    v = rng.standard_normal((n, d))
    full, full_lse = ora.attend(q, k.reshape(-1), v.reshape(-1), _rows(n, d), _rows(n, d), d, 0.3)
    for cuts in ([0, 40], [0, 13, 40], [0, 1, 2, 30, 40], [0, 20, 20, 40]):
        parts, lses = [], []
        for a, b in zip(cuts[:-1], cuts[1:]):
            rows = np.arange(a, b, dtype=np.int64) * d
            o, l = ora.attend(q, k.reshape(-1), v.reshape(-1), rows, rows, d, 0.3)
            parts.append(o)
            lses.append(l)
        out, lse = ora.combine(np.stack(parts), np.array(lses))
        np.testing.assert_allclose(out, full, rtol=1e-12, atol=1e-15)
        assert abs(float(lse) - full_lse) < 1e-12
    # closed form for two parts: lse = ln(e^a + e^b), weights e^{a-lse}, e^{b-lse}
    o, l = ora.combine(np.array([[1.0, 0.0], [0.0, 1.0]]), np.array([math.log(3.0), math.log(1.0)]))
    np.testing.assert_allclose(o, [0.75, 0.25], rtol=1e-15)
    assert abs(float(l) - math.log(4.0)) < 1e-15
    o, l = ora.combine(np.zeros((2, 3)), np.array([-math.inf, -math.inf]))
    assert float(l) == -math.inf and not o.any()


def test_select_argmin_over_decode_keys_only():
    rng = np.random.default_rng(8)
    d, n = 8, 10
    q = rng.standard_normal(d)
    k = rng.standard_normal((n, d))
    rows = np.array([1, 3, 4, 8], dtype=np.int64) * d
    j, w = ora.select_argmin(q, k.reshape(-1), rows, d, 0.5)
    logits = [0.5 * float(q @ k[i]) for i in (1, 3, 4, 8)]
    assert j == int(np.argmin(logits))          # softmax is monotone: argmin w = argmin logit
    np.testing.assert_allclose(w, torch.softmax(torch.tensor(logits, dtype=torch.float64), 0).numpy(),
                               rtol=1e-12)
    k2 = np.tile(k[0], (n, 1))
    j2, _ = ora.select_argmin(q, k2.reshape(-1), rows, d, 0.5)
    assert j2 == 0                               # ties: lowest cache index


def test_replay_with_argmin_selection_against_distance_space_simulation():
    rng = np.random.default_rng(21)
    for n_r, n_att, n_sink, d in ((12, 4, 0, 8), (20, 7, 2, 5), (9, 2, 1, 16), (16, 15, 0, 4)):
        steps = 2 * n_r + 3
        q = rng.standard_normal((steps, d))
        k = rng.standard_normal((steps, d))
        want = brute.argmin_trace(q.tolist(), k.tolist(), n_r, n_att, 0.4, n_sink)
        for t in (0, n_att - 1, n_att, n_r - 2, n_r - 1, steps - 1):
            idx, tr = ora.replay_argmin(t, n_r, n_att, q, d, k.reshape(-1), np.arange(steps) * d, d, 0.4, n_sink)
            n_sel = min(max(t - (n_att - 1) + 1, 0), n_r - n_att)
            assert tr.tolist() == want[:n_sel]
            # the same trace fed back as an input reproduces the attended set
            idx2, _ = ora.replay(t, n_r, n_att, ora.SEL_TRACE, want)
            assert idx.tolist() == idx2.tolist()
    # the selected key really carries the lowest softmax weight among the attended decode keys
    n_r, n_att, d = 10, 4, 6
    q = rng.standard_normal((30, d))
    k = rng.standard_normal((30, d))
    _, tr = ora.replay_argmin(29, n_r, n_att, q, d, k.reshape(-1), np.arange(30) * d, d, 1.0)
    for i, o in enumerate(tr.tolist()):
        s_step = n_att - 1 + i
        idx, _ = ora.replay(s_step, n_r, n_att, ora.SEL_TRACE, tr.tolist())
        w = torch.softmax(torch.from_numpy(k[idx] @ q[s_step]), 0)
        assert int(idx[int(torch.argmin(w))]) == s_step - o


# ---------------------------------------------------------------- the batched driver

def _brute_decode(inp, kept_fn):
    """Per (request, head) pure-Python attention over kept positions, any layout."""
    q = synth.bf16_bits_to_f32(inp["q"]).astype(np.float64)
    kc = synth.bf16_bits_to_f32(inp["k_cache"]).astype(np.float64)
    vc = synth.bf16_bits_to_f32(inp["v_cache"]).astype(np.float64)
    b, hq, d = q.shape
    hkv = inp["workload"].num_kv_heads
    g_sz = hq // hkv
    sb, st, sh = inp["strides"]
    outs = np.zeros((b, hq, d))
    lses = np.zeros((b, hq))
    for i in range(b):
        for h in range(hq):
            g = h // g_sz
            rows = []
            for s in kept_fn(i, h):
                if inp["block_table"] is not None:
                    blk = int(inp["block_table"][i, s // inp["block_size"]])
                    rows.append(blk * sb + (s % inp["block_size"]) * st + g * sh)
                else:
                    rows.append(i * sb + s * st + g * sh)
            ks = [kc[r:r + d].tolist() for r in rows]
            vs = [vc[r:r + d].tolist() for r in rows]
            o, l = brute.attention(q[i, h].tolist(), ks, vs, 1.0 / math.sqrt(d))
            outs[i, h] = o
            lses[i, h] = l
    return outs, lses


def _tiny(paged, hq=6, hkv=2, d=8, batch=5):
    w = synth.Workload("t", 9, batch, hq, hkv, d, 3, 4, 5, 1, 10, 4, 1, 24, positional=True,
                       paged=paged, block_size=4)
    return synth.make_inputs(w, seed=1234 + int(paged))


@pytest.mark.parametrize("paged", [False, True])
def test_decode_driver_gqa_layouts_against_brute_force(paged):
    inp = _tiny(paged)
    w = inp["workload"]
    l_p = w.prompt_len
    common = dict(num_kv_heads=w.num_kv_heads, strides=inp["strides"],
                  block_table=inp["block_table"], block_size=inp["block_size"])
    # dense
    r = ora.decode(inp["q"], inp["k_cache"], inp["v_cache"], inp["seq_len"], inp["prompt_len"],
                   mode=ora.MODE_DENSE, **common)
    bo, bl = _brute_decode(inp, lambda i, h: range(int(inp["seq_len"][i])))
    np.testing.assert_allclose(r["out"], bo, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(r["lse"], bl, rtol=1e-12)
    assert np.isfinite(r["out"]).all()          # NaN rows past seq_len never enter
    # grid
    r = ora.decode(inp["q"], inp["k_cache"], inp["v_cache"], inp["seq_len"], inp["prompt_len"],
                   mode=ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride_grid=w.stride,
                   want_kept=True, **common)

    def grid_kept(i, h):
        p = int(inp["position"][i])
        return list(range(l_p)) + sorted(l_p + p - 1 - o for o in
                                         brute.kept_offsets_grid(p - 1, w.window, w.n_att, w.stride))
    bo, bl = _brute_decode(inp, grid_kept)
    np.testing.assert_allclose(r["out"], bo, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(r["lse"], bl, rtol=1e-12)
    for i in range(w.batch):
        n = int(r["kept_cnt"][i, 0])
        assert r["kept_idx"][i, 0, :n].tolist() == grid_kept(i, 0)
    # per-query-head traces
    rng = np.random.default_rng(99)
    for mask_heads in (1, w.num_kv_heads, w.num_q_heads):
        trace = synth.random_valid_trace(rng, w.window, w.n_att, (w.batch, mask_heads))
        r = ora.decode(inp["q"], inp["k_cache"], inp["v_cache"], inp["seq_len"], inp["prompt_len"],
                       mode=ora.MODE_LIST, n_r=w.window, n_att=w.n_att, trace=trace, **common)
        g_sz = w.num_q_heads // w.num_kv_heads

        def list_kept(i, h):
            mh = 0 if mask_heads == 1 else (h // g_sz if mask_heads == w.num_kv_heads else h)
            p = int(inp["position"][i])
            offs = brute.kept_offsets_from_trace(p - 1, w.window, w.n_att, trace[i, mh].tolist())
            return list(range(l_p)) + sorted(l_p + p - 1 - o for o in offs)
        bo, bl = _brute_decode(inp, list_kept)
        np.testing.assert_allclose(r["out"], bo, rtol=1e-11, atol=1e-13)
        np.testing.assert_allclose(r["lse"], bl, rtol=1e-12)


def test_paged_and_contiguous_agree():
    # same tokens, two layouts: results must be identical
    inp = _tiny(True)
    w = inp["workload"]
    hkv, d, bs = w.num_kv_heads, w.head_dim, w.block_size
    s_max = inp["block_table"].shape[1] * bs
    kc = inp["k_cache"].reshape(-1, bs, hkv, d)[inp["block_table"]].reshape(w.batch, s_max, hkv, d)
    vc = inp["v_cache"].reshape(-1, bs, hkv, d)[inp["block_table"]].reshape(w.batch, s_max, hkv, d)
    a = ora.decode(inp["q"], inp["k_cache"], inp["v_cache"], inp["seq_len"], inp["prompt_len"],
                   num_kv_heads=hkv, strides=inp["strides"], block_table=inp["block_table"],
                   block_size=bs, mode=ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride_grid=w.stride)
    b = ora.decode(inp["q"], np.ascontiguousarray(kc).reshape(-1), np.ascontiguousarray(vc).reshape(-1),
                   inp["seq_len"], inp["prompt_len"], num_kv_heads=hkv,
                   strides=(s_max * hkv * d, hkv * d, d), mode=ora.MODE_GRID, n_r=w.window,
                   n_att=w.n_att, stride_grid=w.stride)
    assert np.array_equal(a["out"], b["out"]) and np.array_equal(a["lse"], b["lse"])


def test_degenerate_requests():
    inp = _tiny(False, batch=3)
    w = inp["workload"]
    seq = inp["seq_len"].copy()
    pl = inp["prompt_len"].copy()
    seq[0] = 0                      # empty request
    seq[1] = pl[1]                  # no decode token yet: prompt only
    r = ora.decode(inp["q"], inp["k_cache"], inp["v_cache"], seq, pl, num_kv_heads=w.num_kv_heads,
                   strides=inp["strides"], mode=ora.MODE_GRID, n_r=w.window, n_att=w.n_att,
                   stride_grid=w.stride, want_kept=True)
    assert np.all(r["lse"][0] == -np.inf) and not r["out"][0].any()
    assert r["kept_cnt"][1, 0] == pl[1]
    assert np.isfinite(r["lse"][1:]).all()


def test_oracle_reports_threads():
    assert ora.num_threads() >= 1
