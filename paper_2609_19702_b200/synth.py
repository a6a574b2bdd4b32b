"""Seeded synthetic decode-attention workloads.

This module only DRAWS INPUTS: random tensors with the shapes, value distributions and position
mixes of the five benchmark configurations, block tables, and valid skip traces.  It holds none
of the method's arithmetic (no mask, no attention), so both the CUDA binding and the CPU oracle
can be fed from it without sharing anything else.

Everything is generated on the host with ``numpy.random.default_rng(seed)`` and rounded to
bfloat16 (stored as uint16 bit patterns); the very same arrays go to the GPU and to the oracle,
so input rounding is not part of any error budget.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional

import numpy as np

BF16_NAN = np.uint16(0x7FC0)
BASE_SEED = 19702


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest even); returns the uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    bits = x.view(np.uint32)
    rounded = (bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass(frozen=True)
class Workload:
    """One benchmark configuration (shapes follow the token counts of the paper's Table 1)."""
    name: str
    index: int                 # 1..5, seeds the generator
    batch: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    prompt_len: int            # L_p
    grid_h: int
    grid_w: int
    row_extra: int             # row-end / separator tokens per image row (0 or 1)
    window: int                # N_r
    n_att: int                 # N_att
    pos_lo: int                # decode position p drawn uniformly from [pos_lo, pos_hi]
    pos_hi: int
    positional: bool = False   # add 0.5 x a 2-D sin-cos embedding to image-token q/k/v
    paged: bool = False
    block_size: int = 16
    share_cache: bool = False  # all requests read one cache (batch stride 0); positions 1..batch

    @property
    def stride(self) -> int:   # tokens per image row in raster order
        return self.grid_w + self.row_extra

    @property
    def image_tokens(self) -> int:
        return self.grid_h * self.stride

    @property
    def max_seq_len(self) -> int:
        return self.prompt_len + self.image_tokens


def workload(index: int, batch: Optional[int] = None, window: Optional[int] = None,
             n_att: Optional[int] = None) -> Workload:
    """The five configurations.  N_att is 5 % of the image tokens (95 % sparsity) unless given."""
    table = {
        1: Workload("tiny", 1, 256, 8, 8, 64, 32, 16, 16, 0, 64, 13, 1, 256, share_cache=True),
        2: Workload("mid_mha", 2, 32, 20, 20, 64, 120, 32, 32, 0, 256, 52, 1, 1024, positional=True),
        3: Workload("mha_7b", 3, 64, 32, 32, 128, 600, 24, 24, 0, 128, 29, 289, 576),
        4: Workload("gqa_long", 4, 8, 32, 8, 128, 64, 90, 90, 1, 1024, 410, 4096, 8190, positional=True),
        5: Workload("paged_sweep", 5, 256, 32, 32, 128, 200, 64, 64, 1, 512, 208, 1, 4160, paged=True),
    }
    w = table[index]
    if batch is not None:
        w = replace(w, batch=batch)
    if window is not None:
        w = replace(w, window=window)
    if n_att is not None:
        w = replace(w, n_att=n_att)
    return w


def _positional(w: Workload) -> np.ndarray:
    """[image_tokens, D] float32: textbook 2-D sin-cos embedding, rows from r, columns from c."""
    d = w.head_dim
    half = d // 2
    tok = np.arange(w.image_tokens)
    r = (tok // w.stride).astype(np.float64)
    c = (tok % w.stride).astype(np.float64)
    is_grid = (tok % w.stride) < w.grid_w
    i = np.arange(half // 2, dtype=np.float64)
    freq = 10000.0 ** (-2.0 * i / half)
    emb = np.zeros((w.image_tokens, d), dtype=np.float64)
    emb[:, 0:half:2] = np.sin(r[:, None] * freq[None, :])
    emb[:, 1:half:2] = np.cos(r[:, None] * freq[None, :])
    emb[:, half::2] = np.sin(c[:, None] * freq[None, :])
    emb[:, half + 1::2] = np.cos(c[:, None] * freq[None, :])
    emb[~is_grid] = 0.0
    return (0.5 * emb).astype(np.float32)


def random_valid_trace(rng: np.random.Generator, window: int, n_att: int, shape=()) -> np.ndarray:
    """Random skip traces [..., window - n_att]: entry k (0-based) is an offset in
    [0, n_att - 1 + k] that no earlier entry used -- the only constraint a trace must meet."""
    m = window - n_att
    n = int(np.prod(shape)) if shape else 1
    out = np.zeros((n, max(m, 0)), dtype=np.int32)
    for i in range(n):
        used = np.zeros(window, dtype=bool)
        for k in range(m):
            free = np.flatnonzero(~used[: n_att + k])
            o = int(free[rng.integers(len(free))])
            used[o] = True
            out[i, k] = o
    return out.reshape(tuple(shape) + (max(m, 0),))


_DRAWN: Dict[tuple, Dict[str, object]] = {}
_DRAWN_BYTES = [0]
_DRAWN_LIMIT = 3 << 30


def make_inputs(w: Workload, seed: Optional[int] = None, poison: bool = True) -> Dict[str, object]:
    """The batch of inputs for workload ``w`` (see _draw_inputs).  Drawing a few hundred million normal
    variates takes seconds and the same (workload, seed) is asked for again and again, so batches are
    kept per process (up to 3 GB) and every caller gets its own copy of the arrays."""
    key = (w, seed, poison)
    hit = _DRAWN.get(key)
    if hit is None:
        hit = _draw_inputs(w, seed, poison)
        size = sum(v.nbytes for v in hit.values() if isinstance(v, np.ndarray))
        if _DRAWN_BYTES[0] + size <= _DRAWN_LIMIT:
            _DRAWN[key] = hit
            _DRAWN_BYTES[0] += size
        else:
            return hit
    return {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in hit.items()}


def _draw_inputs(w: Workload, seed: Optional[int] = None, poison: bool = True) -> Dict[str, object]:
    """Draw one batch of inputs for workload ``w`` on the host.

    Returns a dict with
      q            uint16 [B, H_q, D]   bf16 bits
      k_cache/v_cache uint16, flat view of  [B, S_max, H_kv, D]  (contiguous)  or
                                            [num_blocks, block_size, H_kv, D]  (paged)
      strides      (stride_b_or_block, stride_token, stride_head) in elements
      seq_len, prompt_len  int32 [B];  position int32 [B] (= seq_len - prompt_len)
      block_table  int32 [B, max_blocks] or None;  block_size
    Cache rows at positions >= seq_len are NaN when ``poison`` (never for a shared cache).
    """
    rng = np.random.default_rng(BASE_SEED + w.index if seed is None else seed)
    b, hq, hkv, d = w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim
    s_max = w.max_seq_len
    pos_emb = _positional(w) if w.positional else None

    if w.share_cache:
        position = (np.arange(b, dtype=np.int32) % w.image_tokens) + 1
    else:
        position = rng.integers(w.pos_lo, w.pos_hi + 1, size=b, dtype=np.int32)
    prompt_len = np.full(b, w.prompt_len, dtype=np.int32)
    seq_len = prompt_len + position

    q = rng.standard_normal((b, hq, d), dtype=np.float32)
    if pos_emb is not None:
        q += pos_emb[position - 1][:, None, :]
    q_bits = f32_to_bf16_bits(q)

    def draw_seq() -> np.ndarray:
        x = rng.standard_normal((s_max, hkv, d), dtype=np.float32)
        if pos_emb is not None:
            x[w.prompt_len:] += pos_emb[:, None, :]
        return f32_to_bf16_bits(x)

    row = hkv * d
    block_table = None
    if w.paged:
        bs = w.block_size
        max_blocks = (s_max + bs - 1) // bs
        num_blocks = b * max_blocks
        block_table = rng.permutation(num_blocks).astype(np.int32).reshape(b, max_blocks)
        k_cache = np.empty((num_blocks, bs, hkv, d), dtype=np.uint16)
        v_cache = np.empty((num_blocks, bs, hkv, d), dtype=np.uint16)
        pad = max_blocks * bs - s_max
        for i in range(b):
            for cache in (k_cache, v_cache):
                x = draw_seq()
                if poison:
                    x[seq_len[i]:] = BF16_NAN
                if pad:
                    x = np.concatenate([x, np.full((pad, hkv, d), BF16_NAN, dtype=np.uint16)])
                cache[block_table[i]] = x.reshape(max_blocks, bs, hkv, d)
        strides = (bs * row, row, d)
    elif w.share_cache:
        k_cache = draw_seq().reshape(1, s_max, hkv, d)
        v_cache = draw_seq().reshape(1, s_max, hkv, d)
        strides = (0, row, d)
    else:
        k_cache = np.empty((b, s_max, hkv, d), dtype=np.uint16)
        v_cache = np.empty((b, s_max, hkv, d), dtype=np.uint16)
        for i in range(b):
            for cache in (k_cache, v_cache):
                x = draw_seq()
                if poison:
                    x[seq_len[i]:] = BF16_NAN
                cache[i] = x
        strides = (s_max * row, row, d)

    return {
        "workload": w,
        "q": q_bits,
        "k_cache": k_cache.reshape(-1),
        "v_cache": v_cache.reshape(-1),
        "cache_shape": k_cache.shape,
        "strides": strides,
        "seq_len": seq_len.astype(np.int32),
        "prompt_len": prompt_len,
        "position": position.astype(np.int32),
        "block_table": block_table,
        "block_size": w.block_size if w.paged else 0,
        "max_seq_len": s_max,
    }


def shard_requests(batch: int, world_size: int, rank: int) -> range:
    """Contiguous slice of request ids owned by ``rank`` (requests are independent units)."""
    base, extra = divmod(batch, world_size)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def make_inputs_device(w: Workload, device, seed: Optional[int] = None, poison: bool = True) -> Dict[str, object]:
    """Full-size batches for benchmarking: same shapes, layouts and position mix as
    ``make_inputs`` but K/V/q are drawn on ``device`` with a seeded torch generator (a paged pool
    at batch 256 is 18 GB, too slow to draw on the host).  Values are N(0,1) (+ the positional
    component where the workload has one) rounded to bf16; cache rows at positions >= seq_len are
    NaN when ``poison`` (never for a shared cache), as in ``make_inputs``.  Returns torch tensors;
    positions, lengths and the block table are also returned as numpy arrays under ``host``.
    """
    import torch

    seed = BASE_SEED + w.index if seed is None else seed
    rng = np.random.default_rng(seed)
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    b, hq, hkv, d = w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim
    s_max = w.max_seq_len
    row = hkv * d
    if w.share_cache:
        position = (np.arange(b, dtype=np.int32) % w.image_tokens) + 1
    else:
        position = rng.integers(w.pos_lo, w.pos_hi + 1, size=b, dtype=np.int32)
    prompt_len = np.full(b, w.prompt_len, dtype=np.int32)
    seq_len = (prompt_len + position).astype(np.int32)
    pos_emb = torch.from_numpy(_positional(w)).to(device) if w.positional else None

    q = torch.randn((b, hq, d), generator=gen, device=device, dtype=torch.float32)
    if pos_emb is not None:
        q += pos_emb[torch.from_numpy(position.astype(np.int64) - 1).to(device)][:, None, :]
    q = q.to(torch.bfloat16)

    def draw(n_seq: int):
        """[n_seq, s_pad, hkv, d] bf16, one sequence at a time to bound temporaries."""
        s_pad = s_max if not w.paged else ((s_max + w.block_size - 1) // w.block_size) * w.block_size
        out = torch.empty((n_seq, s_pad, hkv, d), device=device, dtype=torch.bfloat16)
        for i in range(n_seq):
            x = torch.randn((s_pad, hkv, d), generator=gen, device=device, dtype=torch.float32)
            if pos_emb is not None:
                x[w.prompt_len:s_max] += pos_emb[:, None, :]
            out[i] = x.to(torch.bfloat16)
        return out

    block_table = None
    nan = float("nan")
    if w.paged:
        bs = w.block_size
        max_blocks = (s_max + bs - 1) // bs
        num_blocks = b * max_blocks
        block_table = rng.permutation(num_blocks).astype(np.int32).reshape(b, max_blocks)
        bt = torch.from_numpy(block_table.astype(np.int64)).to(device)
        if not w.positional:
            # the pool is i.i.d. noise, so drawing it in pool order is the same distribution as
            # drawing per sequence and scattering through the table
            k_cache = draw(b).reshape(num_blocks, bs, hkv, d)
            v_cache = draw(b).reshape(num_blocks, bs, hkv, d)
        else:
            k_cache = torch.empty((num_blocks, bs, hkv, d), device=device, dtype=torch.bfloat16)
            v_cache = torch.empty_like(k_cache)
            for i in range(b):
                k_cache[bt[i]] = draw(1).reshape(max_blocks, bs, hkv, d)
                v_cache[bt[i]] = draw(1).reshape(max_blocks, bs, hkv, d)
        if poison:
            # tokens at positions >= seq_len: the tail of the block that holds position seq_len,
            # then every later block of the request (one masked fill per request and cache)
            for i in range(b):
                n = int(seq_len[i])
                first, within = divmod(n, bs)
                for cache in (k_cache, v_cache):
                    if within and first < max_blocks:
                        cache[bt[i, first], within:] = nan
                    lo = first + (1 if within else 0)
                    if lo < max_blocks:
                        cache[bt[i, lo:]] = nan
        strides = (bs * row, row, d)
    elif w.share_cache:
        k_cache, v_cache = draw(1), draw(1)
        strides = (0, row, d)
    else:
        k_cache, v_cache = draw(b), draw(b)
        if poison:
            for i in range(b):
                k_cache[i, int(seq_len[i]):] = nan
                v_cache[i, int(seq_len[i]):] = nan
        strides = (s_max * row, row, d)

    return {
        "workload": w,
        "q": q,
        "k_cache": k_cache.reshape(-1),
        "v_cache": v_cache.reshape(-1),
        "cache_shape": tuple(k_cache.shape),
        "strides": strides,
        "seq_len": torch.from_numpy(seq_len).to(device),
        "prompt_len": torch.from_numpy(prompt_len).to(device),
        "block_table": None if block_table is None else torch.from_numpy(block_table).to(device),
        "block_size": w.block_size if w.paged else 0,
        "max_seq_len": s_max,
        "host": {"seq_len": seq_len, "prompt_len": prompt_len, "position": position.astype(np.int32),
                 "block_table": block_table},
    }


def host_subset(dev: Dict[str, object], requests) -> Dict[str, object]:
    """Copy the given requests of a device batch (``make_inputs_device``) to the host, in the
    dict layout of ``make_inputs`` (bf16 bit patterns; paged pools are compacted to the blocks
    these requests own and the block table renumbered).  Pure data movement."""
    import torch

    w: Workload = dev["workload"]
    req = [int(r) for r in requests]
    n = len(req)
    hkv, d = w.num_kv_heads, w.head_dim
    ridx = torch.tensor(req, dtype=torch.int64, device=dev["q"].device)

    def bits(t):
        return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)

    host = dev["host"]
    out = {
        "workload": replace(w, batch=n, share_cache=False) if not w.share_cache else replace(w, batch=n),
        "q": bits(dev["q"][ridx]),
        "seq_len": host["seq_len"][req].copy(),
        "prompt_len": host["prompt_len"][req].copy(),
        "position": host["position"][req].copy(),
        "block_size": dev["block_size"],
        "max_seq_len": dev["max_seq_len"],
        "block_table": None,
    }
    if w.paged:
        bs = w.block_size
        bt = dev["block_table"][ridx].to(torch.int64)
        max_blocks = bt.shape[1]
        kc = dev["k_cache"].view(-1, bs, hkv, d)[bt.reshape(-1)]
        vc = dev["v_cache"].view(-1, bs, hkv, d)[bt.reshape(-1)]
        out["k_cache"], out["v_cache"] = bits(kc).reshape(-1), bits(vc).reshape(-1)
        out["block_table"] = np.arange(n * max_blocks, dtype=np.int32).reshape(n, max_blocks)
        out["strides"] = dev["strides"]
    elif w.share_cache:
        out["k_cache"], out["v_cache"] = bits(dev["k_cache"]).reshape(-1), bits(dev["v_cache"]).reshape(-1)
        out["strides"] = dev["strides"]
    else:
        s_max = dev["max_seq_len"]
        kc = dev["k_cache"].view(-1, s_max, hkv, d)[ridx]
        vc = dev["v_cache"].view(-1, s_max, hkv, d)[ridx]
        out["k_cache"], out["v_cache"] = bits(kc).reshape(-1), bits(vc).reshape(-1)
        out["strides"] = dev["strides"]
    return out
