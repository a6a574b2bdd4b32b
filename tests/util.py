"""Shared helpers of the GPU parity tests: run the oracle and the CUDA library on the same host
batch and compare.  Tolerances are the ones the task states: kept positions bit-exact,
|gpu - ref| <= 1e-2 + 1e-2 |ref| for bf16 outputs, |lse_gpu - lse_ref| <= 1e-3."""
from __future__ import annotations

import zlib

import numpy as np

from oracle import oracle as ora
from paper_2609_19702_b200 import synth

OUT_ATOL, OUT_RTOL, LSE_ATOL = 1e-2, 1e-2, 1e-3
# float32: the worst measured error is 4.4e-7 on the outputs and 9e-7 on the LSE (0.04 / 0.09 of these bounds)
F32_ATOL, F32_RTOL, F32_LSE_ATOL = 1e-5, 1e-5, 1e-5


_ORACLE_MEMO = {}


def _crc(x):
    return None if x is None else (x.shape, str(x.dtype), zlib.crc32(np.ascontiguousarray(x).view(np.uint8).reshape(-1)))


def oracle_run(inp, mode, *, n_r=0, n_att=0, stride=0, trace=None, n_sink=0, want_kept=False, requests=None):
    """Oracle on a host batch (optionally on a subset of requests).  Several modules run the same
    cases under different kernel plans, so results are kept per process, keyed by checksums of every
    input array and by the arguments (the oracle itself is untouched)."""
    w = inp["workload"]
    key = (mode, n_r, n_att, stride, n_sink, want_kept, None if requests is None else tuple(int(r) for r in requests),
           w.num_kv_heads, tuple(inp["strides"]), inp["block_size"], _crc(trace),
           tuple(_crc(inp[k]) for k in ("q", "k_cache", "v_cache", "seq_len", "prompt_len", "block_table")))
    if key in _ORACLE_MEMO:
        return _ORACLE_MEMO[key]
    ref = _oracle_run(inp, mode, n_r=n_r, n_att=n_att, stride=stride, trace=trace, n_sink=n_sink, want_kept=want_kept,
                      requests=requests)
    if len(_ORACLE_MEMO) < 4096:
        _ORACLE_MEMO[key] = ref
    return ref


def _oracle_run(inp, mode, *, n_r=0, n_att=0, stride=0, trace=None, n_sink=0, want_kept=False, requests=None):
    w = inp["workload"]
    q, seq, pl, bt = inp["q"], inp["seq_len"], inp["prompt_len"], inp["block_table"]
    if requests is not None:
        req = np.asarray(requests)
        q, seq, pl = q[req], seq[req], pl[req]
        if bt is not None:
            bt = bt[req]
        else:
            raise ValueError("request subsets need a paged cache")
        if trace is not None:
            trace = trace[req]
    return ora.decode(q, inp["k_cache"], inp["v_cache"], seq, pl, num_kv_heads=w.num_kv_heads,
                      strides=inp["strides"], block_table=bt, block_size=inp["block_size"],
                      mode=mode, n_r=n_r, n_att=n_att, stride_grid=stride, trace=trace, n_sink=n_sink,
                      want_kept=want_kept)


def assert_close(out_gpu, lse_gpu, ref, f32=False, what=""):
    out = out_gpu.float().cpu().numpy().astype(np.float64)
    lse = lse_gpu.cpu().numpy().astype(np.float64)
    atol, rtol, latol = (F32_ATOL, F32_RTOL, F32_LSE_ATOL) if f32 else (OUT_ATOL, OUT_RTOL, LSE_ATOL)
    assert np.isfinite(out).all(), what + ": non-finite output (a masked or poisoned row leaked)"
    err = np.abs(out - ref["out"]) - (atol + rtol * np.abs(ref["out"]))
    assert err.max() <= 0, "%s: out off by %.3g beyond tolerance at %s" % (
        what, err.max(), np.unravel_index(err.argmax(), err.shape))
    ref_lse = ref["lse"]
    both_inf = np.isneginf(lse) & np.isneginf(ref_lse)
    with np.errstate(invalid="ignore"):
        lerr = np.where(both_inf, 0.0, np.abs(lse - ref_lse))
    assert np.nanmax(lerr) <= latol and not np.isnan(lerr).any(), "%s: lse off by %.3g" % (what, np.nanmax(lerr))


def assert_kept_equal(idx_gpu, cnt_gpu, ref, what=""):
    idx = idx_gpu.cpu().numpy()
    cnt = cnt_gpu.cpu().numpy()
    assert np.array_equal(cnt, ref["kept_cnt"]), what + ": kept counts differ"
    b, mh = cnt.shape
    for i in range(b):
        for h in range(mh):
            n = int(cnt[i, h])
            assert np.array_equal(idx[i, h, :n], ref["kept_idx"][i, h, :n]), \
                "%s: kept positions differ at request %d mask head %d" % (what, i, h)
