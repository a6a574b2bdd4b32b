"""ctypes loader for the float64 CPU oracle (``dsa_oracle.c``).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the tests, the smoke check and the benchmark's
CPU-baseline leg import this module.  It imports nothing from the CUDA package and the CUDA
package imports nothing from here.

The wrappers only marshal numpy arrays into the C entry points; every piece of arithmetic is in
``dsa_oracle.c`` (Algorithm 1 replay, softmax attention over the kept rows, log-sum-exp merge).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dsa_oracle.c")
_LIB = os.path.join(_HERE, "libdsa_oracle.so")

F64, F32, BF16 = 0, 1, 2
SEL_TRACE, SEL_GRID, SEL_ARGMIN = 0, 1, 2
MODE_DENSE, MODE_WINDOW, MODE_GRID, MODE_LIST = 0, 1, 2, 3

_lib = None


def build(force: bool = False) -> str:
    """Compile ``dsa_oracle.c`` with gcc into ``libdsa_oracle.so`` next to it."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-Wall", "-Wextra",
           "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        i32, i64, dbl, vp = ctypes.c_int32, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        _lib.dsa_oracle_num_threads.restype = ctypes.c_int
        _lib.dsa_oracle_replay.restype = ctypes.c_int
        _lib.dsa_oracle_replay.argtypes = [i32, i32, i32, i32, vp, i32, i32, vp, vp, vp, vp]
        _lib.dsa_oracle_replay_argmin.restype = ctypes.c_int
        _lib.dsa_oracle_replay_argmin.argtypes = [i32, i32, i32, i32, vp, i64, vp, ctypes.c_int, vp, i32, dbl,
                                                  vp, vp, vp, vp]
        _lib.dsa_oracle_select_argmin.restype = ctypes.c_int
        _lib.dsa_oracle_select_argmin.argtypes = [vp, vp, ctypes.c_int, vp, i32, i32, dbl, vp, vp]
        _lib.dsa_oracle_attend.restype = ctypes.c_int
        _lib.dsa_oracle_attend.argtypes = [vp, vp, vp, ctypes.c_int, vp, vp, i32, i32, dbl, vp, vp]
        _lib.dsa_oracle_combine.restype = ctypes.c_int
        _lib.dsa_oracle_combine.argtypes = [vp, vp, i64, i32, i32, vp, vp]
        _lib.dsa_oracle_kept.restype = ctypes.c_int
        _lib.dsa_oracle_kept.argtypes = [i32, i32, i32, i32, i32, i32, vp, i32, i32, vp, vp]
        _lib.dsa_oracle_decode.restype = ctypes.c_int
        _lib.dsa_oracle_decode.argtypes = [i32, i32, i32, i32, i32, vp, vp, vp, i64, i64, i64,
                                           vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, i32, i32, i32,
                                           dbl, vp, vp, vp, vp, i32, i32]
    return _lib


def num_threads() -> int:
    return int(lib().dsa_oracle_num_threads())


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float64:
        return F64
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16  # bfloat16 bit patterns
    raise TypeError("oracle takes float64, float32 or uint16 (bf16 bits) arrays, got %s" % a.dtype)


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise RuntimeError("%s failed with oracle status %d" % (what, rc))


def replay(t: int, n_r: int, n_att: int, selector: int = SEL_TRACE,
           trace: Optional[Sequence[int]] = None, stride: int = 0):
    """Algorithm 1 up to step ``t``: returns (idx attended at step t, skip_idx after step t)."""
    tr = np.ascontiguousarray(np.asarray([] if trace is None else trace, dtype=np.int32))
    idx = np.zeros(n_r + 1, dtype=np.int32)
    skip = np.zeros(n_r + 1, dtype=np.int32)
    n_idx = ctypes.c_int32(0)
    n_skip = ctypes.c_int32(0)
    rc = lib().dsa_oracle_replay(t, n_r, n_att, selector, _ptr(tr), len(tr), stride, _ptr(idx),
                                 ctypes.addressof(n_idx), _ptr(skip), ctypes.addressof(n_skip))
    _check(rc, "dsa_oracle_replay")
    return idx[: n_idx.value].copy(), skip[: n_skip.value].copy()


def replay_argmin(t: int, n_r: int, n_att: int, q_steps: np.ndarray, q_step_stride: int, k: np.ndarray,
                  k_rows: np.ndarray, d: int, sm_scale: float, n_sink: int = 0):
    """Algorithm 1 with its argmin selection for one head: query of step s at element
    ``s * q_step_stride`` of ``q_steps``, decode key j at element ``k_rows[j]`` of ``k``.
    Returns (idx attended at step t, trace of distances selected so far)."""
    assert q_steps.flags.c_contiguous and k.flags.c_contiguous
    assert _dtype_code(q_steps) == _dtype_code(k)
    rows = np.ascontiguousarray(k_rows, dtype=np.int64)
    idx = np.zeros(n_r + 1, dtype=np.int32)
    tr = np.zeros(max(n_r - n_att, 1), dtype=np.int32)
    n_idx = ctypes.c_int32(0)
    n_tr = ctypes.c_int32(0)
    rc = lib().dsa_oracle_replay_argmin(t, n_r, n_att, n_sink, _ptr(q_steps), int(q_step_stride), _ptr(k),
                                        _dtype_code(k), _ptr(rows), d, float(sm_scale), _ptr(idx),
                                        ctypes.addressof(n_idx), _ptr(tr), ctypes.addressof(n_tr))
    _check(rc, "dsa_oracle_replay_argmin")
    return idx[: n_idx.value].copy(), tr[: n_tr.value].copy()


def kept(mode: int, l_p: int, p: int, n_r: int = 0, n_att: int = 0, stride: int = 0,
         trace: Optional[Sequence[int]] = None, n_sink: int = 0) -> np.ndarray:
    """Kept cache positions (prompt + attended decode keys) of one request at decode position p."""
    tr = np.ascontiguousarray(np.asarray([] if trace is None else trace, dtype=np.int32))
    outbuf = np.zeros(l_p + p + 1, dtype=np.int32)
    n = ctypes.c_int32(0)
    rc = lib().dsa_oracle_kept(mode, l_p, p, n_r, n_att, stride, _ptr(tr), len(tr), n_sink, _ptr(outbuf),
                               ctypes.addressof(n))
    _check(rc, "dsa_oracle_kept")
    return outbuf[: n.value].copy()


def select_argmin(q_row: np.ndarray, k: np.ndarray, k_rows: np.ndarray, d: int, sm_scale: float):
    """Phase-2 selection for one step: returns (position of the argmin within idx, weights w)."""
    q_row = np.ascontiguousarray(q_row)
    k = np.ascontiguousarray(k)
    rows = np.ascontiguousarray(k_rows, dtype=np.int64)
    w = np.zeros(len(rows), dtype=np.float64)
    j = ctypes.c_int32(-1)
    rc = lib().dsa_oracle_select_argmin(_ptr(q_row), _ptr(k), _dtype_code(k), _ptr(rows), len(rows),
                                        d, float(sm_scale), ctypes.addressof(j), _ptr(w))
    _check(rc, "dsa_oracle_select_argmin")
    return int(j.value), w


def attend(q_row: np.ndarray, k: np.ndarray, v: np.ndarray, k_rows: np.ndarray, v_rows: np.ndarray,
           d: int, sm_scale: float):
    """Softmax attention of one query over the given rows: returns (out[D], lse)."""
    q_row = np.ascontiguousarray(q_row)
    assert k.flags.c_contiguous and v.flags.c_contiguous
    assert _dtype_code(q_row) == _dtype_code(k) == _dtype_code(v)
    kr = np.ascontiguousarray(k_rows, dtype=np.int64)
    vr = np.ascontiguousarray(v_rows, dtype=np.int64)
    out = np.zeros(d, dtype=np.float64)
    lse = ctypes.c_double(0.0)
    rc = lib().dsa_oracle_attend(_ptr(q_row), _ptr(k), _ptr(v), _dtype_code(k), _ptr(kr), _ptr(vr),
                                 len(kr), d, float(sm_scale), _ptr(out), ctypes.addressof(lse))
    _check(rc, "dsa_oracle_attend")
    return out, float(lse.value)


def combine(out_part: np.ndarray, lse_part: np.ndarray):
    """Merge partial results: out_part [..., n_split, D], lse_part [..., n_split] (float64)."""
    out_part = np.ascontiguousarray(out_part, dtype=np.float64)
    lse_part = np.ascontiguousarray(lse_part, dtype=np.float64)
    n_split, d = out_part.shape[-2], out_part.shape[-1]
    lead = out_part.shape[:-2]
    rows = int(np.prod(lead)) if lead else 1
    out = np.zeros(lead + (d,), dtype=np.float64)
    lse = np.zeros(lead, dtype=np.float64)
    rc = lib().dsa_oracle_combine(_ptr(out_part), _ptr(lse_part), rows, n_split, d, _ptr(out), _ptr(lse))
    _check(rc, "dsa_oracle_combine")
    return out, lse


def decode(q: np.ndarray, k_cache: np.ndarray, v_cache: np.ndarray, seq_len: np.ndarray,
           prompt_len: np.ndarray, *, num_kv_heads: int, strides: Sequence[int],
           block_table: Optional[np.ndarray] = None, block_size: int = 0,
           mode: int = MODE_DENSE, n_r: int = 0, n_att: int = 0, stride_grid: int = 0,
           trace: Optional[np.ndarray] = None, n_sink: int = 0, sm_scale: Optional[float] = None,
           want_kept: bool = False, n_threads: int = 0):
    """One decode-attention call over a batch.

    q [B, H_q, D]; caches are flat arrays addressed with ``strides`` = (stride_b_or_block,
    stride_token, stride_head) in elements.  ``trace`` [B, mask_heads, m] for MODE_LIST.
    Returns dict(out [B,H_q,D] f64, lse [B,H_q] f64, kept_idx, kept_cnt).
    """
    q = np.ascontiguousarray(q)
    b, h_q, d = q.shape
    assert k_cache.flags.c_contiguous and v_cache.flags.c_contiguous
    code = _dtype_code(q)
    assert code == _dtype_code(k_cache) == _dtype_code(v_cache)
    seq_len = np.ascontiguousarray(seq_len, dtype=np.int32)
    prompt_len = np.ascontiguousarray(prompt_len, dtype=np.int32)
    if sm_scale is None:
        sm_scale = 1.0 / float(np.sqrt(d))
    bt = None
    max_blocks = 0
    if block_table is not None:
        bt = np.ascontiguousarray(block_table, dtype=np.int32)
        max_blocks = bt.shape[1]
    mask_heads, trace_len, tr = 1, 0, None
    if mode == MODE_LIST:
        tr = np.ascontiguousarray(trace, dtype=np.int32)
        assert tr.ndim == 3 and tr.shape[0] == b
        mask_heads, trace_len = tr.shape[1], tr.shape[2]
    out = np.zeros((b, h_q, d), dtype=np.float64)
    lse = np.zeros((b, h_q), dtype=np.float64)
    kept_idx = kept_cnt = None
    max_kept = 0
    if want_kept:
        max_kept = int(seq_len.max()) if b else 0
        kept_idx = np.full((b, mask_heads, max(max_kept, 1)), -1, dtype=np.int32)
        kept_cnt = np.zeros((b, mask_heads), dtype=np.int32)
        max_kept = max(max_kept, 1)
    rc = lib().dsa_oracle_decode(b, h_q, num_kv_heads, d, code, _ptr(q), _ptr(k_cache), _ptr(v_cache),
                                 int(strides[0]), int(strides[1]), int(strides[2]),
                                 _ptr(seq_len), _ptr(prompt_len), _ptr(bt), max_blocks, block_size,
                                 mode, n_r, n_att, stride_grid, _ptr(tr), mask_heads, trace_len, n_sink,
                                 float(sm_scale), _ptr(out), _ptr(lse), _ptr(kept_idx), _ptr(kept_cnt),
                                 max_kept, n_threads)
    _check(rc, "dsa_oracle_decode")
    return {"out": out, "lse": lse, "kept_idx": kept_idx, "kept_cnt": kept_cnt}
