"""ctypes binding of ``libdsa.so``: the same entry-point names as ``include/dsa.h``.

Argument marshalling only -- every step of the attention path runs in the CUDA kernels behind
the C ABI.  PyTorch is used for device memory and streams.  There is no fallback: if the
library has not been built (``python -m paper_2609_19702_b200.build``) importing this module
raises, and every call raises on a non-zero status.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdsa.so")

DSA_BF16, DSA_F32 = 0, 1
DSA_MASK_WINDOW, DSA_MASK_GRID, DSA_MASK_LIST = 0, 1, 2
# dsa_problem.plan_flags: 0 lets the library plan; the bits force single decisions (comparison runs, tests)
DSA_PLAN_CUDA_CORES, DSA_PLAN_NO_ITEM_WARPS, DSA_PLAN_RING_DEEP, DSA_PLAN_RING_SHALLOW = 0x1, 0x2, 0x4, 0x8
DSA_PLAN_GROUP, DSA_PLAN_NO_GROUP, DSA_PLAN_GROUP_W4 = 0x10, 0x20, 0x40
DSA_PLAN_HEADS_PER_WARP_SHIFT = 8
DSA_PLAN_NO_CLUSTER, DSA_PLAN_CLUSTER2, DSA_PLAN_CLUSTER4 = 0x80, 0x10000, 0x20000
DSA_PLAN_GATHER, DSA_PLAN_NO_GATHER = 0x40000, 0x80000
DSA_PLAN_PRODUCERS, DSA_PLAN_NO_PRODUCERS = 0x100000, 0x200000
DSA_PLAN_METADATA_STABLE = 0x800000


def plan_group(warps: int, heads_per_warp: int) -> int:
    """plan_flags that force the head-group kernel with `warps` (2 or 4) warps per block, each
    streaming `heads_per_warp` kv heads."""
    assert warps in (2, 4) and 1 <= heads_per_warp <= 255
    return DSA_PLAN_GROUP | (DSA_PLAN_GROUP_W4 if warps == 4 else 0) | (heads_per_warp << DSA_PLAN_HEADS_PER_WARP_SHIFT)

EXPORTS = ["dsa_version", "dsa_status_string", "dsa_last_cuda_error", "dsa_workspace_size",
           "dsa_query_plan", "dsa_decode_attention_dense", "dsa_decode_attention_sparse",
           "dsa_combine_splits", "dsa_debug_kept_indices",
           "dsa_decode_attention_static_scratch", "dsa_append_kv", "dsa_decode_attention_host_io",
           "dsa_decode_attention_host_mapped", "dsa_decode_step", "dsa_advance_seq_len", "dsa_prepare",
           "dsa_wait_timeouts", "dsa_debug_wait_giveup", "dsa_debug_copy_only", "dsa_build_skip_bitmap"]


class dsa_problem(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("num_q_heads", ctypes.c_int32),
                ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("sm_scale", ctypes.c_float),
                ("q", ctypes.c_void_p), ("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p),
                ("stride_batch", ctypes.c_int64), ("stride_token", ctypes.c_int64),
                ("stride_head", ctypes.c_int64),
                ("seq_len", ctypes.c_void_p), ("prompt_len", ctypes.c_void_p),
                ("block_table", ctypes.c_void_p),
                ("max_blocks", ctypes.c_int32), ("block_size", ctypes.c_int32),
                ("num_blocks", ctypes.c_int32), ("max_seq_len", ctypes.c_int32),
                ("max_prompt_len", ctypes.c_int32), ("split_tokens", ctypes.c_int32),
                ("ring_size", ctypes.c_int32), ("ring_sinks", ctypes.c_int32),
                ("plan_flags", ctypes.c_uint32)]


class dsa_diag_params(ctypes.Structure):
    _fields_ = [("mode", ctypes.c_int32), ("window", ctypes.c_int32), ("n_att", ctypes.c_int32),
                ("grid_w", ctypes.c_int32), ("row_extra", ctypes.c_int32),
                ("skip_offsets", ctypes.c_void_p), ("mask_heads", ctypes.c_int32),
                ("trace_len", ctypes.c_int32), ("n_sink", ctypes.c_int32),
                ("select", ctypes.c_int32), ("skip_bitmap", ctypes.c_void_p)]


class dsa_plan_info(ctypes.Structure):
    _fields_ = [("split_tokens", ctypes.c_int32), ("n_split", ctypes.c_int32),
                ("launches", ctypes.c_int32), ("grid_blocks", ctypes.c_int32),
                ("smem_bytes", ctypes.c_int32), ("tile_tokens", ctypes.c_int32),
                ("stages", ctypes.c_int32), ("tensor_cores", ctypes.c_int32), ("work_items", ctypes.c_int32),
                ("item_warps", ctypes.c_int32), ("heads_per_block", ctypes.c_int32),
                ("block_warps", ctypes.c_int32), ("per_head_lists", ctypes.c_int32),
                ("cluster_blocks", ctypes.c_int32), ("tensor_map_copies", ctypes.c_int32),
                ("producer_warps", ctypes.c_int32)]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError("libdsa.so is not built: run `python -m paper_2609_19702_b200.build` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32 = ctypes.c_void_p, ctypes.c_int32
    lib.dsa_version.restype = i32
    lib.dsa_status_string.restype = ctypes.c_char_p
    lib.dsa_status_string.argtypes = [i32]
    lib.dsa_last_cuda_error.restype = i32
    lib.dsa_workspace_size.restype = i32
    lib.dsa_workspace_size.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_size_t)]
    lib.dsa_query_plan.restype = i32
    lib.dsa_query_plan.argtypes = [vp, vp, ctypes.POINTER(dsa_plan_info)]
    lib.dsa_decode_attention_dense.restype = i32
    lib.dsa_decode_attention_dense.argtypes = [vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.dsa_decode_attention_sparse.restype = i32
    lib.dsa_decode_attention_sparse.argtypes = [vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.dsa_combine_splits.restype = i32
    lib.dsa_combine_splits.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, i32, vp]
    lib.dsa_decode_attention_static_scratch.restype = i32
    lib.dsa_decode_attention_static_scratch.argtypes = [vp, vp, vp, vp, vp]
    lib.dsa_decode_attention_host_io.restype = i32
    lib.dsa_decode_attention_host_io.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.dsa_wait_timeouts.restype = i32
    lib.dsa_wait_timeouts.argtypes = [ctypes.POINTER(i32)]
    lib.dsa_debug_copy_only.restype = i32
    lib.dsa_debug_copy_only.argtypes = [vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.dsa_build_skip_bitmap.restype = i32
    lib.dsa_build_skip_bitmap.argtypes = [vp, vp, vp]
    lib.dsa_debug_wait_giveup.restype = i32
    lib.dsa_debug_wait_giveup.argtypes = [vp]
    lib.dsa_prepare.restype = i32
    lib.dsa_prepare.argtypes = []
    lib.dsa_decode_step.restype = i32
    lib.dsa_decode_step.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.dsa_advance_seq_len.restype = i32
    lib.dsa_advance_seq_len.argtypes = [vp, i32, i32, vp]
    lib.dsa_decode_attention_host_mapped.restype = i32
    lib.dsa_decode_attention_host_mapped.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.dsa_append_kv.restype = i32
    lib.dsa_append_kv.argtypes = [vp, vp, vp, i32, vp]
    lib.dsa_debug_kept_indices.restype = i32
    lib.dsa_debug_kept_indices.argtypes = [vp, vp, vp, vp, i32, vp]
    return lib


_lib = _load()


class DsaError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        msg = _lib.dsa_status_string(status).decode()
        extra = ""
        if status == -4:
            extra = " (cuda error %d)" % _lib.dsa_last_cuda_error()
        super().__init__("%s: %s%s" % (fn, msg, extra))


def _check(fn: str, status: int) -> None:
    if status != 0:
        raise DsaError(fn, status)


def _dptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return DSA_BF16
    if t.dtype == torch.float32:
        return DSA_F32
    raise TypeError("q/k/v must be bfloat16 or float32")


@dataclass
class Problem:
    """Device tensors and host-side sizes of one decode-attention call (see dsa_problem)."""
    q: torch.Tensor                       # [B, H_q, D]
    k_cache: torch.Tensor                 # any shape; addressed through `strides`
    v_cache: torch.Tensor
    strides: tuple                        # (stride_batch_or_block, stride_token, stride_head), elements
    seq_len: torch.Tensor                 # int32 [B]
    prompt_len: torch.Tensor              # int32 [B]
    num_kv_heads: int
    max_seq_len: int
    max_prompt_len: int = 0
    block_table: Optional[torch.Tensor] = None   # int32 [B, max_blocks]
    block_size: int = 0
    num_blocks: int = 0
    sm_scale: float = 0.0
    split_tokens: int = 0
    ring_size: int = 0                    # > 0: bounded cache, decode tokens live in a ring
    ring_sinks: int = 0
    plan_flags: int = 0                   # DSA_PLAN_* bits; 0 = the library chooses the launch plan

    def c_struct(self) -> dsa_problem:
        b, hq, d = self.q.shape
        assert self.q.is_contiguous() and self.q.is_cuda
        assert self.seq_len.dtype == torch.int32 and self.prompt_len.dtype == torch.int32
        p = dsa_problem()
        p.batch, p.num_q_heads, p.num_kv_heads, p.head_dim = b, hq, self.num_kv_heads, d
        p.dtype = _dtype_code(self.q)
        p.sm_scale = float(self.sm_scale)
        p.q, p.k_cache, p.v_cache = self.q.data_ptr(), self.k_cache.data_ptr(), self.v_cache.data_ptr()
        p.stride_batch, p.stride_token, p.stride_head = (int(s) for s in self.strides)
        p.seq_len, p.prompt_len = self.seq_len.data_ptr(), self.prompt_len.data_ptr()
        if self.block_table is not None:
            assert self.block_table.dtype == torch.int32 and self.block_table.is_contiguous()
            p.block_table = self.block_table.data_ptr()
            p.max_blocks = self.block_table.shape[1]
            p.block_size = self.block_size
            p.num_blocks = self.num_blocks
        p.max_seq_len = int(self.max_seq_len)
        p.max_prompt_len = int(self.max_prompt_len)
        p.split_tokens = int(self.split_tokens)
        p.ring_size, p.ring_sinks = int(self.ring_size), int(self.ring_sinks)
        p.plan_flags = int(self.plan_flags)
        return p


@dataclass
class Diag:
    """Mask parameters of the sparse call (see dsa_diag_params)."""
    mode: int
    window: int
    n_att: int = 0
    grid_w: int = 0
    row_extra: int = 0
    skip_offsets: Optional[torch.Tensor] = None   # int32 [B, mask_heads, trace_len] (LIST)
    n_sink: int = 0
    select: bool = False                          # LIST: also append the next trace entry (in place)
    skip_bitmap: Optional[torch.Tensor] = None    # int32 [B, mask_heads, ceil(window / 32)]: the lists as bits

    def c_struct(self) -> dsa_diag_params:
        d = dsa_diag_params()
        d.mode, d.window, d.n_att = self.mode, self.window, self.n_att
        d.grid_w, d.row_extra = self.grid_w, self.row_extra
        d.n_sink = self.n_sink
        d.select = 1 if self.select else 0
        if self.skip_offsets is not None:
            t = self.skip_offsets
            assert t.dtype == torch.int32 and t.is_contiguous() and t.dim() == 3
            d.skip_offsets = t.data_ptr()
            d.mask_heads, d.trace_len = t.shape[1], t.shape[2]
        if self.skip_bitmap is not None:
            bm = self.skip_bitmap
            assert self.skip_offsets is not None and bm.dtype == torch.int32 and bm.is_contiguous()
            assert tuple(bm.shape) == (self.skip_offsets.shape[0], self.skip_offsets.shape[1], (self.window + 31) // 32)
            d.skip_bitmap = bm.data_ptr()
        return d


def _ref(s):
    return None if s is None else ctypes.addressof(s)


def dsa_version() -> int:
    return int(_lib.dsa_version())


def dsa_workspace_size(problem: Problem, diag: Optional[Diag] = None) -> int:
    p = problem.c_struct()
    d = diag.c_struct() if diag is not None else None
    n = ctypes.c_size_t(0)
    _check("dsa_workspace_size", _lib.dsa_workspace_size(_ref(p), _ref(d), ctypes.byref(n)))
    return int(n.value)


def dsa_prepare() -> None:
    """Configure every kernel variant for the current CUDA device (needed only before capturing
    calls that would otherwise be the first of their shape on this device)."""
    _check("dsa_prepare", _lib.dsa_prepare())


def dsa_wait_timeouts() -> int:
    """Bounded waits of the tensor-map kernel that gave up on the current device (0 in a healthy run)."""
    n = ctypes.c_int32(0)
    _check("dsa_wait_timeouts", _lib.dsa_wait_timeouts(ctypes.byref(n)))
    return int(n.value)


def dsa_build_skip_bitmap(problem: Problem, diag: Diag, stream: Optional[torch.cuda.Stream] = None) -> None:
    """Fill diag.skip_bitmap from diag.skip_offsets for the requests' current seq_len."""
    p, d = problem.c_struct(), diag.c_struct()
    _check("dsa_build_skip_bitmap", _lib.dsa_build_skip_bitmap(_ref(p), _ref(d), _stream(stream)))


def dsa_debug_wait_giveup(stream: Optional[torch.cuda.Stream] = None) -> None:
    """Launch the one-warp kernel whose bounded wait runs out (about a second); dsa_wait_timeouts() then
    counts one more."""
    _check("dsa_debug_wait_giveup", _lib.dsa_debug_wait_giveup(_stream(stream)))


def dsa_query_plan(problem: Problem, diag: Optional[Diag] = None) -> dsa_plan_info:
    p = problem.c_struct()
    d = diag.c_struct() if diag is not None else None
    info = dsa_plan_info()
    _check("dsa_query_plan", _lib.dsa_query_plan(_ref(p), _ref(d), ctypes.byref(info)))
    return info


def alloc_outputs(problem: Problem):
    b, hq, d = problem.q.shape
    out = torch.empty((b, hq, d), dtype=problem.q.dtype, device=problem.q.device)
    lse = torch.empty((b, hq), dtype=torch.float32, device=problem.q.device)
    return out, lse


def alloc_workspace(problem: Problem, diag: Optional[Diag] = None) -> Optional[torch.Tensor]:
    n = dsa_workspace_size(problem, diag)
    if n == 0:
        return None
    return torch.empty(n, dtype=torch.uint8, device=problem.q.device)


def dsa_decode_attention_dense(problem: Problem, out: torch.Tensor, lse: torch.Tensor,
                               workspace: Optional[torch.Tensor] = None,
                               stream: Optional[torch.cuda.Stream] = None) -> None:
    p = problem.c_struct()
    ws_n = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check("dsa_decode_attention_dense",
           _lib.dsa_decode_attention_dense(_ref(p), _dptr(out), _dptr(lse), _dptr(workspace), ws_n,
                                           _stream(stream)))


def dsa_decode_attention_sparse(problem: Problem, diag: Diag, out: torch.Tensor, lse: torch.Tensor,
                                workspace: Optional[torch.Tensor] = None,
                                stream: Optional[torch.cuda.Stream] = None) -> None:
    p = problem.c_struct()
    d = diag.c_struct()
    ws_n = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check("dsa_decode_attention_sparse",
           _lib.dsa_decode_attention_sparse(_ref(p), _ref(d), _dptr(out), _dptr(lse), _dptr(workspace),
                                            ws_n, _stream(stream)))


def dsa_debug_copy_only(problem: Problem, diag: Optional[Diag], out: torch.Tensor, lse: torch.Tensor,
                        workspace: Optional[torch.Tensor] = None,
                        stream: Optional[torch.cuda.Stream] = None) -> None:
    """The attention call with the arithmetic taken out (same grid, lists and K / V staging; out and lse
    come back meaningless): what the staging alone costs.  Raises DsaError (unsupported) unless the plan
    is the four-warp head-group kernel."""
    p = problem.c_struct()
    d = diag.c_struct() if diag is not None else None
    ws_n = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check("dsa_debug_copy_only",
           _lib.dsa_debug_copy_only(_ref(p), _ref(d), _dptr(out), _dptr(lse), _dptr(workspace), ws_n,
                                    _stream(stream)))


def dsa_decode_attention_static_scratch(problem: Problem, diag: Optional[Diag], out: torch.Tensor,
                                        lse: torch.Tensor,
                                        stream: Optional[torch.cuda.Stream] = None) -> None:
    """Dense (diag None) or sparse attention whose split partials use the library's built-in
    fixed-size scratch array: for callers that may not allocate device memory around the call.
    Raises DsaError (workspace too small) when the partials would not fit the array."""
    p = problem.c_struct()
    d = diag.c_struct() if diag is not None else None
    _check("dsa_decode_attention_static_scratch",
           _lib.dsa_decode_attention_static_scratch(_ref(p), _ref(d), _dptr(out), _dptr(lse), _stream(stream)))


def dsa_decode_attention_host_io(problem: Problem, diag: Optional[Diag], host_q: torch.Tensor,
                                 host_seq_len: torch.Tensor, host_prompt_len: torch.Tensor,
                                 host_block_table: Optional[torch.Tensor], dev_out: torch.Tensor,
                                 dev_lse: torch.Tensor, host_out: torch.Tensor, host_lse: torch.Tensor,
                                 workspace: Optional[torch.Tensor] = None,
                                 stream: Optional[torch.cuda.Stream] = None) -> None:
    """One decode step with the step's inputs and results in (pinned) host tensors; the device
    tensors inside ``problem`` are overwritten with the host inputs.  Asynchronous: synchronise the
    stream before reading ``host_out`` / ``host_lse``."""
    for t in (host_q, host_seq_len, host_prompt_len, host_out, host_lse):
        assert not t.is_cuda and t.is_contiguous()
    p = problem.c_struct()
    d = diag.c_struct() if diag is not None else None
    ws_n = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check("dsa_decode_attention_host_io",
           _lib.dsa_decode_attention_host_io(_ref(p), _ref(d), _dptr(host_q), _dptr(host_seq_len),
                                             _dptr(host_prompt_len), _dptr(host_block_table), _dptr(dev_out),
                                             _dptr(dev_lse), _dptr(host_out), _dptr(host_lse), _dptr(workspace),
                                             ws_n, _stream(stream)))


def dsa_decode_attention_host_mapped(problem: Problem, diag: Optional[Diag], host_q: torch.Tensor,
                                     host_seq_len: torch.Tensor, host_prompt_len: torch.Tensor,
                                     host_block_table: Optional[torch.Tensor], host_out: torch.Tensor,
                                     host_lse: torch.Tensor, workspace: Optional[torch.Tensor] = None,
                                     stream: Optional[torch.cuda.Stream] = None) -> None:
    """One decode step whose kernels read ``host_q`` from and write ``host_out`` / ``host_lse`` to
    pinned host tensors directly; lengths and block table are copied into the device tensors of
    ``problem`` (and ``problem.q`` may be used as scratch).  Raises DsaError (invalid argument) for
    host tensors that are not pinned.  Asynchronous: synchronise the stream before reading the
    results."""
    for t in (host_q, host_seq_len, host_prompt_len, host_out, host_lse):
        assert not t.is_cuda and t.is_contiguous()
    p = problem.c_struct()
    d = diag.c_struct() if diag is not None else None
    ws_n = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check("dsa_decode_attention_host_mapped",
           _lib.dsa_decode_attention_host_mapped(_ref(p), _ref(d), _dptr(host_q), _dptr(host_seq_len),
                                                 _dptr(host_prompt_len), _dptr(host_block_table),
                                                 _dptr(host_out), _dptr(host_lse), _dptr(workspace),
                                                 ws_n, _stream(stream)))


def dsa_combine_splits(out_part: torch.Tensor, lse_part: torch.Tensor, out: torch.Tensor,
                       lse: Optional[torch.Tensor] = None,
                       stream: Optional[torch.cuda.Stream] = None) -> None:
    """out_part [B, H_q, n_split, D] f32, lse_part [B, H_q, n_split] f32 -> out [B, H_q, D], lse."""
    assert out_part.dtype == torch.float32 and lse_part.dtype == torch.float32
    assert out_part.is_contiguous() and lse_part.is_contiguous() and out.is_contiguous()
    b, hq, n_split, d = out_part.shape
    _check("dsa_combine_splits",
           _lib.dsa_combine_splits(_dptr(out_part), _dptr(lse_part), b, hq, d, n_split, _dptr(out),
                                   _dptr(lse), _dtype_code(out), _stream(stream)))


def dsa_append_kv(problem: Problem, k_new: torch.Tensor, v_new: torch.Tensor, advance: bool = False,
                  stream: Optional[torch.cuda.Stream] = None) -> None:
    """Write the new token's K/V rows [B, H_kv, D] at logical position seq_len[b]; optionally
    increment seq_len on the device afterwards."""
    assert k_new.is_contiguous() and v_new.is_contiguous() and k_new.dtype == problem.q.dtype
    p = problem.c_struct()
    _check("dsa_append_kv", _lib.dsa_append_kv(_ref(p), _dptr(k_new), _dptr(v_new), 1 if advance else 0,
                                               _stream(stream)))


def dsa_decode_step(problem: Problem, diag: Optional[Diag], k_new: torch.Tensor, v_new: torch.Tensor,
                    out: torch.Tensor, lse: torch.Tensor, workspace: Optional[torch.Tensor] = None,
                    stream: Optional[torch.cuda.Stream] = None) -> None:
    """Append + attention of one decode step in one call: ``problem.seq_len`` counts the tokens
    already cached (it is not advanced), ``k_new`` / ``v_new`` [B, H_kv, D] are the current token."""
    b, _, d = problem.q.shape
    for t in (k_new, v_new):
        assert t.is_cuda and t.is_contiguous() and t.dtype == problem.q.dtype
        assert tuple(t.shape) == (b, problem.num_kv_heads, d)
    p = problem.c_struct()
    dg = diag.c_struct() if diag is not None else None
    ws_n = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check("dsa_decode_step",
           _lib.dsa_decode_step(_ref(p), _ref(dg), _dptr(k_new), _dptr(v_new), _dptr(out), _dptr(lse),
                                _dptr(workspace), ws_n, _stream(stream)))


def dsa_advance_seq_len(seq_len: torch.Tensor, max_seq_len: int,
                        stream: Optional[torch.cuda.Stream] = None) -> None:
    """seq_len[b] += 1 on the device for every request below ``max_seq_len``."""
    assert seq_len.is_cuda and seq_len.dtype == torch.int32 and seq_len.is_contiguous()
    _check("dsa_advance_seq_len",
           _lib.dsa_advance_seq_len(_dptr(seq_len), seq_len.numel(), int(max_seq_len), _stream(stream)))


def dsa_debug_kept_indices(problem: Problem, diag: Optional[Diag], max_kept: int,
                           stream: Optional[torch.cuda.Stream] = None):
    """Kept cache positions per (request, mask head): returns (idx [B, mh, max_kept], count [B, mh])."""
    p = problem.c_struct()
    d = diag.c_struct() if diag is not None else None
    mh = 1
    if diag is not None and diag.mode == DSA_MASK_LIST and diag.skip_offsets is not None:
        mh = diag.skip_offsets.shape[1]
    b = problem.q.shape[0]
    idx = torch.full((b, mh, max(max_kept, 1)), -1, dtype=torch.int32, device=problem.q.device)
    cnt = torch.zeros((b, mh), dtype=torch.int32, device=problem.q.device)
    _check("dsa_debug_kept_indices",
           _lib.dsa_debug_kept_indices(_ref(p), _ref(d), _dptr(idx), _dptr(cnt), max_kept, _stream(stream)))
    return idx, cnt


def problem_from_host(inp: dict, device: str = "cuda", dtype: torch.dtype = torch.bfloat16,
                      split_tokens: int = 0, plan_flags: int = 0) -> Problem:
    """Copy one host batch (as made by ``synth.make_inputs``: bf16 bit patterns) to the device."""
    w = inp["workload"]

    def dev(bits):
        t = torch.from_numpy(bits).view(torch.bfloat16).to(device)
        return t if dtype == torch.bfloat16 else t.to(dtype)

    bt = inp["block_table"]
    return Problem(
        q=dev(inp["q"]), k_cache=dev(inp["k_cache"]), v_cache=dev(inp["v_cache"]),
        strides=inp["strides"],
        seq_len=torch.from_numpy(inp["seq_len"]).to(device),
        prompt_len=torch.from_numpy(inp["prompt_len"]).to(device),
        num_kv_heads=w.num_kv_heads, max_seq_len=inp["max_seq_len"], max_prompt_len=w.prompt_len,
        block_table=None if bt is None else torch.from_numpy(bt).to(device),
        block_size=inp["block_size"], num_blocks=0 if bt is None else int(bt.size),
        split_tokens=split_tokens, plan_flags=plan_flags)
