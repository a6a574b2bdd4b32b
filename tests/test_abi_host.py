"""Host-only checks of the C-ABI library: it loads, exports every symbol the header declares,
and rejects bad arguments before touching a device.  No compute call is made here."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "dsa.h")


@pytest.fixture(scope="module")
def dsa():
    from paper_2609_19702_b200 import build
    build.build()
    from paper_2609_19702_b200 import binding
    return binding


def _declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dsa_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(dsa):
    names = _declared_functions()
    assert "dsa_decode_attention_dense" in names and "dsa_decode_attention_sparse" in names
    assert "dsa_combine_splits" in names
    lib = ctypes.CDLL(dsa.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), "libdsa.so does not export %s" % n
    assert sorted(names) == sorted(dsa.EXPORTS)
    for n in names:
        assert hasattr(dsa, n) or n in ("dsa_status_string", "dsa_last_cuda_error"), n


def test_wait_timeouts_validates_its_argument(dsa):
    lib = ctypes.CDLL(dsa.LIB_PATH)
    lib.dsa_wait_timeouts.restype = ctypes.c_int32
    lib.dsa_wait_timeouts.argtypes = [ctypes.c_void_p]
    assert lib.dsa_wait_timeouts(None) == -1


def test_version_and_status_strings(dsa):
    assert dsa.dsa_version() == 101
    lib = ctypes.CDLL(dsa.LIB_PATH)
    lib.dsa_status_string.restype = ctypes.c_char_p
    assert lib.dsa_status_string(0) == b"ok"
    assert lib.dsa_status_string(-3) == b"workspace too small"


def _problem(dsa, **kw):
    p = dsa.dsa_problem()
    p.batch, p.num_q_heads, p.num_kv_heads, p.head_dim = 4, 32, 8, 128
    p.dtype = dsa.DSA_BF16
    # fake, aligned, never dereferenced on the host
    p.q = p.k_cache = p.v_cache = 0x10000
    p.seq_len = p.prompt_len = 0x20000
    p.stride_batch, p.stride_token, p.stride_head = 8254 * 1024, 1024, 128
    p.max_seq_len, p.max_prompt_len = 8254, 64
    for k, v in kw.items():
        setattr(p, k, v)
    return p


def _plan(dsa, p, d=None):
    lib = ctypes.CDLL(dsa.LIB_PATH)
    info = dsa.dsa_plan_info()
    rc = lib.dsa_query_plan(ctypes.byref(p), ctypes.byref(d) if d is not None else None, ctypes.byref(info))
    return rc, info


def _diag(dsa, **kw):
    d = dsa.dsa_diag_params()
    d.mode, d.window, d.n_att, d.grid_w, d.row_extra = dsa.DSA_MASK_GRID, 1024, 410, 90, 1
    for k, v in kw.items():
        setattr(d, k, v)
    return d


def test_argument_validation_on_host(dsa):
    ok, info = _plan(dsa, _problem(dsa))
    assert ok == 0 and info.n_split >= 1 and info.split_tokens % info.tile_tokens == 0
    assert _plan(dsa, _problem(dsa, head_dim=96))[0] == -2
    assert _plan(dsa, _problem(dsa, num_kv_heads=5))[0] == -1
    assert _plan(dsa, _problem(dsa, num_q_heads=48, num_kv_heads=16))[0] == -2      # group of 3
    assert _plan(dsa, _problem(dsa, q=0))[0] == -1
    assert _plan(dsa, _problem(dsa, k_cache=0x10004))[0] == -1                    # misaligned
    assert _plan(dsa, _problem(dsa, stride_token=100))[0] == -1
    assert _plan(dsa, _problem(dsa, stride_head=12))[0] == -1
    assert _plan(dsa, _problem(dsa, dtype=7))[0] == -2
    assert _plan(dsa, _problem(dsa, plan_flags=0x80000000))[0] == -1              # unknown planner switch
    assert _plan(dsa, _problem(dsa, plan_flags=dsa.DSA_PLAN_NO_ITEM_WARPS))[0] == 0
    rc, info = _plan(dsa, _problem(dsa, batch=64, num_q_heads=32, num_kv_heads=32, max_seq_len=4360, max_prompt_len=200,
                                   plan_flags=dsa.plan_group(4, 2)), _diag(dsa, window=512, n_att=208, grid_w=64))
    assert rc == 0 and info.heads_per_block == 8 and info.block_warps == 4 and info.grid_blocks == 64 * 4
    rc, info = _plan(dsa, _problem(dsa, batch=64, num_q_heads=32, num_kv_heads=32, max_seq_len=4360, max_prompt_len=200,
                                   plan_flags=dsa.DSA_PLAN_NO_GROUP), _diag(dsa, window=512, n_att=208, grid_w=64))
    assert rc == 0 and info.heads_per_block == 0
    assert _plan(dsa, _problem(dsa, block_table=0x30000, block_size=16, max_blocks=10, num_blocks=99))[0] == -1
    assert _plan(dsa, _problem(dsa), _diag(dsa, n_att=2000))[0] == -1
    assert _plan(dsa, _problem(dsa), _diag(dsa, window=0))[0] == -1
    assert _plan(dsa, _problem(dsa), _diag(dsa, grid_w=0))[0] == -1
    assert _plan(dsa, _problem(dsa), _diag(dsa, mode=dsa.DSA_MASK_LIST, mask_heads=3, trace_len=614,
                                           skip_offsets=0x40000))[0] == -1
    assert _plan(dsa, _problem(dsa), _diag(dsa, mode=dsa.DSA_MASK_LIST, mask_heads=32, trace_len=10,
                                           skip_offsets=0x40000))[0] == -1


def test_plan_sizes(dsa):
    # sparse: prompt + N_att rows per kv head fit one block -> no split, one launch
    rc, info = _plan(dsa, _problem(dsa, batch=256, num_q_heads=32, num_kv_heads=32, max_seq_len=4360,
                                   max_prompt_len=200), _diag(dsa, window=512, n_att=208, grid_w=64))
    assert rc == 0 and info.n_split == 1 and info.launches == 1
    if info.heads_per_block:                                     # one row list per block, shared by these heads
        assert info.grid_blocks * info.heads_per_block == 256 * 32 and info.block_warps in (2, 4)
        assert info.heads_per_block % info.block_warps == 0
    else:
        assert info.grid_blocks in (256 * 32, 256 * 16)          # 1 or 2 kv heads per block
    # dense on the same problem needs splits and the combine kernel
    rc, info = _plan(dsa, _problem(dsa, batch=256, num_q_heads=32, num_kv_heads=32, max_seq_len=4360))
    assert rc == 0 and info.n_split * info.split_tokens >= 4360 and info.launches == 2
    # workspace covers the partials
    lib = ctypes.CDLL(dsa.LIB_PATH)
    n = ctypes.c_size_t(0)
    p = _problem(dsa, batch=256, num_q_heads=32, num_kv_heads=32, max_seq_len=4360)
    assert lib.dsa_workspace_size(ctypes.byref(p), None, ctypes.byref(n)) == 0
    assert n.value >= 256 * 32 * info.n_split * (128 + 1) * 4
    # explicit split size is honoured, rounded to the tile
    rc, info = _plan(dsa, _problem(dsa, split_tokens=100))
    assert rc == 0 and 100 <= info.split_tokens < 100 + info.tile_tokens
    assert info.split_tokens % info.tile_tokens == 0
    # a few requests with long sequences are split to fill the machine
    rc, info = _plan(dsa, _problem(dsa, batch=1))
    assert rc == 0 and info.grid_blocks >= 148


def test_small_launch_plan_shares_items_between_warps(dsa):
    # 8 requests x 8 kv heads cannot fill the device: four warps per item, no split, one launch
    rc, info = _plan(dsa, _problem(dsa, batch=8), _diag(dsa))
    assert rc == 0 and info.tensor_cores == 1 and info.item_warps == 4
    # ... and a cluster of four such blocks per item (64 x 4 blocks fit the device at once), each block a
    # quarter of the rows; still one launch and no partial results
    assert info.n_split == 1 and info.launches == 1 and info.cluster_blocks == 4
    assert info.split_tokens * info.cluster_blocks >= 64 + 410 and info.grid_blocks == 64 * 4
    rc, info = _plan(dsa, _problem(dsa, batch=8, plan_flags=dsa.DSA_PLAN_NO_CLUSTER), _diag(dsa))
    assert rc == 0 and info.item_warps == 4 and info.cluster_blocks == 1 and info.split_tokens >= 64 + 410
    # the same requests without a mask are longer than one row list: split, one warp per item
    rc, info = _plan(dsa, _problem(dsa, batch=8))
    assert rc == 0 and info.item_warps == 1 and info.n_split > 1 and info.launches == 2
    # a full device keeps one warp per item
    rc, info = _plan(dsa, _problem(dsa, batch=256, num_q_heads=32, num_kv_heads=32, max_seq_len=4360,
                                   max_prompt_len=200), _diag(dsa, window=512, n_att=208, grid_w=64))
    assert rc == 0 and info.item_warps == 1
    # the CUDA-core kernel (float32) has no such form
    rc, info = _plan(dsa, _problem(dsa, batch=8, dtype=dsa.DSA_F32), _diag(dsa))
    assert rc == 0 and info.tensor_cores == 0 and info.item_warps == 1


def test_newer_entry_points_validate_before_touching_a_device(dsa):
    lib = ctypes.CDLL(dsa.LIB_PATH)
    p, d = _problem(dsa), _diag(dsa)
    fake = ctypes.c_void_p(0x50000)
    # fused step: the current token's rows are required, and must be 16-byte aligned
    step = lib.dsa_decode_step
    step.argtypes = [ctypes.c_void_p] * 7 + [ctypes.c_size_t, ctypes.c_void_p]
    assert step(ctypes.byref(p), ctypes.byref(d), None, fake, fake, fake, None, 0, None) == -1
    assert step(ctypes.byref(p), ctypes.byref(d), fake, None, fake, fake, None, 0, None) == -1
    assert step(ctypes.byref(p), ctypes.byref(d), ctypes.c_void_p(0x50004), fake, fake, fake, None, 0, None) == -1
    bad = _problem(dsa, head_dim=96)
    assert step(ctypes.byref(bad), ctypes.byref(d), fake, fake, fake, fake, None, 0, None) == -2
    # seq_len advance
    adv = lib.dsa_advance_seq_len
    adv.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p]
    assert adv(None, 4, 100, None) == -1
    assert adv(fake, -1, 100, None) == -1
    assert adv(fake, 4, -5, None) == -1
    assert adv(None, 0, 100, None) == 0
    # host-buffer steps: every host pointer is required; pointers that are not page-locked host
    # memory the device can address are refused (here: no such memory exists at all)
    mapped = lib.dsa_decode_attention_host_mapped
    mapped.argtypes = [ctypes.c_void_p] * 9 + [ctypes.c_size_t, ctypes.c_void_p]
    host = (ctypes.c_char * 4096)()
    hp = ctypes.cast(host, ctypes.c_void_p)
    assert mapped(ctypes.byref(p), ctypes.byref(d), None, hp, hp, None, hp, hp, None, 0, None) == -1
    assert mapped(ctypes.byref(p), ctypes.byref(d), hp, hp, hp, None, hp, hp, None, 0, None) == -1
    assert mapped(ctypes.byref(p), ctypes.byref(d), hp, hp, hp, hp, hp, hp, None, 0, None) == -1   # table without a paged cache
    host_io = lib.dsa_decode_attention_host_io
    host_io.argtypes = [ctypes.c_void_p] * 11 + [ctypes.c_size_t, ctypes.c_void_p]
    assert host_io(ctypes.byref(p), ctypes.byref(d), None, hp, hp, None, fake, fake, hp, hp, None, 0, None) == -1


def test_copy_only_hook_refuses_plans_without_the_four_warp_head_group_kernel(dsa):
    lib = ctypes.CDLL(dsa.LIB_PATH)
    hook = lib.dsa_debug_copy_only
    hook.argtypes = [ctypes.c_void_p] * 5 + [ctypes.c_size_t, ctypes.c_void_p]
    fake = ctypes.c_void_p(0x50000)
    d = _diag(dsa)
    small = _problem(dsa, batch=8)                      # several warps per item: another kernel
    assert hook(ctypes.byref(small), ctypes.byref(d), fake, fake, None, 0, None) == -2
    f32 = _problem(dsa, batch=256, dtype=dsa.DSA_F32)   # CUDA cores
    assert hook(ctypes.byref(f32), ctypes.byref(d), fake, fake, None, 0, None) == -2
    bad = _problem(dsa, batch=256, head_dim=96)
    assert hook(ctypes.byref(bad), ctypes.byref(d), fake, fake, None, 0, None) == -2
    assert hook(None, ctypes.byref(d), fake, fake, None, 0, None) == -1


def test_tensor_map_copies_only_on_request_and_only_with_a_2d_view(dsa):
    big = dict(batch=256, num_q_heads=32, num_kv_heads=32, max_seq_len=4360, max_prompt_len=200,
               stride_batch=4360 * 4096, stride_token=4096, stride_head=128)
    diag = _diag(dsa, window=512, n_att=208, grid_w=64)
    rc, info = _plan(dsa, _problem(dsa, **big), diag)
    assert rc == 0 and info.heads_per_block > 0 and info.tensor_map_copies == 0      # never by itself
    rc, info = _plan(dsa, _problem(dsa, plan_flags=dsa.DSA_PLAN_GATHER, **big), diag)
    assert rc == 0 and info.tensor_map_copies == 1 and info.block_warps == 4
    rc, info = _plan(dsa, _problem(dsa, plan_flags=dsa.DSA_PLAN_GATHER | dsa.DSA_PLAN_NO_GATHER, **big), diag)
    assert rc == 0 and info.tensor_map_copies == 0
    # head-major cache (a head's tokens contiguous): rows of different heads are not columns of one matrix
    head_major = dict(big, stride_batch=32 * 4360 * 128, stride_token=128, stride_head=4360 * 128)
    rc, info = _plan(dsa, _problem(dsa, plan_flags=dsa.DSA_PLAN_GATHER, **head_major), diag)
    assert rc == 0 and info.tensor_map_copies == 0
    # requests that do not start a whole number of token rows apart
    rc, info = _plan(dsa, _problem(dsa, plan_flags=dsa.DSA_PLAN_GATHER, **dict(big, stride_batch=4360 * 4096 + 8)), diag)
    assert rc == 0 and info.tensor_map_copies == 0
    # float32 and the two-warp head-group form have no such kernel
    rc, info = _plan(dsa, _problem(dsa, dtype=dsa.DSA_F32, plan_flags=dsa.DSA_PLAN_GATHER, **big), diag)
    assert rc == 0 and info.tensor_map_copies == 0
    rc, info = _plan(dsa, _problem(dsa, plan_flags=dsa.plan_group(2, 1) | dsa.DSA_PLAN_GATHER, **big), diag)
    assert rc == 0 and info.block_warps == 2 and info.tensor_map_copies == 0


def test_producer_warps_only_for_grids_of_more_than_one_wave(dsa):
    shape = dict(num_q_heads=32, num_kv_heads=32, max_seq_len=4360, max_prompt_len=200,
                 stride_batch=4360 * 4096, stride_token=4096, stride_head=128)
    diag = _diag(dsa, window=512, n_att=208, grid_w=64)

    def plan(batch, flags=0, d=diag):
        rc, info = _plan(dsa, _problem(dsa, batch=batch, plan_flags=flags, **shape), d)
        assert rc == 0
        return info
    big = plan(256)                       # 512 deep-ring blocks on 296 slots
    assert big.block_warps == 4 and big.stages == 3 and big.grid_blocks > 296 and big.producer_warps == 4
    assert plan(256, dsa.DSA_PLAN_NO_PRODUCERS).producer_warps == 0
    small = plan(128)                     # every block resident from the start
    assert small.grid_blocks <= 296 and small.producer_warps == 0
    assert plan(128, dsa.DSA_PLAN_PRODUCERS).producer_warps == 4
    shallow = plan(192)                   # three blocks to an SM: the registers of 8 warps a block do not fit
    assert shallow.stages == 2 and shallow.producer_warps == 0
    dense = plan(256, d=None)             # split plans keep the plain form
    assert dense.n_split > 1 and dense.producer_warps == 0
    # the tensor-map form has no producer warps, and the two-warp head-group form neither
    assert plan(256, dsa.DSA_PLAN_GATHER).producer_warps == 0
    assert plan(256, dsa.plan_group(2, 1) | dsa.DSA_PLAN_PRODUCERS).producer_warps == 0


def test_no_plan_spills_a_few_blocks_into_a_second_wave(dsa):
    """304 deep-ring blocks on 296 slots ran 21 % slower than a plan that fits (batch 152; batch 232 likewise
    with the shallow ring): the estimate must not round such a spill away."""
    shape = dict(num_q_heads=32, num_kv_heads=32, max_seq_len=4360, max_prompt_len=200,
                 stride_batch=4360 * 4096, stride_token=4096, stride_head=128)
    diag = _diag(dsa, window=512, n_att=208, grid_w=64)
    for batch in range(8, 264, 4):
        rc, info = _plan(dsa, _problem(dsa, batch=batch, **shape), diag)
        assert rc == 0
        if info.heads_per_block == 0:
            continue
        slots = 148 * (2 if info.stages == 3 else 3)
        waves = info.grid_blocks / slots
        assert not 1.0 < waves < 1.1, (batch, info.grid_blocks, info.stages)


def test_ring_depth_follows_the_wave_estimate(dsa):
    def stages(batch):
        rc, info = _plan(dsa, _problem(dsa, batch=batch, num_q_heads=32, num_kv_heads=32, max_seq_len=4360,
                                       max_prompt_len=200), _diag(dsa, window=512, n_att=208, grid_w=64))
        assert rc == 0 and info.n_split == 1 and info.item_warps == 1
        return info.stages
    # 592 two-head blocks fit at once with the deep ring, 888 with the shallow one
    assert stages(36) == 3          # 576 blocks: one wave either way
    assert stages(40) == 2          # 640: a second wave of 48 blocks, or one shallow wave
    assert stages(48) == 2
    assert stages(64) == 3          # 1024: two waves either way, the deep ones are shorter
    assert stages(256) == 3         # many waves: no difference worth the shallower pipeline
    # split plans keep the deep ring
    rc, info = _plan(dsa, _problem(dsa, batch=8, num_q_heads=32, num_kv_heads=32, max_seq_len=4360))
    assert rc == 0 and info.n_split > 1 and info.stages == 3
