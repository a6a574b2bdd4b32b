"""GPU parity: the CUDA library (through its C ABI) against the float64 oracle on the same seeded
inputs.  Kept positions must match bit-exactly; outputs within the stated tolerances."""
import numpy as np
import pytest
import torch

from oracle import oracle as ora
from paper_2609_19702_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dsa():
    from paper_2609_19702_b200 import binding
    return binding


def _run_gpu(dsa, prob, diag):
    out, lse = dsa.alloc_outputs(prob)
    out.fill_(float("nan"))
    lse.fill_(float("nan"))
    ws = dsa.alloc_workspace(prob, diag)
    if ws is not None:
        ws.fill_(0xFF)                       # stale workspace contents must not matter
    if diag is None:
        dsa.dsa_decode_attention_dense(prob, out, lse, ws)
    else:
        dsa.dsa_decode_attention_sparse(prob, diag, out, lse, ws)
    torch.cuda.synchronize()
    return out, lse


def _check_all_modes(dsa, inp, *, f32=False, split_tokens=0, list_heads=(1,), seed=0, what="",
                     max_prompt_len=None, plan_flags=0):
    """Dense, window-only, grid and list masks of one host batch against the oracle."""
    w = inp["workload"]
    dtype = torch.float32 if f32 else torch.bfloat16
    prob = dsa.problem_from_host(inp, dtype=dtype, split_tokens=split_tokens, plan_flags=plan_flags)
    if max_prompt_len is not None:
        prob.max_prompt_len = max_prompt_len
    s_max = inp["max_seq_len"]

    ref = util.oracle_run(inp, ora.MODE_DENSE, want_kept=True)
    out, lse = _run_gpu(dsa, prob, None)
    util.assert_close(out, lse, ref, f32, what + " dense")
    idx, cnt = dsa.dsa_debug_kept_indices(prob, None, s_max)
    util.assert_kept_equal(idx, cnt, ref, what + " dense")

    diag = dsa.Diag(dsa.DSA_MASK_WINDOW, w.window)
    ref = util.oracle_run(inp, ora.MODE_WINDOW, n_r=w.window, want_kept=True)
    out, lse = _run_gpu(dsa, prob, diag)
    util.assert_close(out, lse, ref, f32, what + " window")
    idx, cnt = dsa.dsa_debug_kept_indices(prob, diag, s_max)
    util.assert_kept_equal(idx, cnt, ref, what + " window")

    diag = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
    ref = util.oracle_run(inp, ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride=w.stride, want_kept=True)
    out, lse = _run_gpu(dsa, prob, diag)
    util.assert_close(out, lse, ref, f32, what + " grid")
    idx, cnt = dsa.dsa_debug_kept_indices(prob, diag, s_max)
    util.assert_kept_equal(idx, cnt, ref, what + " grid")

    # sink variants: StreamingLLM (window + sinks) and Diagonal + sink4
    for mode_gpu, mode_ora, tag in ((dsa.DSA_MASK_WINDOW, ora.MODE_WINDOW, "streaming"),
                                    (dsa.DSA_MASK_GRID, ora.MODE_GRID, "grid+sink")):
        diag = dsa.Diag(mode_gpu, w.window, w.n_att, w.grid_w, w.row_extra, n_sink=4)
        ref = util.oracle_run(inp, mode_ora, n_r=w.window, n_att=w.n_att, stride=w.stride, n_sink=4,
                              want_kept=True)
        out, lse = _run_gpu(dsa, prob, diag)
        util.assert_close(out, lse, ref, f32, what + " " + tag)
        idx, cnt = dsa.dsa_debug_kept_indices(prob, diag, s_max)
        util.assert_kept_equal(idx, cnt, ref, what + " " + tag)

    rng = np.random.default_rng(1000 + seed)
    for mh in list_heads:
        trace = synth.random_valid_trace(rng, w.window, w.n_att, (w.batch, mh))
        n_sink = 4 if mh == list_heads[-1] else 0
        diag = dsa.Diag(dsa.DSA_MASK_LIST, w.window, w.n_att,
                        skip_offsets=torch.from_numpy(trace).cuda(), n_sink=n_sink)
        ref = util.oracle_run(inp, ora.MODE_LIST, n_r=w.window, n_att=w.n_att, trace=trace, n_sink=n_sink,
                              want_kept=True)
        out, lse = _run_gpu(dsa, prob, diag)
        util.assert_close(out, lse, ref, f32, what + " list mh=%d" % mh)
        idx, cnt = dsa.dsa_debug_kept_indices(prob, diag, s_max)
        util.assert_kept_equal(idx, cnt, ref, what + " list mh=%d" % mh)


# ---------------------------------------------------------------- the five configurations

def test_config1_every_position(dsa):
    # 16x16 grid, one query at every image position 1..256, all sharing one cache
    w = synth.workload(1)
    inp = synth.make_inputs(w)
    assert inp["position"].tolist() == list(range(1, 257))
    _check_all_modes(dsa, inp, list_heads=(1, 8), what="config1")
    _check_all_modes(dsa, inp, f32=True, list_heads=(8,), what="config1 f32")


def test_config1_paper_trace_from_oracle_argmin(dsa):
    # LIST trace produced by the oracle's own replay of the selection on this data is covered in
    # the selection tests; here the grid trace is fed back as a LIST and must equal GRID mode.
    from tests import brute
    w = synth.workload(1)
    inp = synth.make_inputs(w)
    prob = dsa.problem_from_host(inp)
    tr = np.asarray(brute.grid_trace(w.window, w.n_att, w.stride), dtype=np.int32)
    trace = np.broadcast_to(tr, (w.batch, 1, len(tr))).copy()
    d_list = dsa.Diag(dsa.DSA_MASK_LIST, w.window, w.n_att, skip_offsets=torch.from_numpy(trace).cuda())
    d_grid = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
    i1, c1 = dsa.dsa_debug_kept_indices(prob, d_list, inp["max_seq_len"])
    i2, c2 = dsa.dsa_debug_kept_indices(prob, d_grid, inp["max_seq_len"])
    assert torch.equal(c1, c2) and torch.equal(i1, i2)


@pytest.mark.parametrize("index", [2, 3, 4])
def test_configs_2_3_4(dsa, index):
    w = synth.workload(index)
    inp = synth.make_inputs(w)
    heads = (w.num_q_heads,) if index == 4 else (1,)
    _check_all_modes(dsa, inp, list_heads=heads, seed=index, what="config%d" % index)


@pytest.mark.parametrize("batch", [1, 8])
def test_config5_paged_small_batches(dsa, batch):
    for window, n_att in ((512, 208), (1024, 416)):
        w = synth.workload(5, batch=batch, window=window, n_att=n_att)
        inp = synth.make_inputs(w)
        _check_all_modes(dsa, inp, list_heads=(w.num_q_heads,), seed=batch, what="config5 B=%d" % batch)


# ---------------------------------------------------------------- properties on small shapes

SMALL = [
    # hq, hkv, d, l_p, grid_h, grid_w, extra, n_r, n_att, paged, bs
    (4, 4, 64, 7, 9, 10, 0, 40, 9, False, 16),
    (8, 2, 128, 33, 12, 7, 1, 50, 17, True, 16),
    (8, 1, 64, 1, 20, 20, 0, 200, 31, True, 8),
    (16, 2, 128, 130, 6, 33, 1, 64, 64, False, 16),
    (2, 1, 128, 0, 15, 15, 0, 33, 1, True, 32),
    (6, 3, 64, 300, 10, 12, 0, 100, 2, False, 16),
]


@pytest.mark.parametrize("case", range(len(SMALL)))
@pytest.mark.parametrize("f32", [False, True])
def test_small_shapes_all_masks_and_splits(dsa, case, f32):
    hq, hkv, d, l_p, gh, gw, extra, n_r, n_att, paged, bs = SMALL[case]
    w = synth.Workload("small%d" % case, 10 + case, 7, hq, hkv, d, l_p, gh, gw, extra, n_r, n_att,
                       1, gh * (gw + extra), positional=bool(case % 2), paged=paged, block_size=bs)
    inp = synth.make_inputs(w)
    heads = sorted({1, hkv, hq})
    for split in (0, 32, 96, 1024):
        _check_all_modes(dsa, inp, f32=f32, split_tokens=split, list_heads=heads, seed=case,
                         what="small%d split=%d" % (case, split))


def test_split_counts_agree(dsa):
    # any split size gives the same result up to fp32 rounding of the merge
    w = synth.Workload("splits", 31, 3, 8, 2, 128, 50, 30, 30, 1, 512, 200, 600, 930, paged=True)
    inp = synth.make_inputs(w)
    diag = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
    base = None
    for split in (1024, 512, 128, 64, 32):
        prob = dsa.problem_from_host(inp, dtype=torch.float32, split_tokens=split)
        for dg in (None, diag):
            out, lse = _run_gpu(dsa, prob, dg)
            key = dg is None
            if base is None or key not in base:
                base = base or {}
                base[key] = (out, lse)
            else:
                assert torch.allclose(out, base[key][0], atol=1e-5, rtol=1e-5)
                assert torch.allclose(lse, base[key][1], atol=1e-5, rtol=0)


def test_degenerate_requests(dsa):
    w = synth.Workload("degen", 41, 6, 4, 2, 64, 20, 8, 8, 0, 16, 5, 1, 64)
    inp = synth.make_inputs(w, poison=False)
    inp["seq_len"][0] = 0                       # empty request
    inp["prompt_len"][0] = 0
    inp["seq_len"][1] = inp["prompt_len"][1]    # prompt only, no decode token yet
    inp["prompt_len"][2] = 0                    # no prompt
    inp["seq_len"][2] = 3
    inp["prompt_len"][3] = inp["seq_len"][3] + 5  # prompt_len above seq_len reads as seq_len
    _check_all_modes(dsa, inp, list_heads=(1, 4), what="degenerate", max_prompt_len=0)
    _check_all_modes(dsa, inp, split_tokens=32, list_heads=(2,), what="degenerate split", max_prompt_len=0)


def test_empty_batch_and_bad_arguments(dsa):
    w = synth.Workload("args", 42, 2, 4, 4, 64, 4, 4, 4, 0, 8, 3, 1, 16)
    inp = synth.make_inputs(w)
    prob = dsa.problem_from_host(inp)
    out, lse = dsa.alloc_outputs(prob)
    empty = dsa.Problem(q=prob.q[:0].contiguous(), k_cache=prob.k_cache, v_cache=prob.v_cache,
                        strides=prob.strides, seq_len=prob.seq_len[:0], prompt_len=prob.prompt_len[:0],
                        num_kv_heads=4, max_seq_len=prob.max_seq_len)
    dsa.dsa_decode_attention_dense(empty, out[:0], lse[:0])
    with pytest.raises(dsa.DsaError):
        dsa.dsa_decode_attention_sparse(prob, dsa.Diag(dsa.DSA_MASK_GRID, 8, 9, 4, 0), out, lse)
    with pytest.raises(dsa.DsaError):
        dsa.dsa_decode_attention_sparse(prob, dsa.Diag(dsa.DSA_MASK_LIST, 8, 3), out, lse)
    torch.cuda.synchronize()


def test_combine_splits_standalone(dsa):
    rng = np.random.default_rng(5)
    b, hq, n_split, d = 3, 5, 7, 128
    out_part = rng.standard_normal((b, hq, n_split, d)).astype(np.float32)
    lse_part = (3.0 * rng.standard_normal((b, hq, n_split))).astype(np.float32)
    lse_part[0, 0, :] = -np.inf              # a query with nothing kept
    lse_part[1, 2, 3] = -np.inf              # an empty part whose out_i is garbage
    out_part[1, 2, 3] = np.nan
    ref_out, ref_lse = ora.combine(out_part.astype(np.float64), lse_part.astype(np.float64))
    for dt, tol in ((torch.float32, 1e-5), (torch.bfloat16, 1e-2)):
        out = torch.empty((b, hq, d), dtype=dt, device="cuda")
        lse = torch.empty((b, hq), dtype=torch.float32, device="cuda")
        dsa.dsa_combine_splits(torch.from_numpy(out_part).cuda(), torch.from_numpy(lse_part).cuda(), out, lse)
        torch.cuda.synchronize()
        util.assert_close(out, lse, {"out": ref_out, "lse": ref_lse}, f32=(dt == torch.float32))


def test_skipped_rows_are_never_read(dsa):
    # poison every row the mask drops: a finite, in-tolerance result proves they never enter
    w = synth.workload(5, batch=4)
    inp = synth.make_inputs(w)
    ref = util.oracle_run(inp, ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride=w.stride, want_kept=True)
    hkv, d, bs = w.num_kv_heads, w.head_dim, w.block_size
    kc = inp["k_cache"].reshape(-1, bs, hkv, d).copy()
    vc = inp["v_cache"].reshape(-1, bs, hkv, d).copy()
    for i in range(w.batch):
        keep = np.zeros(inp["block_table"].shape[1] * bs, dtype=bool)
        keep[ref["kept_idx"][i, 0, : ref["kept_cnt"][i, 0]]] = True
        drop = np.flatnonzero(~keep)
        blk = inp["block_table"][i, drop // bs]
        kc[blk, drop % bs] = synth.BF16_NAN
        vc[blk, drop % bs] = synth.BF16_NAN
    inp2 = dict(inp, k_cache=kc.reshape(-1), v_cache=vc.reshape(-1))
    prob = dsa.problem_from_host(inp2)
    diag = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
    out, lse = _run_gpu(dsa, prob, diag)
    util.assert_close(out, lse, ref, what="poisoned")


def test_kept_index_export_truncates_but_counts_everything(dsa):
    w = synth.workload(1)
    inp = synth.make_inputs(w)
    prob = dsa.problem_from_host(inp)
    diag = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
    full_idx, full_cnt = dsa.dsa_debug_kept_indices(prob, diag, inp["max_seq_len"])
    idx, cnt = dsa.dsa_debug_kept_indices(prob, diag, 20)
    torch.cuda.synchronize()
    assert torch.equal(cnt, full_cnt) and int(cnt.max()) > 20
    assert torch.equal(idx[:, :, :20], full_idx[:, :, :20])
