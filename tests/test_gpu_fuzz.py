"""Randomised parity: many small problems with random shapes, layouts and mask parameters, the
CUDA library against the oracle.  Seeds are fixed, so a failure reproduces."""
import numpy as np
import pytest
import torch

from oracle import oracle as ora
from paper_2609_19702_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu


def _random_case(rng):
    g = int(rng.choice([1, 2, 4, 8]))
    hkv = int(rng.choice([1, 2, 3, 4, 6]))
    d = int(rng.choice([64, 128]))
    grid_w = int(rng.integers(1, 40))
    extra = int(rng.integers(0, 2))
    grid_h = int(rng.integers(1, max(2, 400 // (grid_w + extra))))
    n_img = grid_h * (grid_w + extra)
    n_r = int(rng.integers(1, min(n_img, 300) + 1))
    n_att = int(rng.integers(1, n_r + 1))
    l_p = int(rng.choice([0, 1, 5, 17, 64, 200]))
    paged = bool(rng.integers(0, 2))
    bs = int(rng.choice([1, 4, 16, 32]))
    batch = int(rng.integers(1, 6))
    return synth.Workload("fuzz", 0, batch, g * hkv, hkv, d, l_p, grid_h, grid_w, extra, n_r, n_att, 1, n_img,
                          positional=bool(rng.integers(0, 2)), paged=paged, block_size=bs)


def _random_large_case(rng):
    """Up to 3000 image tokens and windows up to 1500: several tiles per warp, several splits,
    the four-warps-per-item plans, long row lists."""
    g = int(rng.choice([1, 2, 4, 8]))
    hkv = int(rng.choice([1, 2, 4, 8]))
    d = int(rng.choice([64, 128]))
    grid_w = int(rng.integers(8, 70))
    extra = int(rng.integers(0, 2))
    grid_h = int(rng.integers(8, max(9, 3000 // (grid_w + extra))))
    n_img = grid_h * (grid_w + extra)
    n_r = int(rng.integers(64, min(n_img, 1500) + 1))
    n_att = int(rng.integers(1, n_r + 1))
    l_p = int(rng.choice([0, 33, 200, 700]))
    return synth.Workload("fuzzbig", 0, int(rng.integers(1, 9)), g * hkv, hkv, d, l_p, grid_h, grid_w, extra, n_r,
                          n_att, 1, n_img, positional=bool(rng.integers(0, 2)), paged=bool(rng.integers(0, 2)),
                          block_size=int(rng.choice([4, 16, 64])))


@pytest.mark.parametrize("seed", list(range(24)) + list(range(1000, 1010)))
def test_random_problem(seed):
    from paper_2609_19702_b200 import binding as dsa
    rng = np.random.default_rng(9000 + seed)
    w = _random_case(rng) if seed < 1000 else _random_large_case(rng)
    inp = synth.make_inputs(w, seed=500 + seed)
    f32 = bool(rng.integers(0, 4) == 0)
    split = int(rng.choice([0, 0, 16, 48, 130]))
    prob = dsa.problem_from_host(inp, dtype=torch.float32 if f32 else torch.bfloat16, split_tokens=split)
    n_sink = int(rng.choice([0, 0, 1, 4]))
    hq, hkv = w.num_q_heads, w.num_kv_heads
    mh = int(rng.choice(sorted({1, hkv, hq})))
    trace = synth.random_valid_trace(rng, w.window, w.n_att, (w.batch, mh))
    cases = [
        (None, ora.MODE_DENSE, {}),
        (dsa.Diag(dsa.DSA_MASK_WINDOW, w.window, n_sink=n_sink), ora.MODE_WINDOW, dict(n_r=w.window, n_sink=n_sink)),
        (dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra, n_sink=n_sink), ora.MODE_GRID,
         dict(n_r=w.window, n_att=w.n_att, stride=w.stride, n_sink=n_sink)),
        (dsa.Diag(dsa.DSA_MASK_LIST, w.window, w.n_att, skip_offsets=torch.from_numpy(trace).cuda(), n_sink=n_sink),
         ora.MODE_LIST, dict(n_r=w.window, n_att=w.n_att, trace=trace, n_sink=n_sink)),
    ]
    tag = "seed %d: %s f32=%s split=%d sinks=%d mh=%d" % (seed, w, f32, split, n_sink, mh)
    for diag, mode, kw in cases:
        ref = util.oracle_run(inp, mode, want_kept=True, **kw)
        out, lse = dsa.alloc_outputs(prob)
        out.fill_(float("nan"))
        ws = dsa.alloc_workspace(prob, diag)
        if diag is None:
            dsa.dsa_decode_attention_dense(prob, out, lse, ws)
        else:
            dsa.dsa_decode_attention_sparse(prob, diag, out, lse, ws)
        torch.cuda.synchronize()
        util.assert_close(out, lse, ref, f32, "%s mode %d" % (tag, mode))
        idx, cnt = dsa.dsa_debug_kept_indices(prob, diag, inp["max_seq_len"])
        util.assert_kept_equal(idx, cnt, ref, "%s mode %d" % (tag, mode))


def test_long_single_sequence_many_splits():
    # one request, 20 000 cached tokens, grouped heads: 20+ splits per kv head and a wide LIST window
    from paper_2609_19702_b200 import binding as dsa
    w = synth.Workload("long", 0, 1, 8, 2, 128, 300, 100, 197, 0, 4096, 1500, 19000, 19700)
    inp = synth.make_inputs(w, seed=77)
    prob = dsa.problem_from_host(inp)
    assert dsa.dsa_query_plan(prob, None).n_split >= 20
    rng = np.random.default_rng(3)
    trace = synth.random_valid_trace(rng, w.window, w.n_att, (1, 8))
    for diag, mode, kw in (
            (None, ora.MODE_DENSE, {}),
            (dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, 0), ora.MODE_GRID,
             dict(n_r=w.window, n_att=w.n_att, stride=w.stride)),
            (dsa.Diag(dsa.DSA_MASK_LIST, w.window, w.n_att, skip_offsets=torch.from_numpy(trace).cuda()),
             ora.MODE_LIST, dict(n_r=w.window, n_att=w.n_att, trace=trace))):
        ref = util.oracle_run(inp, mode, want_kept=True, **kw)
        out, lse = dsa.alloc_outputs(prob)
        ws = dsa.alloc_workspace(prob, diag)
        if diag is None:
            dsa.dsa_decode_attention_dense(prob, out, lse, ws)
        else:
            dsa.dsa_decode_attention_sparse(prob, diag, out, lse, ws)
        torch.cuda.synchronize()
        util.assert_close(out, lse, ref, what="long mode %d" % mode)
        idx, cnt = dsa.dsa_debug_kept_indices(prob, diag, inp["max_seq_len"])
        util.assert_kept_equal(idx, cnt, ref, "long mode %d" % mode)


@pytest.mark.parametrize("seed", list(range(12)) + list(range(2000, 2006)))
def test_random_fused_decode_step(seed):
    """Random shapes through the fused append + attention call: the current token's rows are taken
    out of a complete cache (slots poisoned), handed over as k_new / v_new with seq_len one lower,
    and the oracle's result on the complete cache is expected, with the cache restored bit for bit."""
    from paper_2609_19702_b200 import binding as dsa
    from tests.test_gpu_decode_step import _bits, _take_out_current_token
    rng = np.random.default_rng(9500 + seed)
    w = _random_case(rng) if seed < 1000 else _random_large_case(rng)
    inp = synth.make_inputs(w, seed=700 + seed)
    split = int(rng.choice([0, 0, 32, 96]))
    n_sink = int(rng.choice([0, 0, 2]))
    hq = w.num_q_heads
    mh = int(rng.choice(sorted({1, w.num_kv_heads, hq})))
    trace = synth.random_valid_trace(rng, w.window, w.n_att, (w.batch, mh))
    cases = [
        (lambda: None, ora.MODE_DENSE, {}),
        (lambda: dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra, n_sink=n_sink), ora.MODE_GRID,
         dict(n_r=w.window, n_att=w.n_att, stride=w.stride, n_sink=n_sink)),
        (lambda: dsa.Diag(dsa.DSA_MASK_LIST, w.window, w.n_att, skip_offsets=torch.from_numpy(trace.copy()).cuda(),
                          n_sink=n_sink), ora.MODE_LIST, dict(n_r=w.window, n_att=w.n_att, trace=trace, n_sink=n_sink)),
    ]
    tag = "seed %d: %s split=%d sinks=%d mh=%d" % (seed, w, split, n_sink, mh)
    for make_diag, mode, kw in cases:
        ref = util.oracle_run(inp, mode, **kw)
        prob = dsa.problem_from_host(inp, split_tokens=split)
        original = (_bits(prob.k_cache).clone(), _bits(prob.v_cache).clone())
        diag = make_diag()
        k_new, v_new = _take_out_current_token(prob, inp)
        out, lse = dsa.alloc_outputs(prob)
        out.fill_(float("nan"))
        dsa.dsa_decode_step(prob, diag, k_new, v_new, out, lse, dsa.alloc_workspace(prob, diag))
        torch.cuda.synchronize()
        util.assert_close(out, lse, ref, what="%s mode %d" % (tag, mode))
        assert torch.equal(_bits(prob.k_cache), original[0]) and torch.equal(_bits(prob.v_cache), original[1]), tag


def test_two_streams_use_the_library_at_once():
    """The library keeps no state between calls: two streams with their own problems, outputs and
    workspaces run interleaved and each gets its own oracle result."""
    from paper_2609_19702_b200 import binding as dsa
    jobs = []
    for i, (index, batch) in enumerate(((5, 3), (4, 2))):
        w = synth.workload(index, batch=batch)
        inp = synth.make_inputs(w, seed=40 + i)
        prob = dsa.problem_from_host(inp)
        diag = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
        ref_sparse = util.oracle_run(inp, ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride=w.stride)
        ref_dense = util.oracle_run(inp, ora.MODE_DENSE)
        jobs.append(dict(prob=prob, diag=diag, refs=(ref_sparse, ref_dense), stream=torch.cuda.Stream(),
                         outs=[dsa.alloc_outputs(prob) for _ in range(2)],
                         ws=(dsa.alloc_workspace(prob, diag), dsa.alloc_workspace(prob, None))))
    torch.cuda.synchronize()
    for _ in range(5):                                   # interleave the launches of the two streams
        for j in jobs:
            (o_s, l_s), (o_d, l_d) = j["outs"]
            dsa.dsa_decode_attention_sparse(j["prob"], j["diag"], o_s, l_s, j["ws"][0], stream=j["stream"])
            dsa.dsa_decode_attention_dense(j["prob"], o_d, l_d, j["ws"][1], stream=j["stream"])
    torch.cuda.synchronize()
    for n, j in enumerate(jobs):
        (o_s, l_s), (o_d, l_d) = j["outs"]
        util.assert_close(o_s, l_s, j["refs"][0], what="stream %d sparse" % n)
        util.assert_close(o_d, l_d, j["refs"][1], what="stream %d dense" % n)
