"""Small launches of the tensor-core kernel put four warps on one work item and merge their
softmax states in shared memory instead of splitting the item and combining in a second launch.

Checked here: the plan really takes that path for the small configurations, every mask mode on it
matches the oracle (kept sets are untouched by it), requests so short that some of the four warps
get no tile at all are handled, and the result -- the entries picked by the fused selection
included, which the selection tests pin to the oracle on the one-warp plan -- agrees with the
one-warp-per-item plan of the same library within the summation-order difference."""
import numpy as np
import pytest
import torch

from oracle import oracle as ora
from paper_2609_19702_b200 import synth
from tests import util
from tests.test_gpu_parity import _check_all_modes

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dsa():
    from paper_2609_19702_b200 import binding
    return binding


def _plan(dsa, inp, diag):
    return dsa.dsa_query_plan(dsa.problem_from_host(inp), diag)


@pytest.mark.parametrize("name,make", [
    ("config3, batch 2", lambda: synth.workload(3, batch=2)),
    ("config4 GQA, batch 3", lambda: synth.workload(4, batch=3)),
    ("config5 paged, batch 2", lambda: synth.workload(5, batch=2)),
    ("head_dim 64, 3 kv heads x 2", lambda: synth.Workload("kw", 91, 4, 6, 3, 64, 150, 20, 19, 1, 200, 60, 1, 400)),
])
def test_all_masks_on_the_shared_item_path(dsa, name, make):
    w = make()
    inp = synth.make_inputs(w)
    grid = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
    # (longer bounds still split, each split then shared by four warps: covered by the same cases)
    for diag in (grid, dsa.Diag(dsa.DSA_MASK_WINDOW, w.window)):
        plan = _plan(dsa, inp, diag)
        assert plan.tensor_cores == 1 and plan.item_warps == 4, name
        assert plan.launches == (1 if plan.n_split == 1 else 2)
    heads = (1, w.num_q_heads) if w.num_q_heads != w.num_kv_heads else (w.num_q_heads,)
    _check_all_modes(dsa, inp, list_heads=heads, seed=7, what=name)


def test_requests_shorter_than_one_tile_per_warp(dsa):
    # bound 40 + 300 rows, but most requests hold 1..40 rows: warps 1-3 of their items stay idle
    w = synth.Workload("short", 92, 12, 8, 8, 128, 0, 20, 15, 0, 300, 80, 1, 300)
    inp = synth.make_inputs(w, poison=False)              # (lengths are rewritten below: no NaN tail)
    inp["position"][:8] = np.arange(1, 9) * 5
    inp["seq_len"][:8] = inp["prompt_len"][:8] + inp["position"][:8]
    diag = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
    assert _plan(dsa, inp, diag).item_warps == 4
    _check_all_modes(dsa, inp, list_heads=(8,), seed=3, what="short requests")


@pytest.mark.parametrize("name,make,splits", [
    ("paged, one split", lambda: synth.workload(5, batch=4), 1),
    # 600 kept rows for 4 pairs: two splits, each shared by four warps, then the combine kernel
    ("long list, two splits", lambda: synth.Workload("kw2", 94, 2, 4, 2, 128, 200, 30, 29, 1, 600, 400, 500, 880), 2),
])
def test_shared_item_path_agrees_with_one_warp_per_item(dsa, name, make, splits):
    w = make()
    inp = synth.make_inputs(w)
    rng = np.random.default_rng(4)
    trace = synth.random_valid_trace(rng, w.window, w.n_att, (w.batch, w.num_q_heads))
    results = {}
    for setting in ("1", "0"):
        prob = dsa.problem_from_host(inp, plan_flags=0 if setting == "1" else dsa.DSA_PLAN_NO_ITEM_WARPS)
        outs = []
        for diag in (None, dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra),
                     dsa.Diag(dsa.DSA_MASK_LIST, w.window, w.n_att,
                              skip_offsets=torch.from_numpy(trace.copy()).cuda(), select=True)):
            plan = dsa.dsa_query_plan(prob, diag)
            if diag is not None:
                assert plan.item_warps == (4 if setting == "1" else 1), name
                if setting == "1":
                    # (a cluster of blocks takes the place of HBM splits where the mask allows one)
                    assert plan.n_split == (1 if plan.cluster_blocks > 1 else splits), name
            out, lse = dsa.alloc_outputs(prob)
            ws = dsa.alloc_workspace(prob, diag)
            if diag is None:
                dsa.dsa_decode_attention_dense(prob, out, lse, ws)
            else:
                dsa.dsa_decode_attention_sparse(prob, diag, out, lse, ws)
            torch.cuda.synchronize()
            outs.append((out.float().cpu(), lse.cpu(), None if diag is None else diag.skip_offsets))
        results[setting] = outs
    for (o1, l1, t1), (o0, l0, t0) in zip(results["1"], results["0"]):
        assert torch.allclose(o1, o0, atol=2e-2, rtol=2e-2)
        assert torch.allclose(l1, l0, atol=1e-4, rtol=0)
        if t1 is not None:
            # the selected distances (one new trace entry per head) must be the same keys
            assert torch.equal(t1.cpu(), t0.cpu())


def test_shallow_ring_form_matches_the_oracle(dsa):
    """The two-heads-per-block kernel with a two-stage ring: chosen by the planner when the deep
    ring would spill a few blocks into another wave, and forced here on the standard cases."""
    # 40 requests x 32 kv heads = 640 blocks: 1.08 waves with the deep ring, 0.72 with the shallow one
    w = synth.Workload("shallow", 95, 40, 32, 32, 128, 20, 10, 10, 0, 64, 20, 1, 100)
    inp = synth.make_inputs(w)
    grid = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
    plan = _plan(dsa, inp, grid)
    assert plan.stages == 2 and plan.item_warps == 1 and plan.n_split == 1
    _check_all_modes(dsa, inp, list_heads=(1,), seed=5, what="shallow ring, chosen")
    for make in (lambda: synth.workload(5, batch=3), lambda: synth.workload(2, batch=8)):
        w2 = make()
        inp2 = synth.make_inputs(w2)
        prob = dsa.problem_from_host(inp2, split_tokens=0, plan_flags=dsa.DSA_PLAN_RING_SHALLOW)
        g2 = dsa.Diag(dsa.DSA_MASK_GRID, w2.window, w2.n_att, w2.grid_w, w2.row_extra)
        if w2.num_kv_heads % 2 == 0 and dsa.dsa_query_plan(prob, g2).item_warps == 1:
            assert dsa.dsa_query_plan(prob, g2).stages == 2
        _check_all_modes(dsa, inp2, list_heads=(1,), seed=6, what="shallow ring, forced",
                         plan_flags=dsa.DSA_PLAN_RING_SHALLOW)


# ---------------------------------------------------------------- clusters: several blocks per work item

@pytest.mark.parametrize("name,make", [
    ("config4 GQA, batch 3", lambda: synth.workload(4, batch=3)),
    ("config5 paged, batch 1", lambda: synth.workload(5, batch=1)),
    ("config5 paged, window 1024, batch 2 (in place of two splits)", lambda: synth.workload(5, batch=2, window=1024, n_att=416)),
    ("config3 long prompt, batch 1", lambda: synth.workload(3, batch=1)),
])
def test_cluster_form_is_chosen_for_the_smallest_launches_and_matches_the_oracle(dsa, name, make):
    """The blocks of a thread-block cluster take row ranges of one work item and block 0 collects
    their softmax states through distributed shared memory: same results as every other plan."""
    w = make()
    inp = synth.make_inputs(w)
    grid = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
    plan = _plan(dsa, inp, grid)
    assert plan.cluster_blocks in (2, 4) and plan.item_warps == 4 and plan.n_split == 1 and plan.launches == 1, name
    assert plan.grid_blocks == plan.work_items * plan.cluster_blocks
    _check_all_modes(dsa, inp, list_heads=(1,), seed=11, what=name)
    # and switched off: the plan without clusters, same results within the summation-order difference
    prob_on = dsa.problem_from_host(inp)
    prob_off = dsa.problem_from_host(inp, plan_flags=dsa.DSA_PLAN_NO_CLUSTER)
    assert dsa.dsa_query_plan(prob_off, grid).cluster_blocks == 1
    res = []
    for prob in (prob_on, prob_off):
        out, lse = dsa.alloc_outputs(prob)
        dsa.dsa_decode_attention_sparse(prob, grid, out, lse, dsa.alloc_workspace(prob, grid))
        torch.cuda.synchronize()
        res.append((out.float().cpu(), lse.cpu()))
    assert torch.allclose(res[0][0], res[1][0], atol=2e-2, rtol=2e-2) and torch.allclose(res[0][1], res[1][1], atol=1e-4, rtol=0)


@pytest.mark.parametrize("flag", ["DSA_PLAN_CLUSTER2", "DSA_PLAN_CLUSTER4"])
def test_forced_cluster_sizes_on_short_ragged_and_empty_ranges(dsa, flag):
    """Forced onto requests so short that some blocks of a cluster (and some warps of a block) get no
    rows at all, with and without the fused decode step."""
    from tests import test_gpu_decode_step as t_step
    flags = getattr(dsa, flag)
    w = synth.Workload("clshort", 93, 6, 8, 2, 128, 3, 20, 15, 0, 300, 80, 1, 300)
    inp = synth.make_inputs(w, poison=False)
    inp["position"][:4] = np.array([1, 7, 20, 33])
    inp["seq_len"][:4] = inp["prompt_len"][:4] + inp["position"][:4]
    grid = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
    prob = dsa.problem_from_host(inp, plan_flags=flags)
    plan = dsa.dsa_query_plan(prob, grid)
    assert plan.cluster_blocks == (2 if flag.endswith("2") else 4) and plan.item_warps == 4
    _check_all_modes(dsa, inp, list_heads=(1,), seed=12, what=flag, plan_flags=flags)
    # the fused decode step through the same plans
    orig = dsa.Problem.c_struct

    def patched(self):
        p = orig(self)
        p.plan_flags |= flags
        return p

    dsa.Problem.c_struct = patched
    try:
        for name in ("gqa_long", "paged", "gqa8_paged_small"):
            for mask in ("dense", "grid_sink", "window"):
                t_step.test_fused_step_matches_oracle_and_the_two_calls(dsa, name, mask, 0)
    finally:
        dsa.Problem.c_struct = orig
