"""The bounded mbarrier waits of the producer-warp and tensor-map kernels.

Runs last in the suite: first it checks that no wait of any earlier test gave up, then it makes one
wait run out on purpose (a barrier nothing arrives on, the library's own test hook) and checks that
the kernel ends by itself, the give-up is counted and the context still computes.
"""
import time

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


def test_a_wait_that_runs_out_is_counted_and_the_context_survives(dsa):
    torch.cuda.synchronize()
    before = dsa.dsa_wait_timeouts()
    assert before == 0, "a bounded wait of an earlier call gave up"
    t0 = time.time()
    dsa.dsa_debug_wait_giveup()
    torch.cuda.synchronize()
    took = time.time() - t0
    assert dsa.dsa_wait_timeouts() == before + 1
    assert 0.3 < took < 10.0, "the wait is bounded at about a second, it took %.2f s" % took
    # the context is intact: a producer-warp launch afterwards matches the oracle
    w = synth.workload(5, batch=2)
    inp = synth.make_inputs(w)
    prob = dsa.problem_from_host(inp, plan_flags=dsa.plan_group(4, 1) | dsa.DSA_PLAN_PRODUCERS)
    diag = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
    assert dsa.dsa_query_plan(prob, diag).producer_warps == 4
    out, lse = dsa.alloc_outputs(prob)
    dsa.dsa_decode_attention_sparse(prob, diag, out, lse, dsa.alloc_workspace(prob, diag))
    torch.cuda.synchronize()
    ref = util.oracle_run(inp, ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride=w.stride)
    util.assert_close(out, lse, ref, what="after a give-up")
    assert dsa.dsa_wait_timeouts() == before + 1


def test_copy_only_hook_runs_and_leaves_the_library_as_it_was(dsa):
    """The measuring form of the head-group kernel: same plan, no arithmetic.  Its outputs mean nothing;
    what is checked is that it runs, is not slower than the attention call it mirrors, and that the
    attention call after it still matches the oracle."""
    w = synth.workload(5, batch=32)
    inp = synth.make_inputs(w)
    prob = dsa.problem_from_host(inp)
    diag = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
    plan = dsa.dsa_query_plan(prob, diag)
    assert plan.block_warps == 4 and plan.per_head_lists == 0
    out, lse = dsa.alloc_outputs(prob)
    ws = dsa.alloc_workspace(prob, diag)

    def timed(fn):
        for _ in range(3):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(20):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    t_copy = timed(lambda: dsa.dsa_debug_copy_only(prob, diag, out, lse, ws))
    t_real = timed(lambda: dsa.dsa_decode_attention_sparse(prob, diag, out, lse, ws))
    assert t_copy < 1.25 * t_real, "copy-only %.3f ms against %.3f ms with the arithmetic" % (t_copy, t_real)
    ref = util.oracle_run(inp, ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride=w.stride, requests=[0, 7, 31])
    util.assert_close(out[[0, 7, 31]], lse[[0, 7, 31]], ref, what="after the copy-only form")
    small = dsa.problem_from_host(synth.make_inputs(synth.workload(5, batch=2)))
    with pytest.raises(dsa.DsaError):
        dsa.dsa_debug_copy_only(small, diag, *dsa.alloc_outputs(small))

