"""The multi-head forms of the tensor-core kernel: blocks of W warps, every warp streaming U kv heads
back to back through one ring.  With a mask that does not depend on the head the block builds ONE
row list for all of them (head-group kernel); with per-head list masks and the fused selection it
builds the tables the heads share and every head derives its own list of kept window candidates
(per-head-list kernel, 4 warps per block).

The planner chooses W, U and the ring depth by itself; here several (W, U) shapes are forced onto
the cases of the other GPU test modules -- the five configurations, the small shapes with and
without splits, degenerate requests, poisoned skipped rows, the fused decode step and its loops,
the phase-2 selection, bounded ring caches, the randomised problems -- so that what those modules
pin to the oracle is pinned for every shape of these kernels.  (Calls they cannot serve -- float32,
head counts that W x U does not divide -- run on the other kernels as before.)"""
import pytest
import torch

from paper_2609_19702_b200 import synth
from tests import test_gpu_decode_step as t_step
from tests import test_gpu_fuzz as t_fuzz
from tests import test_gpu_parity as t_parity
from tests import test_gpu_ring_append as t_ring
from tests import test_gpu_selection as t_sel

pytestmark = pytest.mark.gpu

# (warps per block, kv heads per warp, form: "" cp.async by the computing warps, "tma" tensor-map gather
# copies, "ws" producer warps)
SHAPES = [(2, 1, ""), (4, 1, ""), (2, 2, ""), (4, 2, ""), (2, 4, ""), (4, 1, "tma"), (4, 2, "tma"), (4, 1, "ws"),
          (4, 2, "ws")]


@pytest.fixture(scope="module")
def dsa():
    from paper_2609_19702_b200 import binding
    return binding


@pytest.fixture(params=SHAPES, ids=["w%du%d%s" % s for s in SHAPES])
def forced(request, dsa, monkeypatch):
    """Every problem handed to the library carries the head-group switch."""
    w, u, form = request.param
    flags = dsa.plan_group(w, u) | (dsa.DSA_PLAN_GATHER if form == "tma" else dsa.DSA_PLAN_NO_GATHER) | \
        (dsa.DSA_PLAN_PRODUCERS if form == "ws" else dsa.DSA_PLAN_NO_PRODUCERS)
    orig = dsa.Problem.c_struct

    def patched(self):
        p = orig(self)
        p.plan_flags |= flags
        return p

    monkeypatch.setattr(dsa.Problem, "c_struct", patched)
    return request.param


def test_the_switch_really_selects_the_head_group_kernel(dsa, forced):
    w_, u_, form_ = forced
    for w in (synth.workload(5, batch=2), synth.workload(4, batch=2), synth.workload(2, batch=4)):
        inp = synth.make_inputs(w)
        prob = dsa.problem_from_host(inp)
        trace = synth.random_valid_trace(__import__("numpy").random.default_rng(0), w.window, w.n_att, (w.batch, 1))
        for diag in (None, dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra),
                     dsa.Diag(dsa.DSA_MASK_WINDOW, w.window),
                     dsa.Diag(dsa.DSA_MASK_LIST, w.window, w.n_att, skip_offsets=torch.from_numpy(trace).cuda())):
            plan = dsa.dsa_query_plan(prob, diag)
            if w.num_kv_heads % (w_ * u_) == 0:
                assert plan.heads_per_block == w_ * u_ and plan.block_warps == w_ and plan.tensor_cores == 1
                assert plan.grid_blocks * w_ * u_ == plan.work_items and plan.item_warps == 1
                # (all three workloads keep tokens outermost, so the caches have the 2-D view)
                assert plan.tensor_map_copies == (1 if form_ == "tma" else 0)
                assert plan.producer_warps == (4 if form_ == "ws" else 0)
            else:
                assert plan.heads_per_block == 0
        # one mask per query head, with and without the fused selection: the per-head-list kernel (4 warps)
        per_head = synth.random_valid_trace(__import__("numpy").random.default_rng(0), w.window, w.n_att,
                                            (w.batch, w.num_q_heads))
        for select in (False, True):
            diag = dsa.Diag(dsa.DSA_MASK_LIST, w.window, w.n_att, skip_offsets=torch.from_numpy(per_head).cuda(),
                            select=select)
            plan = dsa.dsa_query_plan(prob, diag)
            if w_ == 4 and w.num_kv_heads % (4 * u_) == 0 and w.index != 4:
                assert plan.per_head_lists == 1 and plan.heads_per_block == 4 * u_ and plan.block_warps == 4
            elif w.index != 4:
                assert plan.per_head_lists == 0
            # (window 1024 with four masks per kv head: the per-head tables leave no room for two blocks
            # per SM, so that configuration stays with the one-warp-per-item kernel)
    # float32 has no tensor-core path: the switch is ignored
    w = synth.workload(1)
    prob = dsa.problem_from_host(synth.make_inputs(w), dtype=torch.float32)
    assert dsa.dsa_query_plan(prob, None).heads_per_block == 0


def test_no_wait_ever_gave_up(dsa):
    """The tensor-map kernel bounds its mbarrier waits and counts the ones that ran out."""
    torch.cuda.synchronize()
    assert dsa.dsa_wait_timeouts() == 0


def test_five_configurations(dsa, forced):
    t_parity.test_config1_every_position(dsa)
    for index in (2, 3, 4):
        t_parity.test_configs_2_3_4(dsa, index)
    for batch in (1, 8):
        t_parity.test_config5_paged_small_batches(dsa, batch)


@pytest.mark.parametrize("case", range(len(t_parity.SMALL)))
def test_small_shapes_all_masks_and_splits(dsa, forced, case):
    t_parity.test_small_shapes_all_masks_and_splits(dsa, case, False)


def test_splits_degenerate_requests_and_poisoned_rows(dsa, forced):
    t_parity.test_split_counts_agree(dsa)
    t_parity.test_degenerate_requests(dsa)
    t_parity.test_skipped_rows_are_never_read(dsa)


@pytest.mark.parametrize("mask", ["dense", "grid_sink", "window", "list_heads", "list_select"])
@pytest.mark.parametrize("name", sorted(t_step.WORKLOADS))
def test_fused_decode_step(dsa, forced, name, mask):
    for split in (0, 48):
        t_step.test_fused_step_matches_oracle_and_the_two_calls(dsa, name, mask, split)


def test_fused_decode_step_full_request_and_loops(dsa, forced):
    t_step.test_a_full_request_drops_its_token(dsa)
    for use_graph in (False, True):
        t_step.test_fused_decode_loop_two_layers_one_seq_len(dsa, use_graph)


def test_phase2_selection(dsa, forced):
    params = [mk.args[1] for mk in t_sel.test_every_step_of_one_sequence.pytestmark if mk.name == "parametrize"][0]
    for hq, hkv, d, split, n_sink, positional in params:
        t_sel.test_every_step_of_one_sequence(dsa, hq, hkv, d, split, n_sink, positional)
    t_sel.test_free_running_decode_loop_grows_a_valid_trace(dsa)


def test_bounded_ring_caches(dsa, forced):
    for hq, hkv, d in ((8, 8, 64), (8, 2, 128)):
        t_ring.test_attention_over_a_bounded_cache_equals_the_full_cache(dsa, hq, hkv, d)
    for use_graph in (False, True):
        t_ring.test_decode_loop_with_append_into_a_ring(dsa, use_graph)
    t_ring.test_append_into_a_paged_linear_cache(dsa)
    t_ring.test_prompt_length_above_its_bound_stays_inside_the_request_region(dsa)


@pytest.mark.parametrize("seed", list(range(12)) + list(range(1000, 1006)))
def test_random_problems(forced, seed):
    t_fuzz.test_random_problem(seed)


@pytest.mark.parametrize("seed", list(range(8)) + list(range(2000, 2004)))
def test_random_fused_decode_steps(forced, seed):
    t_fuzz.test_random_fused_decode_step(seed)


def test_long_sequence_many_splits(forced):
    t_fuzz.test_long_single_sequence_many_splits()
