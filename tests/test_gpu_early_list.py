"""DSA_PLAN_METADATA_STABLE: the caller's promise that the launch before a call does not write the
lengths, the block table or the skip lists, which lets the head-group, per-head-list, several-warps-
per-item and cluster kernels work out their rows BEFORE they wait for that launch.

Two things are checked.  (1) The early-list kernels compute the same as the others: the cases of the
other parity modules run with the promise set on every problem (and, so that it is kept whatever a
case does between its calls, with the device idle before each call).  (2) The overlap itself: token
loops as a model runs them -- every layer's fused step back to back, only the first layer of a token
follows the launch that advances the lengths and goes without the promise -- replayed as a CUDA
graph and compared with the oracle step by step.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as ora
from paper_2609_19702_b200 import synth
from tests import test_gpu_decode_step as t_step
from tests import test_gpu_parity as t_parity
from tests import test_gpu_selection as t_sel
from tests import util

pytestmark = pytest.mark.gpu

ENTRY_POINTS = ["dsa_decode_attention_dense", "dsa_decode_attention_sparse", "dsa_decode_step",
                "dsa_decode_attention_static_scratch"]


@pytest.fixture(scope="module")
def dsa():
    from paper_2609_19702_b200 import binding
    return binding


@pytest.fixture(params=[1, 2, 0], ids=["u1", "u2", "planned"])
def promised(request, dsa, monkeypatch):
    """Every problem carries the promise, with the four-warp multi-head kernels forced (1 or 2 heads per
    warp) or with the library's own plan (the small cases then take the several-warps-per-item and
    cluster kernels, which honour it as well); the device is idle when a call is made."""
    flags = dsa.DSA_PLAN_METADATA_STABLE | (dsa.plan_group(4, request.param) if request.param else 0)
    orig = dsa.Problem.c_struct

    def patched(self):
        p = orig(self)
        p.plan_flags |= flags
        return p

    monkeypatch.setattr(dsa.Problem, "c_struct", patched)
    for name in ENTRY_POINTS:
        fn = getattr(dsa, name)

        def idle_first(*args, _fn=fn, **kw):
            torch.cuda.synchronize()
            return _fn(*args, **kw)

        monkeypatch.setattr(dsa, name, idle_first)
    return request.param


def test_five_configurations(dsa, promised):
    t_parity.test_config1_every_position(dsa)
    for index in (2, 3, 4):
        t_parity.test_configs_2_3_4(dsa, index)
    for batch in (1, 8):
        t_parity.test_config5_paged_small_batches(dsa, batch)


def test_splits_degenerate_requests_and_poisoned_rows(dsa, promised):
    t_parity.test_split_counts_agree(dsa)
    t_parity.test_degenerate_requests(dsa)
    t_parity.test_skipped_rows_are_never_read(dsa)


@pytest.mark.parametrize("mask", ["dense", "grid_sink", "window", "list_heads", "list_select"])
@pytest.mark.parametrize("name", ["gqa_long", "paged", "mha_d64"])
def test_fused_decode_step(dsa, promised, name, mask):
    t_step.test_fused_step_matches_oracle_and_the_two_calls(dsa, name, mask, 0)


def test_phase2_selection(dsa, promised):
    params = [mk.args[1] for mk in t_sel.test_every_step_of_one_sequence.pytestmark if mk.name == "parametrize"][0]
    for hq, hkv, d, split, n_sink, positional in params:
        t_sel.test_every_step_of_one_sequence(dsa, hq, hkv, d, split, n_sink, positional)


@pytest.mark.parametrize("use_graph", [False, True])
def test_token_loop_of_three_layers_with_the_promise_on_all_but_the_first(dsa, use_graph):
    """Layer 0 (follows the launch that advances seq_len: no promise): ring cache, grid mask.  Layer 1:
    ring cache, grid mask with sinks, promise.  Layer 2: linear cache, per-head lists grown by the fused
    selection, promise.  Back to back, so the lists of layers 1 and 2 are built while the layer before
    still runs."""
    ring, ring_sinks, steps = 24, 2, 60
    w = synth.Workload("loop", 85, 6, 8, 4, 64, 9, 10, 6, 0, 24, 7, steps, steps)
    inp = synth.make_inputs(w, poison=False)
    rng = np.random.default_rng(8)
    hq, hkv, d, l_p, b = w.num_q_heads, w.num_kv_heads, w.head_dim, w.prompt_len, w.batch
    q_bits = synth.f32_to_bf16_bits(rng.standard_normal((steps, b, hq, d), dtype=np.float32))
    s_max = inp["max_seq_len"]
    k_lin = torch.from_numpy(inp["k_cache"].reshape(b, s_max, hkv, d)).view(torch.bfloat16).cuda()
    v_lin = torch.from_numpy(inp["v_cache"].reshape(b, s_max, hkv, d)).view(torch.bfloat16).cuda()
    q_steps = torch.from_numpy(q_bits).view(torch.bfloat16).cuda()
    row = hkv * d
    seq = torch.full((b,), l_p, dtype=torch.int32, device="cuda")
    pl = torch.full((b,), l_p, dtype=torch.int32, device="cuda")
    q = torch.empty((b, hq, d), dtype=torch.bfloat16, device="cuda")
    k_new = torch.empty((b, hkv, d), dtype=torch.bfloat16, device="cuda")
    v_new = torch.empty_like(k_new)
    promise = dsa.plan_group(4, 1) | dsa.DSA_PLAN_METADATA_STABLE

    def cache(tokens):
        kc = torch.full((b, tokens, hkv, d), float("nan"), dtype=torch.bfloat16, device="cuda")
        vc = torch.full_like(kc, float("nan"))
        kc[:, :l_p], vc[:, :l_p] = k_lin[:, :l_p], v_lin[:, :l_p]
        return kc, vc

    layers = []
    for index, sinks in ((0, 0), (1, ring_sinks), (2, None)):
        bounded = sinks is not None
        cap = l_p + sinks + ring if bounded else s_max
        kc, vc = cache(cap)
        prob = dsa.Problem(q=q, k_cache=kc.view(-1), v_cache=vc.view(-1), strides=(cap * row, row, d), seq_len=seq,
                           prompt_len=pl, num_kv_heads=hkv, max_seq_len=s_max, max_prompt_len=l_p,
                           ring_size=ring if bounded else 0, ring_sinks=sinks if bounded else 0,
                           plan_flags=dsa.plan_group(4, 1) if index == 0 else promise)
        trace = None
        if bounded:
            diag = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra, n_sink=sinks)
        else:
            trace = torch.zeros((b, hq, w.window - w.n_att), dtype=torch.int32, device="cuda")
            diag = dsa.Diag(dsa.DSA_MASK_LIST, w.window, w.n_att, skip_offsets=trace, select=True)
        plan = dsa.dsa_query_plan(prob, diag)
        assert plan.block_warps == 4 and plan.per_head_lists == (0 if bounded else 1)
        out, lse = dsa.alloc_outputs(prob)
        layers.append((prob, diag, out, lse, dsa.alloc_workspace(prob, diag), sinks, (kc, vc), trace))

    def token_step():
        for prob, diag, out, lse, ws, _, _, _ in layers:
            dsa.dsa_decode_step(prob, diag, k_new, v_new, out, lse, ws)
        dsa.dsa_advance_seq_len(seq, s_max)

    graph, got = None, []
    for t in range(steps):
        q.copy_(q_steps[t])
        k_new.copy_(k_lin[:, l_p + t])
        v_new.copy_(v_lin[:, l_p + t])
        if use_graph and t == 1:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                token_step()
            graph.replay()
        elif graph is not None:
            graph.replay()
        else:
            token_step()
        got.append([(out.clone(), lse.clone()) for _, _, out, lse, _, _, _, _ in layers])
    torch.cuda.synchronize()
    assert seq.cpu().tolist() == [l_p + steps] * b
    assert dsa.dsa_wait_timeouts() == 0
    final_trace = layers[2][7].cpu().numpy()
    for t in range(steps):
        step_inp = dict(inp, q=q_bits[t], seq_len=np.full(b, l_p + t + 1, dtype=np.int32))
        for index in (0, 1):
            ref = util.oracle_run(step_inp, ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride=w.stride,
                                  n_sink=layers[index][5])
            util.assert_close(got[t][index][0], got[t][index][1], ref, what="layer %d, step %d" % (index, t))
        ref = util.oracle_run(step_inp, ora.MODE_LIST, n_r=w.window, n_att=w.n_att, trace=final_trace)
        util.assert_close(got[t][2][0], got[t][2][1], ref, what="selecting layer, step %d" % t)
    # the linear cache holds every token bit for bit
    kc2, vc2 = layers[2][6]
    for got_c, want_c, what in ((kc2, k_lin, "K"), (vc2, v_lin, "V")):
        diff = (t_step._bits(got_c) != t_step._bits(want_c)).reshape(b, s_max, hkv, d).any(dim=3).nonzero().cpu().tolist()
        assert not diff, "%s cache differs at (request, position, head) %s ..." % (what, diff[:8])
