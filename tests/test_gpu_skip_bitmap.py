"""dsa_diag_params.skip_bitmap: the skip lists as bits, for the per-head-list kernel.

(1) Reading: the other modules' list-mask cases run with a bitmap that dsa_build_skip_bitmap makes from
the list right before every call, on the per-head-list kernel; results must still match the oracle, which
knows only the lists.  (2) Keeping it in step: a token loop with the fused selection starts from an empty
list and an empty bitmap and lets the library grow both; every step is compared with the oracle, and at
the end the bitmap must be exactly what dsa_build_skip_bitmap makes of the final list.
"""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import oracle as ora
from paper_2609_19702_b200 import synth
from tests import test_gpu_parity as t_parity
from tests import test_gpu_selection as t_sel
from tests import util

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dsa():
    from paper_2609_19702_b200 import binding
    return binding


def _words(window):
    return (window + 31) // 32


@pytest.fixture(params=[1, 2], ids=["u1", "u2"])
def bitmapped(request, dsa, monkeypatch):
    """Every list-mask call gets the bitmap form of its lists, freshly built, and the four-warp
    multi-head kernels."""
    flags = dsa.plan_group(4, request.param)
    orig = dsa.Problem.c_struct

    def patched(self):
        p = orig(self)
        p.plan_flags |= flags
        return p

    monkeypatch.setattr(dsa.Problem, "c_struct", patched)
    build = dsa.dsa_build_skip_bitmap

    def with_bitmap(prob, diag):
        if diag is None or diag.mode != dsa.DSA_MASK_LIST or diag.skip_offsets is None or diag.skip_bitmap is not None:
            return diag
        t = diag.skip_offsets
        bm = torch.full((t.shape[0], t.shape[1], _words(diag.window)), -1, dtype=torch.int32, device=t.device)
        diag = dataclasses.replace(diag, skip_bitmap=bm)
        build(prob, diag)
        return diag

    sparse = dsa.dsa_decode_attention_sparse
    monkeypatch.setattr(dsa, "dsa_decode_attention_sparse",
                        lambda prob, diag, *a, **k: sparse(prob, with_bitmap(prob, diag), *a, **k))
    scratch = dsa.dsa_decode_attention_static_scratch
    monkeypatch.setattr(dsa, "dsa_decode_attention_static_scratch",
                        lambda prob, diag, *a, **k: scratch(prob, with_bitmap(prob, diag), *a, **k))
    return request.param


def test_list_masks_of_the_five_configurations(dsa, bitmapped):
    t_parity.test_config1_every_position(dsa)
    for index in (2, 3, 4):
        t_parity.test_configs_2_3_4(dsa, index)
    for batch in (1, 8):
        t_parity.test_config5_paged_small_batches(dsa, batch)


def test_phase2_selection_reads_the_bitmap(dsa, bitmapped):
    params = [mk.args[1] for mk in t_sel.test_every_step_of_one_sequence.pytestmark if mk.name == "parametrize"][0]
    for hq, hkv, d, split, n_sink, positional in params:
        t_sel.test_every_step_of_one_sequence(dsa, hq, hkv, d, split, n_sink, positional)


def test_the_bitmap_really_is_what_the_kernel_reads(dsa):
    """With a bitmap made from ANOTHER valid list, the per-head-list kernel follows the bitmap."""
    w = synth.workload(2, batch=12)
    inp = synth.make_inputs(w)
    prob = dsa.problem_from_host(inp, plan_flags=dsa.plan_group(4, 1))
    trace = synth.random_valid_trace(np.random.default_rng(3), w.window, w.n_att, (w.batch, w.num_q_heads))
    other = synth.random_valid_trace(np.random.default_rng(4), w.window, w.n_att, (w.batch, w.num_q_heads))
    assert not np.array_equal(trace, other)
    tr = torch.from_numpy(trace.copy()).cuda()
    bm = torch.zeros((w.batch, w.num_q_heads, _words(w.window)), dtype=torch.int32, device="cuda")
    diag = dsa.Diag(dsa.DSA_MASK_LIST, w.window, w.n_att, skip_offsets=tr, skip_bitmap=bm)
    assert dsa.dsa_query_plan(prob, diag).per_head_lists == 1
    out, lse = dsa.alloc_outputs(prob)
    ws = dsa.alloc_workspace(prob, diag)
    dsa.dsa_build_skip_bitmap(prob, dataclasses.replace(diag, skip_offsets=torch.from_numpy(other.copy()).cuda()))
    dsa.dsa_decode_attention_sparse(prob, diag, out, lse, ws)            # list says `trace`, bitmap says `other`
    torch.cuda.synchronize()
    ref_other = util.oracle_run(inp, ora.MODE_LIST, n_r=w.window, n_att=w.n_att, trace=other)
    util.assert_close(out, lse, ref_other, what="bitmap of another list")
    dsa.dsa_build_skip_bitmap(prob, diag)
    dsa.dsa_decode_attention_sparse(prob, diag, out, lse, ws)
    torch.cuda.synchronize()
    ref = util.oracle_run(inp, ora.MODE_LIST, n_r=w.window, n_att=w.n_att, trace=trace)
    util.assert_close(out, lse, ref, what="bitmap built from the list")
    # the builder: bit o of a row is set iff o is one of the row's first n_act entries
    got = bm.cpu().numpy().view(np.uint32)
    pos = inp["seq_len"] - inp["prompt_len"]
    for b in range(w.batch):
        n_act = int(np.clip(pos[b] - 1 - (w.n_att - 1), 0, w.window - w.n_att))
        for h in range(w.num_q_heads):
            want = np.zeros(_words(w.window), dtype=np.uint32)
            for o in trace[b, h, :n_act]:
                if 0 <= o < w.window:
                    want[o >> 5] |= np.uint32(1) << np.uint32(o & 31)
            assert np.array_equal(got[b, h], want), (b, h)


@pytest.mark.parametrize("split", [0, 16])
def test_selection_keeps_list_and_bitmap_in_step(dsa, split):
    steps = 60
    w = synth.Workload("loop", 86, 5, 8, 4, 64, 9, 10, 6, 0, 24, 7, steps, steps)
    inp = synth.make_inputs(w, poison=False)
    rng = np.random.default_rng(9)
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
    kc = torch.full((b, s_max, hkv, d), float("nan"), dtype=torch.bfloat16, device="cuda")
    vc = torch.full_like(kc, float("nan"))
    kc[:, :l_p], vc[:, :l_p] = k_lin[:, :l_p], v_lin[:, :l_p]
    prob = dsa.Problem(q=q, k_cache=kc.view(-1), v_cache=vc.view(-1), strides=(s_max * row, row, d), seq_len=seq,
                       prompt_len=pl, num_kv_heads=hkv, max_seq_len=s_max, max_prompt_len=l_p, split_tokens=split,
                       plan_flags=dsa.plan_group(4, 1))
    trace = torch.zeros((b, hq, w.window - w.n_att), dtype=torch.int32, device="cuda")
    bm = torch.zeros((b, hq, _words(w.window)), dtype=torch.int32, device="cuda")
    diag = dsa.Diag(dsa.DSA_MASK_LIST, w.window, w.n_att, skip_offsets=trace, select=True, skip_bitmap=bm)
    plan = dsa.dsa_query_plan(prob, diag)
    assert plan.per_head_lists == 1 and (plan.n_split > 1) == (split > 0)
    out, lse = dsa.alloc_outputs(prob)
    ws = dsa.alloc_workspace(prob, diag)
    k_new = torch.empty((b, hkv, d), dtype=torch.bfloat16, device="cuda")
    v_new = torch.empty_like(k_new)
    got = []
    for t in range(steps):
        q.copy_(q_steps[t])
        k_new.copy_(k_lin[:, l_p + t])
        v_new.copy_(v_lin[:, l_p + t])
        dsa.dsa_decode_step(prob, diag, k_new, v_new, out, lse, ws)
        dsa.dsa_advance_seq_len(seq, s_max)
        got.append((out.clone(), lse.clone()))
    torch.cuda.synchronize()
    final_trace = trace.cpu().numpy()
    for t in range(steps):
        step_inp = dict(inp, q=q_bits[t], seq_len=np.full(b, l_p + t + 1, dtype=np.int32))
        ref = util.oracle_run(step_inp, ora.MODE_LIST, n_r=w.window, n_att=w.n_att, trace=final_trace)
        util.assert_close(got[t][0], got[t][1], ref, what="step %d" % t)
    rebuilt = torch.full_like(bm, -1)
    dsa.dsa_build_skip_bitmap(prob, dataclasses.replace(diag, skip_bitmap=rebuilt))
    torch.cuda.synchronize()
    assert torch.equal(bm, rebuilt), "the bitmap the selection kept is not the bitmap of the final list"
    assert int((bm != 0).sum()) > 0
