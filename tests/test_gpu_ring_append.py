"""Bounded (ring) KV cache with eviction, and the K/V append that fills it.

The oracle always works on the full linear cache -- Algorithm 1 never attends an evicted key, so
attention over the bounded cache must give exactly what the oracle gives on the full one.  The
ring layout used to build test caches is re-stated here from the header's description, not
taken from the library."""
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


def _phys(l_p, ring_sinks, ring, s):
    first = l_p + ring_sinks
    return s if s < first else first + (s - first) % ring


def _ring_cache(inp, ring, ring_sinks):
    """Contiguous bounded cache [B, cap, H_kv, D] holding, for every request, what a decode loop
    would have left there at its position; never-written slots are NaN."""
    w = inp["workload"]
    hkv, d = w.num_kv_heads, w.head_dim
    cap = w.prompt_len + ring_sinks + ring
    s_max = inp["max_seq_len"]
    out = []
    for name in ("k_cache", "v_cache"):
        src = inp[name].reshape(w.batch, s_max, hkv, d)
        dst = np.full((w.batch, cap, hkv, d), synth.BF16_NAN, dtype=np.uint16)
        for b in range(w.batch):
            l_p = int(inp["prompt_len"][b])
            for s in range(int(inp["seq_len"][b])):
                dst[b, _phys(l_p, ring_sinks, ring, s)] = src[b, s]
        out.append(dst)
    return out[0], out[1], cap


@pytest.mark.parametrize("hq,hkv,d", [(8, 8, 64), (8, 2, 128)])
def test_attention_over_a_bounded_cache_equals_the_full_cache(dsa, hq, hkv, d):
    ring, ring_sinks = 40, 4
    w = synth.Workload("ring", 71, 9, hq, hkv, d, 11, 12, 9, 1, 40, 9, 1, 120)
    inp = synth.make_inputs(w)
    kc, vc, cap = _ring_cache(inp, ring, ring_sinks)
    row = hkv * d

    def dev(bits):
        return torch.from_numpy(bits.reshape(-1)).view(torch.bfloat16).cuda()

    prob = dsa.Problem(q=dev(inp["q"]).view(w.batch, hq, d), k_cache=dev(kc), v_cache=dev(vc),
                       strides=(cap * row, row, d), seq_len=torch.from_numpy(inp["seq_len"]).cuda(),
                       prompt_len=torch.from_numpy(inp["prompt_len"]).cuda(), num_kv_heads=hkv,
                       max_seq_len=inp["max_seq_len"], max_prompt_len=w.prompt_len,
                       ring_size=ring, ring_sinks=ring_sinks)
    rng = np.random.default_rng(3)
    trace = synth.random_valid_trace(rng, w.window, w.n_att, (w.batch, hq))
    cases = [
        (dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra),
         dict(mode=ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride=w.stride)),
        (dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra, n_sink=4),
         dict(mode=ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride=w.stride, n_sink=4)),
        (dsa.Diag(dsa.DSA_MASK_WINDOW, 25, n_sink=3), dict(mode=ora.MODE_WINDOW, n_r=25, n_sink=3)),
        (dsa.Diag(dsa.DSA_MASK_LIST, w.window, w.n_att, skip_offsets=torch.from_numpy(trace).cuda()),
         dict(mode=ora.MODE_LIST, n_r=w.window, n_att=w.n_att, trace=trace)),
    ]
    for split in (0, 16):
        prob.split_tokens = split
        for diag, kw in cases:
            mode = kw.pop("mode") if "mode" in kw else None
            ref = util.oracle_run(inp, mode, **kw)
            kw["mode"] = mode
            out, lse = dsa.alloc_outputs(prob)
            dsa.dsa_decode_attention_sparse(prob, diag, out, lse, dsa.alloc_workspace(prob, diag))
            torch.cuda.synchronize()
            util.assert_close(out, lse, ref, what="ring cache mode %d split %d" % (mode, split))
    # what cannot work on a bounded cache is refused
    out, lse = dsa.alloc_outputs(prob)
    with pytest.raises(dsa.DsaError):
        dsa.dsa_decode_attention_dense(prob, out, lse)
    with pytest.raises(dsa.DsaError):
        dsa.dsa_decode_attention_sparse(prob, dsa.Diag(dsa.DSA_MASK_WINDOW, ring + 1), out, lse)
    with pytest.raises(dsa.DsaError):
        dsa.dsa_decode_attention_sparse(prob, dsa.Diag(dsa.DSA_MASK_WINDOW, 8, n_sink=5), out, lse)
    torch.cuda.synchronize()


def _decode_loop(dsa, w, inp, prob_of, steps, use_graph):
    """Run `steps` decode steps of a batch whose request i decodes one shared trajectory... no:
    every request decodes its own sequence; step t appends token t and attends at p = t + 1."""
    hq, hkv, d = w.num_q_heads, w.num_kv_heads, w.head_dim
    s_max = inp["max_seq_len"]
    k_lin = torch.from_numpy(inp["k_cache"].reshape(w.batch, s_max, hkv, d)).view(torch.bfloat16).cuda()
    v_lin = torch.from_numpy(inp["v_cache"].reshape(w.batch, s_max, hkv, d)).view(torch.bfloat16).cuda()
    q_steps = torch.from_numpy(inp["q_steps"]).view(torch.bfloat16).cuda()       # [steps, B, hq, d]
    prob, diag = prob_of(k_lin, v_lin)
    k_new = torch.empty((w.batch, hkv, d), dtype=torch.bfloat16, device="cuda")
    v_new = torch.empty_like(k_new)
    out, lse = dsa.alloc_outputs(prob)
    ws = dsa.alloc_workspace(prob, diag)
    outs, lses = [], []

    def one_step():
        dsa.dsa_append_kv(prob, k_new, v_new, advance=True)
        dsa.dsa_decode_attention_sparse(prob, diag, out, lse, ws)

    graph = None
    for t in range(steps):
        prob.q.copy_(q_steps[t])
        k_new.copy_(k_lin[:, w.prompt_len + t])
        v_new.copy_(v_lin[:, w.prompt_len + t])
        if use_graph and t == 1:
            # the first step ran eagerly (it also does the library's one-time kernel set-up);
            # capture the second one and replay it from then on
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                one_step()
            graph.replay()
        elif graph is not None:
            graph.replay()
        else:
            one_step()
        outs.append(out.clone())
        lses.append(lse.clone())
    torch.cuda.synchronize()
    return torch.stack(outs), torch.stack(lses), prob


@pytest.mark.parametrize("use_graph", [False, True])
def test_decode_loop_with_append_into_a_ring(dsa, use_graph):
    ring, ring_sinks, steps = 24, 2, 70
    w = synth.Workload("loop", 72, 5, 8, 4, 64, 9, 10, 7, 0, 24, 7, steps, steps)
    inp = synth.make_inputs(w, poison=False)
    rng = np.random.default_rng(5)
    hq, hkv, d = w.num_q_heads, w.num_kv_heads, w.head_dim
    inp["q_steps"] = synth.f32_to_bf16_bits(rng.standard_normal((steps, w.batch, hq, d), dtype=np.float32))
    row = hkv * d
    cap = w.prompt_len + ring_sinks + ring

    def prob_of(k_lin, v_lin):
        kc = torch.full((w.batch, cap, hkv, d), float("nan"), dtype=torch.bfloat16, device="cuda")
        vc = torch.full_like(kc, float("nan"))
        kc[:, :w.prompt_len] = k_lin[:, :w.prompt_len]          # the prefill left the prompt there
        vc[:, :w.prompt_len] = v_lin[:, :w.prompt_len]
        prob = dsa.Problem(q=torch.empty((w.batch, hq, d), dtype=torch.bfloat16, device="cuda"),
                           k_cache=kc.view(-1), v_cache=vc.view(-1), strides=(cap * row, row, d),
                           seq_len=torch.full((w.batch,), w.prompt_len, dtype=torch.int32, device="cuda"),
                           prompt_len=torch.full((w.batch,), w.prompt_len, dtype=torch.int32, device="cuda"),
                           num_kv_heads=hkv, max_seq_len=inp["max_seq_len"], max_prompt_len=w.prompt_len,
                           ring_size=ring, ring_sinks=ring_sinks)
        diag = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra, n_sink=ring_sinks)
        return prob, diag

    outs, lses, prob = _decode_loop(dsa, w, inp, prob_of, steps, use_graph)
    assert prob.seq_len.cpu().tolist() == [w.prompt_len + steps] * w.batch
    # the oracle, step by step, on the full linear cache
    for t in range(steps):
        step_inp = dict(inp, q=inp["q_steps"][t],
                        seq_len=np.full(w.batch, w.prompt_len + t + 1, dtype=np.int32))
        ref = util.oracle_run(step_inp, ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride=w.stride,
                              n_sink=ring_sinks)
        util.assert_close(outs[t], lses[t], ref, what="loop step %d" % t)
    # final cache contents, bit for bit: prompt, sinks, and the last `ring` tokens in their slots
    kc = prob.k_cache.view(w.batch, cap, hkv, d).view(torch.int16).cpu().numpy().view(np.uint16)
    src = inp["k_cache"].reshape(w.batch, -1, hkv, d)
    for s in range(w.prompt_len + steps - ring, w.prompt_len + steps):
        assert np.array_equal(kc[:, _phys(w.prompt_len, ring_sinks, ring, s)], src[:, s])
    for s in range(w.prompt_len + ring_sinks):
        assert np.array_equal(kc[:, s], src[:, s])


def test_append_into_a_paged_linear_cache(dsa):
    w = synth.Workload("app", 73, 4, 4, 2, 128, 6, 5, 5, 0, 8, 3, 1, 10, paged=True, block_size=4)
    inp = synth.make_inputs(w, poison=False)
    prob = dsa.problem_from_host(inp)
    before_k = prob.k_cache.clone()
    rng = np.random.default_rng(9)
    k_new = torch.from_numpy(synth.f32_to_bf16_bits(rng.standard_normal((4, 2, 128), dtype=np.float32))) \
        .view(torch.bfloat16).cuda()
    v_new = torch.from_numpy(synth.f32_to_bf16_bits(rng.standard_normal((4, 2, 128), dtype=np.float32))) \
        .view(torch.bfloat16).cuda()
    prob.seq_len[3] = inp["max_seq_len"]                 # a full request: must be left alone
    seq = prob.seq_len.cpu().numpy().copy()
    dsa.dsa_append_kv(prob, k_new, v_new, advance=True)
    torch.cuda.synchronize()
    assert prob.seq_len.cpu().tolist() == [seq[0] + 1, seq[1] + 1, seq[2] + 1, seq[3]]
    kc = prob.k_cache.view(-1, 4, 2, 128)
    vc = prob.v_cache.view(-1, 4, 2, 128)
    expect = before_k.view(-1, 4, 2, 128).clone()
    for b in range(3):
        blk = int(inp["block_table"][b, seq[b] // 4])
        expect[blk, seq[b] % 4] = k_new[b]
        assert torch.equal(vc[blk, seq[b] % 4].view(torch.int16), v_new[b].view(torch.int16))
    assert torch.equal(kc.view(torch.int16), expect.view(torch.int16))


def test_host_io_call_matches_device_call(dsa):
    w = synth.workload(5, batch=3)
    inp = synth.make_inputs(w)
    prob = dsa.problem_from_host(inp)
    diag = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
    for dg in (None, diag):
        ref_out, ref_lse = dsa.alloc_outputs(prob)
        ws = dsa.alloc_workspace(prob, dg)
        if dg is None:
            dsa.dsa_decode_attention_dense(prob, ref_out, ref_lse, ws)
        else:
            dsa.dsa_decode_attention_sparse(prob, dg, ref_out, ref_lse, ws)
        torch.cuda.synchronize()
        h_q = prob.q.cpu().pin_memory()
        h_seq, h_pl = prob.seq_len.cpu().pin_memory(), prob.prompt_len.cpu().pin_memory()
        h_bt = prob.block_table.cpu().pin_memory()
        # scramble the device copies: the call must restore them from the host buffers
        prob.q.zero_()
        prob.seq_len.zero_()
        prob.block_table.zero_()
        out, lse = dsa.alloc_outputs(prob)
        h_out = torch.empty(out.shape, dtype=out.dtype).pin_memory()
        h_lse = torch.empty(lse.shape, dtype=lse.dtype).pin_memory()
        dsa.dsa_decode_attention_host_io(prob, dg, h_q, h_seq, h_pl, h_bt, out, lse, h_out, h_lse, ws)
        torch.cuda.synchronize()
        assert torch.equal(h_out.view(torch.int16), ref_out.cpu().view(torch.int16))
        assert torch.equal(h_lse, ref_lse.cpu())


def test_prompt_length_above_its_bound_stays_inside_the_request_region(dsa):
    """A device prompt_len[b] above max_prompt_len is read as max_prompt_len when the cache is a
    ring: append, fused step and attention then touch only the request's own
    max_prompt_len + ring_sinks + ring_size tokens (wrong numbers for that request, but no row
    of a neighbour or beyond the allocation)."""
    b, h, d, l_p, ring, sinks = 4, 4, 64, 5, 16, 2
    cap = l_p + sinks + ring
    row = h * d
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5)
    # one spare region behind the last request as a guard
    kc = torch.randn(((b + 1) * cap, h, d), generator=gen, device="cuda").to(torch.bfloat16)
    vc = torch.randn(((b + 1) * cap, h, d), generator=gen, device="cuda").to(torch.bfloat16)
    q = torch.randn((b, h, d), generator=gen, device="cuda").to(torch.bfloat16)
    k_new, v_new = q.clone() + 1, q.clone() - 1
    seq = torch.tensor([60, 70, 23, 40], dtype=torch.int32, device="cuda")
    bad_prompt = torch.tensor([5, 12, 5, 23], dtype=torch.int32, device="cuda")     # two of them above the bound of 5
    prob = dsa.Problem(q=q, k_cache=kc.view(-1), v_cache=vc.view(-1), strides=(cap * row, row, d), seq_len=seq,
                       prompt_len=bad_prompt, num_kv_heads=h, max_seq_len=100, max_prompt_len=l_p,
                       ring_size=ring, ring_sinks=sinks)
    diag = dsa.Diag(dsa.DSA_MASK_GRID, ring, 6, 5, 0, n_sink=sinks)
    out, lse = dsa.alloc_outputs(prob)
    ws = dsa.alloc_workspace(prob, diag)

    def changed_rows(before_k, before_v):
        ck = (kc.view(torch.int16) != before_k).any(dim=2).any(dim=1)
        cv = (vc.view(torch.int16) != before_v).any(dim=2).any(dim=1)
        assert torch.equal(ck, cv)
        return torch.nonzero(ck).flatten().tolist()

    for fused in (False, True):
        bk, bv = kc.view(torch.int16).clone(), vc.view(torch.int16).clone()
        if fused:
            dsa.dsa_decode_step(prob, diag, k_new, v_new, out, lse, ws)
        else:
            dsa.dsa_append_kv(prob, k_new, v_new, advance=False)
            dsa.dsa_decode_attention_sparse(prob, diag, out, lse, ws)
        torch.cuda.synchronize()
        rows = changed_rows(bk, bv)
        assert len(rows) == b and [r // cap for r in rows] == list(range(b)), rows   # one row per request, in its own region
        assert torch.isfinite(out.float()).all()
        k_new, v_new = k_new + 1, v_new + 1
