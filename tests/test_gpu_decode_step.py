"""The fused decode step (append + attention in one call).

The oracle knows nothing about appending: it attends over a cache that already holds the current
token.  So every case starts from such a cache, takes the current token's rows out of it (the
slots are poisoned with NaN), hands them to the step as k_new / v_new with seq_len one lower, and
expects the oracle's result, the result of the two separate calls bit for bit, and the cache
restored bit for bit."""
import numpy as np
import pytest
import torch

from oracle import oracle as ora
from paper_2609_19702_b200 import synth
from tests import util
from tests.test_gpu_ring_append import _phys

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dsa():
    from paper_2609_19702_b200 import binding
    return binding


def _last_row_offsets(inp):
    """Element offset of (request b, kv head 0) of the newest cached token, from the layout rules
    of the header (contiguous [B, S_max, H_kv, D] or token-major paged pool)."""
    sb, st, _ = inp["strides"]
    offs = []
    for b in range(inp["workload"].batch):
        pos = int(inp["seq_len"][b]) - 1
        if inp["block_table"] is not None:
            bs = inp["block_size"]
            offs.append(int(inp["block_table"][b, pos // bs]) * sb + (pos % bs) * st)
        else:
            offs.append(b * sb + pos * st)
    return offs


def _take_out_current_token(prob, inp):
    """k_new, v_new [B, H_kv, D] gathered from the cache; their slots NaN; seq_len one lower."""
    w = inp["workload"]
    sh, d = inp["strides"][2], w.head_dim
    news = []
    for cache in (prob.k_cache, prob.v_cache):
        flat = cache.view(-1)
        new = torch.empty((w.batch, w.num_kv_heads, d), dtype=flat.dtype, device=flat.device)
        for b, off in enumerate(_last_row_offsets(inp)):
            for h in range(w.num_kv_heads):
                new[b, h] = flat[off + h * sh: off + h * sh + d]
                flat[off + h * sh: off + h * sh + d] = float("nan")
        news.append(new)
    prob.seq_len -= 1
    return news[0], news[1]


def _bits(t):
    return t.contiguous().view(torch.int16 if t.element_size() == 2 else torch.int32)


WORKLOADS = {
    "mha_d64": lambda: synth.workload(2, batch=5),
    "gqa_long": lambda: synth.workload(4, batch=2),
    "paged": lambda: synth.workload(5, batch=3),
    "gqa8_paged_small": lambda: synth.Workload("step", 81, 4, 16, 2, 128, 17, 12, 9, 1, 40, 9, 1, 120,
                                               paged=True, block_size=4),
    "odd_heads": lambda: synth.Workload("step", 82, 3, 6, 3, 64, 0, 9, 7, 0, 30, 11, 1, 63),
}


@pytest.mark.parametrize("mask", ["dense", "grid_sink", "window", "list_heads", "list_select"])
@pytest.mark.parametrize("name", sorted(WORKLOADS))
@pytest.mark.parametrize("split", [0, 48])
def test_fused_step_matches_oracle_and_the_two_calls(dsa, name, mask, split):
    w = WORKLOADS[name]()
    inp = synth.make_inputs(w)
    hq = w.num_q_heads
    rng = np.random.default_rng(11)
    trace = synth.random_valid_trace(rng, w.window, w.n_att, (w.batch, hq))

    def diag_of():
        if mask == "dense":
            return None, dict(mode=ora.MODE_DENSE)
        if mask == "grid_sink":
            return (dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra, n_sink=2),
                    dict(mode=ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride=w.stride, n_sink=2))
        if mask == "window":
            return dsa.Diag(dsa.DSA_MASK_WINDOW, w.window), dict(mode=ora.MODE_WINDOW, n_r=w.window)
        t = torch.from_numpy(trace.copy()).cuda()
        return (dsa.Diag(dsa.DSA_MASK_LIST, w.window, w.n_att, skip_offsets=t, select=(mask == "list_select")),
                dict(mode=ora.MODE_LIST, n_r=w.window, n_att=w.n_att, trace=trace))

    _, kw = diag_of()
    ref = util.oracle_run(inp, kw.pop("mode"), **kw)
    results = []
    for fused in (True, False):
        prob = dsa.problem_from_host(inp, split_tokens=split)
        original = (_bits(prob.k_cache).clone(), _bits(prob.v_cache).clone())
        diag, _ = diag_of()
        k_new, v_new = _take_out_current_token(prob, inp)
        out, lse = dsa.alloc_outputs(prob)
        out.fill_(float("nan"))
        ws = dsa.alloc_workspace(prob, diag)
        if fused:
            dsa.dsa_decode_step(prob, diag, k_new, v_new, out, lse, ws)
            dsa.dsa_advance_seq_len(prob.seq_len, inp["max_seq_len"])
        else:
            dsa.dsa_append_kv(prob, k_new, v_new, advance=True)
            if diag is None:
                dsa.dsa_decode_attention_dense(prob, out, lse, ws)
            else:
                dsa.dsa_decode_attention_sparse(prob, diag, out, lse, ws)
        torch.cuda.synchronize()
        what = "%s %s split %d %s" % (name, mask, split, "fused" if fused else "two calls")
        util.assert_close(out, lse, ref, what=what)
        assert torch.equal(_bits(prob.k_cache), original[0]), what + ": K cache not restored"
        assert torch.equal(_bits(prob.v_cache), original[1]), what + ": V cache not restored"
        assert prob.seq_len.cpu().numpy().tolist() == inp["seq_len"].tolist()
        results.append((out, lse, None if diag is None or diag.skip_offsets is None else diag.skip_offsets))
    (o1, l1, t1), (o2, l2, t2) = results
    assert torch.equal(_bits(o1), _bits(o2)) and torch.equal(l1, l2)
    if t1 is not None:
        assert torch.equal(t1, t2), "the fused selection wrote a different trace entry"


def test_fused_step_in_float32_goes_through_the_append_launch(dsa):
    w = WORKLOADS["odd_heads"]()
    inp = synth.make_inputs(w)
    ref = util.oracle_run(inp, ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride=w.stride)
    prob = dsa.problem_from_host(inp, dtype=torch.float32)
    original = _bits(prob.k_cache).clone()
    diag = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
    k_new, v_new = _take_out_current_token(prob, inp)
    out, lse = dsa.alloc_outputs(prob)
    dsa.dsa_decode_step(prob, diag, k_new, v_new, out, lse, dsa.alloc_workspace(prob, diag))
    torch.cuda.synchronize()
    util.assert_close(out, lse, ref, f32=True, what="float32 fused step")
    assert torch.equal(_bits(prob.k_cache), original)


def test_a_full_request_drops_its_token(dsa):
    """seq_len == max_seq_len: nothing is written and attention covers what is cached."""
    w = synth.Workload("full", 83, 2, 4, 4, 64, 5, 6, 5, 0, 16, 5, 30, 30)      # every request at the last position
    inp = synth.make_inputs(w, poison=False)
    assert (inp["seq_len"] == inp["max_seq_len"]).all()
    diag = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
    ref = util.oracle_run(inp, ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride=w.stride)
    prob = dsa.problem_from_host(inp)
    original = _bits(prob.k_cache).clone()
    junk = torch.full((w.batch, w.num_kv_heads, w.head_dim), 3.0, dtype=torch.bfloat16, device="cuda")
    out, lse = dsa.alloc_outputs(prob)
    dsa.dsa_decode_step(prob, diag, junk, junk, out, lse, dsa.alloc_workspace(prob, diag))
    dsa.dsa_advance_seq_len(prob.seq_len, inp["max_seq_len"])
    torch.cuda.synchronize()
    util.assert_close(out, lse, ref, what="full request")
    assert torch.equal(_bits(prob.k_cache), original)
    assert prob.seq_len.cpu().numpy().tolist() == inp["seq_len"].tolist()


@pytest.mark.parametrize("use_graph", [False, True])
def test_fused_decode_loop_two_layers_one_seq_len(dsa, use_graph):
    """A token step = every layer's fused step, then one seq_len advance; layers share seq_len.
    Layer 0: bounded ring cache, grid mask with sinks.  Layer 1: linear cache, per-head list masks
    grown by the fused selection.  Each against the oracle, step by step."""
    ring, ring_sinks, steps = 24, 2, 60
    w = synth.Workload("loop", 84, 4, 8, 4, 64, 9, 10, 6, 0, 24, 7, steps, steps)
    inp = synth.make_inputs(w, poison=False)
    rng = np.random.default_rng(6)
    hq, hkv, d, l_p, b = w.num_q_heads, w.num_kv_heads, w.head_dim, w.prompt_len, w.batch
    q_steps_bits = synth.f32_to_bf16_bits(rng.standard_normal((steps, b, hq, d), dtype=np.float32))
    s_max = inp["max_seq_len"]
    k_lin = torch.from_numpy(inp["k_cache"].reshape(b, s_max, hkv, d)).view(torch.bfloat16).cuda()
    v_lin = torch.from_numpy(inp["v_cache"].reshape(b, s_max, hkv, d)).view(torch.bfloat16).cuda()
    q_steps = torch.from_numpy(q_steps_bits).view(torch.bfloat16).cuda()
    row = hkv * d
    cap = l_p + ring_sinks + ring
    seq = torch.full((b,), l_p, dtype=torch.int32, device="cuda")
    pl = torch.full((b,), l_p, dtype=torch.int32, device="cuda")
    q = torch.empty((b, hq, d), dtype=torch.bfloat16, device="cuda")

    def cache(tokens):
        kc = torch.full((b, tokens, hkv, d), float("nan"), dtype=torch.bfloat16, device="cuda")
        vc = torch.full_like(kc, float("nan"))
        kc[:, :l_p], vc[:, :l_p] = k_lin[:, :l_p], v_lin[:, :l_p]
        return kc, vc

    kc0, vc0 = cache(cap)
    kc1, vc1 = cache(s_max)
    prob0 = dsa.Problem(q=q, k_cache=kc0.view(-1), v_cache=vc0.view(-1), strides=(cap * row, row, d), seq_len=seq,
                        prompt_len=pl, num_kv_heads=hkv, max_seq_len=s_max, max_prompt_len=l_p,
                        ring_size=ring, ring_sinks=ring_sinks)
    prob1 = dsa.Problem(q=q, k_cache=kc1.view(-1), v_cache=vc1.view(-1), strides=(s_max * row, row, d), seq_len=seq,
                        prompt_len=pl, num_kv_heads=hkv, max_seq_len=s_max, max_prompt_len=l_p)
    diag0 = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra, n_sink=ring_sinks)
    trace = torch.zeros((b, hq, w.window - w.n_att), dtype=torch.int32, device="cuda")
    diag1 = dsa.Diag(dsa.DSA_MASK_LIST, w.window, w.n_att, skip_offsets=trace, select=True)
    k_new = torch.empty((b, hkv, d), dtype=torch.bfloat16, device="cuda")
    v_new = torch.empty_like(k_new)
    out0, lse0 = dsa.alloc_outputs(prob0)
    out1, lse1 = dsa.alloc_outputs(prob1)
    ws0, ws1 = dsa.alloc_workspace(prob0, diag0), dsa.alloc_workspace(prob1, diag1)

    def token_step():
        dsa.dsa_decode_step(prob0, diag0, k_new, v_new, out0, lse0, ws0)
        dsa.dsa_decode_step(prob1, diag1, k_new, v_new, out1, lse1, ws1)
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
        got.append((out0.clone(), lse0.clone(), out1.clone(), lse1.clone()))
    torch.cuda.synchronize()
    assert seq.cpu().tolist() == [l_p + steps] * b
    for t in range(steps):
        step_inp = dict(inp, q=q_steps_bits[t], seq_len=np.full(b, l_p + t + 1, dtype=np.int32))
        ref0 = util.oracle_run(step_inp, ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride=w.stride,
                               n_sink=ring_sinks)
        util.assert_close(got[t][0], got[t][1], ref0, what="ring layer, step %d" % t)
    # layer 1: replay the selection with the oracle (Algorithm 1's argmin) and compare step by step
    final_trace = trace.cpu().numpy()
    for t in range(steps):
        step_inp = dict(inp, q=q_steps_bits[t], seq_len=np.full(b, l_p + t + 1, dtype=np.int32))
        ref1 = util.oracle_run(step_inp, ora.MODE_LIST, n_r=w.window, n_att=w.n_att, trace=final_trace)
        util.assert_close(got[t][2], got[t][3], ref1, what="selecting layer, step %d" % t)
    # caches: the linear one holds every token, the ring its last `ring` ones
    assert torch.equal(_bits(kc1), _bits(k_lin)) and torch.equal(_bits(vc1), _bits(v_lin))
    for s in range(l_p + steps - ring, l_p + steps):
        assert torch.equal(_bits(kc0[:, _phys(l_p, ring_sinks, ring, s)]), _bits(k_lin[:, s]))
