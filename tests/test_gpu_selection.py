"""Fused phase-2 selection (Algorithm 1, "select newly skipped KV"): the sparse call with
`select` set appends the next trace entry per query head.  The oracle replays Algorithm 1 with
its argmin literally in float64; the kernel decides on float32 logits, so where the two lowest
logits are closer than float32 can tell apart either key is a valid choice -- the test accepts
a different entry only if the oracle's logits of the two keys differ by less than 1e-4."""
import numpy as np
import pytest
import torch

from oracle import oracle as ora
from paper_2609_19702_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu

SENTINEL = -7


@pytest.fixture(scope="module")
def dsa():
    from paper_2609_19702_b200 import binding
    return binding


def _trajectory(w, inp):
    """Config-1 style batch: request i is decode step t = i of ONE sequence (shared cache).
    Returns float64 views of q [T, H_q, D] and k rows [S, H_kv, D]."""
    q = synth.bf16_bits_to_f32(inp["q"]).astype(np.float64)
    k = synth.bf16_bits_to_f32(inp["k_cache"]).astype(np.float64).reshape(-1, w.num_kv_heads, w.head_dim)
    return q, k


def _oracle_traces(w, inp, n_sink=0):
    """Per query head: the full trace of the sequence, by the oracle's literal replay."""
    hq, hkv, d = w.num_q_heads, w.num_kv_heads, w.head_dim
    g_sz = hq // hkv
    steps = w.batch
    _, st, sh = inp["strides"]
    traces = np.zeros((hq, w.window - w.n_att), dtype=np.int32)
    for h in range(hq):
        rows = (w.prompt_len + np.arange(steps, dtype=np.int64)) * st + (h // g_sz) * sh
        _, tr = ora.replay_argmin(steps - 1, w.window, w.n_att, inp["q"].reshape(-1)[h * d:], hq * d,
                                  inp["k_cache"], rows, d, 1.0 / np.sqrt(d), n_sink)
        traces[h, :len(tr)] = tr
    return traces


def _near_tie(w, q, k, t, h, o_gpu, o_ref):
    g = h // (w.num_q_heads // w.num_kv_heads)
    scale = 1.0 / np.sqrt(w.head_dim)
    lg = scale * float(q[t, h] @ k[w.prompt_len + t - o_gpu, g])
    lr = scale * float(q[t, h] @ k[w.prompt_len + t - o_ref, g])
    return abs(lg - lr) <= 1e-4 * max(1.0, abs(lr))


@pytest.mark.parametrize("hq,hkv,d,split,n_sink,positional", [
    (8, 8, 64, 0, 0, False), (8, 2, 128, 0, 0, False), (4, 4, 128, 16, 0, False), (8, 4, 64, 24, 2, False),
    (8, 8, 64, 0, 0, True), (8, 2, 128, 16, 0, True)])
def test_every_step_of_one_sequence(dsa, hq, hkv, d, split, n_sink, positional):
    # 16x16 grid like the tiny configuration: one call holds every decode step of the sequence,
    # each request with the oracle's trace up to its own step.  With the positional component in
    # q and k, tokens of the same image column score higher, so the selection is no longer a
    # draw among equals.
    w = synth.Workload("sel", 61, 256, hq, hkv, d, 32, 16, 16, 0, 64, 13, 1, 256, share_cache=True,
                       positional=positional)
    inp = synth.make_inputs(w)
    q, k = _trajectory(w, inp)
    traces = _oracle_traces(w, inp, n_sink)
    m = w.window - w.n_att
    buf = np.full((w.batch, hq, m), SENTINEL, dtype=np.int32)
    n_act = np.clip(np.arange(w.batch) - (w.n_att - 1), 0, m)
    for b in range(w.batch):
        buf[b, :, :n_act[b]] = traces[:, :n_act[b]]
    dev_buf = torch.from_numpy(buf).cuda()
    prob = dsa.problem_from_host(inp, split_tokens=split)
    diag = dsa.Diag(dsa.DSA_MASK_LIST, w.window, w.n_att, skip_offsets=dev_buf, n_sink=n_sink, select=True)
    if split:
        assert dsa.dsa_query_plan(prob, diag).n_split > 1
    out, lse = dsa.alloc_outputs(prob)
    dsa.dsa_decode_attention_sparse(prob, diag, out, lse, dsa.alloc_workspace(prob, diag))
    torch.cuda.synchronize()
    got = dev_buf.cpu().numpy()

    # attention itself: the entry written at this step is not skipped at this step
    full = np.broadcast_to(traces, (w.batch, hq, m)).copy()
    ref = util.oracle_run(inp, ora.MODE_LIST, n_r=w.window, n_att=w.n_att, trace=full, n_sink=n_sink)
    util.assert_close(out, lse, ref, what="select attention")

    exact = flips = 0
    for b in range(w.batch):
        t = b
        selecting = w.n_att - 1 <= t <= w.window - 2
        for h in range(hq):
            row = got[b, h]
            keep = np.ones(m, dtype=bool)
            if selecting:
                kk = t - (w.n_att - 1)
                keep[kk] = False
                if row[kk] == traces[h, kk]:
                    exact += 1
                else:
                    assert 0 <= row[kk] <= t and row[kk] not in traces[h, :kk], (b, h, row[kk])
                    assert t - row[kk] >= n_sink
                    assert _near_tie(w, q, k, t, h, int(row[kk]), int(traces[h, kk])), (b, h)
                    flips += 1
            assert np.array_equal(row[keep], buf[b, h][keep]), "entries of other steps were touched"
    assert exact > 0 and flips <= 0.01 * (exact + flips)


def test_free_running_decode_loop_grows_a_valid_trace(dsa):
    # one sequence, one call per decode step, the library extends its own trace
    w = synth.Workload("loop", 62, 160, 4, 2, 64, 16, 10, 16, 0, 48, 10, 1, 160, share_cache=True)
    inp = synth.make_inputs(w)
    q, k = _trajectory(w, inp)
    traces = _oracle_traces(w, inp)
    m = w.window - w.n_att
    full = dsa.problem_from_host(inp)
    dev_buf = torch.full((1, w.num_q_heads, m), SENTINEL, dtype=torch.int32, device="cuda")
    diag = dsa.Diag(dsa.DSA_MASK_LIST, w.window, w.n_att, skip_offsets=dev_buf, select=True)
    outs = []
    for t in range(w.batch):
        step = dsa.Problem(q=full.q[t:t + 1], k_cache=full.k_cache, v_cache=full.v_cache, strides=full.strides,
                           seq_len=full.seq_len[t:t + 1], prompt_len=full.prompt_len[t:t + 1],
                           num_kv_heads=w.num_kv_heads, max_seq_len=full.max_seq_len,
                           max_prompt_len=w.prompt_len)
        out, lse = dsa.alloc_outputs(step)
        dsa.dsa_decode_attention_sparse(step, diag, out, lse, dsa.alloc_workspace(step, diag))
        outs.append((out, lse))
    torch.cuda.synchronize()
    got = dev_buf.cpu().numpy()[0]
    for h in range(w.num_q_heads):
        # a valid trace: Algorithm 1's replay accepts it at every step
        ora.replay(w.batch - 1, w.window, w.n_att, ora.SEL_TRACE, got[h])
        diff = np.flatnonzero(got[h] != traces[h])
        if len(diff):                       # the first divergence must be a float32 near-tie
            kk = int(diff[0])
            assert _near_tie(w, q, k, kk + w.n_att - 1, h, int(got[h, kk]), int(traces[h, kk]))
    # outputs of the loop equal the oracle's attention under the trace the library built
    tr = np.broadcast_to(got, (w.batch, w.num_q_heads, m)).copy()
    ref = util.oracle_run(inp, ora.MODE_LIST, n_r=w.window, n_att=w.n_att, trace=tr)
    out = torch.cat([o for o, _ in outs])
    lse = torch.cat([l for _, l in outs])
    util.assert_close(out, lse, ref, what="decode loop")


def test_selection_needs_per_head_masks(dsa):
    w = synth.Workload("selargs", 63, 2, 8, 2, 64, 4, 4, 4, 0, 8, 3, 1, 16)
    inp = synth.make_inputs(w)
    prob = dsa.problem_from_host(inp)
    out, lse = dsa.alloc_outputs(prob)
    buf = torch.zeros((2, 2, 5), dtype=torch.int32, device="cuda")        # per kv head: refused
    with pytest.raises(dsa.DsaError):
        dsa.dsa_decode_attention_sparse(prob, dsa.Diag(dsa.DSA_MASK_LIST, 8, 3, skip_offsets=buf, select=True),
                                        out, lse)
    buf = torch.zeros((2, 8, 5), dtype=torch.int32, device="cuda")        # sinks >= N_att: refused
    with pytest.raises(dsa.DsaError):
        dsa.dsa_decode_attention_sparse(prob, dsa.Diag(dsa.DSA_MASK_LIST, 8, 3, skip_offsets=buf, select=True,
                                                       n_sink=3), out, lse)
    torch.cuda.synchronize()
