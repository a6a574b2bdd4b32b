"""Parity at the benchmark's full size and launch configuration: the paged throughput workload
at batch 32, 128 and 256 (up to 18 GB of K/V drawn on the device, rows past each request's length
NaN-filled), checked on sampled requests that the oracle computes one by one from a host copy of
just their blocks, plus the kept-count closed form on every request."""
import numpy as np
import pytest
import torch

from oracle import oracle as ora
from paper_2609_19702_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("batch", [32, 128, 256])
def test_config5_large_batches_sampled_requests(batch):
    """The paged sweep at batch 32, 128 and 256 (batch 1 and 8 are compared in full elsewhere)."""
    from paper_2609_19702_b200 import binding as dsa
    free, _ = torch.cuda.mem_get_info()
    if free < (24 << 30) * batch // 256 + (2 << 30):
        pytest.skip("needs %d GB of free device memory" % (24 * batch // 256 + 2))
    w = synth.workload(5, batch=batch)
    dev = synth.make_inputs_device(w, torch.device("cuda"))
    prob = dsa.Problem(q=dev["q"], k_cache=dev["k_cache"], v_cache=dev["v_cache"], strides=dev["strides"],
                       seq_len=dev["seq_len"], prompt_len=dev["prompt_len"], num_kv_heads=w.num_kv_heads,
                       max_seq_len=dev["max_seq_len"], max_prompt_len=w.prompt_len,
                       block_table=dev["block_table"], block_size=dev["block_size"],
                       num_blocks=dev["block_table"].numel())
    pos = dev["host"]["position"]
    # shortest, longest, around the phase boundaries of both windows, and a few at random
    order = np.argsort(pos)
    sample = sorted({int(order[0]), int(order[-1]), int(order[len(order) // 2]),
                     int(np.argmin(np.abs(pos - 208))), int(np.argmin(np.abs(pos - 512))),
                     int(np.argmin(np.abs(pos - 1024))), 0, 17 % batch, 101 % batch, batch - 1})
    sub = synth.host_subset(dev, sample)
    out, lse = dsa.alloc_outputs(prob)
    sidx = torch.tensor(sample, device="cuda")

    cases = [(None, ora.MODE_DENSE, dict())]
    for window, n_att in ((512, 208), (1024, 416)):
        cases.append((dsa.Diag(dsa.DSA_MASK_GRID, window, n_att, w.grid_w, w.row_extra), ora.MODE_GRID,
                      dict(n_r=window, n_att=n_att, stride=w.stride)))
    for diag, mode, kw in cases:
        out.fill_(float("nan"))
        ws = dsa.alloc_workspace(prob, diag)
        if diag is None:
            dsa.dsa_decode_attention_dense(prob, out, lse, ws)
        else:
            dsa.dsa_decode_attention_sparse(prob, diag, out, lse, ws)
        torch.cuda.synchronize()
        assert torch.isfinite(out.float()).all()
        ref = util.oracle_run(sub, mode, want_kept=True, **kw)
        util.assert_close(out[sidx], lse[sidx], ref, what="full size mode %d" % mode)
        idx, cnt = dsa.dsa_debug_kept_indices(prob, diag, dev["max_seq_len"])
        util.assert_kept_equal(idx[sidx], cnt[sidx], ref, "full size mode %d" % mode)
        # property that holds for every request: kept count = prompt + min(p, N_att) (or p)
        want = w.prompt_len + (pos if diag is None else np.minimum(pos, diag.n_att))
        assert np.array_equal(cnt.cpu().numpy()[:, 0], want)
    # the paper's own setting at this size: one skip list per attention head, with the fused selection
    # (sampled requests against the oracle's kept sets and outputs; every request's kept count)
    rng = np.random.default_rng(40 + batch)
    few = synth.random_valid_trace(rng, 512, 208, (16,))
    trace = np.ascontiguousarray(few[rng.integers(0, 16, size=(batch, w.num_q_heads))])
    trace_dev = torch.from_numpy(trace.copy()).cuda()
    diag = dsa.Diag(dsa.DSA_MASK_LIST, 512, 208, skip_offsets=trace_dev, select=True)
    plan = dsa.dsa_query_plan(prob, diag)
    assert plan.per_head_lists == 1 and plan.n_split == 1
    out.fill_(float("nan"))
    dsa.dsa_decode_attention_sparse(prob, diag, out, lse, dsa.alloc_workspace(prob, diag))
    torch.cuda.synchronize()
    assert torch.isfinite(out.float()).all()
    ref = util.oracle_run(sub, ora.MODE_LIST, n_r=512, n_att=208, trace=trace[sample], want_kept=True)
    util.assert_close(out[sidx], lse[sidx], ref, what="full size per-head lists")
    diag_ro = dsa.Diag(dsa.DSA_MASK_LIST, 512, 208, skip_offsets=torch.from_numpy(trace.copy()).cuda())
    idx, cnt = dsa.dsa_debug_kept_indices(prob, diag_ro, dev["max_seq_len"])
    util.assert_kept_equal(idx[sidx], cnt[sidx], ref, "full size per-head lists")
    assert np.array_equal(cnt.cpu().numpy(), np.broadcast_to((w.prompt_len + np.minimum(pos, 208))[:, None], cnt.shape))
    # requests in phase 2 got one new trace entry per head (a valid one), the others none
    t = pos - 1
    selecting = (t >= 207) & (t <= 510)
    new = trace_dev.cpu().numpy()
    changed = (new != trace).any(axis=2)
    assert not changed[~selecting].any()
    for i in np.flatnonzero(selecting)[:8]:
        k = int(t[i]) - 207
        assert (new[i, :, :k] == trace[i, :, :k]).all() and (new[i, :, k] >= 0).all() and (new[i, :, k] <= t[i]).all()
        for h in (0, w.num_q_heads - 1):
            assert new[i, h, k] not in set(trace[i, h, :k].tolist())       # an attended key, not one already skipped
    if batch != 256:
        return
    # the end-to-end call of the benchmark at this size (step inputs and results in pinned host
    # memory): bit for bit what the device-buffer call gives
    diag = dsa.Diag(dsa.DSA_MASK_GRID, 512, 208, w.grid_w, w.row_extra)
    ws = dsa.alloc_workspace(prob, diag)
    dsa.dsa_decode_attention_sparse(prob, diag, out, lse, ws)
    torch.cuda.synchronize()
    h_q, h_seq, h_pl = prob.q.cpu().pin_memory(), prob.seq_len.cpu().pin_memory(), prob.prompt_len.cpu().pin_memory()
    h_bt = prob.block_table.cpu().pin_memory()
    h_out = torch.full(out.shape, float("nan"), dtype=out.dtype).pin_memory()
    h_lse = torch.full(lse.shape, float("nan"), dtype=lse.dtype).pin_memory()
    dsa.dsa_decode_attention_host_mapped(prob, diag, h_q, h_seq, h_pl, h_bt, h_out, h_lse, ws)
    torch.cuda.synchronize()
    assert torch.equal(h_out.view(torch.int16), out.cpu().view(torch.int16)) and torch.equal(h_lse, lse.cpu())
