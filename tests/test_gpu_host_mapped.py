"""The decode step whose kernels read q from, and write out / lse to, pinned host memory.

Checked against the oracle (same tolerances as every other parity test) and, bit for bit, against
the device-buffer entry points, on plans with one work item per (request, kv head) -- q is then
read straight from the host buffer -- and on split plans, where q is staged on the device."""
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


def _pinned_step(prob):
    h = {"q": prob.q.cpu().pin_memory(), "seq": prob.seq_len.cpu().pin_memory(),
         "pl": prob.prompt_len.cpu().pin_memory(),
         "bt": None if prob.block_table is None else prob.block_table.cpu().pin_memory()}
    h["out"] = torch.full(prob.q.shape, float("nan"), dtype=prob.q.dtype).pin_memory()
    h["lse"] = torch.full(prob.q.shape[:2], float("nan"), dtype=torch.float32).pin_memory()
    return h


# (config, batch, mode, forced rows per split): plans with one work item per (request, kv head) read q
# from the host buffer; plans with several splits stage it on the device first
CASES = [(2, None, "sparse", 0), (2, None, "dense", 0), (5, 3, "sparse", 0), (5, 3, "dense", 0),
         (4, None, "sparse", 0), (5, 3, "sparse", 96), (2, None, "dense", 128)]


@pytest.mark.parametrize("index,batch,mode,split", CASES)
def test_host_mapped_step_matches_oracle_and_device_call(dsa, index, batch, mode, split):
    w = synth.workload(index) if batch is None else synth.workload(index, batch=batch)
    inp = synth.make_inputs(w)
    prob = dsa.problem_from_host(inp, split_tokens=split)
    diag = None if mode == "dense" else dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
    ref_out, ref_lse = dsa.alloc_outputs(prob)
    ws = dsa.alloc_workspace(prob, diag)
    if diag is None:
        dsa.dsa_decode_attention_dense(prob, ref_out, ref_lse, ws)
        ref = util.oracle_run(inp, ora.MODE_DENSE)
    else:
        dsa.dsa_decode_attention_sparse(prob, diag, ref_out, ref_lse, ws)
        ref = util.oracle_run(inp, ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride=w.stride)
    torch.cuda.synchronize()
    h = _pinned_step(prob)
    n_split = dsa.dsa_query_plan(prob, diag).n_split
    # scramble what the call must bring over itself; q only matters when it is staged
    q_before = torch.full_like(prob.q, 7.0)
    prob.q.copy_(q_before)
    prob.seq_len.zero_()
    prob.prompt_len.zero_()
    if prob.block_table is not None:
        prob.block_table.zero_()
    for _ in range(2):                                   # twice: nothing may depend on a first call
        h["out"].fill_(float("nan"))
        dsa.dsa_decode_attention_host_mapped(prob, diag, h["q"], h["seq"], h["pl"], h["bt"], h["out"], h["lse"], ws)
        torch.cuda.synchronize()
        util.assert_close(h["out"], h["lse"], ref, what="host-mapped %s config %d" % (mode, index))
        assert torch.equal(h["out"].view(torch.int16), ref_out.cpu().view(torch.int16))
        assert torch.equal(h["lse"], ref_lse.cpu())
    assert torch.equal(prob.seq_len.cpu(), h["seq"])
    # the host rewrites its buffers between steps: the next call must see the new q (here: -q)
    flipped = dict(inp, q=inp["q"] ^ np.uint16(0x8000))
    h["q"].view(torch.int16).copy_(torch.from_numpy(flipped["q"].view(np.int16)))
    ref2 = (util.oracle_run(flipped, ora.MODE_DENSE) if diag is None else
            util.oracle_run(flipped, ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride=w.stride))
    dsa.dsa_decode_attention_host_mapped(prob, diag, h["q"], h["seq"], h["pl"], h["bt"], h["out"], h["lse"], ws)
    torch.cuda.synchronize()
    util.assert_close(h["out"], h["lse"], ref2, what="host-mapped %s config %d, rewritten q" % (mode, index))
    if n_split == 1:
        assert torch.equal(prob.q, q_before), "q is read from the host buffer: the device copy stays untouched"
    else:
        assert torch.equal(prob.q.cpu().view(torch.int16), h["q"].view(torch.int16))


def test_host_mapped_plans_cover_both_q_paths(dsa):
    """The cases above must exercise the direct read of q (one split) and the staged copy (several)."""
    seen = set()
    for index, batch, mode, split in CASES:
        w = synth.workload(index) if batch is None else synth.workload(index, batch=batch)
        inp = synth.make_inputs(w)
        prob = dsa.problem_from_host(inp, split_tokens=split)
        diag = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra) if mode == "sparse" else None
        seen.add(min(dsa.dsa_query_plan(prob, diag).n_split, 2))
    assert seen == {1, 2}


def test_host_mapped_rejects_pageable_buffers(dsa):
    w = synth.workload(5, batch=2)
    inp = synth.make_inputs(w)
    prob = dsa.problem_from_host(inp)
    diag = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
    ws = dsa.alloc_workspace(prob, diag)
    h = _pinned_step(prob)
    seq_before = prob.seq_len.clone()
    prob.seq_len.fill_(1)
    for name in ("q", "out", "lse"):
        bad = dict(h)
        bad[name] = h[name].clone()                      # same contents, ordinary pageable memory
        assert not bad[name].is_pinned()
        with pytest.raises(dsa.DsaError) as ei:
            dsa.dsa_decode_attention_host_mapped(prob, diag, bad["q"], bad["seq"], bad["pl"], bad["bt"],
                                                 bad["out"], bad["lse"], ws)
        assert ei.value.status == -1                   # DSA_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert int(prob.seq_len.max()) == 1, "a rejected call must not have queued anything"
    # and the context is still usable
    prob.seq_len.copy_(seq_before)
    dsa.dsa_decode_attention_host_mapped(prob, diag, h["q"], h["seq"], h["pl"], h["bt"], h["out"], h["lse"], ws)
    torch.cuda.synchronize()
    assert np.isfinite(h["out"].float().numpy()).all()
