"""The allocation-free entry point (collected last on purpose).

Some users of the library cannot allocate device memory around the call -- code running inside
an allocation-free section of a host application, or a server whose memory pool is fully handed
out -- so `dsa_decode_attention_static_scratch` keeps the split-KV partials in a fixed array
inside the library.  It must give what the workspace-based entry points give, call after call,
although the array still holds the previous call's partials."""
import pytest
import torch

from oracle import oracle as ora
from paper_2609_19702_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_matches_workspace_entry_twice_in_a_row():
    from paper_2609_19702_b200 import binding as dsa
    # long grouped-query sequences, few requests: the plan splits every (request, kv head)
    w = synth.Workload("noalloc", 77, 3, 16, 4, 128, 40, 40, 30, 1, 256, 100, 700, 1240, paged=True)
    inp = synth.make_inputs(w)
    prob = dsa.problem_from_host(inp, split_tokens=128)
    diag = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
    assert dsa.dsa_query_plan(prob, None).n_split > 1          # the scratch really is used
    assert 0 < dsa.dsa_workspace_size(prob, None) <= (8 << 20)

    def reference(dg):
        out, lse = dsa.alloc_outputs(prob)
        ws = dsa.alloc_workspace(prob, dg)
        if dg is None:
            dsa.dsa_decode_attention_dense(prob, out, lse, ws)
        else:
            dsa.dsa_decode_attention_sparse(prob, dg, out, lse, ws)
        torch.cuda.synchronize()
        return out.float(), lse

    ref_dense, ref_sparse = reference(None), reference(diag)
    # what the paper's definitions give for the same batch (float64 oracle)
    ora_dense = util.oracle_run(inp, ora.MODE_DENSE)
    ora_sparse = util.oracle_run(inp, ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride=w.stride)
    # two calls in a row, alternating problems so that each sees the other's leftovers
    for _ in range(2):
        for dg, (ref_out, ref_lse), ora_ref in ((None, ref_dense, ora_dense), (diag, ref_sparse, ora_sparse)):
            out, lse = dsa.alloc_outputs(prob)
            out.fill_(float("nan"))
            lse.fill_(float("nan"))
            dsa.dsa_decode_attention_static_scratch(prob, dg, out, lse)
            torch.cuda.synchronize()
            err = (out.float() - ref_out).abs() - (1e-2 + 1e-2 * ref_out.abs())
            assert torch.isfinite(out.float()).all() and err.max().item() <= 0
            assert (lse - ref_lse).abs().max().item() <= 1e-3
            util.assert_close(out, lse, ora_ref, what="static scratch against the oracle")

    # a problem whose partials do not fit the fixed array is refused, nothing is launched
    big = synth.workload(5, batch=256)
    fake = dsa.Problem(q=torch.empty((256, 32, 128), dtype=torch.bfloat16, device="cuda"),
                       k_cache=prob.k_cache, v_cache=prob.v_cache, strides=prob.strides,
                       seq_len=torch.zeros(256, dtype=torch.int32, device="cuda"),
                       prompt_len=torch.zeros(256, dtype=torch.int32, device="cuda"),
                       num_kv_heads=32, max_seq_len=big.max_seq_len, block_table=None)
    assert dsa.dsa_workspace_size(fake, None) > (8 << 20)
    out, lse = dsa.alloc_outputs(fake)
    with pytest.raises(dsa.DsaError) as ei:
        dsa.dsa_decode_attention_static_scratch(fake, None, out, lse)
    assert ei.value.status == -3
    torch.cuda.synchronize()
