"""dsa_prepare(): after it, calls that are the first of their shape in the process can be captured.

Runs in a child process, because in the test process other tests have long configured the kernels."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import torch
from paper_2609_19702_b200 import binding as dsa, synth

w = synth.workload(5, batch=3)
inp = synth.make_inputs(w, poison=False)
prob = dsa.problem_from_host(inp)
diag = dsa.Diag(dsa.DSA_MASK_GRID, w.window, w.n_att, w.grid_w, w.row_extra)
outs = [dsa.alloc_outputs(prob) for _ in range(3)]
ws_s, ws_d = dsa.alloc_workspace(prob, diag), dsa.alloc_workspace(prob, None)
k_new = torch.randn((w.batch, w.num_kv_heads, w.head_dim), device="cuda").to(torch.bfloat16)
v_new = torch.randn_like(k_new)
prob.seq_len -= 1                      # room for the fused step's token
torch.cuda.synchronize()

dsa.dsa_prepare()
graph = torch.cuda.CUDAGraph()
with torch.cuda.graph(graph):          # the very first attention calls of this process
    dsa.dsa_decode_attention_sparse(prob, diag, outs[0][0], outs[0][1], ws_s)
    dsa.dsa_decode_attention_dense(prob, outs[1][0], outs[1][1], ws_d)
    dsa.dsa_decode_step(prob, diag, k_new, v_new, outs[2][0], outs[2][1], ws_s)
graph.replay()
torch.cuda.synchronize()
got = [(o.clone(), l.clone()) for o, l in outs]

# the same three calls eagerly
dsa.dsa_decode_attention_sparse(prob, diag, outs[0][0], outs[0][1], ws_s)
dsa.dsa_decode_attention_dense(prob, outs[1][0], outs[1][1], ws_d)
dsa.dsa_decode_step(prob, diag, k_new, v_new, outs[2][0], outs[2][1], ws_s)
torch.cuda.synchronize()
for (o, l), (o2, l2) in zip(got, outs):
    assert torch.isfinite(o.float()).all()
    assert torch.equal(o.view(torch.int16), o2.view(torch.int16)) and torch.equal(l, l2)
print("CAPTURED-FIRST-CALLS-OK")
"""


def test_first_calls_of_a_process_can_be_captured_after_prepare():
    env = dict(os.environ, PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    res = subprocess.run([sys.executable, "-c", CHILD], cwd=ROOT, env=env, capture_output=True, text=True,
                         timeout=600)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-4000:]
    assert "CAPTURED-FIRST-CALLS-OK" in res.stdout
