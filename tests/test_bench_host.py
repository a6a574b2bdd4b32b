"""Host-side pieces of bench.py: the algorithmic-byte formula against the oracle's kept sets, and
the workload naming.  No GPU."""
import numpy as np

import bench
from oracle import oracle as ora
from paper_2609_19702_b200 import synth


def test_algorithmic_bytes_match_the_oracle_kept_sets():
    w = synth.Workload("bytes", 3, 9, 8, 2, 128, 21, 12, 10, 1, 40, 9, 1, 132, paged=True, block_size=16)
    rng = np.random.default_rng(1)
    position = rng.integers(w.pos_lo, w.pos_hi + 1, size=w.batch).astype(np.int32)
    host = {"position": position, "prompt_len": np.full(w.batch, w.prompt_len, dtype=np.int32)}
    for mode, ora_mode in (("dense", ora.MODE_DENSE), ("sparse", ora.MODE_GRID)):
        rows = blocks = 0
        for p in position:
            kept = ora.kept(ora_mode, w.prompt_len, int(p), w.window, w.n_att, w.stride)
            rows += len(kept)
            blocks += len(set((kept // w.block_size).tolist()))
        got, got_rows = bench.algorithmic_bytes(w, host, mode, blocks)
        want = rows * w.num_kv_heads * w.head_dim * 2 * 2             # K and V rows, bf16
        want += w.batch * w.num_q_heads * (w.head_dim * 2 * 2 + 4)    # q, out, lse
        want += 4 * blocks                                            # block-table entries
        assert got_rows == rows and got == want


def test_workload_names_are_distinct():
    names = {bench.workload_name(synth.workload(i), m) for i in range(1, 6) for m in ("dense", "sparse")}
    assert len(names) == 10
    w = synth.workload(5, batch=256)
    assert bench.workload_name(w, "sparse") in bench.NCU_TRAFFIC_BYTES


def test_oracle_baseline_reports_all_threads_and_one_thread():
    import torch
    w = synth.workload(5, batch=2)
    inputs = synth.make_inputs_device(w, torch.device("cpu"), seed=3)
    res = bench.oracle_baseline(synth, inputs, w, "sparse", sample=2, min_seconds=0.5)
    assert res["kind"] == "oracle" and res["cores"] >= 1 and res["unit"] == bench.UNIT
    assert res["value"] > 0 and res["single_thread_value"] > 0
