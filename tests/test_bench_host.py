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


def test_device_batches_poison_exactly_the_rows_past_each_request():
    """make_inputs_device NaN-fills cache rows at positions >= seq_len (and nothing else), paged and
    contiguous, so that a read past a request's length shows up at full size too."""
    import torch
    for w in (synth.Workload("pz", 8, 5, 4, 2, 64, 7, 6, 5, 1, 16, 5, 1, 36, paged=True, block_size=8),
              synth.Workload("cz", 9, 4, 4, 4, 64, 3, 5, 5, 0, 16, 5, 1, 25)):
        dev = synth.make_inputs_device(w, torch.device("cpu"), seed=11)
        hkv, d = w.num_kv_heads, w.head_dim
        for name in ("k_cache", "v_cache"):
            for b in range(w.batch):
                n = int(dev["host"]["seq_len"][b])
                if w.paged:
                    bt = torch.from_numpy(dev["host"]["block_table"][b].astype(np.int64))
                    seq = dev[name].view(-1, w.block_size, hkv, d)[bt].reshape(-1, hkv, d)
                else:
                    seq = dev[name].view(w.batch, -1, hkv, d)[b]
                assert torch.isfinite(seq[:n].float()).all()
                assert torch.isnan(seq[n:].float()).all() and seq.shape[0] >= w.max_seq_len


def test_list_mask_bytes_match_the_oracle_per_head_kept_sets():
    """Per-query-head list masks under grouped queries: K/V bytes are those of the union of the
    group's kept sets, and every mask head reads its active trace entries."""
    w = synth.Workload("lbytes", 4, 6, 8, 2, 128, 9, 12, 10, 1, 40, 9, 1, 132, paged=True, block_size=16)
    group = w.num_q_heads // w.num_kv_heads
    rng = np.random.default_rng(2)
    position = rng.integers(w.pos_lo, w.pos_hi + 1, size=w.batch).astype(np.int32)
    position[0], position[1] = 3, w.n_att + 4                 # phase 1 and early phase 2 are in the mix
    host = {"position": position, "prompt_len": np.full(w.batch, w.prompt_len, dtype=np.int32)}
    trace = synth.random_valid_trace(rng, w.window, w.n_att, (w.batch, w.num_q_heads))
    max_kept = w.prompt_len + w.window
    idx = np.full((w.batch, w.num_q_heads, max_kept), -1, dtype=np.int32)
    cnt = np.zeros((w.batch, w.num_q_heads), dtype=np.int32)
    rows = entries = 0
    for i, p in enumerate(position):
        for g0 in range(0, w.num_q_heads, group):
            union = set()
            for h in range(g0, g0 + group):
                kept = ora.kept(ora.MODE_LIST, w.prompt_len, int(p), w.window, w.n_att, trace=trace[i, h])
                idx[i, h, :len(kept)], cnt[i, h] = kept, len(kept)
                union.update(kept.tolist())
                # active entries = the window keys of this head that its mask drops
                entries += min(int(p), w.window) - (len(kept) - w.prompt_len)
            rows += len(union)
    assert bench.union_rows(idx, cnt, group) == rows
    assert int(bench.list_active_entries(position, w.window, w.n_att).sum()) * w.num_q_heads == entries
    lmask = {"mask_heads": w.num_q_heads, "union_rows": rows}
    got, _ = bench.algorithmic_bytes(w, host, "sparse", 0, lmask)
    want = rows * w.head_dim * 2 * 2 + w.batch * w.num_q_heads * (w.head_dim * 2 * 2 + 4) + 4 * entries
    assert got == want
    # one shared list, no grouping effect: the rows of the grid formula plus one trace per request
    got1, _ = bench.algorithmic_bytes(w, host, "sparse", 0, {"mask_heads": 1, "union_rows": None})
    base, _ = bench.algorithmic_bytes(w, host, "sparse", 0)
    assert got1 == base + 4 * entries // w.num_q_heads


def test_whole_job_value_is_all_ranks_work_over_the_slowest_rank():
    # two ranks, 256 queries per step each, 20 steps; rank 1 is the slower one
    assert bench.aggregate_value(2, 256, 20, [0.0051, 0.0064]) == 2 * 256 * 20 / 0.0064
    assert bench.aggregate_value(1, 256, 20, [0.005]) == 256 * 20 / 0.005
    # doubling the ranks at equal per-rank time doubles the value (weak scaling)
    assert bench.aggregate_value(8, 32, 10, [0.01] * 8) == 8 * bench.aggregate_value(1, 32, 10, [0.01])
