#!/usr/bin/env python
"""Benchmark of the decode-attention hot path.

    python bench.py --gpus 1 --steps K --warmup W            # this library (CUDA, sm_100a)
    python bench.py --impl reference --steps K --warmup W    # the float64 CPU oracle

A "step" is one sparse decode-attention call (mask generation, K/V staging, scores, online
softmax, partial write and split combine where the plan needs one) over one batch of the paged
throughput workload at its largest batch: 256 requests, 32/32 heads, head_dim 128, bf16, 200
prompt tokens + a 64x64 grid with one separator per row, 16-token blocks in a shuffled block
table, decode positions uniform in [1, 4160], window 512 / N_att 208.  Inputs are seeded and
synthetic and already resident in HBM when the timed region starts; every step reads ~1.7 GB of
distinct K/V, far more than the L2, so no flush is needed between steps.

One JSON line is printed by rank 0.  With torchrun (N > 1) every rank owns its own batch of the
same shape (requests are independent: weak scaling, no collective on the data path) and the
time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "decode_attention_queries_per_sec"
UNIT = "queries/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
L2_BYTES = 126 << 20
# DRAM bytes per launch of the timed kernel (dram__bytes_read.sum + dram__bytes_write.sum of an ncu
# capture), keyed by the workload string of the JSON line; None until a capture of that launch exists.
NCU_TRAFFIC_BYTES = {
    # measured with ncu at batch 32 (head-group kernel with producer warps, the form a batch-256 launch
    # takes): 209.39 MB read + 4.48 MB written per launch; traffic grows in proportion to the batch, so
    # a batch-256 launch moves 8 x that
    "config5_paged_sweep B=256 Hq=32 Hkv=32 D=128 Lp=200 grid=64x64+1 paged16 sparse grid-mask window=512 n_att=208":
        8 * 213_865_600,
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=5, help="workload 1..5")
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--window", type=int, default=None)
    ap.add_argument("--n-att", type=int, default=None)
    ap.add_argument("--mode", default="sparse", choices=["sparse", "dense"])
    ap.add_argument("--split-tokens", type=int, default=0)
    ap.add_argument("--plan-flags", type=lambda x: int(x, 0), default=0,
                    help="dsa_problem.plan_flags for comparison runs (DSA_PLAN_* bits of dsa.h; 0: the library plans)")
    ap.add_argument("--no-variants", action="store_true", help="skip the dense / other-window timings")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-decode-loop", action="store_true",
                    help="skip the whole-image decode loop at batch 128 (the paper's shape: 50 prompt tokens, 1024 "
                         "image tokens, N_att 52)")
    ap.add_argument("--no-per-config", action="store_true",
                    help="skip the table of every configuration (dense and sparse, L2 flushed between calls)")
    ap.add_argument("--all-configs", action="store_true",
                    help="also run the whole-image decode loops and the mask-variant comparison")
    return ap.parse_args()


def workload_name(w, mode):
    s = "config%d_%s B=%d Hq=%d Hkv=%d D=%d Lp=%d grid=%dx%d+%d %s" % (
        w.index, w.name, w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.prompt_len,
        w.grid_h, w.grid_w, w.row_extra, "paged%d" % w.block_size if w.paged else "contiguous")
    if mode == "sparse":
        s += " sparse grid-mask window=%d n_att=%d" % (w.window, w.n_att)
    else:
        s += " dense"
    return s


def kernel_name(plan):
    """Which attention kernel a plan launches (see dsa_plan_info)."""
    if not plan.tensor_cores:
        return "dsa_attn_kernel"
    if plan.per_head_lists:
        return "dsa_attn_heads_kernel"
    if plan.heads_per_block:
        if plan.tensor_map_copies:
            return "dsa_attn_gather_kernel"
        return "dsa_attn_group_ws_kernel" if plan.producer_warps else "dsa_attn_group_kernel"
    return "dsa_attn_mma_kernel"


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, torch_device_index: int):
        self.samples, self.reasons, self.max_mhz, self.err = [], set(), None, None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            props = torch.cuda.get_device_properties(torch_device_index)
            handle = None
            try:
                bus = "%08x:%02x:%02x.0" % (props.pci_domain_id, props.pci_bus_id, props.pci_device_id)
                handle = pynvml.nvmlDeviceGetHandleByPciBusId(bus.encode())
            except Exception:
                vis = os.environ.get("CUDA_VISIBLE_DEVICES")
                idx = torch_device_index
                if vis:
                    try:
                        idx = int(vis.split(",")[torch_device_index])
                    except ValueError:
                        pass
                handle = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self._nv, self._h = pynvml, handle
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # pragma: no cover
            self.err = repr(e)
            self._nv = None

    def _run(self):
        nv, h = self._nv, self._h
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(h))
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception as e:  # pragma: no cover
                self.err = repr(e)
                break
            time.sleep(0.0005)

    def start(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        out = {"sm_mhz": int(np.median(self.samples)) if self.samples else None,
               "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}
        if self.err:
            out["error"] = self.err
        return out


def list_active_entries(position, window, n_att):
    """Trace entries a LIST-mask request reads at decode position p (its active skips): with
    t = p - 1, the selections of steps N_att-1 .. t-1, at most window - N_att of them."""
    t = np.asarray(position, dtype=np.int64) - 1
    return np.clip(t - (n_att - 1), 0, window - n_att)


def union_rows(kept_idx, kept_cnt, group):
    """Rows a LIST-mask call reads per (request, kv head) when every query head has its own mask:
    the union of the kept sets of the `group` query heads that share the kv head (a row is fetched
    once if any of them keeps it).  kept_idx [B, H_q, max_kept], kept_cnt [B, H_q] (numpy); returns
    the total over requests and kv heads."""
    b, hq, _ = kept_idx.shape
    total = 0
    for i in range(b):
        for g0 in range(0, hq, group):
            rows = set()
            for h in range(g0, g0 + group):
                rows.update(kept_idx[i, h, :int(kept_cnt[i, h])].tolist())
            total += len(rows)
    return total


def algorithmic_bytes(w, host, mode, blocks_touched, list_mask=None):
    """Bytes one call must move: kept K and V rows, q, out, lse, and the block-table entries of
    the blocks it touches.  Kept rows per kv head: the whole prompt plus min(p, N_att) decode
    keys for the sparse call (the attended count of Algorithm 1), p for the dense call.
    list_mask (LIST masks): {"mask_heads": 1 | H_kv | H_q, "union_rows": total rows over
    (request, kv head) when query heads of a group keep different rows, else None}; adds the
    trace entries every mask head reads, mask_heads x n_act x 4 bytes per request -- or, with
    "bitmap_words" (the lists given as bitmaps, dsa_diag_params.skip_bitmap), the bitmap rows read instead:
    mask_heads x bitmap_words x 4 bytes per request."""
    esize = 2
    p = host["position"].astype(np.int64)
    lp = host["prompt_len"].astype(np.int64)
    dec = p if mode == "dense" else np.minimum(p, w.n_att)
    kept_rows = int((lp + dec).sum())
    kv_rows = kept_rows * w.num_kv_heads
    trace = 0
    if list_mask is not None:
        if list_mask.get("union_rows") is not None:
            kv_rows = int(list_mask["union_rows"])
        if list_mask.get("bitmap_words"):
            trace = 4 * int(list_mask["mask_heads"]) * int(list_mask["bitmap_words"]) * len(p)
        else:
            trace = 4 * int(list_mask["mask_heads"]) * int(list_active_entries(p, w.window, w.n_att).sum())
    kv = kv_rows * w.head_dim * esize * 2
    qo = w.batch * w.num_q_heads * (2 * w.head_dim * esize + 4)
    table = 4 * int(blocks_touched)
    return kv + qo + table + trace, kept_rows


def aggregate_value(world, batch_per_rank, steps, rank_seconds):
    """Whole-job throughput of a weak-scaling run: every rank processed batch_per_rank x steps
    queries and the job took as long as its slowest rank."""
    return world * batch_per_rank * steps / max(rank_seconds)


def time_calls(torch, fn, steps, warmup, sampler=None, barrier=None):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    if barrier:
        barrier()
        torch.cuda.synchronize()
    if sampler:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    if barrier:
        barrier()
        torch.cuda.synchronize()
    clocks = sampler.stop() if sampler else None
    return e0.elapsed_time(e1) / 1e3, clocks          # seconds for `steps` calls


def time_calls_flushed(torch, fn, steps, warmup, flush, sampler=None, barrier=None):
    """Like time_calls for working sets that would stay in L2: a write larger than L2 precedes every
    call and only the calls are timed (one event pair each, summed)."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    if barrier:
        barrier()
        torch.cuda.synchronize()
    if sampler:
        sampler.start()
    pairs = []
    for _ in range(steps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        pairs.append((e0, e1))
    torch.cuda.synchronize()
    if barrier:
        barrier()
        torch.cuda.synchronize()
    clocks = sampler.stop() if sampler else None
    return sum(a.elapsed_time(b) for a, b in pairs) / 1e3, clocks


def time_flushed(torch, fn, flush, iters=30, warmup=3):
    """Median device time of single calls with the L2 flushed (a 512 MB write) before each."""
    times = []
    for i in range(warmup + iters):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        if i >= warmup:
            times.append(e0.elapsed_time(e1) / 1e3)
    return float(np.median(times)), float(np.min(times))


def per_config_table(torch, dsa, synth, dev, peak, plan_flags=0, only=None):
    """Every configuration, dense and sparse from the same library, one call at a time.
    plan_flags: planner switches for comparison runs (0: the library chooses); only: restrict to
    these (config, batch) pairs."""
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    rows = []
    todo = [(synth.workload(i), None) for i in (1, 2, 3, 4)]
    for b in (1, 8, 32, 128, 256):
        todo.append((synth.workload(5, batch=b), [(512, 208), (1024, 416)]))
    for w, windows in todo:
        if only is not None and (w.index, w.batch) not in only:
            continue
        inputs = synth.make_inputs_device(w, dev)
        host = inputs["host"]
        prob = dsa.Problem(
            q=inputs["q"], k_cache=inputs["k_cache"], v_cache=inputs["v_cache"], strides=inputs["strides"],
            seq_len=inputs["seq_len"], prompt_len=inputs["prompt_len"], num_kv_heads=w.num_kv_heads,
            max_seq_len=inputs["max_seq_len"], max_prompt_len=w.prompt_len,
            block_table=inputs["block_table"], block_size=inputs["block_size"],
            num_blocks=0 if inputs["block_table"] is None else inputs["block_table"].numel(),
            plan_flags=plan_flags)
        out, lse = dsa.alloc_outputs(prob)
        ws = dsa.alloc_workspace(prob, None)
        plan = dsa.dsa_query_plan(prob, None)
        t_dense, t_dense_min = time_flushed(torch, lambda: dsa.dsa_decode_attention_dense(prob, out, lse, ws), flush)
        b_dense, _ = algorithmic_bytes(w, host, "dense", 0)
        row = {"config": w.index, "name": w.name, "batch": w.batch,
               "dense": {"us": round(t_dense * 1e6, 2), "us_min": round(t_dense_min * 1e6, 2),
                         "queries_per_sec": round(w.batch / t_dense, 1),
                         "bytes": b_dense, "GBs": round(b_dense / t_dense / 1e9, 1),
                         "frac_of_peak": round(b_dense / t_dense / 1e9 / peak, 4),
                         "n_split": plan.n_split, "launches": plan.launches, "kernel": kernel_name(plan),
                         "heads_per_block": plan.heads_per_block, "item_warps": plan.item_warps,
                         "cluster_blocks": plan.cluster_blocks, "tensor_map_copies": plan.tensor_map_copies,
                         "producer_warps": plan.producer_warps},
               "sparse": []}
        for window, n_att in (windows or [(w.window, w.n_att)]):
            ww = synth.workload(w.index, batch=w.batch, window=window, n_att=n_att)
            diag = dsa.Diag(dsa.DSA_MASK_GRID, window, n_att, w.grid_w, w.row_extra)
            ws2 = dsa.alloc_workspace(prob, diag)
            plan2 = dsa.dsa_query_plan(prob, diag)
            t_sp, t_sp_min = time_flushed(torch, lambda: dsa.dsa_decode_attention_sparse(prob, diag, out, lse, ws2), flush)
            b_sp, _ = algorithmic_bytes(ww, host, "sparse", 0)
            row["sparse"].append({"window": window, "n_att": n_att, "us": round(t_sp * 1e6, 2),
                                  "us_min": round(t_sp_min * 1e6, 2),
                                  "queries_per_sec": round(w.batch / t_sp, 1), "bytes": b_sp,
                                  "GBs": round(b_sp / t_sp / 1e9, 1),
                                  "frac_of_peak": round(b_sp / t_sp / 1e9 / peak, 4),
                                  "speedup_over_dense": round(t_dense / t_sp, 3),
                                  "ideal_byte_ratio": round(b_dense / b_sp, 3),
                                  "n_split": plan2.n_split, "launches": plan2.launches,
                                  "kernel": kernel_name(plan2), "heads_per_block": plan2.heads_per_block,
                                  "item_warps": plan2.item_warps, "cluster_blocks": plan2.cluster_blocks,
                                  "tensor_map_copies": plan2.tensor_map_copies,
                                  "producer_warps": plan2.producer_warps})
        rows.append(row)
        del inputs, prob, out, lse, ws
        torch.cuda.empty_cache()
    return rows


def selection_overhead(torch, dsa, synth, dev):
    """Cost of the fused phase-2 selection: config 5 at batch 256 with per-head LIST masks, every
    request at a phase-2 position (N_att <= p < N_r), the sparse call with and without `select`."""
    w = synth.workload(5, batch=256)
    inputs = synth.make_inputs_device(w, dev)
    rng = np.random.default_rng(synth.BASE_SEED + 5)
    p = rng.integers(w.n_att, w.window, size=w.batch).astype(np.int32)
    seq = torch.from_numpy(w.prompt_len + p).to(dev)
    few = synth.random_valid_trace(rng, w.window, w.n_att, (8,))
    trace = torch.from_numpy(np.ascontiguousarray(
        few[rng.integers(0, 8, size=(w.batch, w.num_q_heads))])).to(dev)
    prob = dsa.Problem(
        q=inputs["q"], k_cache=inputs["k_cache"], v_cache=inputs["v_cache"], strides=inputs["strides"],
        seq_len=seq, prompt_len=inputs["prompt_len"], num_kv_heads=w.num_kv_heads,
        max_seq_len=inputs["max_seq_len"], max_prompt_len=w.prompt_len, block_table=inputs["block_table"],
        block_size=inputs["block_size"], num_blocks=inputs["block_table"].numel())
    out, lse = dsa.alloc_outputs(prob)
    res = {"batch": w.batch, "window": w.window, "n_att": w.n_att, "mask": "per-head list"}
    for name, sel in (("without_select", False), ("with_select", True)):
        diag = dsa.Diag(dsa.DSA_MASK_LIST, w.window, w.n_att, skip_offsets=trace, select=sel)
        ws = dsa.alloc_workspace(prob, diag)
        secs, _ = time_calls(torch, lambda: dsa.dsa_decode_attention_sparse(prob, diag, out, lse, ws), 50, 5)
        res[name + "_us"] = round(secs / 50 * 1e6, 2)
    res["overhead_pct"] = round(100.0 * (res["with_select_us"] / res["without_select_us"] - 1.0), 2)
    return res


def mask_variants(torch, dsa, synth, dev, peak):
    """The mask variants of the paper's comparison at one attention budget (Section 5: sliding
    window, StreamingLLM, diagonal, diagonal + 4 sinks; here N_att = 208 of window 512 on the paged
    batch-256 workload), from the same kernel: time and bandwidth on the rows each one keeps."""
    w = synth.workload(5, batch=256)
    inputs = synth.make_inputs_device(w, dev)
    prob = dsa.Problem(
        q=inputs["q"], k_cache=inputs["k_cache"], v_cache=inputs["v_cache"], strides=inputs["strides"],
        seq_len=inputs["seq_len"], prompt_len=inputs["prompt_len"], num_kv_heads=w.num_kv_heads,
        max_seq_len=inputs["max_seq_len"], max_prompt_len=w.prompt_len, block_table=inputs["block_table"],
        block_size=inputs["block_size"], num_blocks=inputs["block_table"].numel())
    out, lse = dsa.alloc_outputs(prob)
    n = w.n_att
    cases = [
        ("sliding_window", dsa.Diag(dsa.DSA_MASK_WINDOW, n)),
        ("streaming_llm_4_sinks", dsa.Diag(dsa.DSA_MASK_WINDOW, n - 4, n_sink=4)),
        ("diagonal_grid", dsa.Diag(dsa.DSA_MASK_GRID, w.window, n, w.grid_w, w.row_extra)),
        ("diagonal_grid_4_sinks", dsa.Diag(dsa.DSA_MASK_GRID, w.window, n - 4, w.grid_w, w.row_extra, n_sink=4)),
    ]
    res = {"batch": w.batch, "n_att": n, "window": w.window}
    row_bytes = w.num_kv_heads * w.head_dim * 2 * 2
    for name, diag in cases:
        ws = dsa.alloc_workspace(prob, diag)
        _, cnt = dsa.dsa_debug_kept_indices(prob, diag, 0)
        kept = int(cnt.sum().item())
        secs, _ = time_calls(torch, lambda: dsa.dsa_decode_attention_sparse(prob, diag, out, lse, ws), 50, 5)
        t = secs / 50
        res[name] = {"us": round(t * 1e6, 2), "kept_rows_mean": round(kept / w.batch, 1),
                     "GBs": round(kept * row_bytes / t / 1e9, 1), "frac_of_peak": round(kept * row_bytes / t / 1e9 / peak, 4)}
    return res


def decode_loop_bench(torch, dsa, synth, dev, n_layers=8, batch=16,
                      modes=("dense", "sparse", "sparse_select", "dense_two_calls", "sparse_two_calls"),
                      plan_flags=0):
    """Whole-image decode loop: 1024 image tokens after a 50-token prompt, `batch` requests (16: the
    shape of the paper's Lumina-mGPT latency runs), 32/32 heads, head_dim 128, over `n_layers`
    layers, each with its own KV cache (together larger than the L2).  Every step appends the new
    token's K/V and attends, layer after layer: one fused dsa_decode_step per layer, the layers
    sharing one seq_len array that is advanced once per token ("_two_calls" modes: dsa_append_kv +
    attention per layer instead); layers 2 ... n of a token carry DSA_PLAN_METADATA_STABLE.  The step is captured once as a CUDA graph and replayed 1024
    times.  Sparse: bounded ring cache, window 512, N_att 52 (95 % sparsity), grid mask.  Dense:
    full linear cache."""
    b, h, d, l_p, grid = batch, 32, 128, 50, 32
    steps = grid * grid
    s_max = l_p + steps
    row = h * d
    gen = torch.Generator(device=dev)
    gen.manual_seed(synth.BASE_SEED + 77)
    res = {"batch": b, "heads": h, "head_dim": d, "prompt_len": l_p, "image_tokens": steps, "layers": n_layers}
    # "sparse": grid-derived diagonals (no selection work); "sparse_select": the paper's own method,
    # per-head list masks grown step by step by the fused phase-2 selection (argmin) in the call
    # "_two_calls": dsa_append_kv + attention per layer (each layer advancing its own seq_len);
    # otherwise the fused dsa_decode_step per layer and one dsa_advance_seq_len per token
    for mode in modes:
        fused = not mode.endswith("_two_calls")
        kind = mode.replace("_two_calls", "")
        ring = 0 if kind == "dense" else 512
        cap = l_p + ring if ring else s_max
        diag = dsa.Diag(dsa.DSA_MASK_GRID, 512, 52, grid, 0) if kind == "sparse" else None
        q = torch.randn((b, h, d), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
        k_new, v_new = q.clone(), q.clone()
        shared_seq = torch.full((b,), l_p, dtype=torch.int32, device=dev)
        layers = []
        for index in range(n_layers):
            kc = torch.randn((b, cap, h, d), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
            vc = torch.randn((b, cap, h, d), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
            seq = shared_seq if fused else torch.full((b,), l_p, dtype=torch.int32, device=dev)
            pl = torch.full((b,), l_p, dtype=torch.int32, device=dev)
            # Every fused step but a token's first follows another layer's step, which writes neither the
            # lengths nor a skip list of this layer: those calls carry the promise that lets the kernel
            # build its row list before it waits for the launch in front of it.  (The first layer follows
            # dsa_advance_seq_len, which writes seq_len.)
            promise = dsa.DSA_PLAN_METADATA_STABLE if (fused and index > 0) else 0
            prob = dsa.Problem(q=q, k_cache=kc.view(-1), v_cache=vc.view(-1), strides=(cap * row, row, d),
                               seq_len=seq, prompt_len=pl, num_kv_heads=h, max_seq_len=s_max,
                               max_prompt_len=l_p, ring_size=ring, plan_flags=plan_flags | promise)
            out, lse = dsa.alloc_outputs(prob)
            ldiag = diag
            if kind == "sparse_select":
                # the lists and their bitmap form (dsa_diag_params.skip_bitmap), both grown by the selection
                trace = torch.zeros((b, h, 512 - 52), dtype=torch.int32, device=dev)
                bitmap = torch.zeros((b, h, 512 // 32), dtype=torch.int32, device=dev)
                ldiag = dsa.Diag(dsa.DSA_MASK_LIST, 512, 52, skip_offsets=trace, select=True, skip_bitmap=bitmap)
            layers.append((prob, out, lse, dsa.alloc_workspace(prob, ldiag), ldiag))

        def step():
            for prob, out, lse, ws, ldiag in layers:
                if fused:
                    dsa.dsa_decode_step(prob, ldiag, k_new, v_new, out, lse, ws)
                    continue
                dsa.dsa_append_kv(prob, k_new, v_new, advance=True)
                if ldiag is None:
                    dsa.dsa_decode_attention_dense(prob, out, lse, ws)
                else:
                    dsa.dsa_decode_attention_sparse(prob, ldiag, out, lse, ws)
            if fused:
                dsa.dsa_advance_seq_len(shared_seq, s_max)

        def reset(value):
            for prob, _, _, _, ldiag in layers:
                prob.seq_len.fill_(value)
                if value == l_p and ldiag is not None and ldiag.skip_bitmap is not None:
                    ldiag.skip_offsets.zero_()             # the image starts over: empty lists, empty bitmaps
                    ldiag.skip_bitmap.zero_()

        step()                                             # eager warm-up (one-time kernel set-up)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
        best = None
        for _ in range(3):
            reset(l_p)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(steps):
                graph.replay()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
            best = ms if best is None else min(best, ms)
        assert int(layers[0][0].seq_len[0].item()) == s_max
        # the last step alone (the paper's per-step breakdown is taken there)
        reps, last = 20, 0.0
        for _ in range(reps):
            reset(s_max - 1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            graph.replay()
            e1.record()
            torch.cuda.synchronize()
            last += e0.elapsed_time(e1)
        plan = dsa.dsa_query_plan(layers[0][0], layers[0][4])
        cache_gb = n_layers * 2 * b * cap * row * 2 / 1e9
        res[mode] = {"ms_per_image": round(best, 3), "us_per_step": round(best / steps * 1e3, 2),
                     "us_per_layer_step": round(best / steps / n_layers * 1e3, 2),
                     "us_last_step": round(last / reps * 1e3, 2), "cache_GB": round(cache_gb, 3),
                     "n_split": plan.n_split, "heads_per_block": plan.heads_per_block,
                     "launches_per_layer_step": plan.launches + (0 if fused else 1)}
        del layers, graph
        torch.cuda.empty_cache()
    if "sparse_select" in res:
        res["speedup_per_image_with_selection"] = round(
            res["dense"]["ms_per_image"] / res["sparse_select"]["ms_per_image"], 3)
    res["speedup_per_image"] = round(res["dense"]["ms_per_image"] / res["sparse"]["ms_per_image"], 3)
    res["speedup_last_step"] = round(res["dense"]["us_last_step"] / res["sparse"]["us_last_step"], 3)
    res["cache_ratio"] = round(res["dense"]["cache_GB"] / res["sparse"]["cache_GB"], 3)
    res["ideal_last_step_byte_ratio"] = round((l_p + steps) / (l_p + 52), 3)
    return res


def run_ours(args):
    import torch
    from paper_2609_19702_b200 import build as cuda_build
    cuda_build.build()
    from paper_2609_19702_b200 import binding as dsa, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()

    w = synth.workload(args.config, batch=args.batch, window=args.window, n_att=args.n_att)
    inputs = synth.make_inputs_device(w, dev, seed=synth.BASE_SEED + w.index + 1000 * rank)
    host = inputs["host"]

    def problem(split_tokens=0):
        return dsa.Problem(
            q=inputs["q"], k_cache=inputs["k_cache"], v_cache=inputs["v_cache"], strides=inputs["strides"],
            seq_len=inputs["seq_len"], prompt_len=inputs["prompt_len"], num_kv_heads=w.num_kv_heads,
            max_seq_len=inputs["max_seq_len"], max_prompt_len=w.prompt_len,
            block_table=inputs["block_table"], block_size=inputs["block_size"],
            num_blocks=0 if inputs["block_table"] is None else inputs["block_table"].numel(),
            split_tokens=split_tokens, plan_flags=args.plan_flags)

    prob = problem(args.split_tokens)
    out, lse = dsa.alloc_outputs(prob)

    def make_call(mode, ww):
        diag = None if mode == "dense" else dsa.Diag(dsa.DSA_MASK_GRID, ww.window, ww.n_att, ww.grid_w, ww.row_extra)
        ws = dsa.alloc_workspace(prob, diag)
        plan = dsa.dsa_query_plan(prob, diag)
        if diag is None:
            return (lambda: dsa.dsa_decode_attention_dense(prob, out, lse, ws)), plan, diag
        return (lambda: dsa.dsa_decode_attention_sparse(prob, diag, out, lse, ws)), plan, diag

    call, plan, diag = make_call(args.mode, w)

    # ---- algorithmic bytes of one step (rank-local; also decides how L2 is kept out of the timing)
    idx, cnt = dsa.dsa_debug_kept_indices(prob, diag, inputs["max_seq_len"])
    torch.cuda.synchronize()
    if inputs["block_table"] is not None:
        valid = torch.arange(idx.shape[2], device=dev)[None, None, :] < cnt[:, :, None]
        blk = torch.where(valid, idx // inputs["block_size"], -1)
        blocks_touched = sum(int(torch.unique(blk[i][blk[i] >= 0]).numel()) for i in range(blk.shape[0]))
    else:
        blocks_touched = 0
    del idx
    abytes, kept_rows = algorithmic_bytes(w, host, args.mode, blocks_touched)

    # ---- the timed step ------------------------------------------------------------------
    # One timed region is EXACTLY args.steps calls between two events.  A region of 20 steps lasts
    # 5 ms, too short for the clock sampler, so the region is repeated (each repeat bracketed the same
    # way) until 150 ms have been timed and the MEDIAN region is reported; the sampler runs across
    # all repeats.
    sampler = ClockSampler(local_rank)
    flush_l2 = abytes < 2 * L2_BYTES
    flush = torch.empty(4 * L2_BYTES, dtype=torch.uint8, device=dev) if flush_l2 else None
    if flush_l2:
        l2_note = ("working set (%.3f GB per step) would stay in the %d MB L2: a %d MB write precedes every timed "
                   "call and only the calls are timed" % (abytes / 1e9, L2_BYTES >> 20, 4 * L2_BYTES >> 20))
    else:
        l2_note = "inputs larger than L2: each step reads %.2f GB of distinct K/V" % (abytes / 1e9)

    def region(warmup):
        if flush_l2:
            return time_calls_flushed(torch, call, args.steps, warmup, flush, None, barrier)[0]
        return time_calls(torch, call, args.steps, warmup, None, barrier)[0]

    first = region(args.warmup)                            # (also the warm-up of the repeats)
    repeats = int(min(200, max(1, np.ceil(0.15 / max(first, 1e-6)))))
    sampler.start()
    regions = [region(0) for _ in range(repeats)]
    clocks = sampler.stop()
    regions_max = torch.tensor(regions, dtype=torch.float64, device=dev)
    if dist is not None:
        dist.all_reduce(regions_max, op=dist.ReduceOp.MAX)  # per repeat: the slowest rank
    secs = float(np.median(regions))                       # this rank (roofline of its own launches)
    secs_max = float(regions_max.median().item())
    ms_per_step = secs_max / args.steps * 1e3
    value = aggregate_value(world, w.batch, args.steps, [secs_max])
    del flush

    # ---- roofline of the attention kernel (rank-local numbers) ----------------------------
    peak, peak_kind = measured_peak()
    peak_gbs = peak
    launch_secs = secs / args.steps                       # one attention launch (+ combine) per step
    achieved = abytes / launch_secs / 1e9
    name = workload_name(w, args.mode)
    roofline = {"bound": "hbm", "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                "frac": round(achieved / peak, 4), "traffic": NCU_TRAFFIC_BYTES.get(name),
                "peak_kind": "of " + peak_kind, "algorithmic_bytes": abytes,
                "frac_of_nominal_8TBs": round(achieved / NOMINAL_HBM_GBS, 4),
                "kernel": kernel_name(plan) + (" + dsa_combine_kernel" if plan.launches > 1 else "")}

    # ---- the launch's own speed of light: the same call with the arithmetic taken out (same grid, same
    # row lists, same K / V tiles staged through the same rings; dsa_debug_copy_only), timed in regions
    # that alternate with regions of the real call so that clock drift hits both alike
    if plan.block_warps == 4 and not plan.per_head_lists and not flush_l2 and world == 1:
        ws_copy = dsa.alloc_workspace(prob, diag)

        def copy_call():
            dsa.dsa_debug_copy_only(prob, diag, out, lse, ws_copy)

        real_t, copy_t = [], []
        time_calls(torch, copy_call, args.steps, 3, None, barrier)
        for _ in range(5):
            real_t.append(time_calls(torch, call, args.steps, 0, None, barrier)[0])
            copy_t.append(time_calls(torch, copy_call, args.steps, 0, None, barrier)[0])
        c_secs, r_secs = float(np.median(copy_t)) / args.steps, float(np.median(real_t)) / args.steps
        roofline["copy_only"] = {"ms_per_launch": round(c_secs * 1e3, 5), "GBs": round(abytes / c_secs / 1e9, 1),
                                 "attention_ms_in_the_same_regions": round(r_secs * 1e3, 5),
                                 "attention_over_copy_only": round(r_secs / c_secs, 4),
                                 "note": "the same launch without the arithmetic (plain four-warp head-group "
                                         "kernel with the plan's grid): lists built, tiles staged and read once"}
        call()                                              # (out / lse hold the attention result again)
        torch.cuda.synchronize()

    # ---- the same step as a single call with a cold L2 (launch latency and first misses included)
    iso_flush = torch.empty(4 * L2_BYTES, dtype=torch.uint8, device=dev)
    iso_med, iso_min = time_flushed(torch, call, iso_flush, iters=30, warmup=3)
    del iso_flush

    # ---- variants: dense, the other window, and the paper's per-head list masks; same library,
    # same batch, timed like the step
    variants = {}
    if not args.no_variants and args.mode == "sparse":
        vsteps = max(5, args.steps // 4)

        def time_variant(vcall, vbytes):
            if vbytes < 2 * L2_BYTES:                       # same rule as the timed step
                vflush = torch.empty(4 * L2_BYTES, dtype=torch.uint8, device=dev)
                vsecs, _ = time_calls_flushed(torch, vcall, vsteps, 3, vflush)
                del vflush
            else:
                vsecs, _ = time_calls(torch, vcall, vsteps, 3)
            return vsecs / vsteps

        todo = [("dense", w)]
        if w.index == 5:
            todo.append(("sparse", synth.workload(5, batch=w.batch, window=1024, n_att=416)))
        for mode, ww in todo:
            vcall, vplan, _ = make_call(mode, ww)
            vb, _ = algorithmic_bytes(ww, host, mode, 0)
            vt = time_variant(vcall, vb)
            key = "dense" if mode == "dense" else "sparse_w%d_a%d" % (ww.window, ww.n_att)
            variants[key] = {"ms_per_step": round(vt * 1e3, 4), "queries_per_sec": round(w.batch / vt, 1),
                             "achieved_GBs": round(vb / vt / 1e9, 1), "frac_of_peak": round(vb / vt / 1e9 / peak_gbs, 4),
                             "launches_per_step": vplan.launches, "n_split": vplan.n_split}
        if "dense" in variants:
            variants["sparse_over_dense_speedup"] = round(variants["dense"]["ms_per_step"] / (secs / args.steps * 1e3), 3)
            dense_bytes, _ = algorithmic_bytes(w, host, "dense", 0)
            variants["ideal_byte_ratio"] = round(dense_bytes / abytes, 3)
        # The paper's own setting: one skip list per attention head (random valid traces here), without
        # and with the fused phase-2 selection (which appends the next trace entry of every head whose
        # request is in phase 2).  Same positions, same budget, same kernel family.
        lrng = np.random.default_rng(synth.BASE_SEED + 500 + w.index)
        few = synth.random_valid_trace(lrng, w.window, w.n_att, (8,))
        trace = torch.from_numpy(np.ascontiguousarray(
            few[lrng.integers(0, 8, size=(w.batch, w.num_q_heads))])).to(dev)
        group = w.num_q_heads // w.num_kv_heads
        words = (w.window + 31) // 32
        bitmap = torch.zeros((w.batch, w.num_q_heads, words), dtype=torch.int32, device=dev)
        for key, sel, bm in (("list_per_head", False, None), ("list_per_head_select", True, None),
                             ("list_per_head_bitmap", False, bitmap), ("list_per_head_bitmap_select", True, bitmap)):
            ldiag = dsa.Diag(dsa.DSA_MASK_LIST, w.window, w.n_att, skip_offsets=trace, select=sel, skip_bitmap=bm)
            if bm is not None:
                dsa.dsa_build_skip_bitmap(prob, ldiag)      # (the lists as they stand now, as bits)
            lws = dsa.alloc_workspace(prob, ldiag)
            lplan = dsa.dsa_query_plan(prob, ldiag)
            lmask = {"mask_heads": w.num_q_heads, "union_rows": None, "bitmap_words": words if bm is not None else 0}
            if group > 1:
                lidx, lcnt = dsa.dsa_debug_kept_indices(prob, ldiag, inputs["max_seq_len"])
                lmask["union_rows"] = union_rows(lidx.cpu().numpy(), lcnt.cpu().numpy(), group)
            lb, _ = algorithmic_bytes(w, host, "sparse", blocks_touched, lmask)
            lt = time_variant(lambda: dsa.dsa_decode_attention_sparse(prob, ldiag, out, lse, lws), lb)
            variants[key] = {"ms_per_step": round(lt * 1e3, 4), "queries_per_sec": round(w.batch / lt, 1),
                             "algorithmic_bytes": lb, "achieved_GBs": round(lb / lt / 1e9, 1),
                             "frac_of_peak": round(lb / lt / 1e9 / peak_gbs, 4),
                             "launches_per_step": lplan.launches, "n_split": lplan.n_split}

    # ---- end to end: per-step inputs from pinned host memory, result back to the host ------
    e2e = None
    if not args.no_e2e:
        h_q = inputs["q"].cpu().pin_memory()
        h_seq = inputs["seq_len"].cpu().pin_memory()
        h_pl = inputs["prompt_len"].cpu().pin_memory()
        h_bt = None if inputs["block_table"] is None else inputs["block_table"].cpu().pin_memory()
        h_out = torch.empty(out.shape, dtype=out.dtype).pin_memory()
        h_lse = torch.empty(lse.shape, dtype=lse.dtype).pin_memory()
        e2e_ws = dsa.alloc_workspace(prob, diag)

        def e2e_step():
            # the C-ABI call with host buffers: lengths and block table copied up, q read from and
            # out / lse written to the pinned host buffers by the kernels themselves
            dsa.dsa_decode_attention_host_mapped(prob, diag, h_q, h_seq, h_pl, h_bt, h_out, h_lse, e2e_ws)
            torch.cuda.current_stream().synchronize()      # the caller needs the result to go on

        def e2e_step_copies():
            # same step with every transfer as an explicit copy before / after the kernels
            dsa.dsa_decode_attention_host_io(prob, diag, h_q, h_seq, h_pl, h_bt, out, lse, h_out, h_lse, e2e_ws)
            torch.cuda.current_stream().synchronize()

        def warm(fn, seconds=0.5):
            # The host link leaves its idle state only under traffic: the first few hundred steps
            # after a pause run 30-40 % slower than the steady state (measured), so warm up by time.
            t0 = time.perf_counter()
            while time.perf_counter() - t0 < seconds:
                fn()

        esteps = min(args.steps, 100)
        warm(e2e_step)
        esecs, _ = time_calls(torch, e2e_step, esteps, 3, None, barrier)
        warm(e2e_step_copies)
        csecs, _ = time_calls(torch, e2e_step_copies, esteps, 3, None, barrier)
        te = torch.tensor([esecs, csecs], dtype=torch.float64, device=dev)
        if dist is not None:
            dist.all_reduce(te, op=dist.ReduceOp.MAX)
        h2d = sum(x.numel() * x.element_size() for x in (h_q, h_seq, h_pl) + ((h_bt,) if h_bt is not None else ()))
        d2h = h_out.numel() * h_out.element_size() + h_lse.numel() * h_lse.element_size()
        e2e = {"value": round(world * w.batch * esteps / float(te[0].item()), 1), "unit": UNIT,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": esteps,
               "warmup": "0.5 s of untimed steps, then 3",
               "with_explicit_copies": round(world * w.batch * esteps / float(te[1].item()), 1),
               "note": "dsa_decode_attention_host_mapped per step: seq_len, prompt_len and block table copied "
                       "from pinned host memory, q read from and out / lse written to pinned host memory by "
                       "the kernels, stream synchronised; with_explicit_copies = dsa_decode_attention_host_io "
                       "(every transfer a copy); the KV cache is decode state and stays resident in HBM"}

    # ---- CPU baseline: the oracle on a bounded sample of the same workload ------------------
    cpu = None
    if not args.no_cpu_baseline and rank == 0 and world == 1:
        cpu = oracle_baseline(synth, inputs, w, args.mode)

    per_config = decode_loop = decode_loop_large = selection = masks = None
    if rank == 0 and world == 1 and (not args.no_per_config or not args.no_decode_loop or args.all_configs):
        del inputs, prob, out, lse
        torch.cuda.empty_cache()
        if not args.no_per_config:
            per_config = per_config_table(torch, dsa, synth, dev, peak, plan_flags=args.plan_flags)
        if not args.no_decode_loop or args.all_configs:
            # the paper's own shape at a batch where a B200 step is bandwidth-bound: grid-derived diagonals
            # ("sparse") and the paper's method, per-head lists grown by the fused selection ("sparse_select")
            decode_loop_large = decode_loop_bench(torch, dsa, synth, dev, batch=128,
                                                  modes=("dense", "sparse", "sparse_select"),
                                                  plan_flags=args.plan_flags)
        if args.all_configs:
            decode_loop = decode_loop_bench(torch, dsa, synth, dev, plan_flags=args.plan_flags)
            selection = selection_overhead(torch, dsa, synth, dev)
            masks = mask_variants(torch, dsa, synth, dev, peak)

    if rank == 0:
        line = {
            "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms_per_step, 5),
            "timed_regions": {"repeats": repeats, "reported": "median region of %d steps" % args.steps,
                              "ms_per_step_min": round(float(regions_max.min().item()) / args.steps * 1e3, 5),
                              "ms_per_step_max": round(float(regions_max.max().item()) / args.steps * 1e3, 5),
                              "ms_per_step_first": round(first / args.steps * 1e3, 5)},
            "isolated_ms": {"median": round(iso_med * 1e3, 5), "min": round(iso_min * 1e3, 5),
                            "note": "one call at a time, a %d MB write before each (cold L2), 30 calls; "
                                    "ms_per_step is back-to-back calls, whose launch latency and prologue "
                                    "overlap the previous call" % (4 * L2_BYTES >> 20)},
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": name, "global_batch": world * w.batch,
                       "kept_rows_per_kv_head_mean": round(kept_rows / w.batch, 1),
                       "l2": l2_note,
                       "parallelism": "requests sharded over %d GPU(s), no collective" % world,
                       "plan": {"split_tokens": plan.split_tokens, "n_split": plan.n_split,
                                "grid_blocks": plan.grid_blocks, "smem_bytes": plan.smem_bytes,
                                "tile_tokens": plan.tile_tokens, "stages": plan.stages,
                                "tensor_cores": plan.tensor_cores, "work_items": plan.work_items,
                                "item_warps": plan.item_warps, "heads_per_block": plan.heads_per_block,
                                "block_warps": plan.block_warps, "per_head_lists": plan.per_head_lists,
                                "cluster_blocks": plan.cluster_blocks, "tensor_map_copies": plan.tensor_map_copies,
                                "producer_warps": plan.producer_warps, "plan_flags": args.plan_flags}},
            "clocks": clocks, "e2e": e2e, "gpu_launches": plan.launches * args.steps,
            "roofline": roofline, "cpu_baseline": cpu, "variants": variants,
        }
        if per_config is not None:
            line["per_config"] = per_config
        if decode_loop_large is not None:
            line["decode_loop_batch128"] = decode_loop_large
        if decode_loop is not None:
            line["decode_loop"] = decode_loop
            line["selection_overhead"] = selection
            line["mask_variants"] = masks
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def oracle_baseline(synth, inputs, w, mode, sample=16, min_seconds=10.0):
    """Time the float64 oracle, as it stands, on the first `sample` requests of this batch."""
    from oracle import oracle as ora
    n = min(sample, w.batch)
    sub = synth.host_subset(inputs, range(n))
    kw = dict(num_kv_heads=w.num_kv_heads, strides=sub["strides"], block_table=sub["block_table"],
              block_size=sub["block_size"])
    if mode == "dense":
        kw.update(mode=ora.MODE_DENSE)
    else:
        kw.update(mode=ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride_grid=w.stride)
    def timed(seconds, **extra):
        reps, t0 = 0, time.perf_counter()
        while True:
            ora.decode(sub["q"], sub["k_cache"], sub["v_cache"], sub["seq_len"], sub["prompt_len"], **kw, **extra)
            reps += 1
            el = time.perf_counter() - t0
            if el >= seconds or reps >= 1000:
                return reps, el

    reps, el = timed(min_seconds)                         # all host threads (OpenMP over request x head)
    reps1, el1 = timed(min_seconds / 4, n_threads=1)      # and one thread, for the per-core rate
    return {"value": round(n * reps / el, 2), "unit": UNIT, "cores": ora.num_threads(), "kind": "oracle",
            "sample": "first %d requests of the batch, %d repetitions, %.1f s" % (n, reps, el),
            "single_thread_value": round(n * reps1 / el1, 2)}


def run_reference(args):
    """The reference arm: the float64 CPU oracle on the same workload, metric and unit; each step
    is one oracle call on a bounded sample of requests.  Rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import oracle as ora
    from paper_2609_19702_b200 import synth
    sample = 4
    w_full = synth.workload(args.config, batch=args.batch, window=args.window, n_att=args.n_att)
    w = synth.workload(args.config, batch=sample, window=args.window, n_att=args.n_att)
    inp = synth.make_inputs(w)
    kw = dict(num_kv_heads=w.num_kv_heads, strides=inp["strides"], block_table=inp["block_table"],
              block_size=inp["block_size"])
    if args.mode == "dense":
        kw.update(mode=ora.MODE_DENSE)
    else:
        kw.update(mode=ora.MODE_GRID, n_r=w.window, n_att=w.n_att, stride_grid=w.stride)

    def step():
        ora.decode(inp["q"], inp["k_cache"], inp["v_cache"], inp["seq_len"], inp["prompt_len"], **kw)

    steps = min(args.steps, 50)
    for _ in range(min(args.warmup, 3)):
        step()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    el = time.perf_counter() - t0
    value = round(sample * steps / el, 2)
    cpu = {"value": value, "unit": UNIT, "cores": ora.num_threads(), "kind": "oracle",
           "sample": "%d requests of the workload per step, %d steps" % (sample, steps)}
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": min(args.warmup, 3), "ms_per_step": round(el / steps * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": workload_name(w_full, args.mode) + " (%d-request sample per step)" % sample},
        "cpu_baseline": cpu,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
