"""Multi-rank host logic on CPU (gloo, world size 2): requests are independent units, so ranks
own disjoint request shards, run the same per-rank work with no collective on the data path, and
only the timing (maximum over ranks) and the final gather of results cross ranks."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import oracle as ora
from paper_2609_19702_b200 import synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, batch, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = synth.Workload("dist", 50, batch, 4, 2, 64, 5, 6, 6, 1, 16, 5, 1, 42, paged=True, block_size=8)
        inp = synth.make_inputs(w)                         # every rank draws the same global batch
        mine = list(synth.shard_requests(batch, world, rank))
        kw = dict(num_kv_heads=2, strides=inp["strides"], block_size=8, mode=ora.MODE_GRID,
                  n_r=w.window, n_att=w.n_att, stride_grid=w.stride)
        r = ora.decode(inp["q"][mine], inp["k_cache"], inp["v_cache"], inp["seq_len"][mine],
                       inp["prompt_len"][mine], block_table=inp["block_table"][mine], **kw)
        # gather the shards (the only exchange the path has) and compare with the unsharded run
        parts = [None] * world
        dist.all_gather_object(parts, (mine, r["out"]))
        t = torch.tensor([0.001 * (rank + 1)], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)             # timing rule: maximum over ranks
        if rank == 0:
            full = ora.decode(inp["q"], inp["k_cache"], inp["v_cache"], inp["seq_len"],
                              inp["prompt_len"], block_table=inp["block_table"], **kw)
            got = np.zeros_like(full["out"])
            seen = []
            for ids, o in parts:
                got[ids] = o
                seen += ids
            ret["ok"] = bool(np.array_equal(got, full["out"])) and sorted(seen) == list(range(batch))
            ret["tmax"] = float(t.item())
    finally:
        dist.destroy_process_group()


def test_request_sharding_world_size_2():
    batch = 7
    with mp.Manager() as mgr:
        ret = mgr.dict()
        port = _free_port()
        mp.spawn(_worker, args=(2, port, batch, ret), nprocs=2, join=True)
        assert ret["ok"] is True
        assert abs(ret["tmax"] - 0.002) < 1e-12


def test_shards_partition_the_batch():
    for batch in (0, 1, 7, 256):
        for world in (1, 2, 3, 8):
            ids = [i for r in range(world) for i in synth.shard_requests(batch, world, r)]
            assert ids == list(range(batch))
            sizes = [len(synth.shard_requests(batch, world, r)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
