"""The N > 1 path on CPU: two gloo ranks shard a workload's independent units (rows of an MLP chain) with no
data-path collective, run the oracle on their shard, and combine timing the way bench.py does (barrier, max
over ranks).  Checks that the shards tile the full result exactly and that the reduction plumbing works."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    from oracle import interp
    from paper_2301_01333_b200 import workloads as W
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    full = W.mlp_int8(batch=16, dims=(30, 32, 16, 1), final="none")
    rows = np.array_split(np.arange(16), world)[rank]            # batch rows are independent units
    shard = W.mlp_int8(batch=len(rows), dims=(30, 32, 16, 1), final="none")
    for a, b in zip(shard.graph.inputs, full.graph.inputs):
        shard.feeds[a] = full.feeds[b][rows] if a == shard.graph.inputs[0] else full.feeds[b]
    dist.barrier()
    out = interp.run(shard.graph, shard.feeds)[shard.graph.outputs[0]]
    dist.barrier()
    t = torch.tensor([float(rank + 1)], dtype=torch.float64)     # stand-in for this rank's elapsed time
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    units = torch.tensor([float(len(rows))], dtype=torch.float64)
    dist.all_reduce(units, op=dist.ReduceOp.SUM)
    np.save(os.path.join(out_dir, f"out{rank}.npy"), out)
    if rank == 0:
        np.save(os.path.join(out_dir, "meta.npy"), np.array([t.item(), units.item()]))
    dist.destroy_process_group()


def test_two_rank_sharding_has_no_exchange_step(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    sys.path.insert(0, ROOT)
    from oracle import interp
    from paper_2301_01333_b200 import workloads as W
    full = W.mlp_int8(batch=16, dims=(30, 32, 16, 1), final="none")
    ref = interp.run(full.graph, full.feeds)[full.graph.outputs[0]]
    got = np.concatenate([np.load(tmp_path / f"out{r}.npy") for r in range(world)], axis=0)
    assert np.array_equal(got, ref)                               # shards tile the full result bit for bit
    t_max, units = np.load(tmp_path / "meta.npy")
    assert t_max == 2.0 and units == 16.0                        # max over ranks; whole-job unit count
