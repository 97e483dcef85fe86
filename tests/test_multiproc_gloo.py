"""The N > 1 path on CPU.  Two gloo ranks run the rank plumbing the benchmark uses on GPUs (`paper_2301_01333_b200.multi`:
process-group set-up from the torchrun environment, build on the local root, barrier-bracketed timed region, maximum
over ranks, whole-job totals) with a stub step, split one batch the way `bench.py --split` does, run the oracle on
their shard and check that the shards tile the full result exactly: the path has no exchange step."""
import os
import socket
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    from oracle import interp
    from paper_2301_01333_b200 import multi
    from paper_2301_01333_b200 import workloads as W
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    ranks = multi.init_ranks("gloo")
    assert (ranks.rank, ranks.world, ranks.backend) == (rank, world, "gloo")
    built = []
    multi.build_on_local_root(ranks, lambda: built.append(rank))      # only local rank 0 "builds"
    assert built == ([0] if rank == 0 else [])
    full = W.mlp_int8(batch=16, dims=(30, 32, 16, 1), final="none")
    first, count = multi.split_units(16, world, rank)                  # batch rows are independent units
    shard = W.mlp_int8(batch=count, dims=(30, 32, 16, 1), final="none")
    for a, b in zip(shard.graph.inputs, full.graph.inputs):
        shard.feeds[a] = full.feeds[b][first:first + count] if a == shard.graph.inputs[0] else full.feeds[b]
    result = {}

    def run_steps():                                                   # the stub step: the oracle on this rank's shard
        result["out"] = interp.run(shard.graph, shard.feeds)[shard.graph.outputs[0]]
        return float(rank + 1)                                         # stand-in for this rank's device time in ms

    ms = multi.timed_region(ranks, run_steps)
    job = multi.job_line_fields(ranks, float(count), ms)
    np.save(os.path.join(out_dir, f"out{rank}.npy"), result["out"])
    if ranks.is_root:
        np.save(os.path.join(out_dir, "meta.npy"), np.array([ms, job["units_total"], job["units_per_s"]]))
    multi.finish(ranks)


def test_two_rank_sharding_has_no_exchange_step(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    from oracle import interp
    from paper_2301_01333_b200 import workloads as W
    full = W.mlp_int8(batch=16, dims=(30, 32, 16, 1), final="none")
    ref = interp.run(full.graph, full.feeds)[full.graph.outputs[0]]
    got = np.concatenate([np.load(tmp_path / f"out{r}.npy") for r in range(world)], axis=0)
    assert np.array_equal(got, ref)                               # shards tile the full result bit for bit
    t_max, units, rate = np.load(tmp_path / "meta.npy")
    assert t_max == 2.0 and units == 16.0                         # max over ranks; whole-job unit count
    assert rate == 16.0 / 2e-3


def test_single_process_plumbing_is_a_no_op():
    from paper_2301_01333_b200 import multi
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    r = multi.init_ranks("gloo")
    assert (r.rank, r.world, r.backend) == (0, 1, None) and r.is_root
    multi.barrier(r)
    assert multi.max_over_ranks(r, 3.5) == 3.5 and multi.sum_over_ranks(r, 2.0) == 2.0
    assert multi.timed_region(r, lambda: 1.25) == 1.25
    multi.finish(r)


def test_even_split_tiles_the_units():
    from paper_2301_01333_b200 import multi
    for total in (8192, 64, 32, 128, 7):
        for world in (1, 2, 3, 4, 8):
            parts = [multi.split_units(total, world, r) for r in range(world)]
            assert parts[0][0] == 0 and sum(c for _, c in parts) == total
            for (f0, c0), (f1, _) in zip(parts, parts[1:]):
                assert f0 + c0 == f1
            assert max(c for _, c in parts) - min(c for _, c in parts) <= 1


def test_per_rank_workloads_of_every_config_tile_the_full_one():
    # what `bench.py --split` gives each rank: the per-unit inputs of the ranks, concatenated, are the full
    # workload's; the constants are replicated; the graphs differ only in the unit count
    from paper_2301_01333_b200 import multi
    from paper_2301_01333_b200 import workloads as W
    for name in ("c1", "c2", "c3", "c4", "c5"):
        full = W.CONFIGS[name]()
        total = W.CONFIG_UNITS[name][2]
        assert full.graph.tensors[full.graph.inputs[0]].dims[0] == total
        world = 4
        shards = [W.shard_config(name, full, *multi.split_units(total, world, r)) for r in range(world)]
        assert sum(s.ops for s in shards) == full.ops
        for pos, tid in enumerate(full.graph.inputs):
            lt = full.graph.tensors[tid]
            parts = [s.feeds[s.graph.inputs[pos]] for s in shards]
            if lt.is_constant:
                assert all(p is full.feeds[tid] for p in parts)
            else:
                assert np.array_equal(np.concatenate(parts, axis=0), full.feeds[tid])
                for s in shards:
                    assert s.graph.tensors[s.graph.inputs[pos]].dims[1:] == lt.dims[1:]
