"""The N > 1 path of bench.py on CPU: two gloo ranks.  The path shards layers over ranks with no data-path collective;
what the ranks share is the MAX reduction of their device-measured times and the rule that gives each rank its own layers."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, torch.device("cpu"))
        seeds = [bench.slot_seed(rank, s, 3) for s in range(3)]
        gathered = [None] * world
        dist.all_gather_object(gathered, seeds)
        if rank == 0:
            out.put((ms, gathered))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_time_and_disjoint_layers():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    ms, gathered = out.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert ms == 15.0                                   # the slower rank
    flat = [s for seeds in gathered for s in seeds]
    assert len(set(flat)) == len(flat)                  # no two ranks generate the same layer
    # seeds of the K-like / V-like / appended tensors of a slot (seed, seed + 1, seed + 2) never collide across slots either
    assert all(abs(a - b) >= 3 for i, a in enumerate(flat) for b in flat[i + 1:])


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks(3.5, 1, torch.device("cpu")) == 3.5
