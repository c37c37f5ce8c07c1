"""Rank plumbing of the benchmark on CPU: two gloo ranks.  The data path has no
exchange step (every rank runs its own seeded batch); only the timing is
reduced (max over ranks) behind a barrier."""
import os
import socket
import sys

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


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, rank, world)
    bench.barrier()
    t = bench.reduce_max(10.0 + rank, backend_device="cpu")          # slowest rank decides
    seeds = [None] * world
    dist.all_gather_object(seeds, bench.rank_seed(7, rank))
    # whole-job value = units of all ranks / max time
    value = world * 100 / t
    q.put((rank, t, seeds, value))
    dist.destroy_process_group()


def test_two_gloo_ranks_reduce_timing_and_draw_distinct_batches():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, t, seeds, value in res:
        assert t == 11.0                                   # max over ranks
        assert len(set(seeds)) == world                    # each rank has its own batch
        assert abs(value - world * 100 / 11.0) < 1e-12


def test_single_process_helpers_are_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max(3.5, backend_device="cpu") == 3.5
    bench.barrier()
    from paper_2607_16339_b200.workloads import WORKLOADS
    c = bench.flops_and_bytes(WORKLOADS[2])
    # hand count at the LLaDA-8B shape (N = 768, L_b = 32, 32 heads x 128): a step is 4 d Hq L_b (2N - L_b)
    # = 0.789 GFLOP, a build 4 d Hq (N - L_b)^2 = 8.88 GFLOP
    assert abs(c["step_flops"] / 1e9 - 0.789) < 0.002 and abs(c["build_flops"] / 1e9 - 8.88) < 0.01
    assert abs(c["step_bytes"] / 1e6 - 45.0) < 0.5
