"""The benchmark's N > 1 path on CPU: two gloo ranks, each with its own replica timing; the reported time is
the slowest rank's and the whole-job metric counts one layer per replica and step.  (The path itself has no
collective: replicas only.)"""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = 10.0 + 5.0 * rank                      # rank 1 is slower
    slowest = bench.max_over_ranks(mine, torch.device("cpu"))
    dist.barrier()
    out.put((rank, slowest, bench.per_layer_us(slowest / 4, world)))
    dist.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[1] for g in got] == [15.0, 15.0]
    assert all(abs(g[2] - 15.0 / 4 * 1e3 / 2) < 1e-9 for g in got)


def test_single_process_passes_through():
    import bench
    assert bench.max_over_ranks(3.5, torch.device("cpu")) == 3.5
    assert bench.per_layer_us(2.0, 1) == 2000.0
