"""The N > 1 path is "replicas only": ranks share nothing on the data path; only the timing is reduced
(max over ranks).  Covered here with two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench

    def allmax(x):
        t = torch.tensor([x], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    ms_local = 0.5 + 0.25 * rank          # rank 1 is the slow replica
    dist.barrier()
    ms, mult = bench.aggregate_over_ranks(ms_local, world, allmax)
    layers = 32
    us_per_layer = ms * 1e3 / (layers * mult)
    out.put((rank, ms, mult, us_per_layer))
    dist.destroy_process_group()


def test_two_rank_aggregation_takes_the_slowest_replica():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, mult, us in res:
        assert ms == 0.75 and mult == 2                   # both ranks agree on the job's step time
        assert abs(us - 0.75e3 / 64) < 1e-12               # two replicas: twice the layers per step


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(1.25, 1, None) == (1.25, 1)
