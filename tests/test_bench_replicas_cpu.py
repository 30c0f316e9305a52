"""The multi-GPU arm of bench.py is "replicas only": ranks share nothing on the data path, the
job's time is the slowest rank's and its work the sum over ranks.  Checked here with two gloo
ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms, units = bench.whole_job(10.0 + 5.0 * rank, 7.0, dist, "cpu")
    out.put((rank, ms, units))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_take_the_slowest_time_and_sum_the_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[0] for g in got] == [0, 1]
    for _, ms, units in got:
        assert ms == 15.0          # MAX over ranks
        assert units == 14.0       # whole-job work


def test_single_process_is_the_identity():
    import bench
    assert bench.whole_job(3.5, 2.0) == (3.5, 2.0)
