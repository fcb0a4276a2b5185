"""N > 1 is "replicas only": every rank runs its own pot and the job's rate is the sum of the ranks'
cycles over the slowest rank's time.  The aggregation is checked with two gloo ranks on CPU."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _rank(rank, world, port, q):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms_local = 100.0 if rank == 0 else 250.0   # rank 1 is slower: its time is the job's time
    rate, ms_step = bench.whole_job_rate(ms_local, 50, world, "cpu")
    dist.barrier()
    q.put((rank, rate, ms_step))
    dist.destroy_process_group()


def test_two_gloo_ranks_report_sum_over_max_time():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29000 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for _, rate, ms_step in got:
        assert rate == pytest.approx(2 * 50 * 1e3 / 250.0)
        assert ms_step == pytest.approx(5.0)


def test_single_rank_needs_no_process_group():
    import bench
    rate, ms_step = bench.whole_job_rate(40.0, 20, 1)
    assert rate == pytest.approx(500.0) and ms_step == pytest.approx(2.0)
