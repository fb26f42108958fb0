"""The N > 1 path of bench.py is N independent replicas: no collective on the data path, only a
barrier and a max-over-ranks of the step time.  Checked here with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank)          # rank 1 is the slow replica
    dist.barrier()
    out[rank] = (ms, bench.whole_job_rate(1000.0, world, ms))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_sum_of_work():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, 29731, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, rate = res[0]
    assert ms == 15.0
    assert abs(rate - 2 * 1000.0 / 0.015) < 1e-6


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.whole_job_rate(10.0, 1, 1000.0) == 10.0
    work = torch.tensor([0, 10, 40, 600, 40000, 36]).numpy()
    deg = torch.tensor([0, 3, 5, 40, 9, 5]).numpy()
    w = bench.class_of_rows(work, deg, work)
    assert list(w) == [0, 1, 2, 6, 7, 2]
    # lower-triangle mode classes a light row by its products without the d_i diagonal ones
    w = bench.class_of_rows(work - deg, deg, work)
    assert list(w) == [0, 1, 2, 6, 7, 1]
