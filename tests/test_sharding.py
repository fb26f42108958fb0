"""The 1-D row distribution: slices of A are all-gathered so that every rank holds A, and the output
rows are cut into ranges that tile [0, m).  Two gloo ranks on CPU."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_2608_09713_b200 import sharding as S, workloads as W
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    a = W.small(3)  # has empty rows and very uneven row lengths
    b = S.row_slice_bounds(a.m, world)
    r0, r1 = b[rank], b[rank + 1]
    rp = torch.from_numpy(a.rowptr[r0:r1 + 1] - a.rowptr[r0])
    ci = torch.from_numpy(a.colidx[a.rowptr[r0]:a.rowptr[r1]])
    va = torch.from_numpy(a.vals[a.rowptr[r0]:a.rowptr[r1]])
    full = S.allgather_csr(a.m, rp, ci, va)
    ok = (np.array_equal(full[0].numpy(), a.rowptr) and np.array_equal(full[1].numpy(), a.colidx)
          and np.array_equal(full[2].numpy(), a.vals))
    out[rank] = (ok, S.rank_rows([0, 5, a.m], rank))
    dist.destroy_process_group()


def test_allgather_rebuilds_a_on_every_rank():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, 29741, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] and res[1][0]
    assert res[0][1][1] == res[1][1][0] == 5 and res[0][1][0] == 0


def test_row_slices_tile_the_matrix():
    sys.path.insert(0, ROOT)
    from paper_2608_09713_b200 import sharding as S
    for m in (0, 1, 7, 100):
        for world in (1, 2, 3, 8):
            b = S.row_slice_bounds(m, world)
            assert b[0] == 0 and b[-1] == m and all(x <= y for x, y in zip(b, b[1:]))
