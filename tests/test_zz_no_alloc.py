"""The allocation-free entry point, for callers that may not allocate device memory (a plug-in in a
process whose host application owns the whole GPU memory pool, a loop that cannot afford the
device-wide synchronisation of an allocation) and have no workspace to pass.

It must give exactly what the workspace-based entry point gives, also on a second call that
finds the previous call's leftovers in the shared built-in scratch array.  This file sorts last on
purpose, so that a run stopping at the first failure has already run every other test.
"""
import gc

import numpy as np
import pytest
import torch

from paper_2608_09713_b200 import workloads as W

pytestmark = pytest.mark.gpu


def lower_triangle(B, a):
    d = (torch.from_numpy(a.rowptr).cuda(), torch.from_numpy(a.colidx).cuda(), torch.from_numpy(a.vals).cuda())
    rp, ci, cv, _ = B.tril_syrk(a.m, a.n, *d)
    return rp, ci, cv


def test_no_alloc_rowptr_matches_workspace_entry_point_twice():
    assert torch.cuda.is_available()
    from paper_2608_09713_b200 import binding as B
    # two different matrices back to back: the second call sees the first call's counters
    cases = [W.small(3), W.small(5), W.small(3)]
    for a in cases:
        rp, ci, cv = lower_triangle(B, a)
        ref_rowptr, ref_colidx, _ = B.spsyrk_mirror(a.m, rp, ci, cv)            # existing entry point
        out = torch.full((a.m + 1,), -7, dtype=torch.int64, device="cuda")
        gc.collect()                                                            # no stale tensor is freed in between
        before = torch.cuda.memory_allocated()
        nnz = B.spsyrk_mirror_rowptr_noalloc(a.m, rp, ci, out)
        assert torch.cuda.memory_allocated() <= before                          # nothing taken from torch either
        assert nnz == ref_colidx.numel()
        assert torch.equal(out, ref_rowptr)                                     # integers: exact
        # straight again on the same input
        out2 = torch.empty_like(out)
        assert B.spsyrk_mirror_rowptr_noalloc(a.m, rp, ci, out2) == nnz
        assert torch.equal(out2, ref_rowptr)


def test_no_alloc_rejects_oversize_and_upper_entries():
    from paper_2608_09713_b200 import binding as B
    rp = torch.zeros(2, dtype=torch.int64, device="cuda")
    ci = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(B.SpsyrkError) as e:
        B.spsyrk_mirror_rowptr_noalloc(B.NOALLOC_MAX_ROWS + 1, rp, ci, torch.zeros(B.NOALLOC_MAX_ROWS + 2, dtype=torch.int64, device="cuda"))
    assert e.value.status == 4
    rp = torch.tensor([0, 1, 2], dtype=torch.int64, device="cuda")
    ci = torch.tensor([1, 1], dtype=torch.int32, device="cuda")
    with pytest.raises(B.SpsyrkError) as e:
        B.spsyrk_mirror_rowptr_noalloc(2, rp, ci, torch.zeros(3, dtype=torch.int64, device="cuda"))
    assert e.value.status == 2
    # a decreasing row pointer is reported, not turned into a wrapped row length
    rp = torch.tensor([0, 2, 1, 3], dtype=torch.int64, device="cuda")
    ci = torch.tensor([0, 0, 1], dtype=torch.int32, device="cuda")
    with pytest.raises(B.SpsyrkError) as e:
        B.spsyrk_mirror_rowptr_noalloc(3, rp, ci, torch.zeros(4, dtype=torch.int64, device="cuda"))
    assert e.value.status == 2
    # zero rows
    assert B.spsyrk_mirror_rowptr_noalloc(0, torch.zeros(1, dtype=torch.int64, device="cuda"), ci,
                                          torch.ones(1, dtype=torch.int64, device="cuda")) == 0
