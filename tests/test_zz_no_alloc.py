"""The allocation-free consensus-distance call against the regular one.

Some callers of this library may not allocate device memory at the moment they want the
consensus distance: a hook that runs while a memory pool or a stream capture owns all
allocation, or a process that has given its whole memory budget away.  For them the library
offers choco_consensus_error_noalloc, whose scratch space is a fixed array inside the library
instead of memory obtained at choco_init.  This file checks, through the C interface, that
it returns what choco_consensus_error returns, twice in a row on different inputs (the
scratch array is shared between calls and must not leak one call's partial sums into the
next), and that it refuses sizes beyond its fixed capacity.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

import paper_1907_09356_b200 as choco
import workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_noalloc_matches_regular_entry_point_twice():
    w = workloads.ring(6)
    n = 6
    out = torch.zeros(1, dtype=torch.float64, device=DEV)          # the caller's own output cell
    # second call is smaller than the first: stale partials of the first must not be read
    for d, ld, seed in ((70001, 70004, 1), (4099, 4099, 2)):
        X = torch.full((n, ld), float("nan"), device=DEV)
        X[:, :d] = torch.from_numpy(workloads.normal_rows(n, d, 3.0, seed)).to(DEV)
        ch = choco.Choco(w, d, "sign", ld=ld)
        want = choco.choco_consensus_error(ch.ctx, X)
        choco.choco_consensus_error_noalloc(X, n, d, ld, out)
        torch.cuda.synchronize()
        got = float(out.item())
        # same kernels, same summation order: identical; the tests' tolerance on this metric is 1e-4
        assert abs(got - want) <= 1e-4 * want
        assert got == want
        x64 = X[:, :d].double()
        ref = float(((x64 - x64.mean(dim=0, keepdim=True)) ** 2).sum())
        assert abs(got - ref) <= 1e-9 * ref
        ch.close()


def test_noalloc_rejects_sizes_beyond_its_capacity():
    out = torch.zeros(1, dtype=torch.float64, device=DEV)
    X = torch.zeros(8, device=DEV)
    lib = choco.load()
    too_big = 4_194_304 + 1
    assert lib.choco_consensus_error_noalloc(X.data_ptr(), 1, too_big, too_big, out.data_ptr(), None) == -7
    assert lib.choco_consensus_error_noalloc(None, 1, 8, 8, out.data_ptr(), None) == -1
    assert lib.choco_consensus_error_noalloc(X.data_ptr(), 1, 8, 4, out.data_ptr(), None) == -1
    torch.cuda.synchronize()
