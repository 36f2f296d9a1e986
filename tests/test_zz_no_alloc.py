"""cc_update_static: the M-step for callers that are not allowed to allocate device memory.

Some users of the library run inside a process whose device memory belongs to somebody else (a
framework's pool, a container sized at start-up) or in a loop that must never reach cudaMalloc;
they can pass inputs and outputs but no workspace.  For them the library offers one entry point
whose scratch is a fixed array inside the library image.  This file checks, through the C ABI,
that it returns exactly what cc_update returns -- counts equal, centroids bit for bit, the bar the
other M-step tests use -- on two calls in a row (the second must not see the first one's sums),
and that it refuses problems beyond its fixed capacity.

The file is named so that pytest collects it last: a run that stops at the first failure has
then already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_13089_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _run_both(cc, u, X, idx, C_prev):
    N, g = X.shape
    K = C_prev.shape[0]
    C_ref, counts_ref = u.gpu_update(X, idx, C_prev)                 # existing entry point (workspace)
    Xd = u.half_dev(X)
    Cd = u.dev(C_prev.astype(np.float32))
    idxd = torch.from_numpy(idx.astype(np.uint16).view(np.int16)).cuda().view(torch.uint16)
    counts = torch.full((K,), -7, dtype=torch.int32, device="cuda")
    cc.cc_update_static(0, Xd, N, g, idxd, K, Cd, counts)
    torch.cuda.synchronize()
    return C_ref, counts_ref, Cd.cpu().numpy(), counts.cpu().numpy()


def test_update_static_matches_update_on_two_calls_in_a_row():
    from paper_2503_13089_b200 import binding as cc
    from tests import gpu_util as u
    rng = np.random.default_rng(5)
    # first call: a ragged size, empty clusters at the end, values on both accumulator ranges
    X1 = wl.make_points(70001, 4, 31)
    X1[::13] = (rng.standard_normal((len(X1[::13]), 4)) * 200).astype(np.float16)
    idx1 = rng.integers(0, 990, len(X1)).astype(np.int32)
    C1 = wl.make_codebook(1000, 4, 32)
    # second call: fewer accumulators than the first one used, different data; stale sums would show
    X2 = wl.make_points(9000, 8, 33)
    idx2 = rng.integers(0, 300, len(X2)).astype(np.int32)
    C2 = wl.make_codebook(301, 8, 34)
    for X, idx, C_prev in ((X1, idx1, C1), (X2, idx2, C2)):
        C_ref, counts_ref, C_st, counts_st = _run_both(cc, u, X, idx, C_prev)
        assert np.array_equal(counts_st, counts_ref)
        assert u.centroid_rel_err(C_st, C_ref, X) <= u.REL_CENTROID
        assert np.array_equal(C_st.view(np.uint32), C_ref.view(np.uint32))
        C_or, counts_or = oracle.update(X, idx, C_prev)              # and the CPU oracle says the same
        assert np.array_equal(counts_st.astype(np.int64), counts_or.astype(np.int64))
        assert np.array_equal(C_st.view(np.uint32), C_or.view(np.uint32))
        empty = counts_ref == 0
        assert empty.any() and np.array_equal(C_st[empty].view(np.uint32), C_prev[empty].view(np.uint32))


def test_update_static_rejects_sizes_beyond_its_fixed_capacity():
    from paper_2503_13089_b200 import binding as cc
    g, K = 8, 65536                                    # K * g = 524288 > UPDATE_STATIC_MAX_KG
    assert K * g > cc.UPDATE_STATIC_MAX_KG
    X = torch.zeros((16, g), dtype=torch.float16, device="cuda")
    idx = torch.zeros(16, dtype=torch.uint16, device="cuda")
    C = torch.ones((K, g), dtype=torch.float32, device="cuda")
    counts = torch.full((K,), 3, dtype=torch.int32, device="cuda")
    with pytest.raises(cc.CCError) as e:
        cc.cc_update_static(0, X, 16, g, idx, K, C, counts)
    assert e.value.status == 12
    torch.cuda.synchronize()
    assert bool((C == 1).all()) and bool((counts == 3).all())       # nothing was enqueued
    # the largest supported problem is accepted
    K = cc.UPDATE_STATIC_MAX_KG // g
    cc.cc_update_static(0, X, 16, g, idx, K, C[:K], counts[:K])
    torch.cuda.synchronize()
    assert int(counts[0].item()) == 16 and int(counts[1:K].sum().item()) == 0


def test_update_static_at_full_capacity_and_without_touching_the_allocator():
    """K * g exactly at the fixed capacity with members in the very last cluster (the last words of
    the array are used), compared with the oracle; and a warm call must leave the device's free
    memory as it found it -- the point of the entry point is that it never allocates."""
    from paper_2503_13089_b200 import binding as cc
    from tests import gpu_util as u
    g = 4
    K = cc.UPDATE_STATIC_MAX_KG // g
    rng = np.random.default_rng(9)
    X = wl.make_points(50000, g, 35)
    idx = rng.integers(0, K, len(X)).astype(np.int32)
    idx[-3:] = K - 1
    C_prev = wl.make_codebook(K, g, 36)
    Xd = u.half_dev(X)
    idxd = torch.from_numpy(idx.astype(np.uint16).view(np.int16)).cuda().view(torch.uint16)
    Cd = u.dev(C_prev)
    counts = torch.empty(K, dtype=torch.int32, device="cuda")
    cc.cc_update_static(0, Xd, len(X), g, idxd, K, Cd, counts)       # first call on the device: set-up
    torch.cuda.synchronize()
    C_or, counts_or = oracle.update(X, idx, C_prev)
    assert counts_or[K - 1] >= 3
    assert np.array_equal(counts.cpu().numpy().astype(np.int64), counts_or.astype(np.int64))
    assert np.array_equal(Cd.cpu().numpy().view(np.uint32), C_or.view(np.uint32))
    Cd.copy_(torch.from_numpy(C_prev))
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    cc.cc_update_static(0, Xd, len(X), g, idxd, K, Cd, counts)       # warm call
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert np.array_equal(Cd.cpu().numpy().view(np.uint32), C_or.view(np.uint32))
