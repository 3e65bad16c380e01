"""The workspace-free assign entry point, for callers that cannot allocate device memory.

Such callers (code inside another framework's allocator hook, or a process whose device memory is
fully spoken for) cannot give the library a scratch buffer, so cake_kmeans_assign_static keeps its
scratch in a fixed array inside the library.  This file is collected last on purpose: the static
array is shared, process-wide state, and the test must pass both in a fresh process and after every
other test has used the device.
"""
import numpy as np
import pytest
import torch

import paper_2608_12629_b200 as cake
from paper_2608_12629_b200 import inputs
from tests import grading

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _problem(N, D, K, seed):
    X, _ = inputs.gaussian_mixture(N, D, 48, 1.0, 0.5, seed)
    return X.to(DEV), inputs.sample_init(X, K, seed).to(DEV)


def test_static_assign_matches_workspace_assign_twice_in_a_row():
    # two calls in a row with different K and D: the second must not be affected by what the first
    # left in the shared array (a longer ||c||^2 row and its padding rows)
    for N, D, K, seed in [(3000, 128, 700, 11), (2500, 64, 300, 12)]:
        X, C = _problem(N, D, K, seed)
        idx_ref, dist_ref = cake.cake_kmeans_assign(X, C)          # the existing entry point
        idx, dist = cake.cake_kmeans_assign_static(X, C)           # through the C ABI, no workspace
        torch.cuda.synchronize()
        assert torch.equal(idx, idx_ref)
        assert torch.allclose(dist, dist_ref, rtol=0, atol=0)
    assert cake.cake_kmeans_assign_static_status(DEV) == cake.CAKE_OK


def test_static_assign_rejects_sizes_beyond_its_fixed_scratch():
    X, C = _problem(64, 64, 32, 1)
    big_c = torch.zeros(16385, 64, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(cake.CakeError) as e:
        cake.cake_kmeans_assign_static(X, big_c)
    assert e.value.code == cake.CAKE_ERR_UNSUPPORTED
    idx, _ = cake.cake_kmeans_assign_static(X, C)                  # still usable afterwards
    assert torch.equal(idx, cake.cake_kmeans_assign(X, C)[0])


@pytest.mark.parametrize("N,D,K", [(3000, 96, 700), (2000, 40, 100), (1500, 320, 64), (2500, 72, 300), (1200, 200, 513),
                                   (500, 100, 33), (300, 520, 9), (4096, 64, 16384)])
def test_static_assign_graded_by_the_oracle(N, D, K):
    """Feature counts that are no multiple of 64 (this entry point streams the centroid rows unpadded, which no
    workspace call does any more), the CUDA-core branch (D % 8 != 0, D > 512) and K at the limit of the fixed
    array: graded against the oracle and equal to the workspace entry point wherever both take the same route."""
    X, C = _problem(N, D, K, N + D)
    idx, dist = cake.cake_kmeans_assign_static(X, C)
    torch.cuda.synchronize()
    assert cake.cake_kmeans_assign_static_status(DEV) == cake.CAKE_OK
    rep = grading.grade_assign(inputs.to_bits(X), inputs.to_bits(C), idx.cpu().numpy(), dist.cpu().numpy())
    assert rep["mismatch"] <= 3, rep
    if D % 8 == 0 and D <= 512:      # same arithmetic as the workspace call (padding columns are zeros)
        idx_ref, dist_ref = cake.cake_kmeans_assign(X, C)
        assert torch.equal(idx, idx_ref) and torch.equal(dist, dist_ref)


def test_static_assign_small_problem_right_after_one_at_the_limit():
    """K = 16384 fills the fixed array to its last byte; the K = 40 call after it must see none of it."""
    X, C = _problem(2000, 64, 16384, 5)
    i1, d1 = cake.cake_kmeans_assign_static(X, C)
    X2, C2 = _problem(1500, 128, 40, 6)
    i2, d2 = cake.cake_kmeans_assign_static(X2, C2)
    torch.cuda.synchronize()
    grading.grade_assign(inputs.to_bits(X), inputs.to_bits(C), i1.cpu().numpy(), d1.cpu().numpy())
    grading.grade_assign(inputs.to_bits(X2), inputs.to_bits(C2), i2.cpu().numpy(), d2.cpu().numpy())
    assert cake.cake_kmeans_assign_static_status(DEV) == cake.CAKE_OK


def test_static_assign_allocates_nothing_and_edge_arguments():
    X, C = _problem(3000, 128, 300, 9)
    idx = torch.empty(3000, dtype=torch.int32, device=DEV)
    dist = torch.empty(3000, dtype=torch.float32, device=DEV)
    cake.cake_kmeans_assign_static(X, C, out_idx=idx, out_dist=dist)      # first call on the device: set-up
    torch.cuda.synchronize()
    # a call that allocated would take device memory every time: over several calls the free memory reported by
    # the driver must stay put at least once (other activity of the process may move it now and then) and the
    # framework's own allocator must see no allocation request at all
    import gc
    gc.collect()                                   # tensors of earlier tests must not be freed while we count
    events0 = torch.cuda.memory_stats().get("allocation.all.allocated", 0)
    deltas = []
    for _ in range(4):
        free0, _ = torch.cuda.mem_get_info()
        cake.cake_kmeans_assign_static(X, C, out_idx=idx, out_dist=dist)
        torch.cuda.synchronize()
        deltas.append(free0 - torch.cuda.mem_get_info()[0])
        assert torch.cuda.memory_stats().get("allocation.all.allocated", 0) == events0     # no allocation event at all
    assert min(deltas) <= 0, deltas
    # N = 0 does nothing; no distances wanted; misaligned outputs are refused before anything is enqueued
    e_idx, _ = cake.cake_kmeans_assign_static(X[:0], C)
    assert e_idx.numel() == 0
    i2, none = cake.cake_kmeans_assign_static(X, C, want_dist=False)
    assert none is None and torch.equal(i2, idx)
    L = cake.lib()
    import ctypes
    s = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    rc = L.cake_kmeans_assign_static(ctypes.c_void_p(X.data_ptr()), ctypes.c_void_p(C.data_ptr()), 3000, 128, 300,
                                     ctypes.c_void_p(idx.data_ptr() + 2), ctypes.c_void_p(dist.data_ptr()), s)
    assert rc == cake.CAKE_ERR_ALIGN
    assert np.array_equal(idx.cpu().numpy(), i2.cpu().numpy())
