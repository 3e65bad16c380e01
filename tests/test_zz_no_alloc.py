"""The workspace-free assign entry point, for callers that cannot allocate device memory.

Such callers (code inside another framework's allocator hook, or a process whose device memory is
fully spoken for) cannot give the library a scratch buffer, so cake_kmeans_assign_static keeps its
scratch in a fixed array inside the library.  This file is collected last on purpose: the static
array is shared, process-wide state, and the test must pass both in a fresh process and after every
other test has used the device.
"""
import pytest
import torch

import paper_2608_12629_b200 as cake
from paper_2608_12629_b200 import inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _problem(N, D, K, seed):
    X, _ = inputs.gaussian_mixture(N, D, 48, 1.0, 0.5, seed)
    return X.to(DEV), inputs.sample_init(X, K, seed).to(DEV)


def test_static_assign_matches_workspace_assign_twice_in_a_row():
    # two calls in a row with different K and D: the second must not be affected by what the first
    # left in the shared array (a longer ||c||^2 row and its +inf padding)
    for N, D, K, seed in [(3000, 128, 700, 11), (2500, 64, 300, 12)]:
        X, C = _problem(N, D, K, seed)
        idx_ref, dist_ref = cake.cake_kmeans_assign(X, C)          # the existing entry point
        idx, dist = cake.cake_kmeans_assign_static(X, C)           # through the C ABI, no workspace
        torch.cuda.synchronize()
        assert torch.equal(idx, idx_ref)
        assert torch.allclose(dist, dist_ref, rtol=0, atol=0)


def test_static_assign_rejects_sizes_beyond_its_fixed_scratch():
    X, C = _problem(64, 64, 32, 1)
    big_c = torch.zeros(16385, 64, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(cake.CakeError) as e:
        cake.cake_kmeans_assign_static(X, big_c)
    assert e.value.code == cake.CAKE_ERR_UNSUPPORTED
    idx, _ = cake.cake_kmeans_assign_static(X, C)                  # still usable afterwards
    assert torch.equal(idx, cake.cake_kmeans_assign(X, C)[0])
