"""The single-pass Lloyd iteration (one problem, K <= 128, D <= 128): the assign kernel adds every row tile to
per-cluster sums on the tensor core while the tile is in shared memory, a small kernel adds the per-CTA partials up and
divides.  Checked against the two-pass iteration (bit for bit on integer data, where every sum is exact in any order)
and against the oracle, teacher-forced."""
import numpy as np
import pytest
import torch

import paper_2608_12629_b200 as cake
from oracle import kmeans_oracle as orc
from paper_2608_12629_b200 import inputs
from tests import grading

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

SHAPES = [(1, 64, 1), (100, 64, 5), (127, 8, 3), (128, 64, 128), (129, 128, 100), (5000, 64, 64), (20000, 128, 128),
          (33333, 96, 77), (40000, 72, 128), (70000, 16, 33), (148 * 128 * 3 + 5, 64, 128), (300000, 128, 64), (1 << 20, 64, 100)]


@pytest.mark.parametrize("N,D,K", SHAPES)
def test_fused_iteration_equals_two_pass_iteration_on_integer_data(N, D, K):
    g = torch.Generator().manual_seed(N + D + K)
    X = torch.randint(-4, 5, (N, D), generator=g).to(torch.bfloat16)
    C0 = torch.randint(-4, 5, (K, D), generator=g).to(torch.bfloat16)
    C0[:, 0] += torch.arange(K).to(torch.bfloat16) * 0.5             # distinct centroids
    Xd, Cd = X.to(DEV), C0.to(DEV)
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    n0 = cake.cake_kmeans_kernel_launches()
    a = cake.cake_kmeans_lloyd(Xd, Cd, 4, ws=ws)
    launches = cake.cake_kmeans_kernel_launches() - n0
    torch.cuda.synchronize()
    assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
    assert launches == 1 + 2 * 4, launches                         # the first prologue, then assign + division per iteration
    b = cake.cake_kmeans_lloyd(Xd, Cd, 4, ws=ws, flags=cake.CAKE_LLOYD_NO_FUSE)
    assert torch.equal(a.idx, b.idx) and torch.equal(a.dist, b.dist) and torch.equal(a.counts, b.counts)
    assert torch.equal(a.C, b.C) and torch.equal(a.C_bf16, b.C_bf16)
    np.testing.assert_allclose(a.inertia.cpu().numpy(), b.inertia.cpu().numpy(), rtol=1e-12)
    assert int(a.counts.sum()) == N


@pytest.mark.parametrize("N,D,K", [(3000, 64, 50), (32768, 64, 128), (10000, 128, 100), (5000, 40, 17)])
def test_fused_iteration_teacher_forced_against_the_oracle(N, D, K):
    X, _ = inputs.gaussian_mixture(N, D, K, 2.0, 1.0, N + K)
    C0 = inputs.sample_init(X, K, N)
    Xb = inputs.to_bits(X)
    Xd = X.to(DEV)
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    cur = C0.to(DEV)
    for _ in range(4):
        out = cake.cake_kmeans_lloyd(Xd, cur, 1, ws=ws)
        assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
        cb = inputs.to_bits(cur)
        idx = out.idx.cpu().numpy()
        grading.grade_assign(Xb, cb, idx, out.dist.cpu().numpy())
        grading.grade_update(Xb, idx, K, cb, out.C.cpu().numpy(), inputs.to_bits(out.C_bf16), out.counts.cpu().numpy())
        cur = out.C_bf16
    free = orc.lloyd(Xb, inputs.to_bits(C0), 4, round_centroids=True)
    full = cake.cake_kmeans_lloyd(Xd, C0.to(DEV), 4, ws=ws)
    np.testing.assert_allclose(full.inertia.cpu().numpy(), free.inertia, rtol=grading.INERTIA_TOL)


def test_fused_iteration_empty_clusters_keep_their_centroid_and_repeat_bit_for_bit():
    X, _ = inputs.gaussian_mixture(20000, 64, 10, 2.0, 0.5, 3)
    C0 = inputs.sample_init(X, 100, 3)
    C0[40:60] = (C0[40:60].float() + 500.0).to(torch.bfloat16)      # far away: these clusters stay empty
    Xd, Cd = X.to(DEV), C0.to(DEV)
    a = cake.cake_kmeans_lloyd(Xd, Cd, 3)
    assert int(a.counts[40:60].sum()) == 0 and torch.equal(a.C_bf16[40:60], Cd[40:60])
    b = cake.cake_kmeans_lloyd(Xd, Cd, 3)
    assert torch.equal(a.idx, b.idx) and torch.equal(a.counts, b.counts)
    np.testing.assert_allclose(a.C.cpu().numpy(), b.C.cpu().numpy(), rtol=1e-5, atol=1e-6)    # fp32 summation order only
