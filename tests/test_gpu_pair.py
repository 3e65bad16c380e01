"""The CTA-pair assign kernel (flags = CAKE_ASSIGN_TCGEN05_PAIR: tcgen05.mma.cta_group::2, two SMs share every
256 x 256 tile): graded by the oracle, and bit-identical to the single-CTA kernel, whose arithmetic and epilogue it
shares.  Shapes cover three to many centroid tiles per row tile, ragged row and centroid tails, a row tile whose second
CTA holds no row at all, feature counts that need padding (D % 64 != 0), several ring layouts (D = 64 ... 512),
batches, and the full-precision epilogue."""
import numpy as np
import pytest
import torch

import paper_2608_12629_b200 as cake
from paper_2608_12629_b200 import inputs
from tests import grading

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

SHAPES = [(1, 64, 513), (100, 128, 700), (128, 64, 1024), (129, 128, 769), (255, 64, 513), (257, 192, 600), (1000, 128, 1000),
          (4096, 64, 700), (777, 128, 2048), (5000, 256, 1030), (3000, 320, 800), (2000, 512, 520), (33333, 96, 3000),
          (40000, 72, 1500), (148 * 128 * 2 + 77, 128, 1024), (20000, 128, 16384)]


@pytest.mark.parametrize("N,D,K", SHAPES)
def test_pair_assign_graded_and_identical_to_single_cta(N, D, K):
    X, _ = inputs.gaussian_mixture(N, D, 32, 1.0, 0.5, N + K)
    C = inputs.sample_init(X, K, N)
    Xd, Cd = X.to(DEV), C.to(DEV)
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    idx, dist = cake.cake_kmeans_assign(Xd, Cd, ws=ws, flags=cake.CAKE_ASSIGN_TCGEN05_PAIR)
    torch.cuda.synchronize()
    assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
    rows = None if N * K <= 4e7 else np.sort(np.random.default_rng(1).choice(N, 3000, replace=False))
    grading.grade_assign(inputs.to_bits(X), inputs.to_bits(C), idx.cpu().numpy(), dist.cpu().numpy(), rows=rows)
    i1, d1 = cake.cake_kmeans_assign(Xd, Cd, ws=ws, flags=cake.CAKE_ASSIGN_TCGEN05)
    assert torch.equal(idx, i1) and torch.equal(dist, d1)


@pytest.mark.parametrize("N,D,K", [(1000, 128, 1000), (5000, 64, 600), (2500, 256, 777)])
def test_pair_assign_full_precision_epilogue(N, D, K):
    X, _ = inputs.gaussian_mixture(N, D, 32, 1.0, 0.5, N + K + 1)
    C = inputs.sample_init(X, K, N)
    Xd, Cd = X.to(DEV), C.to(DEV)
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    ie, de = cake.cake_kmeans_assign(Xd, Cd, ws=ws, flags=cake.CAKE_ASSIGN_TCGEN05_EXACT)
    ip, dp = cake.cake_kmeans_assign(Xd, Cd, ws=ws, flags=cake.CAKE_ASSIGN_TCGEN05_PAIR_EXACT)
    torch.cuda.synchronize()
    assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
    grading.grade_assign(inputs.to_bits(X), inputs.to_bits(C), ip.cpu().numpy(), dp.cpu().numpy())
    assert torch.equal(ie, ip) and torch.equal(de, dp)


def test_pair_assign_batched_and_lloyd_equal_single_cta():
    B, N, D, K = 5, 3000, 128, 600
    Xs, Cs = [], []
    for b in range(B):
        X, _ = inputs.gaussian_mixture(N, D, 40, 1.0, 0.5, 77 + b)
        Xs.append(X)
        Cs.append(inputs.sample_init(X, K, 77 + b))
    Xd, Cd = torch.stack(Xs).to(DEV), torch.stack(Cs).to(DEV)
    ws = cake.alloc_workspace(B, N, D, K, DEV)
    ip, dp = cake.cake_kmeans_assign(Xd, Cd, ws=ws, flags=cake.CAKE_ASSIGN_TCGEN05_PAIR)
    i1, d1 = cake.cake_kmeans_assign(Xd, Cd, ws=ws)
    assert torch.equal(ip, i1) and torch.equal(dp, d1)
    for b in (0, B - 1):
        grading.grade_assign(inputs.to_bits(Xs[b]), inputs.to_bits(Cs[b]), ip[b].cpu().numpy(), dp[b].cpu().numpy())
    a = cake.cake_kmeans_lloyd(Xd, Cd, 3, ws=ws, flags=cake.CAKE_ASSIGN_TCGEN05_PAIR)
    r = cake.cake_kmeans_lloyd(Xd, Cd, 3, ws=ws)
    torch.cuda.synchronize()
    assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
    assert torch.equal(a.idx, r.idx) and torch.equal(a.C_bf16, r.C_bf16) and torch.equal(a.counts, r.counts)
    np.testing.assert_allclose(a.inertia.cpu().numpy(), r.inertia.cpu().numpy(), rtol=1e-12)


def test_pair_assign_refuses_what_it_does_not_cover():
    # feature counts that only the automatic choice takes to the tensor cores (through a padded copy of X) and
    # cluster counts of at most two centroid tiles (their kernel keeps the centroids resident) are refused with the
    # flag instead of silently taking another kernel; nothing is enqueued and the workspace stays usable
    for N, D, K in [(500, 36, 600), (500, 64, 512), (500, 128, 100)]:
        X, _ = inputs.gaussian_mixture(N, D, 8, 1.0, 0.5, 3)
        C = inputs.sample_init(X, K, 3)
        ws = cake.alloc_workspace(1, N, D, K, DEV)
        n0 = cake.cake_kmeans_kernel_launches()
        with pytest.raises(cake.CakeError) as e:
            cake.cake_kmeans_assign(X.to(DEV), C.to(DEV), ws=ws, flags=cake.CAKE_ASSIGN_TCGEN05_PAIR)
        assert e.value.code == cake.CAKE_ERR_UNSUPPORTED
        assert cake.cake_kmeans_kernel_launches() == n0
        idx, dist = cake.cake_kmeans_assign(X.to(DEV), C.to(DEV), ws=ws)
        grading.grade_assign(inputs.to_bits(X), inputs.to_bits(C), idx.cpu().numpy(), dist.cpu().numpy())
