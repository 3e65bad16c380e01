"""GPU parity of assign on inputs whose norms differ wildly: centroids far larger (or smaller) than the data,
un-centred data, very small and very large magnitudes, a batch where only one problem has an outlier.

The tolerance of a row is relative to |x|^2 + |c_best|^2 of THAT row (tests/grading.py), so a method whose
resolution follows the largest centroid of the whole problem fails here.  Every case goes through the C ABI
on the tensor-core route under both epilogue policies and is graded by the unchanged rules.
"""
import numpy as np
import pytest
import torch

import paper_2608_12629_b200 as cake
from paper_2608_12629_b200 import inputs
from tests import grading

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

POLICIES = {"auto": cake.CAKE_ASSIGN_AUTO, "packed": cake.CAKE_ASSIGN_TCGEN05, "exact": cake.CAKE_ASSIGN_TCGEN05_EXACT}
# (N, D, K): many centroid tiles, one resident tile (K <= 128 and K <= 256), two resident tiles, a split X buffer
SHAPES = [(4000, 64, 600), (3000, 128, 100), (2500, 64, 256), (3000, 128, 400), (1500, 320, 60), (2000, 256, 1100)]


def mixture(N, D, K, seed, sigma=1.0, mean_std=1.0):
    X, _ = inputs.gaussian_mixture(N, D, max(1, min(K, 32)), mean_std, sigma, seed)
    return X, inputs.sample_init(X, K, seed)


def run_and_grade(X, C, flags, max_mismatch=None):
    N, D = X.shape
    K = C.shape[0]
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    idx, dist = cake.cake_kmeans_assign(X.to(DEV), C.to(DEV), ws=ws, flags=flags)
    torch.cuda.synchronize()
    assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
    rep = grading.grade_assign(inputs.to_bits(X), inputs.to_bits(C), idx.cpu().numpy(), dist.cpu().numpy())
    if max_mismatch is not None:
        assert rep["mismatch"] <= max_mismatch, rep
    return rep, idx, dist


@pytest.mark.parametrize("policy", sorted(POLICIES))
@pytest.mark.parametrize("scale", [30.0, 60.0, 1000.0, 1.0e6])
@pytest.mark.parametrize("N,D,K", SHAPES)
def test_one_centroid_far_larger_than_the_data(N, D, K, scale, policy):
    """One centroid `scale` times the data's norm, at a column position in the middle of a tile and once as the
    last real centroid next to the padding rows."""
    X, C = mixture(N, D, K, seed=N + K)
    for where in (K // 3, K - 1):
        C2 = C.clone()
        C2[where] = (C[where].float() * scale).to(torch.bfloat16)
        run_and_grade(X, C2, POLICIES[policy], max_mismatch=max(2, N // 500))


@pytest.mark.parametrize("policy", sorted(POLICIES))
@pytest.mark.parametrize("scale", [60.0, 1000.0])
def test_outlier_row_picked_as_initial_centroid(scale, policy):
    """A few rows of X lie far from the rest and are among the sampled initial centroids: each is nearest to
    itself (distance 0 against norms of scale^2), everything else must be unaffected."""
    N, D, K = 5000, 64, 300
    X, _ = mixture(N, D, K, seed=7)
    far = [11, 2048, 4999]
    for i in far:
        X[i] = (X[i].float() * scale).to(torch.bfloat16)
    pick = np.random.default_rng(3).choice(N, size=K, replace=False)
    pick[:3] = far
    C = X[torch.from_numpy(np.unique(pick))].contiguous()
    rep, idx, dist = run_and_grade(X, C, POLICIES[policy], max_mismatch=10)
    cbits = inputs.to_bits(C)
    for i in far:
        k = int(idx[i])
        assert np.array_equal(cbits[k], inputs.to_bits(X[i:i + 1])[0]) and float(dist[i]) <= 1e-3 * 2 * float((X[i].float() ** 2).sum())


@pytest.mark.parametrize("policy", sorted(POLICIES))
@pytest.mark.parametrize("N,D,K", SHAPES[:4])
def test_centroid_norms_spread_over_many_binades(N, D, K, policy):
    """Centroid k scaled by 2^e_k with e_k uniform in [-12, 12], data rows by 2^e_i likewise: near and far pairs of
    every ratio, no single scale describes the problem."""
    X, C = mixture(N, D, K, seed=D + K)
    rng = np.random.default_rng(N)
    X = (X.float() * torch.from_numpy(2.0 ** rng.integers(-12, 13, size=(N, 1))).float()).to(torch.bfloat16)
    C = (C.float() * torch.from_numpy(2.0 ** rng.integers(-12, 13, size=(K, 1))).float()).to(torch.bfloat16)
    run_and_grade(X, C, POLICIES[policy], max_mismatch=max(4, N // 200))


@pytest.mark.parametrize("policy", sorted(POLICIES))
def test_centroid_at_the_origin_among_unit_centroids(policy):
    """min |c|^2 = 0 next to |c|^2 ~ D: rows close to the origin have a tolerance far below the other centroids' norms."""
    N, D, K = 3000, 64, 300
    X, C = mixture(N, D, K, seed=21)
    X[:500] = (X[:500].float() * 1e-3).to(torch.bfloat16)
    C[5] = 0
    C[6] = (C[6].float() * 1e-3).to(torch.bfloat16)
    run_and_grade(X, C, POLICIES[policy], max_mismatch=6)


@pytest.mark.parametrize("policy", sorted(POLICIES))
@pytest.mark.parametrize("N,D,K", SHAPES[:4])
def test_data_far_from_the_origin(N, D, K, policy):
    """A common offset of 50 sigma in every coordinate: distances are tiny against the norms (the tolerance is
    relative to the norms, so near-ties are excused, anything else is not)."""
    X, _ = mixture(N, D, K, seed=N)
    X = (X.float() + 50.0).to(torch.bfloat16)
    C = inputs.sample_init(X, K, 5)
    run_and_grade(X, C, POLICIES[policy])


@pytest.mark.parametrize("policy", sorted(POLICIES))
@pytest.mark.parametrize("mag", [1.0e-15, 1.0e-9, 1.0e9, 1.0e15])
def test_very_small_and_very_large_magnitudes(mag, policy):
    N, D, K = 3000, 64, 300
    X, _ = mixture(N, D, K, seed=33)
    X = (X.float() * mag).to(torch.bfloat16)
    C = inputs.sample_init(X, K, 9)
    run_and_grade(X, C, POLICIES[policy], max_mismatch=6)


@pytest.mark.parametrize("policy", sorted(POLICIES))
@pytest.mark.parametrize("B,N,D,K", [(4, 1500, 64, 600), (5, 1200, 128, 100), (3, 2000, 128, 400)])
def test_batch_where_one_problem_has_the_outlier(B, N, D, K, policy):
    """Problems of a batch share nothing: an outlier centroid in problem 1 must not change the resolution of the
    others (every problem graded on its own, and equal to the same problem run alone)."""
    Xs, Cs = zip(*(mixture(N, D, K, seed=90 + b) for b in range(B)))
    Cs = [c.clone() for c in Cs]
    Cs[1][K // 2] = (Cs[1][K // 2].float() * 1000.0).to(torch.bfloat16)
    X, C = torch.stack(Xs).to(DEV), torch.stack(Cs).to(DEV)
    ws = cake.alloc_workspace(B, N, D, K, DEV)
    idx, dist = cake.cake_kmeans_assign(X, C, ws=ws, flags=POLICIES[policy])
    assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
    for b in range(B):
        grading.grade_assign(inputs.to_bits(Xs[b]), inputs.to_bits(Cs[b]), idx[b].cpu().numpy(), dist[b].cpu().numpy())
        i1, d1 = cake.cake_kmeans_assign(X[b].contiguous(), C[b].contiguous(), flags=POLICIES[policy])
        assert torch.equal(i1, idx[b]) and torch.equal(d1, dist[b])


def test_lloyd_with_an_outlier_centroid_teacher_forced():
    """Three Lloyd iterations from an initialisation that contains a far outlier row; every iteration's assignment is
    graded against the oracle from the GPU's own centroids (through stepwise calls, which the one-call loop equals)."""
    N, D, K = 6000, 64, 200
    X, _ = mixture(N, D, K, seed=55)
    X[100] = (X[100].float() * 500.0).to(torch.bfloat16)
    pick = np.random.default_rng(1).choice(N, size=K, replace=False)
    pick[0] = 100
    C = X[torch.from_numpy(np.unique(pick))].contiguous()
    K = C.shape[0]
    Xd = X.to(DEV)
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    out = cake.cake_kmeans_lloyd(Xd, C.to(DEV), 3, ws=ws)
    Cc = C.to(DEV)
    for _ in range(3):
        idx, dist = cake.cake_kmeans_assign(Xd, Cc, ws=ws)
        grading.grade_assign(inputs.to_bits(X), inputs.to_bits(Cc.cpu()), idx.cpu().numpy(), dist.cpu().numpy())
        Cf, Cb, counts = cake.cake_kmeans_update(Xd, idx, K, C_prev=Cc, ws=ws)
        grading.grade_update(inputs.to_bits(X), idx.cpu().numpy(), K, inputs.to_bits(Cc.cpu()), Cf.cpu().numpy(),
                             inputs.to_bits(Cb.cpu()), counts.cpu().numpy())
        Cc = Cb
    assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
    assert torch.equal(out.idx, idx) and torch.equal(out.C_bf16, Cb)
