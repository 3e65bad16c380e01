"""GPU parity of the exact k-nearest-neighbour search against the fp64 oracle, through the C ABI.

Rule per (query, place p): the GPU's p-th neighbour g differs from the oracle's o only where the two distances are a
near-tie, |d64(q, x_g) - d_oracle[p]| < 1e-3 (|q|^2 + |x_o|^2) (the oracle's p-th distance is unique, the row that
attains it need not be); every GPU row is a valid, distinct database row; every returned distance is within
1e-3 (|q|^2 + |x_g|^2) of d64(q, x_g); the list is ascending.  Integer-valued data must agree exactly, ties included.
"""
import numpy as np
import pytest
import torch

import paper_2608_12629_b200 as cake
from oracle import kmeans_oracle as orc
from paper_2608_12629_b200 import inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def grade_knn(Q, X, k, idx_gpu, dist_gpu):
    Qb, Xb = inputs.to_bits(Q), inputs.to_bits(X)
    idx_o, dist_o = orc.knn(Qb, Xb, k)
    N, M = Q.shape[0], X.shape[0]
    kk = min(k, M)
    assert idx_gpu.shape == (N, k)
    if kk < k:
        assert (idx_gpu[:, kk:] == -1).all() and np.isinf(dist_gpu[:, kk:]).all()
    g = idx_gpu[:, :kk]
    assert g.min() >= 0 and g.max() < M
    assert all(len(set(row)) == kk for row in g), "a database row was returned twice"
    Xf, Qf = orc.bf16_to_f64(Xb), orc.bf16_to_f64(Qb)
    qn, xn = (Qf * Qf).sum(1), (Xf * Xf).sum(1)
    d_g = np.stack([orc.pair_sqdist(Qb, Xf, np.ascontiguousarray(g[:, p])) for p in range(kk)], 1)
    mism = g != idx_o[:, :kk]
    tau = 1e-3 * (qn[:, None] + xn[idx_o[:, :kk]])
    unexcused = mism & ~(np.abs(d_g - dist_o[:, :kk]) < tau)
    rep = {"n": N * kk, "mismatch": int(mism.sum()), "unexcused": int(unexcused.sum())}
    assert not unexcused.any(), rep
    err = np.abs(dist_gpu[:, :kk].astype(np.float64) - d_g)
    assert (err <= 1e-3 * (qn[:, None] + xn[g])).all(), rep
    assert (np.diff(dist_gpu[:, :kk], axis=1) >= 0).all()
    return rep


def data(N, M, D, seed, sigma=0.5):
    X, _ = inputs.gaussian_mixture(M, D, 32, 1.0, sigma, seed)
    Q, _ = inputs.gaussian_mixture(N, D, 32, 1.0, sigma, seed)       # same mixture, its own noise below
    g = torch.Generator().manual_seed(seed + 1)
    Q = (Q.float() + 0.25 * torch.randn(N, D, generator=g)).to(torch.bfloat16)
    return Q, X


@pytest.mark.parametrize("k", [1, 8, 32])
@pytest.mark.parametrize("N,M,D", [(1, 300, 64), (127, 1000, 64), (1000, 5000, 128), (300, 257, 128), (2000, 20000, 64),
                                   (500, 3000, 256), (129, 4097, 96), (400, 2500, 320), (700, 6000, 40), (64, 2000, 100),
                                   (33, 7, 64)])
def test_knn_search_graded_by_the_oracle(N, M, D, k):
    Q, X = data(N, M, D, N + M + D)
    idx, dist = cake.cake_knn_search(Q.to(DEV), X.to(DEV), k)
    torch.cuda.synchronize()
    rep = grade_knn(Q, X, k, idx.cpu().numpy(), dist.cpu().numpy())
    assert rep["mismatch"] <= max(2, rep["n"] // 2000), rep


def test_knn_k1_equals_assign_and_integer_ties_are_exact():
    g = torch.Generator().manual_seed(8)
    Q = torch.randint(-2, 3, (1500, 64), generator=g).to(torch.bfloat16)
    X = torch.randint(-2, 3, (1200, 64), generator=g).to(torch.bfloat16)
    X[600:1200] = X[0:600]                 # every database row twice: across tiles and across the two column halves
    Qd, Xd = Q.to(DEV), X.to(DEV)
    idx, dist = cake.cake_knn_search(Qd, Xd, 16)
    idx_o, dist_o = orc.knn(inputs.to_bits(Q), inputs.to_bits(X), 16)
    assert np.array_equal(idx.cpu().numpy(), idx_o)                  # exact arithmetic: ties go to the lower row everywhere
    assert np.array_equal(dist.cpu().numpy().astype(np.float64), dist_o)
    i1, d1 = cake.cake_knn_search(Qd, Xd, 1)
    ia, da = cake.cake_kmeans_assign(Qd, Xd, flags=cake.CAKE_ASSIGN_TCGEN05_EXACT)
    assert torch.equal(i1[:, 0], ia) and torch.equal(d1[:, 0], da)


def test_knn_self_search_finds_the_point_first_and_repeats_bit_for_bit():
    Q, X = data(10, 30000, 128, 5)
    Xd = X.to(DEV)
    q = Xd[:4000].contiguous()
    idx, dist = cake.cake_knn_search(q, Xd, 8)
    Xb = inputs.to_bits(X)
    first = {}
    for i, r in enumerate(Xb):
        first.setdefault(r.tobytes(), i)
    want = np.array([first[r.tobytes()] for r in Xb[:4000]])
    assert np.array_equal(idx[:, 0].cpu().numpy(), want)
    assert float(dist[:, 0].max()) <= 1e-3 * 2 * float((X.float() ** 2).sum(1).max())
    idx2, dist2 = cake.cake_knn_search(q, Xd, 8)
    assert torch.equal(idx, idx2) and torch.equal(dist, dist2)


def test_knn_argument_checks():
    Q, X = data(16, 64, 64, 1)
    Qd, Xd = Q.to(DEV), X.to(DEV)
    with pytest.raises(cake.CakeError) as e:
        cake.cake_knn_search(Qd, Xd, 33)
    assert e.value.code == cake.CAKE_ERR_UNSUPPORTED
    with pytest.raises(cake.CakeError) as e:
        cake.cake_knn_search(Qd, Xd, 0)
    assert e.value.code == cake.CAKE_ERR_SHAPE
    big = torch.zeros(4, 520, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(cake.CakeError) as e:
        cake.cake_knn_search(big, big, 2)
    assert e.value.code == cake.CAKE_ERR_UNSUPPORTED
    ws = torch.zeros(cake.cake_knn_workspace_bytes(16, 64, 64, 4), dtype=torch.uint8, device=DEV)
    with pytest.raises(cake.CakeError) as e:
        cake.cake_knn_search(Qd, Xd, 4, ws=ws[:512])
    assert e.value.code == cake.CAKE_ERR_WORKSPACE
    idx, dist = cake.cake_knn_search(Qd[:0], Xd, 4)
    assert idx.shape == (0, 4)
    idx, none = cake.cake_knn_search(Qd, Xd, 4, ws=ws, want_dist=False)
    assert none is None and cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
    grade_knn(Q, X, 4, idx.cpu().numpy(), cake.cake_knn_search(Qd, Xd, 4)[1].cpu().numpy())
