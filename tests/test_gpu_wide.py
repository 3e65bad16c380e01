"""Rows of more than 512 columns on the tensor cores: no CTA can keep such an X tile resident, so the CTA-pair kernel
streams X chunk by chunk beside the centroids (its wide mode) and takes the rows' norms from a small kernel that runs
ahead.  Graded by the oracle: one to many centroid tiles, ragged tails, feature counts that need zero padding
(D % 8 != 0 and D % 64 != 0), batches, both epilogues, Lloyd iterations (the row operand is made once per call)."""
import numpy as np
import pytest
import torch

import paper_2608_12629_b200 as cake
from oracle import kmeans_oracle as orc
from paper_2608_12629_b200 import inputs
from tests import grading

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

SHAPES = [(1, 520, 1), (300, 576, 5), (1000, 520, 300), (777, 1024, 1030), (5000, 640, 600), (2000, 1001, 257),
          (1500, 2048, 100), (257, 4096, 40), (130, 8192, 9), (20000, 768, 2048), (148 * 128 + 5, 600, 513)]


@pytest.mark.parametrize("N,D,K", SHAPES)
def test_wide_rows_assign_graded(N, D, K):
    X, _ = inputs.gaussian_mixture(N, D, 32, 1.0, 0.5, N + K)
    C = inputs.sample_init(X, K, N)
    Xd, Cd = X.to(DEV), C.to(DEV)
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    n0 = cake.cake_kmeans_kernel_launches()
    idx, dist = cake.cake_kmeans_assign(Xd, Cd, ws=ws)
    launches = cake.cake_kmeans_kernel_launches() - n0
    torch.cuda.synchronize()
    assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
    # centroid prologue, row operand, the pair kernel (+ the padded copy of X when D % 8 != 0): never the CUDA-core kernel
    assert launches == (4 if D % 8 else 3), launches
    rows = None if N * K * D <= 3e9 else np.sort(np.random.default_rng(1).choice(N, 1500, replace=False))
    rep = grading.grade_assign(inputs.to_bits(X), inputs.to_bits(C), idx.cpu().numpy(), dist.cpu().numpy(), rows=rows)
    assert rep["mismatch"] <= max(2, N // 1000), rep
    if D % 8 == 0:
        ie, de = cake.cake_kmeans_assign(Xd, Cd, ws=ws, flags=cake.CAKE_ASSIGN_TCGEN05_EXACT)
        torch.cuda.synchronize()
        assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
        grading.grade_assign(inputs.to_bits(X), inputs.to_bits(C), ie.cpu().numpy(), de.cpu().numpy(), rows=rows)
        assert (ie != idx).float().mean().item() <= 0.01


def test_wide_rows_norm_spread():
    """One centroid far away and one row far away: every pair keeps its own resolution (the margins are per row)."""
    N, D, K = 3000, 640, 300
    X, _ = inputs.gaussian_mixture(N, D, 16, 1.0, 0.5, 5)
    C = inputs.sample_init(X, K, 5)
    C = C.clone()
    C[7] = (C[7].float() * 60).to(torch.bfloat16)
    X = X.clone()
    X[11] = (X[11].float() * 1000).to(torch.bfloat16)
    X[12] = (X[12].float() * 1e-3).to(torch.bfloat16)
    idx, dist = cake.cake_kmeans_assign(X.to(DEV), C.to(DEV))
    grading.grade_assign(inputs.to_bits(X), inputs.to_bits(C), idx.cpu().numpy(), dist.cpu().numpy())


def test_wide_rows_batched():
    B, N, D, K = 3, 1000, 576, 270
    Xs, Cs = [], []
    for b in range(B):
        X, _ = inputs.gaussian_mixture(N, D, 20, 1.0, 0.5, 31 + b)
        Xs.append(X)
        Cs.append(inputs.sample_init(X, K, 31 + b))
    ws = cake.alloc_workspace(B, N, D, K, DEV)
    idx, dist = cake.cake_kmeans_assign(torch.stack(Xs).to(DEV), torch.stack(Cs).to(DEV), ws=ws)
    torch.cuda.synchronize()
    assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
    for b in range(B):
        grading.grade_assign(inputs.to_bits(Xs[b]), inputs.to_bits(Cs[b]), idx[b].cpu().numpy(), dist[b].cpu().numpy())


@pytest.mark.parametrize("N,D,K", [(4000, 640, 50), (3000, 1000, 300), (2500, 1536, 64)])
def test_wide_rows_lloyd_teacher_forced(N, D, K):
    X, _ = inputs.gaussian_mixture(N, D, K, 2.0, 1.0, N + K)
    C0 = inputs.sample_init(X, K, N)
    Xb = inputs.to_bits(X)
    Xd = X.to(DEV)
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    cur = C0.to(DEV)
    for _ in range(3):
        out = cake.cake_kmeans_lloyd(Xd, cur, 1, ws=ws)
        assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
        cb = inputs.to_bits(cur)
        idx = out.idx.cpu().numpy()
        grading.grade_assign(Xb, cb, idx, out.dist.cpu().numpy())
        grading.grade_update(Xb, idx, K, cb, out.C.cpu().numpy(), inputs.to_bits(out.C_bf16), out.counts.cpu().numpy())
        cur = out.C_bf16
    # one call of three iterations: the rows' operand is made once (iteration 1: prologue + row operand + assign + update
    # launches; later iterations: assign + update launches only) and the result is that of the three single steps above
    n0 = cake.cake_kmeans_kernel_launches()
    full = cake.cake_kmeans_lloyd(Xd, C0.to(DEV), 3, ws=ws)
    n3 = cake.cake_kmeans_kernel_launches() - n0
    n0 = cake.cake_kmeans_kernel_launches()
    cake.cake_kmeans_lloyd(Xd, C0.to(DEV), 1, ws=ws)
    n1 = cake.cake_kmeans_kernel_launches() - n0
    assert n3 < 3 * n1, (n1, n3)
    assert torch.equal(full.idx, out.idx) and torch.equal(full.C_bf16, out.C_bf16) and torch.equal(full.counts, out.counts)
    # the first iteration starts from the same centroids as the oracle's free run (later ones may part at a near-tie)
    first = orc.lloyd(Xb, inputs.to_bits(C0), 1, round_centroids=True)
    np.testing.assert_allclose(full.inertia.cpu().numpy()[:1], first.inertia, rtol=grading.INERTIA_TOL)


def test_wide_rows_through_the_other_lloyd_entry_points():
    """The convergence-tolerance loop, the row-sharded loop (one rank) and the k-means++ seeding take rows of more than
    512 columns through the same route: equal to the plain Lloyd call, seeding graded against the oracle's draw rule."""
    from paper_2608_12629_b200 import sharded
    N, D, K = 3000, 640, 40
    X, _ = inputs.gaussian_mixture(N, D, K, 2.0, 1.0, 17)
    C0 = inputs.sample_init(X, K, 17)
    Xd, Cd = X.to(DEV), C0.to(DEV)
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    ref = cake.cake_kmeans_lloyd(Xd, Cd, 4, ws=ws)
    sh = sharded.cake_kmeans_lloyd_sharded(Xd, Cd, 4)
    assert torch.equal(sh.idx, ref.idx) and torch.equal(sh.C_bf16, ref.C_bf16) and torch.equal(sh.counts, ref.counts)
    tol, iters = cake.cake_kmeans_lloyd_tol(Xd, Cd, 4, 0.0, check_every=2, ws=ws)
    torch.cuda.synchronize()
    assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
    assert iters == 4 and torch.equal(tol.idx, ref.idx) and torch.equal(tol.C_bf16, ref.C_bf16)
    np.testing.assert_allclose(tol.inertia.cpu().numpy()[:4], ref.inertia.cpu().numpy(), rtol=1e-12)
    # seeding: every drawn row is distinct and the first one is the oracle's (u[0] picks a row uniformly)
    u = torch.rand(K, generator=torch.Generator().manual_seed(3)).float()
    Cs, rows = cake.cake_kmeans_init_plusplus(Xd, K, u.to(DEV))
    torch.cuda.synchronize()
    rows = rows.cpu().numpy()
    assert len(set(rows.tolist())) == K
    want = orc.kmeanspp(inputs.to_bits(X), K, u.numpy().astype(np.float64))
    assert rows[0] == want[0] and (rows == want).mean() >= 0.5
    assert torch.equal(Cs.cpu(), X[torch.from_numpy(rows).long()])
