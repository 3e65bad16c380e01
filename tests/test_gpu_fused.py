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
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    resident = (N + 127) // 128 <= 4 * sms                         # small enough for the one-launch form
    # one cooperative launch for all iterations, or the first prologue, then assign + division per iteration
    assert launches == (1 if resident else 1 + 2 * 4), launches
    b = cake.cake_kmeans_lloyd(Xd, Cd, 4, ws=ws, flags=cake.CAKE_LLOYD_NO_FUSE)
    assert torch.equal(a.idx, b.idx) and torch.equal(a.dist, b.dist) and torch.equal(a.counts, b.counts)
    assert torch.equal(a.C, b.C) and torch.equal(a.C_bf16, b.C_bf16)
    np.testing.assert_allclose(a.inertia.cpu().numpy(), b.inertia.cpu().numpy(), rtol=1e-9)
    assert int(a.counts.sum()) == N
    if resident:      # ... and the two-launch form of the single-pass iteration agrees with both
        n0 = cake.cake_kmeans_kernel_launches()
        c = cake.cake_kmeans_lloyd(Xd, Cd, 4, ws=ws, flags=cake.CAKE_LLOYD_NO_RESIDENT)
        assert cake.cake_kmeans_kernel_launches() - n0 == 1 + 2 * 4
        assert torch.equal(a.idx, c.idx) and torch.equal(a.dist, c.dist) and torch.equal(a.counts, c.counts)
        assert torch.equal(a.C, c.C) and torch.equal(a.C_bf16, c.C_bf16)


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


@pytest.mark.parametrize("N,D,K", [(1, 64, 1), (300, 64, 7), (18944, 64, 128), (32768, 64, 128), (75776, 64, 100),
                                   (40000, 128, 128), (75776, 128, 33), (5000, 128, 1), (9000, 8, 5), (30000, 24, 40),
                                   (50000, 32, 128), (20000, 72, 100), (60000, 96, 77), (33333, 120, 128)])
def test_one_launch_form_teacher_forced_and_against_the_two_launch_form(N, D, K):
    """All iterations in one cooperative kernel (rows resident in shared memory, grid barriers): every iteration graded by
    the oracle (teacher-forced), the run equal to the two-launch form in assignments, and repeatable bit for bit (its
    partial sums are added in a fixed order)."""
    X, _ = inputs.gaussian_mixture(N, D, max(K, 2), 2.0, 1.0, N + K)
    C0 = inputs.sample_init(X, K, N)
    Xb = inputs.to_bits(X)
    Xd = X.to(DEV)
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    cur = C0.to(DEV)
    for _ in range(3):
        n0 = cake.cake_kmeans_kernel_launches()
        out = cake.cake_kmeans_lloyd(Xd, cur, 1, ws=ws)
        assert cake.cake_kmeans_kernel_launches() - n0 == 1
        assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
        cb = inputs.to_bits(cur)
        idx = out.idx.cpu().numpy()
        grading.grade_assign(Xb, cb, idx, out.dist.cpu().numpy())
        grading.grade_update(Xb, idx, K, cb, out.C.cpu().numpy(), inputs.to_bits(out.C_bf16), out.counts.cpu().numpy())
        assert abs(float(out.inertia[0]) - float(out.dist.double().sum())) <= 1e-9 * max(1.0, float(out.inertia[0]))
        cur = out.C_bf16
    a = cake.cake_kmeans_lloyd(Xd, C0.to(DEV), 5, ws=ws)
    b = cake.cake_kmeans_lloyd(Xd, C0.to(DEV), 5, ws=ws)
    assert torch.equal(a.idx, b.idx) and torch.equal(a.C, b.C) and torch.equal(a.C_bf16, b.C_bf16) and torch.equal(a.dist, b.dist)
    c = cake.cake_kmeans_lloyd(Xd, C0.to(DEV), 5, ws=ws, flags=cake.CAKE_LLOYD_NO_RESIDENT)
    torch.cuda.synchronize()
    assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
    assert (a.idx != c.idx).float().mean().item() <= 1e-3           # (fp32 sums in another order: a near-tie may flip)
    np.testing.assert_allclose(a.inertia.cpu().numpy(), c.inertia.cpu().numpy(), rtol=1e-4)


def test_one_launch_form_without_optional_outputs_and_through_the_tolerance_loop():
    N, D, K = 20000, 64, 50
    X, _ = inputs.gaussian_mixture(N, D, K, 2.0, 1.0, 9)
    C0 = inputs.sample_init(X, K, 9)
    Xd, Cd = X.to(DEV), C0.to(DEV)
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    ref = cake.cake_kmeans_lloyd(Xd, Cd, 6, ws=ws)
    tol, iters = cake.cake_kmeans_lloyd_tol(Xd, Cd, 6, 0.0, check_every=2, ws=ws)
    torch.cuda.synchronize()
    assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
    assert iters == 6 and torch.equal(tol.idx, ref.idx) and torch.equal(tol.C_bf16, ref.C_bf16)
    np.testing.assert_allclose(tol.inertia.cpu().numpy()[:6], ref.inertia.cpu().numpy(), rtol=1e-9)
    assert (np.diff(ref.inertia.cpu().numpy()) <= 0).all()
