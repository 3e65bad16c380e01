"""GPU tests of the two conveniences around the Lloyd loop: k-means++ seeding and the convergence test.

Seeding is teacher-forced: a draw depends on all earlier ones, and where the target falls within rounding of a
boundary of the running sums several rows are correct.  So for every draw the oracle recomputes, from the rows the
GPU chose before it, the fp64 running sums, and the GPU's row must be one whose interval of the running sum contains
the target up to 1e-5 of the total (the GPU's distances are fp32); what is unique (row 0, rows drawn with a clear
margin, no row drawn twice) is compared exactly.
"""
import numpy as np
import pytest
import torch

import paper_2608_12629_b200 as cake
from oracle import kmeans_oracle as orc
from paper_2608_12629_b200 import inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def check_seeding(X, K, u, rows_gpu, C0_gpu):
    Xb = inputs.to_bits(X)
    Xf = orc.bf16_to_f64(Xb)
    N = X.shape[0]
    assert rows_gpu[0] == min(int(float(u[0]) * N), N - 1)
    assert np.array_equal(inputs.to_bits(C0_gpu), Xb[rows_gpu])               # the centroids ARE the chosen rows
    mind = np.full(N, np.inf)
    clear = 0
    for k in range(1, K):
        diff = Xf - Xf[rows_gpu[k - 1]]
        mind = np.minimum(mind, (diff * diff).sum(1))
        want, cum = orc.kmeanspp_step(mind, float(u[k]))
        total = cum[-1]
        g = int(rows_gpu[k])
        if not total > 0:
            assert g == want
            continue
        target = float(u[k]) * total
        lo = cum[g - 1] if g > 0 else 0.0
        assert lo - 1e-5 * total <= target <= cum[g] + 1e-5 * total, (k, g, want)
        assert mind[g] > 0, "a row at distance 0 from the chosen set was drawn"
        if min(abs(target - (cum[want - 1] if want > 0 else 0.0)), abs(cum[want] - target)) > 3e-5 * total:
            assert g == want, (k, g, want)                                      # clear margin: the draw is unique
            clear += 1
    return clear


@pytest.mark.parametrize("N,D,K", [(5000, 64, 40), (3000, 128, 64), (2000, 24, 30), (1500, 100, 12), (4097, 8, 17), (64, 64, 64)])
def test_kmeanspp_seeding_teacher_forced(N, D, K):
    X, _ = inputs.gaussian_mixture(N, D, 16, 2.0, 0.5, N + K)
    u = torch.rand(K, generator=torch.Generator().manual_seed(K)).float()
    C0, rows = cake.cake_kmeans_init_plusplus(X.to(DEV), K, u.to(DEV))
    torch.cuda.synchronize()
    rows = rows.cpu().numpy()
    assert len(set(rows.tolist())) == K
    clear = check_seeding(X, K, u.numpy(), rows, C0.cpu())
    assert clear >= (K - 1) * 0.3         # (a row's share of the total is about 1/N: many targets lie near a boundary)
    # and where no draw was a close call the free-running oracle agrees on every row
    if clear == K - 1:
        assert np.array_equal(rows, orc.kmeanspp(inputs.to_bits(X), K, u.numpy().astype(np.float64)))


def test_kmeanspp_all_points_equal_and_single_centroid():
    X = torch.ones(300, 64).to(torch.bfloat16)
    u = torch.tensor([0.0, 0.5, 0.99]).float()
    C0, rows = cake.cake_kmeans_init_plusplus(X.to(DEV), 3, u.to(DEV))
    assert rows.cpu().tolist() == [0, 150, 297]                                 # nothing to weigh by: uniform rows
    C1, r1 = cake.cake_kmeans_init_plusplus(X.to(DEV), 1, u[:1].to(DEV))
    assert r1.cpu().tolist() == [0] and torch.equal(C1.cpu(), X[:1])


def test_kmeanspp_seeds_a_lloyd_run_with_lower_inertia_than_sampled_rows():
    X, _ = inputs.gaussian_mixture(20000, 64, 50, 3.0, 0.3, 9)
    Xd = X.to(DEV)
    u = torch.rand(50, generator=torch.Generator().manual_seed(3)).float().to(DEV)
    Cpp, _ = cake.cake_kmeans_init_plusplus(Xd, 50, u)
    a = cake.cake_kmeans_lloyd(Xd, Cpp, 1)
    b = cake.cake_kmeans_lloyd(Xd, inputs.sample_init(X, 50, 9).to(DEV), 1)
    assert float(a.inertia[0]) < float(b.inertia[0])                            # spread-out seeds start closer


@pytest.mark.parametrize("check_every", [1, 3])
def test_lloyd_tol_stops_where_its_own_inertia_says(check_every):
    X, _ = inputs.gaussian_mixture(8000, 64, 20, 3.0, 0.5, 4)
    C0 = inputs.sample_init(X, 20, 4)
    Xd, Cd = X.to(DEV), C0.to(DEV)
    tol, max_iters = 1e-4, 40
    out, n = cake.cake_kmeans_lloyd_tol(Xd, Cd, max_iters, tol, check_every)
    full = cake.cake_kmeans_lloyd(Xd, Cd, max_iters)
    ine = full.inertia.cpu().numpy()
    # the first iteration whose decrease is within tol, rounded up to the end of its block
    hit = next((t for t in range(1, max_iters) if ine[t - 1] - ine[t] <= tol * ine[t - 1]), None)
    assert hit is not None and hit < max_iters - 3
    want = min(max_iters, ((hit + 1 + check_every - 1) // check_every) * check_every)
    assert n == want
    np.testing.assert_allclose(out.inertia.cpu().numpy(), ine[:n], rtol=1e-12)
    ref = cake.cake_kmeans_lloyd(Xd, Cd, n)
    assert torch.equal(out.idx, ref.idx) and torch.equal(out.C_bf16, ref.C_bf16) and torch.equal(out.counts, ref.counts)
    # the oracle's own rounded trajectory stops in the same block (free run: inertia within 1e-3)
    r = orc.lloyd(inputs.to_bits(X), inputs.to_bits(C0), n, round_centroids=True)
    np.testing.assert_allclose(out.inertia.cpu().numpy(), r.inertia, rtol=1e-3)


def test_lloyd_tol_runs_to_max_iters_and_checks_arguments():
    X, _ = inputs.gaussian_mixture(3000, 64, 10, 2.0, 1.0, 2)
    Xd, Cd = X.to(DEV), inputs.sample_init(X, 10, 2).to(DEV)
    out, n = cake.cake_kmeans_lloyd_tol(Xd, Cd, 5, 0.0, 2)         # tol 0: only an exact fixed point would stop it
    assert n == 5 and out.inertia.numel() == 5
    with pytest.raises(cake.CakeError) as e:
        cake.cake_kmeans_lloyd_tol(Xd, Cd, 0, 1e-3, 1)
    assert e.value.code == cake.CAKE_ERR_SHAPE
