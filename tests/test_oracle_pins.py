"""Pins for the fp64 CPU oracle: every check compares it with something other than itself.

The paper (Section 5, "Flash-KMeans clean-start workload") defines the two kernels in words only
and prints no numeric K-means result, so the pins are the mathematics: brute force in other
libraries, exact integer cases, closed forms, invariants, and a hand-worked example carried out in
exact rational arithmetic.
"""
import json
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import kmeans_oracle as orc
from paper_2608_12629_b200 import inputs

HERE = os.path.dirname(os.path.abspath(__file__))


def bits_of(a):
    """float array (values must be bf16-exact or will be rounded) -> bf16 bits via torch."""
    t = torch.as_tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)
    return inputs.to_bits(t)


def vals_of(bits):
    return inputs.from_bits(bits).to(torch.float64).numpy()


def rand_bits(rng, shape, scale=1.0):
    return bits_of(rng.standard_normal(shape) * scale)


# ----------------------------------------------------------------------------- conversions

def test_bf16_widening_matches_torch():
    allbits = np.arange(0, 1 << 16, dtype=np.uint16)
    finite = allbits[((allbits >> 7) & 0xFF) != 0xFF]
    got = orc.bf16_to_f64(finite)
    want = inputs.from_bits(finite).to(torch.float64).numpy()
    assert np.array_equal(got, want)


def test_bf16_rounding_matches_torch_and_hand_values():
    rng = np.random.default_rng(0)
    v = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.integers(-6, 6, 20000),
                        [0.0, -0.0, 1.0, 2 / 3, 32 / 3, 1.00390625, 1.01171875]])
    got = orc.f64_to_bf16(v)
    want = inputs.to_bits(torch.from_numpy(v).to(torch.float32).to(torch.bfloat16))
    assert np.array_equal(got, want)
    # hand values: bf16 keeps 8 significant bits; 2/3 -> 171/256, 32/3 -> 171/16
    assert vals_of(orc.f64_to_bf16(np.array([2 / 3, 32 / 3])).reshape(1, 2)).tolist() == [[171 / 256, 171 / 16]]
    # ties to even: 1 + 2^-8 is halfway between 1 and 1+2^-7 -> 1 ; 1 + 3*2^-8 -> 1 + 2^-6
    assert vals_of(orc.f64_to_bf16(np.array([1 + 2 ** -8, 1 + 3 * 2 ** -8])).reshape(1, 2)).tolist() == \
        [[1.0, 1 + 2 ** -6]]


# ----------------------------------------------------------------------------- assign

@pytest.mark.parametrize("N,K,D", [(1, 1, 1), (7, 3, 2), (64, 8, 4), (33, 5, 3), (50, 50, 16)])
def test_assign_vs_numpy_and_scipy_bruteforce(N, K, D):
    from scipy.spatial.distance import cdist
    rng = np.random.default_rng(N * 100 + K * 10 + D)
    Xb, Cb = rand_bits(rng, (N, D)), rand_bits(rng, (K, D))
    X, C = vals_of(Xb), vals_of(Cb)
    idx, dist, second = orc.assign(Xb, Cb)
    d_np = ((X[:, None, :] - C[None, :, :]) ** 2).sum(-1)
    d_sp = cdist(X, C, "sqeuclidean")
    assert np.array_equal(idx, d_np.argmin(1))
    assert np.array_equal(idx, d_sp.argmin(1))
    np.testing.assert_allclose(dist, d_np.min(1), rtol=1e-13, atol=0)
    np.testing.assert_allclose(dist, d_sp.min(1), rtol=1e-12, atol=1e-300)
    if K > 1:
        np.testing.assert_allclose(second, np.sort(d_np, 1)[:, 1], rtol=1e-13)
    else:
        assert np.all(np.isinf(second))


def test_assign_integer_inputs_are_exact():
    rng = np.random.default_rng(5)
    Xi = rng.integers(-8, 9, (200, 6))
    Ci = rng.integers(-8, 9, (17, 6))
    idx, dist, second = orc.assign(bits_of(Xi), bits_of(Ci))
    d = ((Xi[:, None, :] - Ci[None, :, :]) ** 2).sum(-1)          # int64, exact
    assert np.array_equal(idx, d.argmin(1))                         # first occurrence on ties
    assert np.array_equal(dist, d.min(1).astype(np.float64))
    assert np.array_equal(second, np.sort(d, 1)[:, 1].astype(np.float64))
    assert (d == d.min(1, keepdims=True)).sum(1).max() > 1, "case must contain exact ties"


def test_assign_tie_goes_to_lowest_index():
    idx, dist, second = orc.assign(bits_of([[1.0, 0.0]]), bits_of([[0.0, 0.0], [2.0, 0.0]]))
    assert idx.tolist() == [0] and dist.tolist() == [1.0] and second.tolist() == [1.0]
    # duplicate centroids: the later copy never wins
    idx, _, _ = orc.assign(bits_of([[3.0, 3.0], [0.0, 0.0]]), bits_of([[0, 0], [3, 3], [3, 3], [0, 0]]))
    assert idx.tolist() == [1, 0]


def test_assign_special_cases():
    rng = np.random.default_rng(11)
    Xb = rand_bits(rng, (40, 5))
    # K = 1
    idx, dist, _ = orc.assign(Xb, Xb[:1])
    assert not idx.any()
    np.testing.assert_allclose(dist, ((vals_of(Xb) - vals_of(Xb[:1])) ** 2).sum(1), rtol=1e-14)
    # C = X (distinct rows): identity, zero distance
    assert len({r.tobytes() for r in Xb}) == 40
    idx, dist, second = orc.assign(Xb, Xb)
    assert np.array_equal(idx, np.arange(40)) and not dist.any() and (second > 0).all()
    # D = 1, sorted centroids: decision boundaries are the midpoints
    c = np.array([-4.0, -1.0, 0.5, 3.0])
    x = np.linspace(-6, 6, 193)                       # multiples of 1/16: bf16-exact
    idx, _, _ = orc.assign(bits_of(x[:, None]), bits_of(c[:, None]))
    mids = (c[1:] + c[:-1]) / 2
    want = np.searchsorted(mids, x, side="left")      # x == midpoint -> lower index
    assert np.array_equal(idx, want)


def test_assign_recovers_labels_of_separated_mixture():
    X, labels = inputs.gaussian_mixture(3000, 8, 12, 50.0, 0.01, seed=3)
    means = torch.stack([X[labels == j].float().mean(0) for j in range(12)]).to(torch.bfloat16)
    idx, _, _ = orc.assign(inputs.to_bits(X), inputs.to_bits(means))
    assert np.array_equal(idx, labels.numpy())


def test_assign_invariances():
    rng = np.random.default_rng(21)
    Xb, Cb = rand_bits(rng, (300, 7)), rand_bits(rng, (13, 7))
    idx, dist, _ = orc.assign(Xb, Cb)
    p = rng.permutation(300)
    idx_p, dist_p, _ = orc.assign(Xb[p], Cb)
    assert np.array_equal(idx_p, idx[p]) and np.array_equal(dist_p, dist[p])
    q = rng.permutation(13)
    idx_q, dist_q, _ = orc.assign(Xb, Cb[q])
    assert np.array_equal(q[idx_q], idx) and np.array_equal(dist_q, dist)
    # translating X and C by the same vector leaves distances unchanged; use small integers plus
    # an integer shift so that every translated value is still exact in bf16
    Xi, Ci = rng.integers(-20, 21, (300, 7)), rng.integers(-20, 21, (13, 7))
    shift = rng.integers(-30, 31, 7)
    a = orc.assign(bits_of(Xi), bits_of(Ci))
    b = orc.assign(bits_of(Xi + shift), bits_of(Ci + shift))
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_assign_f64_centroids_and_pair_sqdist():
    rng = np.random.default_rng(8)
    Xb = rand_bits(rng, (100, 6))
    C = rng.standard_normal((9, 6))                   # not bf16-representable
    idx, dist, _ = orc.assign(Xb, C)
    d = ((vals_of(Xb)[:, None] - C[None]) ** 2).sum(-1)
    assert np.array_equal(idx, d.argmin(1))
    np.testing.assert_allclose(dist, d.min(1), rtol=1e-13)
    g = rng.integers(0, 9, 100).astype(np.int32)
    np.testing.assert_allclose(orc.pair_sqdist(Xb, C, g), d[np.arange(100), g], rtol=1e-13)


# ----------------------------------------------------------------------------- update

def test_update_mean_mass_and_huygens():
    rng = np.random.default_rng(31)
    N, D, K = 500, 5, 7
    Xb = rand_bits(rng, (N, D), 3.0)
    X = vals_of(Xb)
    idx = rng.integers(0, K, N).astype(np.int32)
    C_new, counts, sums = orc.update(Xb, idx, K, None, return_sums=True)
    assert counts.sum() == N and np.array_equal(counts, np.bincount(idx, minlength=K))
    for k in range(K):                                 # separate loop, exact rationals
        rows = [i for i in range(N) if idx[i] == k]
        s = [sum(Fraction(float(X[i, d])) for i in rows) for d in range(D)]
        for d in range(D):
            assert abs(Fraction(float(sums[k, d])) - s[d]) <= abs(s[d]) * Fraction(1, 10 ** 13) + Fraction(1, 10 ** 13)
            assert abs(Fraction(float(C_new[k, d])) - s[d] / len(rows)) <= Fraction(1, 10 ** 12)
    # global mass
    np.testing.assert_allclose((counts[:, None] * C_new).sum(0), X.sum(0), rtol=1e-12, atol=1e-10)
    # Huygens: sum_i |x_i - c_a(i)|^2 = sum |x|^2 - sum_k n_k |c_k|^2 for exact means
    lhs = orc.pair_sqdist(Xb, C_new, idx).sum()
    rhs = (X ** 2).sum() - (counts * (C_new ** 2).sum(1)).sum()
    assert abs(lhs - rhs) <= 1e-11 * (X ** 2).sum()


def test_update_k1_closed_form():
    rng = np.random.default_rng(32)
    Xb = rand_bits(rng, (257, 4))
    X = vals_of(Xb)
    C_new, counts = orc.update(Xb, np.zeros(257, np.int32), 1)
    np.testing.assert_allclose(C_new[0], X.mean(0), rtol=1e-13, atol=1e-15)
    assert counts.tolist() == [257]
    inertia = orc.pair_sqdist(Xb, C_new, np.zeros(257, np.int32)).sum()
    assert abs(inertia - ((X ** 2).sum() - 257 * (X.mean(0) ** 2).sum())) < 1e-10


def test_update_empty_cluster_keeps_previous_bits():
    rng = np.random.default_rng(33)
    Xb = rand_bits(rng, (20, 3))
    prev_bits = rand_bits(rng, (4, 3))
    idx = np.array([0, 2] * 10, dtype=np.int32)        # clusters 1 and 3 stay empty
    C_new, counts = orc.update(Xb, idx, 4, prev_bits)
    assert counts.tolist() == [10, 0, 10, 0]
    assert np.array_equal(C_new[[1, 3]], vals_of(prev_bits)[[1, 3]])
    assert np.array_equal(orc.f64_to_bf16(C_new[[1, 3]]), prev_bits[[1, 3]])
    C_zero, _ = orc.update(Xb, idx, 4, None)
    assert not C_zero[[1, 3]].any()
    with pytest.raises(RuntimeError):
        orc.update(Xb, np.full(20, 4, np.int32), 4)


# ----------------------------------------------------------------------------- Lloyd

def test_lloyd_handworked_example_exact_rationals():
    g = json.load(open(os.path.join(HERE, "golden", "handworked_2d.json")))
    F = lambda p: Fraction(p[0], p[1])
    X = [[Fraction(v) for v in r] for r in g["X"]]
    Xb = bits_of(g["X"])
    C0b = Xb[g["C0_rows"]]

    # (a) the stored table is self-consistent under exact rational arithmetic
    def d2(x, c):
        return sum((a - b) ** 2 for a, b in zip(x, c))

    for it in g["iterations"]:
        C = [[F(v) if isinstance(v, list) else Fraction(v) for v in c] for c in it["C"]]
        for i, x in enumerate(X):
            dd = [d2(x, c) for c in C]
            stored = [F(v) if isinstance(v, list) else Fraction(v) for v in it["d"][i]]
            assert dd == stored
            assert it["idx"][i] == dd.index(min(dd))
        assert sum(min(d2(x, c) for c in C) for x in X) == F(it["inertia"])

    # (b) the oracle reproduces it: pure fp64 mode
    for t, it in enumerate(g["iterations"]):
        r = orc.lloyd(Xb, C0b, t + 1, round_centroids=False)
        assert r.idx.tolist() == it["idx"]
        assert r.inertia[t] == float(F(it["inertia"]))
        assert r.counts.tolist() == it["counts_after"]
    r = orc.lloyd(Xb, C0b, 4, round_centroids=False)
    assert r.idx.tolist() == g["t2_pure"]["idx"]
    assert abs(r.inertia[2] - float(F(g["t2_pure"]["inertia"]))) < 1e-13
    assert r.inertia[3] == r.inertia[2]                            # fixed point
    want = np.array([[float(F(v)) for v in c] for c in g["t2_pure"]["C"]])
    np.testing.assert_allclose(r.C, want, rtol=1e-15)

    # (c) bf16-rounded mode: centroids 171/256 and 171/16, inertia 349611/32768 exactly
    r = orc.lloyd(Xb, C0b, 4, round_centroids=True)
    want_b = np.array([[float(F(v)) for v in c] for c in g["t2_bf16_rounded"]["C"]])
    assert np.array_equal(vals_of(r.C_bits), want_b)
    assert r.inertia[0] == 576.0 and r.inertia[1] == 47.75
    assert r.inertia[2] == float(F(g["t2_bf16_rounded"]["inertia"])) == 10.669281005859375
    assert r.idx.tolist() == g["t2_bf16_rounded"]["idx"]

    # (d) K = 1
    r1 = orc.lloyd(Xb, Xb[:1], 2, round_centroids=False)
    np.testing.assert_allclose(r1.C[0], [17 / 3, 17 / 3], rtol=1e-15)
    assert abs(r1.inertia[1] - 932 / 3) < 1e-12


def test_lloyd_inertia_monotone_and_fixed_point():
    X, _ = inputs.gaussian_mixture(2000, 6, 9, 2.0, 1.0, seed=77)
    Xb = inputs.to_bits(X)
    C0b = inputs.to_bits(inputs.sample_init(X, 9, 77))
    r = orc.lloyd(Xb, C0b, 60, round_centroids=False)
    diffs = np.diff(r.inertia)
    assert (diffs <= 1e-12 * r.inertia[:-1]).all(), "inertia must never increase with exact means"
    assert diffs[0] < 0
    # fixed point reached: one more iteration changes nothing
    r2 = orc.lloyd(Xb, C0b, 61, round_centroids=False)
    if np.array_equal(r2.idx, r.idx):
        assert np.array_equal(r2.C, r.C) and r2.inertia[-1] == r2.inertia[-2]
    # rounded mode may rise by a bf16 rounding of the centroids, never by more
    rr = orc.lloyd(Xb, C0b, 30, round_centroids=True)
    assert (np.diff(rr.inertia) <= 1e-4 * rr.inertia[:-1]).all()


def test_lloyd_centroids_are_means_of_their_points():
    X, _ = inputs.gaussian_mixture(1500, 4, 6, 2.0, 1.0, seed=5)
    Xb = inputs.to_bits(X)
    C0b = inputs.to_bits(inputs.sample_init(X, 6, 5))
    r = orc.lloyd(Xb, C0b, 5, round_centroids=True)
    Xv = vals_of(Xb)
    for k in range(6):
        rows = Xv[r.idx == k]
        assert len(rows) == r.counts[k]
        if len(rows):
            np.testing.assert_allclose(r.C[k], rows.mean(0), rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("t", [1, 3, 8])
def test_lloyd_vs_sklearn(t):
    import warnings
    from sklearn.cluster import KMeans
    X, _ = inputs.gaussian_mixture(4000, 8, 10, 2.0, 1.0, seed=123)
    Xb = inputs.to_bits(X)
    C0 = inputs.sample_init(X, 10, 123)
    r = orc.lloyd(Xb, inputs.to_bits(C0), t, round_centroids=False)
    assert r.counts.min() > 0, "sklearn relocates empty clusters; the case must have none"
    with warnings.catch_warnings():
        warnings.simplefilter("ignore")
        km = KMeans(n_clusters=10, init=C0.to(torch.float64).numpy(), n_init=1, algorithm="lloyd",
                    tol=0.0, max_iter=t).fit(vals_of(Xb))
    np.testing.assert_allclose(r.C, km.cluster_centers_, rtol=1e-9, atol=1e-9)


def test_lloyd_teacher_forced_composition():
    """lloyd == assign followed by update, composed by hand (guards the loop's bookkeeping)."""
    X, _ = inputs.gaussian_mixture(800, 5, 7, 2.0, 1.0, seed=9)
    Xb = inputs.to_bits(X)
    Cb = inputs.to_bits(inputs.sample_init(X, 7, 9))
    r = orc.lloyd(Xb, Cb, 3, round_centroids=True)
    cur = Cb
    for t in range(3):
        idx, dist, _ = orc.assign(Xb, cur)
        assert abs(dist.sum() - r.inertia[t]) <= 1e-12 * dist.sum()
        C_new, counts = orc.update(Xb, idx, 7, cur)
        cur = orc.f64_to_bf16(C_new)
    assert np.array_equal(cur, r.C_bits) and np.array_equal(idx, r.idx) and np.array_equal(counts, r.counts)


# ------------------------------------------------------------------------------------ k nearest neighbours

def _knn_brute(Q, X, k):
    q, x = Q.double().numpy(), X.double().numpy()
    d = ((q[:, None, :] - x[None, :, :]) ** 2).sum(-1)
    order = np.stack([np.lexsort((np.arange(x.shape[0]), row)) for row in d])      # by distance, then row number
    idx = np.full((q.shape[0], k), -1, dtype=np.int64)
    dist = np.full((q.shape[0], k), np.inf)
    kk = min(k, x.shape[0])
    idx[:, :kk] = order[:, :kk]
    dist[:, :kk] = np.take_along_axis(d, order[:, :kk], 1)
    return idx, dist


@pytest.mark.parametrize("N,M,D,k", [(7, 50, 3, 1), (20, 200, 5, 8), (5, 64, 16, 32), (9, 10, 2, 10), (4, 6, 4, 9)])
def test_knn_vs_numpy_bruteforce(N, M, D, k):
    g = torch.Generator().manual_seed(N * M + k)
    Q = torch.randn(N, D, generator=g).to(torch.bfloat16)
    X = torch.randn(M, D, generator=g).to(torch.bfloat16)
    idx, dist = orc.knn(inputs.to_bits(Q), inputs.to_bits(X), k)
    bi, bd = _knn_brute(Q, X, k)
    assert np.array_equal(idx, bi)
    np.testing.assert_allclose(dist, bd, rtol=1e-13)
    # a second, independent selection: partition, then order the k survivors
    d = ((Q.double().numpy()[:, None] - X.double().numpy()[None]) ** 2).sum(-1)
    kk = min(k, M)
    part = np.argpartition(d, kk - 1, axis=1)[:, :kk]
    assert all(set(part[i]) == set(idx[i, :kk]) for i in range(N))          # random reals: no ties
    assert (np.diff(dist[:, :kk], axis=1) >= 0).all()


def test_knn_integer_ties_go_to_the_lower_row_and_k1_is_assign():
    g = torch.Generator().manual_seed(2)
    Q = torch.randint(-2, 3, (40, 6), generator=g).to(torch.bfloat16)
    X = torch.randint(-2, 3, (300, 6), generator=g).to(torch.bfloat16)
    X[100:200] = X[0:100]                                    # every one of these rows exists twice
    idx, dist = orc.knn(inputs.to_bits(Q), inputs.to_bits(X), 12)
    bi, bd = _knn_brute(Q, X, 12)
    assert np.array_equal(idx, bi) and np.array_equal(dist, bd)       # integers: exact, ties included
    d = dist
    tied = d[:, 1:] == d[:, :-1]
    assert tied.any() and (idx[:, 1:][tied] > idx[:, :-1][tied]).all()
    i1, d1 = orc.knn(inputs.to_bits(Q), inputs.to_bits(X), 1)
    ia, da, _ = orc.assign(inputs.to_bits(Q), inputs.to_bits(X))
    assert np.array_equal(i1[:, 0], ia) and np.array_equal(d1[:, 0], da)
    # a point that is in the database finds itself first, at distance 0
    i2, d2 = orc.knn(inputs.to_bits(X[:50]), inputs.to_bits(X), 3)
    assert np.array_equal(i2[:, 0], np.arange(50)) and (d2[:, 0] == 0).all()


# ------------------------------------------------------------------------------------ k-means++ seeding

def test_kmeanspp_hand_example_and_brute_force():
    # points 0, 1, 10 on a line: first row floor(0.1 * 3) = 0; then mind = (0, 1, 100), running sums (0, 1, 101):
    # u = 0.5 -> target 50.5 -> row 2; then mind = (0, 1, 0), sums (0, 1, 1): u = 0.999 -> target 0.999 -> row 1
    X = torch.tensor([[0.0], [1.0], [10.0]]).to(torch.bfloat16)
    assert orc.kmeanspp(inputs.to_bits(X), 3, np.array([0.1, 0.5, 0.999])).tolist() == [0, 2, 1]
    # u just below 1/101 still lands on row 1 (sum 1 > target), row 0 has no mass and can never be drawn again
    assert orc.kmeanspp(inputs.to_bits(X), 2, np.array([0.1, 0.009])).tolist() == [0, 1]
    # brute force with python floats and exact fractions of the bf16 values
    g = torch.Generator().manual_seed(5)
    Xr = torch.randint(-3, 4, (40, 3), generator=g).to(torch.bfloat16)
    u = np.random.default_rng(1).random(8)
    rows = orc.kmeanspp(inputs.to_bits(Xr), 8, u)
    pts = [[Fraction(float(v)) for v in row] for row in Xr.tolist()]
    want = [int(u[0] * 40)]
    for k in range(1, 8):
        mind = [min(sum((a - b) ** 2 for a, b in zip(p, pts[r])) for r in want) for p in pts]
        total, run, pick = sum(mind), Fraction(0), None
        for i, m in enumerate(mind):
            run += m
            if run > Fraction(u[k]) * total:
                pick = i
                break
        want.append(pick)
    assert rows.tolist() == want
    assert len(set(rows.tolist())) == 8                       # a chosen row has mind = 0: never drawn twice


def test_kmeanspp_degenerate_inputs():
    X = torch.ones(5, 4).to(torch.bfloat16)                    # all points coincide: draws fall back to uniform rows
    assert orc.kmeanspp(inputs.to_bits(X), 3, np.array([0.0, 0.5, 0.99])).tolist() == [0, 2, 4]
    assert orc.kmeanspp(inputs.to_bits(X[:1]), 1, np.array([0.7])).tolist() == [0]
