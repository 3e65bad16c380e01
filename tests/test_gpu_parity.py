"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU oracle.

Small shapes are compared element by element; the full-size workloads are compared on sampled rows
(assign is independent per row) and in full for update (linear cost).  Tolerances: tests/grading.py.
"""
import numpy as np
import pytest
import torch

import paper_2608_12629_b200 as cake
from oracle import kmeans_oracle as orc
from paper_2608_12629_b200 import inputs
from tests import grading

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def problem(N, D, K, seed, comps=None, mean_std=1.0, sigma=0.5):
    X, _ = inputs.gaussian_mixture(N, D, comps or max(1, min(K, 64)), mean_std, sigma, seed)
    C = inputs.sample_init(X, K, seed)
    return X, C


def sampled_rows(N, n, seed):
    return np.sort(np.random.default_rng(seed).choice(N, size=min(n, N), replace=False))


def check_status(ws, want=cake.CAKE_OK):
    assert cake.cake_kmeans_device_status(ws) == want


# ------------------------------------------------------------------------------------ assign

TC_SHAPES = [
    # N, D, K : single tile, ragged rows, ragged K, several K tiles, D tails (96, 72, 8), D=256, and
    # 256 < D <= 512 (one X buffer; five to eight 64-column chunks, full and partial)
    (1, 64, 1), (127, 64, 2), (128, 64, 256), (129, 128, 257), (1000, 128, 1000), (777, 96, 65),
    (4096, 128, 300), (300, 256, 700), (257, 16, 5), (1000, 8, 3), (2000, 72, 260), (333, 192, 513),
    (20000, 64, 128), (50, 128, 2048),
    (300, 264, 70), (1000, 288, 300), (515, 352, 1000), (2000, 480, 130), (700, 512, 600), (129, 504, 33),
    (40000, 320, 24), (30000, 384, 100), (25000, 264, 128),
]


TC_POLICIES = {"packed": cake.CAKE_ASSIGN_TCGEN05, "exact": cake.CAKE_ASSIGN_TCGEN05_EXACT}


@pytest.mark.parametrize("policy", sorted(TC_POLICIES))
@pytest.mark.parametrize("N,D,K", TC_SHAPES)
def test_assign_tcgen05_small_shapes(N, D, K, policy):
    X, C = problem(N, D, K, seed=N + D + K)
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    idx, dist = cake.cake_kmeans_assign(X.to(DEV), C.to(DEV), ws=ws, flags=TC_POLICIES[policy])
    torch.cuda.synchronize()
    check_status(ws)
    rep = grading.grade_assign(inputs.to_bits(X), inputs.to_bits(C), idx.cpu().numpy(), dist.cpu().numpy())
    assert rep["mismatch"] <= max(2, N // 1000), rep


@pytest.mark.parametrize("N,D,K", [(100, 5, 7), (300, 33, 40), (64, 130, 3), (1000, 64, 100), (200, 520, 9)])
def test_assign_simt_fallback(N, D, K):
    X, C = problem(N, D, K, seed=N * 3 + D)
    idx, dist = cake.cake_kmeans_assign(X.to(DEV), C.to(DEV), flags=cake.CAKE_ASSIGN_SIMT)
    grading.grade_assign(inputs.to_bits(X), inputs.to_bits(C), idx.cpu().numpy(), dist.cpu().numpy())
    if D % 8:  # the tensor path must refuse such D when asked for by name
        with pytest.raises(cake.CakeError) as e:
            cake.cake_kmeans_assign(X.to(DEV), C.to(DEV), flags=cake.CAKE_ASSIGN_TCGEN05)
        assert e.value.code == cake.CAKE_ERR_UNSUPPORTED
    if D > 512:           # rows too long for a resident X tile: the tensor cores stream them (automatically and by name)
        idx2, dist2 = cake.cake_kmeans_assign(X.to(DEV), C.to(DEV))
        grading.grade_assign(inputs.to_bits(X), inputs.to_bits(C), idx2.cpu().numpy(), dist2.cpu().numpy())
        idx3, dist3 = cake.cake_kmeans_assign(X.to(DEV), C.to(DEV), flags=cake.CAKE_ASSIGN_TCGEN05)
        assert torch.equal(idx2, idx3) and torch.equal(dist2, dist3)


@pytest.mark.parametrize("B,N,D,K", [(1, 100, 5, 7), (1, 3000, 33, 40), (2, 640, 130, 300), (1, 20000, 100, 1000),
                                     (3, 257, 1, 2), (1, 1000, 12, 6), (1, 500, 509, 77), (1, 129, 255, 257)])
def test_assign_feature_count_not_multiple_of_8(B, N, D, K):
    """The automatic route copies X and C into zero-padded rows and runs the tensor-core kernel on them:
    same grading as any other shape, and a Lloyd call (which pads X once) agrees with step-by-step calls."""
    g = torch.Generator().manual_seed(N + D)
    X = torch.randint(-4, 5, (B, N, D), generator=g).to(torch.bfloat16)   # small integers: sums exact in any order
    C = torch.randint(-4, 5, (B, K, D), generator=g).to(torch.bfloat16) + 0.25
    ws = cake.alloc_workspace(B, N, D, K, DEV)
    Xd, Cd = X.to(DEV), C.to(DEV)
    launches = cake.cake_kmeans_kernel_launches()
    idx, dist = cake.cake_kmeans_assign(Xd, Cd, ws=ws)
    assert cake.cake_kmeans_kernel_launches() - launches == 3      # copy of X, prologue, tensor-core kernel
    check_status(ws)
    for b in range(B):
        grading.grade_assign(inputs.to_bits(X[b]), inputs.to_bits(C[b]), idx[b].cpu().numpy(), dist[b].cpu().numpy())
    out = cake.cake_kmeans_lloyd(Xd, Cd, 3, ws=ws)
    check_status(ws)
    Cc = Cd
    for _ in range(3):
        i2, d2 = cake.cake_kmeans_assign(Xd, Cc, ws=ws)
        Cf, Cb, counts = cake.cake_kmeans_update(Xd, i2, K, C_prev=Cc, ws=ws)
        Cc = Cb
    assert torch.equal(out.idx, i2) and torch.equal(out.dist, d2) and torch.equal(out.counts, counts)
    assert torch.equal(out.C, Cf) and torch.equal(out.C_bf16, Cb)


@pytest.mark.parametrize("policy", sorted(TC_POLICIES))
def test_assign_exact_ties_lowest_index(policy):
    """Small integers: every product, norm and sum is exact in fp32, so ties are exact on the GPU too."""
    g = torch.Generator().manual_seed(4)
    N, D, K = 3000, 64, 600
    X = torch.randint(-2, 3, (N, D), generator=g).to(torch.bfloat16)
    C = torch.randint(-2, 3, (K, D), generator=g).to(torch.bfloat16)
    C[17] = C[5]
    C[300:600] = C[0:300]            # every centroid duplicated across the two K tiles and column halves
    idx, dist = cake.cake_kmeans_assign(X.to(DEV), C.to(DEV), flags=TC_POLICIES[policy])
    idx_o, dist_o, _ = orc.assign(inputs.to_bits(X), inputs.to_bits(C))
    assert np.array_equal(idx.cpu().numpy(), idx_o)
    assert np.array_equal(dist.cpu().numpy().astype(np.float64), dist_o)
    assert idx_o.max() < 300


def test_assign_batched_matches_per_problem_and_oracle():
    B, N, D, K = 5, 700, 128, 300
    Xs, Cs = zip(*(problem(N, D, K, seed=50 + b) for b in range(B)))
    X, C = torch.stack(Xs).to(DEV), torch.stack(Cs).to(DEV)
    ws = cake.alloc_workspace(B, N, D, K, DEV)
    idx, dist = cake.cake_kmeans_assign(X, C, ws=ws)
    check_status(ws)
    for b in range(B):
        grading.grade_assign(inputs.to_bits(Xs[b]), inputs.to_bits(Cs[b]), idx[b].cpu().numpy(),
                             dist[b].cpu().numpy())
        i1, d1 = cake.cake_kmeans_assign(X[b].contiguous(), C[b].contiguous())
        assert torch.equal(i1, idx[b]) and torch.equal(d1, dist[b])


@pytest.mark.parametrize("B,N,D,K", [(200, 300, 64, 100), (150, 513, 128, 256), (67, 700, 192, 7), (90, 400, 96, 200),
                                     (40, 700, 320, 60), (35, 900, 384, 128)])
def test_assign_many_small_problems_single_centroid_tile(B, N, D, K):
    """One centroid tile per row tile with the tile resident in shared memory: every CTA meets several
    problems (the resident tile is reloaded, both MMA issuers hand it back), row tiles alternate between
    the two issuers / epilogue warpgroups, odd and even tile counts per CTA; inertia per problem."""
    g = torch.Generator().manual_seed(B + N + D)
    X = torch.randn(B, N, D, generator=g).to(torch.bfloat16)
    C = (torch.randn(B, K, D, generator=g) * (1 + torch.arange(B).view(B, 1, 1) % 3)).to(torch.bfloat16)
    Xd, Cd = X.to(DEV), C.to(DEV)
    ws = cake.alloc_workspace(B, N, D, K, DEV)
    idx, dist = cake.cake_kmeans_assign(Xd, Cd, ws=ws)
    check_status(ws)
    for b in range(0, B, max(1, B // 7)):
        grading.grade_assign(inputs.to_bits(X[b]), inputs.to_bits(C[b]), idx[b].cpu().numpy(), dist[b].cpu().numpy())
    # the exact epilogue must agree on the distances it reports, and a second call must reproduce the first
    idx2, dist2 = cake.cake_kmeans_assign(Xd, Cd, ws=ws)
    assert torch.equal(idx, idx2) and torch.equal(dist, dist2)
    out = cake.cake_kmeans_lloyd(Xd, Cd, 1, ws=ws)
    assert torch.equal(out.idx, idx)
    np.testing.assert_allclose(out.inertia[:, 0].cpu().numpy(), dist.double().sum(-1).cpu().numpy(), rtol=1e-9)


def test_assign_many_row_tiles_few_centroids_and_single_buffer_shapes():
    """Row tiles far beyond the SM count with 1-2 centroid tiles (deep X prefetch), and D=256 with
    many centroid tiles (single X buffer)."""
    for N, D, K, sample in [(148 * 128 * 3 + 77, 128, 300, 3000), (40000, 256, 2304, 600), (33333, 64, 64, 3000)]:
        X, C = problem(N, D, K, seed=N % 1000 + K)
        ws = cake.alloc_workspace(1, N, D, K, DEV)
        idx, dist = cake.cake_kmeans_assign(X.to(DEV), C.to(DEV), ws=ws)
        check_status(ws)
        rows = sampled_rows(N, sample, K)
        grading.grade_assign(inputs.to_bits(X), inputs.to_bits(C), idx.cpu().numpy(), dist.cpu().numpy(), rows=rows)


@pytest.mark.parametrize("N,D,K,order", [(3000, 64, 16384, "random"), (2500, 32, 20000, "random"), (1500, 128, 33000, "random"),
                                         (1200, 200, 16400, "random"), (1000, 256, 16500, "random"),
                                         (2000, 64, 16384, "closer_later"), (2000, 128, 16384, "closer_later"),
                                         (2000, 64, 16384, "duplicates"), (1500, 128, 20000, "duplicates")])
def test_assign_gated_epilogue_from_64_centroid_tiles(N, D, K, order):
    """From 64 centroid tiles per row tile the epilogue first takes a 32-column group's smallest raw accumulator and
    builds the keys only where some row can still improve.  Graded by the oracle, and bit-identical to the CTA-pair
    kernel, which has the same arithmetic and no gate: on unordered centroids, on centroids ordered so that later tiles
    keep winning (every group passes the gate), and with every centroid repeated half the table later (an equal value
    in a later tile must not replace the earlier one)."""
    both, _ = inputs.gaussian_mixture(N + K, D, 48, 1.0, 0.5, N + K + D)
    X, C = both[:N].contiguous(), both[N:].contiguous()
    if order == "closer_later":
        far = ((C.float() - X.float().mean(0)) ** 2).sum(1)
        C = C[torch.argsort(far, descending=True)].contiguous()
    if order == "duplicates":
        g = torch.Generator().manual_seed(K)
        X = torch.randint(-3, 4, (N, D), generator=g).to(torch.bfloat16)
        C = torch.randint(-3, 4, (K, D), generator=g).to(torch.bfloat16)
        C[K // 2:] = C[:K - K // 2]
    Xd, Cd = X.to(DEV), C.to(DEV)
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    idx, dist = cake.cake_kmeans_assign(Xd, Cd, ws=ws, flags=cake.CAKE_ASSIGN_TCGEN05)
    check_status(ws)
    grading.grade_assign(inputs.to_bits(X), inputs.to_bits(C), idx.cpu().numpy(), dist.cpu().numpy())
    ip, dp = cake.cake_kmeans_assign(Xd, Cd, ws=ws, flags=cake.CAKE_ASSIGN_TCGEN05_PAIR)
    check_status(ws)
    assert torch.equal(idx, ip) and torch.equal(dist, dp)
    if order == "duplicates":
        assert int(idx.max()) < K - K // 2                      # the first copy of the winning centroid


def test_assign_edge_cases():
    X, C = problem(64, 64, 4, seed=1)
    # N = 0
    idx, dist = cake.cake_kmeans_assign(X[:0].to(DEV), C.to(DEV))
    assert idx.numel() == 0
    # K > N, and C = X gives the identity with zero distance
    Xd = X.to(DEV)
    idx, dist = cake.cake_kmeans_assign(Xd, Xd.clone())
    rows = inputs.to_bits(X)
    first = {}
    for i, r in enumerate(rows):
        first.setdefault(r.tobytes(), i)
    want = np.array([first[r.tobytes()] for r in rows])
    assert np.array_equal(idx.cpu().numpy(), want)
    assert float(dist.max()) <= 1e-3 * float((X.float() ** 2).sum(1).max()) * 2
    # no dist requested
    idx2, none = cake.cake_kmeans_assign(Xd, C.to(DEV), want_dist=False)
    assert none is None
    # workspace too small / misaligned / null
    ws = cake.alloc_workspace(1, 64, 64, 4, DEV)
    with pytest.raises(cake.CakeError) as e:
        cake.cake_kmeans_assign(Xd, C.to(DEV), ws=ws[:1024])
    assert e.value.code == cake.CAKE_ERR_WORKSPACE
    with pytest.raises(cake.CakeError) as e:
        cake.cake_kmeans_assign(Xd, C.to(DEV), ws=ws[8:])
    assert e.value.code == cake.CAKE_ERR_ALIGN


# ------------------------------------------------------------------------------------ update

UPD_SHAPES = [(1, 64, 1), (1000, 64, 128), (5000, 128, 256), (333, 96, 17), (4097, 256, 64), (2500, 8, 3),
              (3000, 128, 3000)]


@pytest.mark.parametrize("path", ["smem", "sort"])
@pytest.mark.parametrize("N,D,K", UPD_SHAPES)
def test_update_paths(path, N, D, K):
    flag = cake.CAKE_UPDATE_SMEM if path == "smem" else cake.CAKE_UPDATE_SORT
    if path == "smem" and K * D * 4 + K * 4 > 227 * 1024:
        pytest.skip("table does not fit in shared memory")
    X, C = problem(N, D, K, seed=N + K)
    g = torch.Generator().manual_seed(N)
    idx = torch.randint(0, K, (N,), generator=g, dtype=torch.int32)
    if K > 4:
        idx[idx == 1] = 0                      # cluster 1 empty, cluster 0 heavy
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    Cf, Cb, counts = cake.cake_kmeans_update(X.to(DEV), idx.to(DEV), K, C_prev=C.to(DEV), ws=ws, flags=flag)
    check_status(ws)
    grading.grade_update(inputs.to_bits(X), idx.numpy(), K, inputs.to_bits(C), Cf.cpu().numpy(),
                         inputs.to_bits(Cb), counts.cpu().numpy())


@pytest.mark.parametrize("N,D,K", [(70001, 64, 100), (9000, 128, 9000), (40000, 32, 20000), (8193, 16, 8193)])
def test_update_sort_route_slab_tails_and_large_k(N, D, K):
    """Ragged slabs (N not a multiple of 4 or of the slab), and K above the shared-memory histogram limit."""
    X, C = problem(N, D, K, seed=N + D)
    g = torch.Generator().manual_seed(K)
    idx = torch.randint(0, K, (N,), generator=g, dtype=torch.int32)
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    Cf, Cb, counts = cake.cake_kmeans_update(X.to(DEV), idx.to(DEV), K, C_prev=C.to(DEV), ws=ws,
                                             flags=cake.CAKE_UPDATE_SORT)
    check_status(ws)
    grading.grade_update(inputs.to_bits(X), idx.numpy(), K, inputs.to_bits(C), Cf.cpu().numpy(),
                         inputs.to_bits(Cb), counts.cpu().numpy())


SLAB_FLAGS = {"auto": cake.CAKE_UPDATE_SLAB, "f1": cake.CAKE_UPDATE_SLAB_F1, "f2": cake.CAKE_UPDATE_SLAB_F2,
              "f4": cake.CAKE_UPDATE_SLAB_F4}


@pytest.mark.parametrize("f", ["auto", "f1", "f2", "f4"])
@pytest.mark.parametrize("N,D,K", [(1, 64, 1), (1000, 64, 128), (70001, 64, 100), (20000, 128, 3000), (8193, 16, 8192),
                                   (50003, 96, 17), (300001, 128, 1024), (33000, 256, 512), (2500, 8, 3),
                                   (20001, 288, 500), (9000, 512, 100), (5000, 1000, 64), (3000, 1024, 7)])
def test_update_slab_route(f, N, D, K):
    """Slab route: ragged last slab, N % 4 != 0, clusters of 1, 2 and 4 CTAs (also with CTAs that get no
    rows), K at the shared-memory limit, D that does not fill the lane group, D > 256 (several column
    passes, the last one partial)."""
    X, C = problem(N, D, K, seed=N + D)
    g = torch.Generator().manual_seed(K)
    idx = torch.randint(0, K, (N,), generator=g, dtype=torch.int32)
    if K > 4:
        idx[idx == 1] = 0                      # cluster 1 empty, cluster 0 heavy
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    Cf, Cb, counts = cake.cake_kmeans_update(X.to(DEV), idx.to(DEV), K, C_prev=C.to(DEV), ws=ws, flags=SLAB_FLAGS[f])
    check_status(ws)
    grading.grade_update(inputs.to_bits(X), idx.numpy(), K, inputs.to_bits(C), Cf.cpu().numpy(),
                         inputs.to_bits(Cb), counts.cpu().numpy())


def test_update_slab_route_refuses_what_it_cannot_run():
    X, C = problem(100, 12, 4, seed=1)
    idx = torch.zeros(100, dtype=torch.int32)
    with pytest.raises(cake.CakeError) as e:
        cake.cake_kmeans_update(X.to(DEV), idx.to(DEV), 4, C_prev=C.to(DEV), flags=cake.CAKE_UPDATE_SLAB)
    assert e.value.code == cake.CAKE_ERR_UNSUPPORTED


@pytest.mark.parametrize("flag", [cake.CAKE_UPDATE_SORT, cake.CAKE_UPDATE_SLAB, cake.CAKE_UPDATE_SLAB_F2])
def test_update_batched_unaligned_problem_size(flag):
    """B > 1 with N % 4 != 0: the per-problem idx slices are not 16-byte aligned."""
    B, N, D, K = 3, 10001, 64, 37
    Xs, Cs = zip(*(problem(N, D, K, seed=20 + b) for b in range(B)))
    X, C = torch.stack(Xs), torch.stack(Cs)
    g = torch.Generator().manual_seed(1)
    idx = torch.randint(0, K, (B, N), generator=g, dtype=torch.int32)
    Cf, Cb, counts = cake.cake_kmeans_update(X.to(DEV), idx.to(DEV), K, C_prev=C.to(DEV), flags=flag)
    for b in range(B):
        grading.grade_update(inputs.to_bits(Xs[b]), idx[b].numpy(), K, inputs.to_bits(Cs[b]), Cf[b].cpu().numpy(),
                             inputs.to_bits(Cb[b]), counts[b].cpu().numpy())


@pytest.mark.parametrize("B,N,D,K", [(5, 40000, 64, 100), (32, 65536, 128, 256), (7, 20001, 24, 33), (3, 70001, 128, 1000),
                                     (9, 16385, 8, 2000)])
def test_update_batch_dealt_over_all_ctas(B, N, D, K):
    """Batches whose problems do not divide the SMs evenly: the slab route deals the rows of all problems to the
    CTAs, so slabs straddle the end of a problem (also with N % 4 != 0, bad indices next to the boundary, an empty
    cluster).  Graded per problem against the oracle, and equal to the route with one grid row per problem."""
    g = torch.Generator().manual_seed(B * N + K)
    X = torch.randint(-4, 5, (B, N, D), generator=g).to(torch.bfloat16)       # integers: any summation order is exact
    C = torch.randint(-4, 5, (B, K, D), generator=g).to(torch.bfloat16)
    idx = torch.randint(0, K, (B, N), generator=g, dtype=torch.int32)
    idx[idx == 1] = 0
    idx[0, N - 1] = K          # last row of problem 0 and first row of problem 1: skipped, status raised
    idx[1, 0] = -5
    Xd, idxd, Cd = X.to(DEV), idx.to(DEV), C.to(DEV)
    ws = cake.alloc_workspace(B, N, D, K, DEV)
    Cf, Cb, counts = cake.cake_kmeans_update(Xd, idxd, K, C_prev=Cd, ws=ws)
    check_status(ws, cake.CAKE_ERR_BAD_INDEX)
    ws2 = cake.alloc_workspace(B, N, D, K, DEV)
    Cf1, Cb1, counts1 = cake.cake_kmeans_update(Xd, idxd, K, C_prev=Cd, ws=ws2, flags=cake.CAKE_UPDATE_SLAB_F1)
    assert torch.equal(Cf, Cf1) and torch.equal(Cb, Cb1) and torch.equal(counts, counts1)
    for b in range(B if B * N * D < 5e7 else 3):
        keep = (idx[b] >= 0) & (idx[b] < K)
        grading.grade_update(inputs.to_bits(X[b])[keep.numpy()], idx[b][keep].numpy(), K, inputs.to_bits(C[b]),
                             Cf[b].cpu().numpy(), inputs.to_bits(Cb[b]), counts[b].cpu().numpy())


@pytest.mark.parametrize("D", [8, 64, 256])
def test_update_many_clusters_few_rows_with_and_without_prev(D):
    """K > 8192 with a few rows per cluster: the sort route hands every cluster to one warp, which writes
    the centroid itself; most clusters are empty here and keep the previous centroid (or zeros)."""
    N, K = 12000, 20000
    X, C = problem(N, D, 64, seed=D)
    g = torch.Generator().manual_seed(D)
    idx = torch.randint(0, K, (N,), generator=g, dtype=torch.int32)
    Cprev = inputs.from_bits(np.random.default_rng(D).integers(0x3C00, 0x4100, size=(K, D), dtype=np.uint16))
    for prev in (Cprev, None):
        Cf, Cb, counts = cake.cake_kmeans_update(X.to(DEV), idx.to(DEV), K, C_prev=None if prev is None else prev.to(DEV),
                                                 flags=cake.CAKE_UPDATE_SORT)
        grading.grade_update(inputs.to_bits(X), idx.numpy(), K, None if prev is None else inputs.to_bits(prev),
                             Cf.cpu().numpy(), inputs.to_bits(Cb), counts.cpu().numpy())


@pytest.mark.parametrize("D", [8, 24, 128, 256, 512, 1024])
def test_update_many_clusters_skewed_sizes(D):
    """K > 8192 with cluster sizes from 0 to several thousand rows: clusters that cross the 64-row windows
    of the sorted order, heavy clusters shared by many warps (partials + arrival count), runs of empty
    clusters at both ends, a few invalid indices, two problems."""
    B, N, K = 2, 40000, 9000 + D
    g = torch.Generator().manual_seed(100 + D)
    X = inputs.from_bits(np.random.default_rng(D).integers(0x3C00, 0x4100, size=(B, N, D), dtype=np.uint16))
    idx = torch.randint(500, K - 700, (B, N), generator=g, dtype=torch.int32)
    idx[0, :6000] = 777                  # heavy
    idx[0, 6000:7500] = K - 701          # heavy, the last cluster with rows
    idx[0, 7500:7700] = 778              # crosses windows, light
    idx[1, 1000:3100] = 500              # heavy, the first cluster with rows
    idx[1, 5000:5065] = 6000
    idx[1, 7] = -1
    idx[1, 9] = K
    perm = torch.randperm(N, generator=g)
    idx = idx[:, perm].contiguous()
    Cprev = inputs.from_bits(np.random.default_rng(D + 1).integers(0x3C00, 0x4100, size=(B, K, D), dtype=np.uint16))
    ws = cake.alloc_workspace(B, N, D, K, DEV)
    for _ in range(2):                  # twice: the arrival counters must start from zero every time
        Cf, Cb, counts = cake.cake_kmeans_update(X.to(DEV), idx.to(DEV), K, C_prev=Cprev.to(DEV), ws=ws,
                                                 flags=cake.CAKE_UPDATE_SORT)
        check_status(ws, cake.CAKE_ERR_BAD_INDEX)
        for b in range(B):
            keep = ((idx[b] >= 0) & (idx[b] < K)).numpy()
            grading.grade_update(inputs.to_bits(X[b])[keep], idx[b].numpy()[keep], K, inputs.to_bits(Cprev[b]),
                                 Cf[b].cpu().numpy(), inputs.to_bits(Cb[b]), counts[b].cpu().numpy())


@pytest.mark.parametrize("case", ["one_row", "few_rows", "all_invalid", "one_cluster", "two_clusters_alternating"])
@pytest.mark.parametrize("D", [24, 40, 256, 520])
def test_update_many_clusters_degenerate(case, D):
    """K > 8192, degenerate index sets: a single row, fewer rows than a window, no valid index at all (every
    centroid keeps its previous value and the status word says so), every row in one heavy cluster, rows
    alternating between the first and the last cluster; granule counts that do not fill the lanes."""
    K = 9001
    N = {"one_row": 1, "few_rows": 50, "all_invalid": 300, "one_cluster": 5000, "two_clusters_alternating": 4100}[case]
    X = inputs.from_bits(np.random.default_rng(D + N).integers(0x3C00, 0x4100, size=(N, D), dtype=np.uint16))
    g = torch.Generator().manual_seed(N)
    if case == "all_invalid":
        idx = torch.full((N,), K + 5, dtype=torch.int32)
        idx[::2] = -1
    elif case == "one_cluster":
        idx = torch.full((N,), 4242, dtype=torch.int32)
    elif case == "two_clusters_alternating":
        idx = torch.where(torch.arange(N) % 2 == 0, 0, K - 1).to(torch.int32)
    else:
        idx = torch.randint(0, K, (N,), generator=g, dtype=torch.int32)
    Cprev = inputs.from_bits(np.random.default_rng(D).integers(0x3C00, 0x4100, size=(K, D), dtype=np.uint16))
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    Cf, Cb, counts = cake.cake_kmeans_update(X.to(DEV), idx.to(DEV), K, C_prev=Cprev.to(DEV), ws=ws,
                                             flags=cake.CAKE_UPDATE_SORT)
    check_status(ws, cake.CAKE_ERR_BAD_INDEX if case == "all_invalid" else cake.CAKE_OK)
    keep = ((idx >= 0) & (idx < K)).numpy()
    grading.grade_update(inputs.to_bits(X)[keep], idx.numpy()[keep], K, inputs.to_bits(Cprev), Cf.cpu().numpy(),
                         inputs.to_bits(Cb), counts.cpu().numpy())


def test_update_odd_feature_count_and_null_prev():
    N, D, K = 500, 7, 9
    X, _ = problem(N, D, K, seed=2)
    idx = (torch.arange(N) % (K - 1)).to(torch.int32)          # last cluster empty
    Cf, Cb, counts = cake.cake_kmeans_update(X.to(DEV), idx.to(DEV), K, C_prev=None)
    grading.grade_update(inputs.to_bits(X), idx.numpy(), K, None, Cf.cpu().numpy(), inputs.to_bits(Cb),
                         counts.cpu().numpy())
    assert not Cf[K - 1].any()


@pytest.mark.parametrize("path", ["smem", "sort", "slab", "slab_f2"])
def test_update_bad_index_is_skipped_and_reported(path):
    flag = {"smem": cake.CAKE_UPDATE_SMEM, "sort": cake.CAKE_UPDATE_SORT, "slab": cake.CAKE_UPDATE_SLAB,
            "slab_f2": cake.CAKE_UPDATE_SLAB_F2}[path]
    N, D, K = 1000, 64, 10
    X, C = problem(N, D, K, seed=3)
    idx = (torch.arange(N) % K).to(torch.int32)
    idx[5], idx[77] = K, -3
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    Cf, _, counts = cake.cake_kmeans_update(X.to(DEV), idx.to(DEV), K, C_prev=C.to(DEV), ws=ws, flags=flag)
    check_status(ws, cake.CAKE_ERR_BAD_INDEX)
    check_status(ws)                                            # reading clears it
    keep = (idx >= 0) & (idx < K)
    C_o, counts_o = orc.update(inputs.to_bits(X)[keep.numpy()], idx[keep].numpy(), K, inputs.to_bits(C))
    assert np.array_equal(counts.cpu().numpy(), counts_o)
    np.testing.assert_allclose(Cf.cpu().numpy(), C_o, rtol=1e-4, atol=1e-5)


def test_update_batched_and_n_zero():
    B, N, D, K = 3, 900, 64, 20
    Xs, Cs = zip(*(problem(N, D, K, seed=70 + b) for b in range(B)))
    X, C = torch.stack(Xs), torch.stack(Cs)
    g = torch.Generator().manual_seed(0)
    idx = torch.randint(0, K, (B, N), generator=g, dtype=torch.int32)
    for flag in (cake.CAKE_UPDATE_SMEM, cake.CAKE_UPDATE_SORT, cake.CAKE_UPDATE_SLAB, cake.CAKE_UPDATE_SLAB_F4):
        Cf, Cb, counts = cake.cake_kmeans_update(X.to(DEV), idx.to(DEV), K, C_prev=C.to(DEV), flags=flag)
        for b in range(B):
            grading.grade_update(inputs.to_bits(Xs[b]), idx[b].numpy(), K, inputs.to_bits(Cs[b]),
                                 Cf[b].cpu().numpy(), inputs.to_bits(Cb[b]), counts[b].cpu().numpy())
    Cf, Cb, counts = cake.cake_kmeans_update(X[0, :0].to(DEV), idx[0, :0].to(DEV), K, C_prev=C[0].to(DEV))
    assert not counts.any() and torch.equal(Cb.cpu(), C[0])


# ------------------------------------------------------------------------------------ Lloyd

def teacher_forced(X, C0, iters, flags=0):
    """Runs iteration by iteration on the GPU; the oracle re-derives each step from the GPU's own state."""
    Xb = inputs.to_bits(X)
    Xd = X.to(DEV)
    cur = C0.to(DEV)
    N, D = X.shape
    K = C0.shape[0]
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    inertia, near_ties = [], 0
    for t in range(iters):
        out = cake.cake_kmeans_lloyd(Xd, cur, 1, ws=ws, flags=flags)
        torch.cuda.synchronize()
        check_status(ws)
        cur_bits = inputs.to_bits(cur)
        idx = out.idx.cpu().numpy()
        rep = grading.grade_assign(Xb, cur_bits, idx, out.dist.cpu().numpy())
        near_ties += rep["mismatch"]
        _, dist_o, _ = orc.assign(Xb, cur_bits)
        assert abs(float(out.inertia[0]) - dist_o.sum()) <= grading.INERTIA_TOL * dist_o.sum()
        grading.grade_update(Xb, idx, K, cur_bits, out.C.cpu().numpy(), inputs.to_bits(out.C_bf16),
                             out.counts.cpu().numpy())
        inertia.append(float(out.inertia[0]))
        cur = out.C_bf16
    return cur, inertia, near_ties


def test_lloyd_c1_teacher_forced_and_free_run():
    w = inputs.WORKLOADS["c1"]
    X, C0 = inputs.make_problem(w)
    cur, inertia, near = teacher_forced(X, C0, w.iters)
    assert near <= 5
    # one call for all iterations follows the same trajectory up to fp32 summation order
    out = cake.cake_kmeans_lloyd(X.to(DEV), C0.to(DEV), w.iters)
    np.testing.assert_allclose(out.inertia.cpu().numpy(), inertia, rtol=1e-4)
    # free-running oracle (its own bf16-rounded trajectory)
    r = orc.lloyd(inputs.to_bits(X), inputs.to_bits(C0), w.iters, round_centroids=True)
    np.testing.assert_allclose(out.inertia.cpu().numpy(), r.inertia, rtol=grading.INERTIA_TOL)
    assert int(out.counts.sum()) == w.N
    assert (np.diff(out.inertia.cpu().numpy()) <= 1e-4 * out.inertia.cpu().numpy()[:-1]).all()


@pytest.mark.parametrize("flags", [cake.CAKE_UPDATE_SMEM, cake.CAKE_UPDATE_SORT,
                                   cake.CAKE_ASSIGN_SIMT | cake.CAKE_UPDATE_SORT])
def test_lloyd_small_all_paths(flags):
    X, C0 = problem(3000, 64, 50, seed=12, comps=50, mean_std=2.0, sigma=1.0)
    teacher_forced(X, C0, 4, flags=flags)


@pytest.mark.parametrize("flags", [0, cake.CAKE_ASSIGN_SIMT, cake.CAKE_UPDATE_SORT, cake.CAKE_ASSIGN_SIMT | cake.CAKE_UPDATE_SORT])
@pytest.mark.parametrize("N,D,K", [(3000, 50, 40), (2500, 7, 9), (1200, 300, 33)])
def test_lloyd_feature_count_not_multiple_of_8_all_paths(N, D, K, flags):
    """Real-valued data, graded against the oracle step by step: padded tensor-core assign + slab update on the
    padded copy (automatic), and every mix with the fallback assign and the sort route (where the update
    has to make the padded copy itself, or none is made at all)."""
    X, C0 = problem(N, D, K, seed=N + D, comps=K, mean_std=2.0, sigma=1.0)
    cur, inertia, near = teacher_forced(X, C0, 3, flags=flags)
    assert near <= 3
    out = cake.cake_kmeans_lloyd(X.to(DEV), C0.to(DEV), 3, flags=flags)
    np.testing.assert_allclose(out.inertia.cpu().numpy(), inertia, rtol=1e-3)


def test_lloyd_handworked_example_on_gpu():
    """The six-point example (golden/handworked_2d.json), padded to D=8 with zero columns."""
    pts = [[0, 0], [0, 2], [2, 0], [10, 10], [10, 12], [12, 10]]
    X = torch.zeros(6, 8)
    X[:, :2] = torch.tensor(pts, dtype=torch.float32)
    X = X.to(torch.bfloat16)
    C0 = X[[0, 2]].contiguous()
    out = cake.cake_kmeans_lloyd(X.to(DEV), C0.to(DEV), 4)
    assert out.idx.cpu().tolist() == [0, 0, 0, 1, 1, 1]
    assert out.counts.cpu().tolist() == [3, 3]
    np.testing.assert_allclose(out.inertia.cpu().numpy(), [576.0, 47.75, 349611 / 32768, 349611 / 32768], rtol=1e-5)
    np.testing.assert_allclose(out.C.cpu().numpy()[:, :2], [[2 / 3, 2 / 3], [32 / 3, 32 / 3]], rtol=1e-6)
    assert out.C_bf16.float().cpu()[:, :2].tolist() == [[171 / 256, 171 / 256], [171 / 16, 171 / 16]]


@pytest.mark.parametrize("B,N,D,K", [(1, 5000, 64, 37), (2, 3000, 128, 300), (1, 2000, 24, 9), (33, 300, 64, 5), (1, 700, 12, 6),
                                       (1, 1500, 320, 40), (2, 900, 512, 300)])
def test_lloyd_call_equals_stepwise_calls(B, N, D, K):
    """Inside a Lloyd call the division kernel prepares the next assign (half-norm operand, max ||c||^2,
    cleared inertia): the result must be bit-identical to assign and update called one by one, where the
    assign computes all that in its own prologue.  Small integer data: the sums are exact in fp32
    whatever their order, so bit-identity is well defined."""
    g = torch.Generator().manual_seed(B * 1000 + D)
    X = torch.randint(-4, 5, (B, N, D), generator=g).to(torch.bfloat16)
    C0 = X[:, :K].contiguous().clone()
    C0[:, :, 0] += torch.arange(K).to(torch.bfloat16)          # distinct centroids
    Xd, C0d = X.to(DEV), C0.to(DEV)
    if B == 1:
        Xd, C0d = Xd[0], C0d[0]
    iters = 4
    out = cake.cake_kmeans_lloyd(Xd, C0d, iters)
    C = C0d
    inertia = []
    for _ in range(iters):
        idx, dist = cake.cake_kmeans_assign(Xd, C)
        inertia.append(dist.double().sum(-1))
        Cf, Cb, counts = cake.cake_kmeans_update(Xd, idx, K, C_prev=C)
        C = Cb
    assert torch.equal(out.idx, idx) and torch.equal(out.dist, dist)
    assert torch.equal(out.C, Cf) and torch.equal(out.C_bf16, Cb) and torch.equal(out.counts, counts)
    np.testing.assert_allclose(out.inertia.cpu().numpy(), torch.stack(inertia, -1).cpu().numpy(), rtol=1e-12)


def test_lloyd_iters_zero_and_batched():
    B, N, D, K = 3, 1500, 64, 24
    Xs, Cs = zip(*(problem(N, D, K, seed=90 + b, comps=24, mean_std=2.0, sigma=1.0) for b in range(B)))
    X, C0 = torch.stack(Xs).to(DEV), torch.stack(Cs).to(DEV)
    out0 = cake.cake_kmeans_lloyd(X, C0, 0)
    assert torch.equal(out0.C_bf16, C0) and torch.equal(out0.C, C0.float())
    out = cake.cake_kmeans_lloyd(X, C0, 5)
    for b in range(B):
        one = cake.cake_kmeans_lloyd(X[b].contiguous(), C0[b].contiguous(), 5)
        np.testing.assert_allclose(out.inertia[b].cpu().numpy(), one.inertia.cpu().numpy(), rtol=1e-4)
        r = orc.lloyd(inputs.to_bits(Xs[b]), inputs.to_bits(Cs[b]), 5, round_centroids=True)
        np.testing.assert_allclose(out.inertia[b].cpu().numpy(), r.inertia, rtol=grading.INERTIA_TOL)


def test_lloyd_host_buffers_match_device_call():
    X, C0 = problem(5000, 128, 40, seed=33, comps=40, mean_std=2.0, sigma=1.0)
    iters = 3
    dev_out = cake.cake_kmeans_lloyd(X.to(DEV), C0.to(DEV), iters)
    Xh, Ch = X.pin_memory(), C0.pin_memory()
    host_out = cake.alloc_lloyd_outputs(Xh, Ch, iters, pin_host=True)
    scratch = torch.empty(cake.cake_kmeans_lloyd_host_device_bytes(1, 5000, 128, 40, iters), dtype=torch.uint8,
                          device=DEV)
    cake.cake_kmeans_lloyd_host(Xh, Ch, iters, host_out, scratch)
    torch.cuda.synchronize()
    assert torch.equal(host_out.idx, dev_out.idx.cpu())
    np.testing.assert_allclose(host_out.inertia.numpy(), dev_out.inertia.cpu().numpy(), rtol=1e-5)
    np.testing.assert_allclose(host_out.C.numpy(), dev_out.C.cpu().numpy(), rtol=1e-4, atol=1e-5)
    assert torch.equal(host_out.counts, dev_out.counts.cpu())


# ------------------------------------------------------------------------------------ full-size workloads

def test_assign_policies_agree_except_near_ties():
    """The packed epilogue orders values that agree to 2^-16 by index; everything else is identical."""
    X, C = problem(30000, 128, 1500, seed=77, comps=200)
    Xd, Cd = X.to(DEV), C.to(DEV)
    ip, dp = cake.cake_kmeans_assign(Xd, Cd, flags=cake.CAKE_ASSIGN_TCGEN05)
    ie, de = cake.cake_kmeans_assign(Xd, Cd, flags=cake.CAKE_ASSIGN_TCGEN05_EXACT)
    differ = (ip != ie).cpu().numpy()
    assert differ.mean() < 1e-3
    rel = ((dp - de).abs() / de.clamp_min(1e-6)).cpu().numpy()
    assert rel[~differ].max() <= 2.0 ** -15
    if differ.any():   # where they differ the two candidates are closer than the packing granularity
        Xb, Cb = inputs.to_bits(X), inputs.to_bits(C)
        rows = np.nonzero(differ)[0]
        d1 = orc.pair_sqdist(Xb[rows], Cb, ip.cpu().numpy()[rows])
        d2 = orc.pair_sqdist(Xb[rows], Cb, ie.cpu().numpy()[rows])
        assert (np.abs(d1 - d2) <= 2.0 ** -14 * np.maximum(d1, d2) + 1e-4).all()


@pytest.mark.parametrize("name,sample", [("c2", 4096), ("c4", 1024)])
def test_full_size_workload_sampled(name, sample):
    """The benchmark's launch configuration: one Lloyd iteration at full size, graded on sampled rows
    (assign) and in full (update)."""
    w = inputs.WORKLOADS[name]
    X, C0 = inputs.make_problem(w, device=DEV)
    ws = cake.alloc_workspace(1, w.N, w.D, w.K, DEV)
    out = cake.cake_kmeans_lloyd(X, C0, 1, ws=ws)
    torch.cuda.synchronize()
    check_status(ws)
    Xb, Cb = inputs.to_bits(X), inputs.to_bits(C0)
    idx = out.idx.cpu().numpy()
    rows = sampled_rows(w.N, sample, w.seed)
    rep = grading.grade_assign(Xb, Cb, idx, out.dist.cpu().numpy(), rows=rows)
    assert rep["mismatch"] <= max(2, sample // 500), rep
    assert int(out.counts.sum()) == w.N
    grading.grade_update(Xb, idx, w.K, Cb, out.C.cpu().numpy(), inputs.to_bits(out.C_bf16), out.counts.cpu().numpy())
    # inertia equals the sum of the per-point distances the same call returned
    assert abs(float(out.inertia[0]) - float(out.dist.double().sum())) <= 1e-6 * float(out.inertia[0])


def test_full_size_batched_workload_sampled():
    w = inputs.WORKLOADS["c3"]
    X, C0 = inputs.make_batch(w, device=DEV)
    ws = cake.alloc_workspace(w.B, w.N, w.D, w.K, DEV)
    out = cake.cake_kmeans_lloyd(X, C0, 1, ws=ws)
    torch.cuda.synchronize()
    check_status(ws)
    for b in (0, 13, 31):
        Xb, Cb = inputs.to_bits(X[b]), inputs.to_bits(C0[b])
        idx = out.idx[b].cpu().numpy()
        grading.grade_assign(Xb, Cb, idx, out.dist[b].cpu().numpy(), rows=sampled_rows(w.N, 2048, b))
        grading.grade_update(Xb, idx, w.K, Cb, out.C[b].cpu().numpy(), inputs.to_bits(out.C_bf16[b]),
                             out.counts[b].cpu().numpy())


@pytest.mark.parametrize("N,D,K", [(1 << 24, 64, 64), (1 << 23, 64, 300)])
def test_assign_many_row_tiles_few_centroid_tiles(N, D, K):
    """Hundreds of row tiles per CTA with one or two centroid tiles each: the X buffers, the norm warps'
    row exponents and the accumulators turn over as fast as they can, which is where a barrier protocol
    that lets any role run a whole buffer cycle ahead of another shows up (as a time-out in the status
    word, or as distances decoded with another row's exponent)."""
    w = inputs.sweep_workload(N, D, K)
    X, _ = inputs.gaussian_mixture(N, D, 4096, w.mean_std, w.sigma, w.seed, device=DEV)
    C0 = inputs.sample_init(X, K, w.seed)
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    for _ in range(2):
        idx, dist = cake.cake_kmeans_assign(X, C0, ws=ws)
        torch.cuda.synchronize()
        check_status(ws)
    rows = sampled_rows(N, 2048, K)
    rows_t = torch.from_numpy(rows).to(DEV)
    Xs = inputs.to_bits(X[rows_t].cpu())
    rep = grading.grade_assign(Xs, inputs.to_bits(C0.cpu()), idx[rows_t].cpu().numpy(), dist[rows_t].cpu().numpy())
    assert rep["mismatch"] <= 4, rep
    # every row was written: a valid index and a finite distance
    assert int(idx.min()) >= 0 and int(idx.max()) < K and bool(torch.isfinite(dist).all())


@pytest.mark.parametrize("N,D,K", [(1 << 21, 64, 64), (1 << 21, 128, 300), (1 << 20, 256, 600), (1 << 21, 96, 1000),
                                   (1 << 20, 128, 1300), (1 << 20, 384, 64), (1 << 20, 512, 32), (1 << 19, 288, 300),
                                   (1 << 20, 256, 256), (1 << 20, 100, 200)])
def test_assign_repeatable_over_many_launches(N, D, K):
    """The assign kernel has no data-dependent order (no atomics on its outputs): repeated launches must
    return identical bits.  A role that gets ahead of a buffer it must not yet reuse (X tile, row
    exponents, half-norm block, accumulator) shows up here as a difference or as a time-out."""
    w = inputs.sweep_workload(N, D, K)
    X, _ = inputs.gaussian_mixture(N, D, 1024, w.mean_std, w.sigma, w.seed, device=DEV)
    C0 = inputs.sample_init(X, K, w.seed)
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    idx0, dist0 = cake.cake_kmeans_assign(X, C0, ws=ws)
    idx0, dist0 = idx0.clone(), dist0.clone()
    for _ in range(6):
        idx, dist = cake.cake_kmeans_assign(X, C0, ws=ws)
        torch.cuda.synchronize()
        check_status(ws)
        assert torch.equal(idx, idx0) and torch.equal(dist, dist0)
    rows = sampled_rows(N, 1024, D)
    rows_t = torch.from_numpy(rows).to(DEV)
    grading.grade_assign(inputs.to_bits(X[rows_t].cpu()), inputs.to_bits(C0.cpu()), idx0[rows_t].cpu().numpy(),
                         dist0[rows_t].cpu().numpy())


# ------------------------------------------------------------------------------------ bounded waits

def test_bounded_wait_expires_and_context_survives():
    ws = cake.alloc_workspace(1, 256, 64, 8, DEV)
    cake.cake_kmeans_selftest_bounded_wait(ws, 20)
    assert cake.cake_kmeans_device_status(ws) == cake.CAKE_ERR_TIMEOUT
    assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
    X, C = problem(256, 64, 8, seed=5)
    idx, _ = cake.cake_kmeans_assign(X.to(DEV), C.to(DEV), ws=ws)
    idx_o, _, _ = orc.assign(inputs.to_bits(X), inputs.to_bits(C))
    assert np.array_equal(idx.cpu().numpy(), idx_o)
