"""GPU tests of the two-part centroid update, the inertia entry point and the row-sharded Lloyd driver
(one GPU: two gloo ranks share it; their kernels never wait on one another, the exchange is on the host side)."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import paper_2608_12629_b200 as cake  # noqa: E402
from paper_2608_12629_b200 import inputs  # noqa: E402
from tests import grading  # noqa: E402

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def int_problem(N, D, K, seed):
    """Small integers: fp32 sums are exact in any order, so results of different routes and splits are bit-identical."""
    g = torch.Generator().manual_seed(seed)
    X = torch.randint(-4, 5, (N, D), generator=g).to(torch.bfloat16)
    C0 = X[:K].clone() if K <= N else torch.randint(-4, 5, (K, D), generator=g).to(torch.bfloat16)
    C0[:, 0] += (torch.arange(K) % 64).to(torch.bfloat16)
    return X, C0


@pytest.mark.parametrize("flags", [0, cake.CAKE_UPDATE_SLAB, cake.CAKE_UPDATE_SORT])
@pytest.mark.parametrize("N,D,K", [(5000, 64, 37), (70001, 128, 1000), (3000, 24, 8192), (900, 12, 5), (4097, 320, 100),
                                   (30000, 64, 20000), (9000, 12, 9000)])
def test_update_partial_of_two_halves_adds_up_to_the_update(N, D, K, flags):
    if flags == cake.CAKE_UPDATE_SLAB and (D % 8 or K > 8192):
        pytest.skip("slab route needs D % 8 == 0 and K <= 8192")
    X, C0 = int_problem(N, D, K, N + D)
    g = torch.Generator().manual_seed(K)
    idx = torch.randint(0, K, (N,), generator=g, dtype=torch.int32)
    idx[idx == 1] = 0
    Xd, idxd, Cd = X.to(DEV), idx.to(DEV), C0.to(DEV)
    h = N // 2 + 3
    s0, c0 = cake.cake_kmeans_update_partial(Xd[:h].clone(), idxd[:h].clone(), K, flags=flags)
    s1, c1 = cake.cake_kmeans_update_partial(Xd[h:].clone(), idxd[h:].clone(), K, flags=flags)
    Cf, Cb = cake.cake_kmeans_update_finish(s0 + s1, c0 + c1, C_prev=Cd)
    Cf_ref, Cb_ref, counts_ref = cake.cake_kmeans_update(Xd, idxd, K, C_prev=Cd)
    assert torch.equal(c0 + c1, counts_ref)
    if K <= 8192 or D % 8:
        assert torch.equal(Cf, Cf_ref) and torch.equal(Cb, Cb_ref)
    else:   # the one-call route for many clusters multiplies by a reciprocal instead of dividing: last-bit differences
        np.testing.assert_allclose(Cf.cpu().numpy(), Cf_ref.cpu().numpy(), rtol=3e-7, atol=0)
    grading.grade_update(inputs.to_bits(X), idx.numpy(), K, inputs.to_bits(C0), Cf.cpu().numpy(), inputs.to_bits(Cb),
                         (c0 + c1).cpu().numpy())


def test_update_partial_limits_and_empty_input():
    X, C0 = int_problem(100, 16, 9000, 1)
    idx = torch.zeros(100, dtype=torch.int32)
    with pytest.raises(cake.CakeError) as e:       # the slab route by name stops at 8,192 clusters
        cake.cake_kmeans_update_partial(X.to(DEV), idx.to(DEV), 9000, flags=cake.CAKE_UPDATE_SLAB)
    assert e.value.code == cake.CAKE_ERR_UNSUPPORTED
    s, c = cake.cake_kmeans_update_partial(X[:0].to(DEV), idx[:0].to(DEV), 7)
    assert int(c.sum()) == 0 and float(s.abs().sum()) == 0.0
    Cf, Cb = cake.cake_kmeans_update_finish(s, c, C_prev=None)
    assert float(Cf.abs().sum()) == 0.0


def test_inertia_entry_point():
    g = torch.Generator().manual_seed(3)
    d = torch.rand(3, 100001, generator=g).to(DEV)
    out = cake.cake_kmeans_inertia(d, stride=2)
    np.testing.assert_allclose(out.cpu().numpy()[::2], d.double().sum(-1).cpu().numpy(), rtol=1e-12)
    one = cake.cake_kmeans_inertia(d[0, :0].contiguous())
    assert float(one[0]) == 0.0


@pytest.mark.parametrize("N,D,K", [(20000, 64, 100), (5000, 128, 1030), (3000, 12, 9)])
def test_lloyd_sharded_without_a_group_equals_lloyd(N, D, K):
    X, C0 = int_problem(N, D, K, N)
    Xd, Cd = X.to(DEV), C0.to(DEV)
    a = cake.cake_kmeans_lloyd_sharded(Xd, Cd, 4)
    b = cake.cake_kmeans_lloyd(Xd, Cd, 4)
    assert torch.equal(a.idx, b.idx) and torch.equal(a.dist, b.dist) and torch.equal(a.counts, b.counts)
    assert torch.equal(a.C, b.C) and torch.equal(a.C_bf16, b.C_bf16)
    np.testing.assert_allclose(a.inertia.cpu().numpy(), b.inertia.cpu().numpy(), rtol=1e-12)


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    torch.cuda.set_device(0)
    X, C0 = int_problem(30001, 64, 300, 5)
    a, b = cake.shard_rows(X.shape[0], rank, world)
    out = cake.cake_kmeans_lloyd_sharded(X[a:b].clone().to(DEV), C0.to(DEV), 4)
    torch.cuda.synchronize()
    q.put((rank, inputs.to_bits(out.C_bf16), out.C.cpu().numpy(), out.counts.cpu().numpy(), out.idx.cpu().numpy(),
           out.inertia.cpu().numpy()))
    dist.barrier()
    dist.destroy_process_group()


def test_lloyd_sharded_two_ranks_equal_the_single_device_iteration():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 33500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict()
    for _ in range(2):
        r = q.get(timeout=300)
        got[r[0]] = r[1:]
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    X, C0 = int_problem(30001, 64, 300, 5)
    ref = cake.cake_kmeans_lloyd(X.to(DEV), C0.to(DEV), 4)
    for rank in range(2):
        Cb, C, counts, idx, inertia = got[rank]
        a, b = cake.shard_rows(X.shape[0], rank, 2)
        assert np.array_equal(Cb, inputs.to_bits(ref.C_bf16)) and np.array_equal(C, ref.C.cpu().numpy())
        assert np.array_equal(counts, ref.counts.cpu().numpy()) and np.array_equal(idx, ref.idx.cpu().numpy()[a:b])
        np.testing.assert_allclose(inertia, ref.inertia.cpu().numpy(), rtol=1e-12)


def _rank_real(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    torch.cuda.set_device(0)
    X, _ = inputs.gaussian_mixture(20001, 64, 40, 2.0, 0.7, 77)
    C0 = inputs.sample_init(X, 150, 77)
    a, b = cake.shard_rows(X.shape[0], rank, world)
    one = cake.cake_kmeans_lloyd_sharded(X[a:b].clone().to(DEV), C0.to(DEV), 1)
    three = cake.cake_kmeans_lloyd_sharded(X[a:b].clone().to(DEV), C0.to(DEV), 3)
    torch.cuda.synchronize()
    q.put((rank, one.idx.cpu().numpy(), one.dist.cpu().numpy(), one.C.cpu().numpy(), inputs.to_bits(one.C_bf16),
           one.counts.cpu().numpy(), one.inertia.cpu().numpy(), three.inertia.cpu().numpy()))
    dist.barrier()
    dist.destroy_process_group()


def test_lloyd_sharded_two_ranks_graded_by_the_oracle():
    """Real-valued data, two ranks: the first iteration is graded against the oracle as any single-device iteration is
    (each rank's assignment of its rows; the update from the indices of both ranks together), three iterations against
    the oracle's own rounded trajectory on the inertia."""
    from oracle import kmeans_oracle as orc
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 35500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_real, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict()
    for _ in range(2):
        r = q.get(timeout=300)
        got[r[0]] = r[1:]
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    X, _ = inputs.gaussian_mixture(20001, 64, 40, 2.0, 0.7, 77)
    C0 = inputs.sample_init(X, 150, 77)
    Xb, Cb = inputs.to_bits(X), inputs.to_bits(C0)
    idx_all = np.empty(X.shape[0], dtype=np.int32)
    for rank in range(2):
        a, b = cake.shard_rows(X.shape[0], rank, 2)
        idx, dist_, C, Cbits, counts, inertia1, inertia3 = got[rank]
        grading.grade_assign(Xb[a:b], Cb, idx, dist_)
        idx_all[a:b] = idx
    for rank in range(2):
        idx, dist_, C, Cbits, counts, inertia1, inertia3 = got[rank]
        grading.grade_update(Xb, idx_all, 150, Cb, C, Cbits, counts)        # the same global result on both ranks
        ref = orc.lloyd(Xb, Cb, 3, round_centroids=True)
        np.testing.assert_allclose(inertia3, ref.inertia, rtol=grading.INERTIA_TOL)
        np.testing.assert_allclose(inertia1, ref.inertia[:1], rtol=grading.INERTIA_TOL)
