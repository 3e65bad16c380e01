"""Host-side logic of the row-sharded Lloyd driver, on CPU: the partition of the rows, and the driver run as two
gloo ranks with the library's per-rank call replaced by a stand-in built on the oracle (what is checked here is the
exchange the driver supplies: what is all-reduced and when, and the empty-cluster rule when a cluster is empty on
one rank only; the library's loop and kernels are checked on the GPU)."""
import os
import sys
import types

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
from paper_2608_12629_b200 import inputs, sharded  # noqa: E402
from paper_2608_12629_b200.sharded import shard_rows  # noqa: E402


@pytest.mark.parametrize("N,world", [(0, 1), (1, 4), (10, 3), (128, 8), (1000003, 7)])
def test_shard_rows_is_a_partition_into_contiguous_near_equal_shares(N, world):
    spans = [shard_rows(N, r, world) for r in range(world)]
    assert spans[0][0] == 0 and spans[-1][1] == N
    assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
    sizes = [b - a for a, b in spans]
    assert max(sizes) - min(sizes) <= 1 and sorted(sizes, reverse=True) == sizes
    with pytest.raises(ValueError):
        shard_rows(N, world, world)


def _oracle_binding():
    """An object with the names sharded.py uses from the binding, computing on CPU tensors through the oracle."""
    from oracle import kmeans_oracle as orc
    from paper_2608_12629_b200 import binding as real

    def assign(X, C, out_idx, out_dist, ws=None, flags=0):
        idx, d, _ = orc.assign(inputs.to_bits(X), inputs.to_bits(C))
        out_idx.copy_(torch.from_numpy(idx))
        out_dist.copy_(torch.from_numpy(d).float())
        return out_idx, out_dist

    def inertia(d, out_inertia, stride=1, stream=None):
        out_inertia[0] = d.double().sum()
        return out_inertia

    def partial(X, idx, K, out_sums, out_counts, ws=None, flags=0):
        _, counts, sums = orc.update(inputs.to_bits(X), idx.numpy(), K, None, return_sums=True)
        out_sums.copy_(torch.from_numpy(sums).float())
        out_counts.copy_(torch.from_numpy(counts).int())
        return out_sums, out_counts

    def finish(sums, counts, C_prev, out_C, out_C_bf16):
        prev = orc.bf16_to_f64(inputs.to_bits(C_prev))
        n = counts.numpy().astype(np.float64)[:, None]
        C = np.where(n > 0, sums.double().numpy() / np.maximum(n, 1.0), prev)
        out_C.copy_(torch.from_numpy(C).float())
        out_C_bf16.copy_(inputs.from_bits(orc.f64_to_bf16(C)))
        return out_C, out_C_bf16

    def sharded_call(X, C0, iters, out, ws, reduce=None, stream=None, flags=0):
        """What the C entry point does, stated with the stand-ins above: per iteration assign, the local inertia, the
        local sums and counts, the caller's exchange, the division."""
        K, D = C0.shape
        sums = torch.empty(K, D, dtype=torch.float32)
        cur = C0
        for t in range(iters):
            assign(X, cur, out.idx, out.dist)
            inertia(out.dist, out.inertia[t:])
            partial(X, out.idx, K, sums, out.counts)
            if reduce is not None:
                reduce(sums, out.counts)
            nxt = torch.empty_like(C0)
            finish(sums, out.counts, cur, out.C, nxt)
            cur = nxt
        out.C_bf16.copy_(cur)
        return out

    return types.SimpleNamespace(alloc_workspace=lambda B, N, D, K, dev: torch.empty(1), alloc_lloyd_outputs=real.alloc_lloyd_outputs,
                                 cake_kmeans_lloyd_sharded_call=sharded_call)


def _problem():
    """Small integers (sums exact in any order and precision).  Cluster 5 has no point anywhere (its centroid is far
    away), and the points near centroid 6 all sit in the second half of the rows: empty on rank 0 only."""
    g = torch.Generator().manual_seed(7)
    N, D, K = 600, 8, 7
    X = torch.randint(-3, 4, (N, D), generator=g).float()
    X[N // 2 + 10:N // 2 + 60] += 40.0
    C0 = X[:K].clone()
    C0[5] = -100.0
    C0[6] = 40.0
    return X.to(torch.bfloat16), C0.to(torch.bfloat16)


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sharded.binding = _oracle_binding()
    X, C0 = _problem()
    a, b = shard_rows(X.shape[0], rank, world)
    out = sharded.cake_kmeans_lloyd_sharded(X[a:b].clone(), C0, 3)
    q.put((rank, inputs.to_bits(out.C_bf16), out.C.numpy(), out.counts.numpy(), out.idx.numpy(), out.inertia.numpy()))
    dist.barrier()
    dist.destroy_process_group()


def test_sharded_lloyd_two_gloo_ranks_follow_the_single_device_iteration():
    from oracle import kmeans_oracle as orc
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict()
    for _ in range(2):
        r = q.get(timeout=180)
        got[r[0]] = r[1:]
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    X, C0 = _problem()
    ref = orc.lloyd(inputs.to_bits(X), inputs.to_bits(C0), 3)
    assert ref.counts[5] == 0 and ref.counts[6] > 0
    for rank in range(2):
        Cb, C, counts, idx, inertia = got[rank]
        a, b = shard_rows(X.shape[0], rank, 2)
        assert np.array_equal(Cb, ref.C_bits) and np.array_equal(counts, ref.counts)
        assert np.array_equal(idx, ref.idx[a:b])
        np.testing.assert_allclose(C, ref.C, rtol=1e-6)
        np.testing.assert_allclose(inertia, ref.inertia, rtol=1e-6)
    assert np.array_equal(got[0][0][5], inputs.to_bits(C0)[5])       # the empty cluster kept its centroid
