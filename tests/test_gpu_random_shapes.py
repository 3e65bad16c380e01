"""Seeded random shapes through the C ABI against the CPU oracle (GPU).

The hand-picked cases of test_gpu_parity.py aim at known edges; these walk over combinations nobody thought
of: batch counts around the header limit of 32, feature counts with and without whole 16-byte granules,
cluster counts around every tile and route boundary (32-column groups, 128, 256, 512, 8192), row counts
around a row tile, one wave and several waves, three input scales, both epilogue policies, all update
routes, invalid indices.  Every draw is seeded; sizes are bounded so that the oracle grades in seconds.
"""
import random

import numpy as np
import pytest
import torch

from tests import grading
import paper_2608_12629_b200 as cake
from paper_2608_12629_b200 import inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("seed", [3, 11, 21])
def test_assign_and_lloyd_random_shapes(seed):
    rnd = random.Random(seed)
    for it in range(25):
        B = rnd.choice([1, 1, 1, 2, 3, 7, 33])
        D = rnd.choice([8, 16, 24, 32, 40, 64, 72, 96, 128, 136, 192, 200, 256, 264, 320, 384, 504, 512, 7, 12, 100, 130, 509])
        K = rnd.choice([1, 2, 3, 17, 31, 32, 33, 64, 65, 100, 127, 128, 129, 200, 255, 256, 257, 300, 511, 512, 513, 700,
                        1000, 1024, 1500])
        N = rnd.choice([1, 5, 127, 128, 129, 300, 1000, 2049, 5000, 20000, 40000, 148 * 128 + 5, 148 * 128 * 2 + 1])
        if B * N * K > 6e7:
            N = max(1, int(6e7 / (B * K)))
        flags = rnd.choice([0, cake.CAKE_ASSIGN_TCGEN05_EXACT])
        if D % 8:
            flags = 0      # the padded route is the automatic choice only; by name the tensor-core path refuses such D
        g = torch.Generator().manual_seed(seed * 1000 + it)
        X = (torch.randn(B, N, D, generator=g) * rnd.choice([0.1, 1.0, 30.0])).to(torch.bfloat16)
        C = (torch.randn(B, K, D, generator=g) * rnd.choice([0.1, 1.0, 30.0])).to(torch.bfloat16)
        Xd, Cd = X.to(DEV), C.to(DEV)
        ws = cake.alloc_workspace(B, N, D, K, DEV)
        where = f"B={B} N={N} D={D} K={K} flags={flags}"
        idx, dist = cake.cake_kmeans_assign(Xd, Cd, ws=ws, flags=flags)
        assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK, where
        for b in range(B):
            rows = None
            if N * K > 4e6:
                rows = np.unique(np.random.default_rng(it).integers(0, N, size=max(1, int(4e6 / K))))
            grading.grade_assign(inputs.to_bits(X[b]), inputs.to_bits(C[b]), idx[b].cpu().numpy(), dist[b].cpu().numpy(),
                                 rows=rows)
        out = cake.cake_kmeans_lloyd(Xd, Cd, 2, ws=ws, flags=flags)
        assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK, where
        assert int(out.counts.sum()) == B * N, where


@pytest.mark.parametrize("seed", [5, 17])
def test_update_random_shapes_and_index_sets(seed):
    rnd = random.Random(seed)
    for it in range(30):
        B = rnd.choice([1, 1, 2, 3])
        D = rnd.choice([8, 16, 24, 32, 40, 64, 96, 128, 136, 256, 264, 512, 520, 1024, 12, 7])
        K = rnd.choice([1, 5, 100, 1000, 4096, 8192, 8193, 9000, 20000, 65536, 70001])
        N = rnd.choice([1, 63, 64, 65, 1000, 5000, 50000, 200000])
        if B * N * D > 4e7:
            N = max(1, int(4e7 / (B * D)))
        if B * K * D > 6e7:
            K = max(1, int(6e7 / (B * D)))
        rng = np.random.default_rng(seed * 1000 + it)
        mode = rnd.choice(["uniform", "skew", "few", "onehot"])
        if mode == "uniform":
            idx = rng.integers(0, K, size=(B, N))
        elif mode == "skew":
            idx = np.minimum((rng.pareto(1.0, size=(B, N)) * K / 50).astype(np.int64), K - 1)
        elif mode == "few":
            idx = rng.choice(rng.integers(0, K, size=max(1, min(K, 7))), size=(B, N))
        else:
            idx = np.full((B, N), rng.integers(0, K))
        idx = idx.astype(np.int32)
        bad = rnd.random() < 0.3 and N > 3
        if bad:
            idx[0, 0] = -1
            idx[-1, N // 2] = K
        flag = rnd.choice([0, cake.CAKE_UPDATE_SORT, cake.CAKE_UPDATE_SORT])
        if flag == 0 and rnd.random() < 0.3 and K <= 8192 and D % 8 == 0 and D <= 1024:
            flag = cake.CAKE_UPDATE_SLAB
        X = inputs.from_bits(rng.integers(0x3C00, 0x4100, size=(B, N, D), dtype=np.uint16))
        prev = None if rnd.random() < 0.3 else inputs.from_bits(rng.integers(0x3C00, 0x4100, size=(B, K, D), dtype=np.uint16))
        ws = cake.alloc_workspace(B, N, D, K, DEV)
        where = f"B={B} N={N} D={D} K={K} {mode} flag={flag >> 4} bad={bad}"
        Cf, Cb, counts = cake.cake_kmeans_update(X.to(DEV), torch.from_numpy(idx).to(DEV), K,
                                                 C_prev=None if prev is None else prev.to(DEV), ws=ws, flags=flag)
        assert cake.cake_kmeans_device_status(ws) == (cake.CAKE_ERR_BAD_INDEX if bad else cake.CAKE_OK), where
        for b in range(B):
            keep = (idx[b] >= 0) & (idx[b] < K)
            grading.grade_update(inputs.to_bits(X[b])[keep], idx[b][keep], K, None if prev is None else inputs.to_bits(prev[b]),
                                 Cf[b].cpu().numpy(), inputs.to_bits(Cb[b]), counts[b].cpu().numpy())
