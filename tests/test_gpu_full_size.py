"""Parity at the full sizes of the named workloads, in the launch configuration the benchmark times.

Teacher-forced: every iteration the oracle starts from the GPU's own bf16 centroids and grades the GPU's
assignment (all rows where the oracle finishes in seconds, else a seeded row sample: assign is independent per
row) and the GPU's update in full (linear cost) from the GPU's own indices.  Later iterations matter: cluster sizes,
the update's route and the density of near-ties all change after the first step from sampled initial centroids.
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


def rows_sample(N, n, seed):
    return np.sort(np.random.default_rng(seed).choice(N, size=min(n, N), replace=False))


def teacher_forced_full_size(X, C0, iters, full_iters, sample, seed):
    """X, C0 on the device (one problem).  Returns per-iteration reports."""
    N, D = X.shape
    K = C0.shape[0]
    ws = cake.alloc_workspace(1, N, D, K, DEV)
    Xb = inputs.to_bits(X)
    cur = C0
    reports = []
    for t in range(iters):
        idx, dist = cake.cake_kmeans_assign(X, cur, ws=ws)
        Cf, Cb, counts = cake.cake_kmeans_update(X, idx, K, C_prev=cur, ws=ws)
        torch.cuda.synchronize()
        assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
        cur_bits = inputs.to_bits(cur)
        idx_h = idx.cpu().numpy()
        rows = None if t < full_iters else rows_sample(N, sample, seed + t)
        rep = grading.grade_assign(Xb, cur_bits, idx_h, dist.cpu().numpy(), rows=rows)
        assert int(counts.sum()) == N
        rep.update(grading.grade_update(Xb, idx_h, K, cur_bits, Cf.cpu().numpy(), inputs.to_bits(Cb), counts.cpu().numpy()))
        reports.append(rep)
        cur = Cb
    return reports, cur


def test_c2_three_iterations_two_of_them_graded_on_every_row():
    w = inputs.WORKLOADS["c2"]
    X, C0 = inputs.make_problem(w, device=DEV)
    reports, last = teacher_forced_full_size(X, C0, 3, 2, 8192, w.seed)
    for t, rep in enumerate(reports):
        assert rep["unexcused"] == 0 and rep["mismatch"] <= max(4, rep["n"] // 20000), (t, rep)
    # the one-call loop follows the same trajectory (fp32 summation order aside)
    out = cake.cake_kmeans_lloyd(X, C0, 3)
    assert (out.C_bf16 != last).float().mean() < 1e-3
    assert (np.diff(out.inertia.cpu().numpy()) < 0).all()


def test_c4_all_five_iterations_sampled_rows_full_update():
    w = inputs.WORKLOADS["c4"]
    X, C0 = inputs.make_problem(w, device=DEV)
    reports, _ = teacher_forced_full_size(X, C0, w.iters, 0, 1024, w.seed)
    for t, rep in enumerate(reports):
        assert rep["unexcused"] == 0 and rep["mismatch"] <= 3, (t, rep)
    assert reports[0]["empty"] > 0 or reports[-1]["empty"] > 0      # the workload is built to leave clusters empty


def batched_one_iteration(name, sample):
    w = inputs.WORKLOADS[name]
    X, C0 = inputs.make_batch(w, device=DEV)
    ws = cake.alloc_workspace(w.B, w.N, w.D, w.K, DEV)
    out = cake.cake_kmeans_lloyd(X, C0, 2, ws=ws)          # iteration 1 is the one graded: from updated centroids
    torch.cuda.synchronize()
    assert cake.cake_kmeans_device_status(ws) == cake.CAKE_OK
    first = cake.cake_kmeans_lloyd(X, C0, 1, ws=ws)
    total = 0
    for b in range(w.B):
        Xb, Cb = inputs.to_bits(X[b]), inputs.to_bits(first.C_bf16[b])
        idx = out.idx[b].cpu().numpy()
        rep = grading.grade_assign(Xb, Cb, idx, out.dist[b].cpu().numpy(), rows=rows_sample(w.N, sample, w.seed + b))
        total += rep["mismatch"]
        grading.grade_update(Xb, idx, w.K, Cb, out.C[b].cpu().numpy(), inputs.to_bits(out.C_bf16[b]), out.counts[b].cpu().numpy())
    assert total <= max(4, w.B * sample // 10000), total


def test_c3_every_problem_of_the_batch():
    batched_one_iteration("c3", 2048)


def test_paper_shape_every_problem_of_the_batch():
    batched_one_iteration("paper", 1024)


def test_w1_wide_rows_three_iterations_sampled():
    """The wide-row workload (D = 1,024: X streamed over D by CTA pairs) at full size, teacher-forced, sampled rows;
    the update of such rows (D = 1,024) graded in full."""
    w = inputs.WORKLOADS["w1"]
    X, C0 = inputs.make_problem(w, device=DEV)
    reports, _ = teacher_forced_full_size(X, C0, 3, 0, 2048, w.seed)
    for t, rep in enumerate(reports):
        assert rep["unexcused"] == 0 and rep["mismatch"] <= 3, (t, rep)
