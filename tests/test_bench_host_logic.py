"""Host-side logic of bench.py that needs no GPU: the reference arm, and the multi-rank reduction
(world_size 2 over gloo on CPU)."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_algorithmic_bytes_and_peaks():
    from paper_2608_12629_b200 import inputs
    w = inputs.WORKLOADS["c2"]
    assert bench.algorithmic_update_bytes(w) == 2 * w.N * w.D + 4 * w.N + 8 * w.K * w.D + 4 * w.K
    p = bench.measured_peaks()
    assert p["hbm_gbs"] > 1000 and p["bf16_tflops"] > 100 and p["source"] in ("measured", "fallback")


def test_repeats_and_clock_bins():
    assert bench.repeats_for(6.0, 1000.0) == 167 and bench.repeats_for(2000.0, 1000.0) == 1 and bench.repeats_for(0.0, 1000.0) == 1
    assert bench.repeats_for(1e-4, 1000.0) == 4000                       # capped
    peaks = {"bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0}
    chunks = [(1965, [1.0, 1.0]), (1650, [2.0]), (None, [4.0])]
    b = bench.bin_by_clock(chunks, peaks, unit_work=1.6e12, peak_key_burst="bf16_tflops",
                           peak_key_settled="bf16_tflops_sustained", scale=1e-12)
    assert b["burst"]["samples"] == 2 and b["burst"]["frac"] == pytest.approx(1.0)          # 1.6e12 FLOP in 1 ms = 1600 TF
    assert b["settled"]["sm_mhz"] == 1650 and b["settled"]["frac"] == pytest.approx(800.0 / 1400.0)
    assert b["unknown"]["rate"] == pytest.approx(400.0)
    from paper_2608_12629_b200 import inputs
    assert "c2: N=1048576 D=128 K=1024 B=1" in bench.workload_string(inputs.WORKLOADS["c2"])
    assert "WARM" in bench.l2_note(inputs.WORKLOADS["c1"], False) and "COLD" in bench.l2_note(inputs.WORKLOADS["c1"], True)
    assert "larger than" in bench.l2_note(inputs.WORKLOADS["c2"], False)


def test_parity_on_sample_counts_near_ties_and_unexcused():
    import numpy as np
    from oracle import kmeans_oracle as orc
    from paper_2608_12629_b200 import inputs
    X = torch.tensor([[0.0, 0.0], [1.0, 0.0], [10.0, 0.0], [5.0, 0.0]]).to(torch.bfloat16)
    C = torch.tensor([[0.0, 0.0], [10.0, 0.0], [10.0078125, 0.0]]).to(torch.bfloat16)   # centroids 1 and 2 nearly coincide
    Xb, Cb = inputs.to_bits(X), inputs.to_bits(C)
    idx_o, dist_o, _ = orc.assign(Xb, Cb)
    sel = np.arange(4)
    gpu = np.array([0, 1, 2, 0], dtype=np.int32)            # row 1: plainly wrong; row 2: the near twin; row 3: exact tie broken right
    rep = bench.parity_on_sample(Xb, Cb, sel, idx_o, dist_o, gpu, orc.pair_sqdist(Xb, Cb, gpu).astype(np.float32))
    assert rep == {"rows": 4, "mismatch": 2, "near_ties": 1, "unexcused": 1, "max_dist_err_rel": 0.0}


def test_reference_arm_prints_one_json_line_and_other_ranks_stay_silent():
    env = dict(os.environ, OMP_NUM_THREADS="4")
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1", "--steps", "2",
           "--warmup", "1"]
    out = subprocess.run(cmd, env=dict(env, RANK="0", WORLD_SIZE="2"), capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["metric"] == bench.METRIC and line["unit"] == bench.UNIT
    assert line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["gpu_launches"] == 0
    other = subprocess.run(cmd, env=dict(env, RANK="1", WORLD_SIZE="2"), capture_output=True, text=True, timeout=300)
    assert other.returncode == 0 and other.stdout.strip() == ""


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    times = [10.0 + rank, 3.0 - rank, 1.0, 7.0 * (rank + 1)]       # ms per quantity, different on each rank
    red = bench.max_over_ranks(times, torch.device("cpu"), world)
    line = bench.assemble_value(world, steps=4, ms_total=red[0])
    dist.barrier()
    if rank == 0:
        q.put((red, line))
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value_with_gloo_world_size_2():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    red, line = q.get(timeout=120)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    assert red == [11.0, 3.0, 1.0, 14.0]                            # the slowest rank decides every time
    assert line["ms_per_step"] == pytest.approx(11.0 / 4)
    assert line["value"] == pytest.approx(2 * 1000.0 / (11.0 / 4))   # units of ALL ranks / max time


def test_roofline_denominator_follows_the_clock_bin_of_the_launches():
    peaks = {"bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0, "source": "measured"}
    p, src = bench.roofline_peak({"settled": {"samples": 900}, "burst": {"samples": 20}}, peaks)
    assert p == 1400.0 and "sustained" in src
    p, src = bench.roofline_peak({"burst": {"samples": 50}}, peaks)
    assert p == 1600.0 and "burst" in src
    p, src = bench.roofline_peak({"settled": {"samples": 10}}, {"bf16_tflops": 1590.0, "source": "fallback"})
    assert p == 1590.0 and src.startswith("fallback")
