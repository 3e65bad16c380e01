#!/usr/bin/env python
"""Benchmark of the Flash-KMeans Lloyd hot path on B200.

A "step" is one Lloyd iteration (assign + centroid update) over the workload's seeded synthetic Gaussian
mixture; the K timed steps are ONE cake_kmeans_lloyd(iters=K) call (the library's own loop, centroids fed
forward on the device) after one warm-up call of W iterations.
Prints ONE JSON line (rank 0):
  value      Lloyd iterations/s with X resident in HBM (whole job, all ranks)
  e2e        the same through cake_kmeans_lloyd_host: pinned HOST buffers, H2D + D2H inside the timing
  roofline   the dominant kernel (assign): 2*N*K*D FLOP / its CUDA-event time inside the timed region,
             against the measured bf16 tensor peak; also update GB/s against measured HBM bandwidth
  cpu_baseline  the fp64 CPU oracle timed on this machine's host cores on a bounded sample
`--impl reference` times the CPU oracle alone (there is no reference implementation to install).
Multi-GPU (`--gpus N` under torchrun): every rank runs its own independent problem of the same
shape (no data-path collective), timed as the max over ranks: weak scaling.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2608_12629_b200 import inputs  # noqa: E402

# dram__bytes_read.sum + dram__bytes_write.sum of ONE launch of the dominant kernel (assign_tc_kernel),
# from the ncu capture summarised in profiles/assign_tc_kernel_c2.md (same workload, same launch shape)
NCU_DRAM_BYTES_PER_ASSIGN_LAUNCH = {"c2": 268921088 + 9016832}
# the same for the dominant update kernel (slab_update_kernel), profiles/update_slab_route_c2.md
NCU_DRAM_BYTES_PER_UPDATE_LAUNCH = {"c2": 273203712 + 4012032}

METRIC = "lloyd_iters_per_sec"
UNIT = "iter/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
        except Exception:
            pass
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.004):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._index, self._period = index, period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None

    def _loop(self):
        nv = self._nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20,
                 "hw_thermal_slowdown": 0x40, "hw_power_brake_slowdown": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                try:
                    r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for n, bit in names.items():
                    if r & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            self._stop.wait(self._period)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        return {"sm_mhz": int(statistics.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


def algorithmic_update_bytes(w):
    # X once, idx once, previous centroids (bf16) read, fp32 + bf16 centroids and counts written
    return w.B * (2 * w.N * w.D + 4 * w.N + 4 * w.K * w.D + 2 * w.K * w.D + 2 * w.K * w.D + 4 * w.K)


def max_over_ranks(values, device, world):
    """Element-wise maximum over all ranks of a list of floats (device times in ms)."""
    t = torch.tensor(values, device=device, dtype=torch.float64)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def assemble_value(world, steps, ms_total):
    """Whole-job throughput: every rank processed `steps` units in the (max over ranks) time."""
    ms_step = ms_total / steps
    return {"value": world * 1000.0 / ms_step, "ms_per_step": ms_step}


def oracle_sample_rate(w, Xb, Cb, budget_s, threads_note):
    """Times the oracle on a bounded row sample; returns (iters_per_s_extrapolated, rows, seconds, cores)."""
    from oracle import kmeans_oracle as orc
    N = Xb.shape[0]
    probe = min(N, 256)
    t0 = time.perf_counter()
    orc.assign(Xb[:probe], Cb)
    per_row = max((time.perf_counter() - t0) / probe, 1e-9)
    rows = int(max(probe, min(N, budget_s / per_row)))
    rows = min(N, rows)
    sel = np.sort(np.random.default_rng(w.seed).choice(N, rows, replace=False)) if rows < N else np.arange(N)
    Xs = np.ascontiguousarray(Xb[sel])
    t0 = time.perf_counter()
    idx, _, _ = orc.assign(Xs, Cb)
    orc.update(Xs, idx, w.K, Cb)
    dt = time.perf_counter() - t0
    iter_s = dt * (N / rows) * w.B
    return 1.0 / iter_s, rows, dt, orc.num_threads()


def run_reference(args, rank, world):
    """The reference arm: the fp64 CPU oracle as it stands, on this machine's host cores, rank 0 only."""
    if rank != 0:
        return
    w = inputs.WORKLOADS[args.workload]
    X, C0 = inputs.make_problem(w, device="cpu")
    Xb, Cb = inputs.to_bits(X), inputs.to_bits(C0)
    steps, warm = args.steps, args.warmup
    budget = min(20.0, 150.0 / max(1, steps + warm))
    vals, rows, cores = [], 0, 0
    for s in range(warm + steps):
        v, rows, dt, cores = oracle_sample_rate(w, Xb, Cb, budget, "")
        if s >= warm:
            vals.append(v)
    value = len(vals) / sum(1.0 / v for v in vals)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": warm, "ms_per_step": 1000.0 / value, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{w.name}: N={w.N} D={w.D} K={w.K} B={w.B}", "note": "CPU oracle, no GPU work"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"{rows} of {w.N} rows per step (assign + update), time scaled by N/rows"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_sweep(args):
    """Shape sweep (3 Lloyd iterations per shape): one markdown table row per shape with the fraction of
    the roofline (the slower of 2NKD at the tensor peak and the bytes moved at HBM bandwidth)."""
    import paper_2608_12629_b200 as cake
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks = measured_peaks()
    Ns = [1 << 16, 1 << 20, 1 << 24] if not args.sweep_full else [1 << e for e in range(16, 25)]
    Ds = [64, 96, 100, 128, 256, 384]
    Ks = [64, 256, 1000, 1024, 4096, 65536] if not args.sweep_full else [64, 128, 256, 512, 1000, 1024, 2048, 4096,
                                                                          8192, 16384, 32768, 65536]
    print("| N | D | K | lloyd it/s | assign ms | TFLOP/s | update ms | GB/s | roofline it/s | fraction |")
    print("|---|---|---|---|---|---|---|---|---|---|", flush=True)
    e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    for D in Ds:
        for N in Ns:
            w0 = inputs.sweep_workload(N, D, 64)
            X, _ = inputs.gaussian_mixture(N, D, 16384, w0.mean_std, w0.sigma, w0.seed, device=dev)
            for K in Ks:
                if K > N:
                    continue
                w = inputs.sweep_workload(N, D, K)
                C0 = inputs.sample_init(X, K, w.seed)
                ws = cake.alloc_workspace(1, N, D, K, dev)
                out = cake.alloc_lloyd_outputs(X, C0, w.iters)
                cake.cake_kmeans_lloyd(X, C0, 1, out=cake.alloc_lloyd_outputs(X, C0, 1), ws=ws)      # warm-up
                e[0].record()
                cake.cake_kmeans_lloyd(X, C0, w.iters, out=out, ws=ws)
                e[1].record()
                cake.cake_kmeans_assign(X, out.C_bf16, out_idx=out.idx, out_dist=out.dist, ws=ws)
                e[2].record()
                cake.cake_kmeans_update(X, out.idx, K, C_prev=out.C_bf16, out_C=out.C, out_C_bf16=out.C_bf16,
                                        out_counts=out.counts, ws=ws)
                e[3].record()
                torch.cuda.synchronize()
                if cake.cake_kmeans_device_status(ws) != cake.CAKE_OK:
                    raise SystemExit("device status raised during the sweep")
                it_ms = e[0].elapsed_time(e[1]) / w.iters
                a_ms, u_ms = e[1].elapsed_time(e[2]), e[2].elapsed_time(e[3])
                flop = 2.0 * N * K * D
                a_bytes = 2 * N * D + 2 * K * D + 8 * N
                u_bytes = algorithmic_update_bytes(w)
                floor_ms = max(flop / (peaks["bf16_tflops"] * 1e12), a_bytes / (peaks["hbm_gbs"] * 1e9)) * 1e3 + \
                    u_bytes / (peaks["hbm_gbs"] * 1e9) * 1e3
                print(f"| {N} | {D} | {K} | {1000.0 / it_ms:.1f} | {a_ms:.4f} | {flop / a_ms / 1e9:.1f} | {u_ms:.4f} | "
                      f"{u_bytes / u_ms / 1e6:.0f} | {1000.0 / floor_ms:.1f} | {floor_ms / it_ms:.3f} |", flush=True)
                del ws, out
            del X
            torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2", choices=sorted(inputs.WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--sweep", action="store_true", help="print the shape-sweep table instead of the JSON line")
    ap.add_argument("--sweep-full", action="store_true", help="with --sweep: every power of two in N and K")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import torch.distributed as dist
    import paper_2608_12629_b200 as cake

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    w = inputs.WORKLOADS[args.workload]
    peaks = measured_peaks()
    # every rank gets its own independent problem (weak scaling, no collective on the data path)
    if w.B == 1:
        X, C0 = inputs.make_problem(w, device=dev, b=rank)
    else:
        import dataclasses
        X, C0 = inputs.make_batch(dataclasses.replace(w, seed=w.seed + 1000 * rank), device=dev)
    B, N, D, K = w.B, w.N, w.D, w.K
    ws = cake.alloc_workspace(B, N, D, K, dev)
    out = cake.alloc_lloyd_outputs(X, C0, 1)
    stream = torch.cuda.current_stream(dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    # ---------------- timed region 1: whole steps through cake_kmeans_lloyd (value)
    # W warm-up iterations in one call, then the K timed iterations in one call that starts from the
    # warm-up's centroids: the library's own Lloyd loop, no host work between the steps
    cur = C0.clone()
    if args.warmup > 0:
        out_w = cake.alloc_lloyd_outputs(X, C0, args.warmup)
        cake.cake_kmeans_lloyd(X, cur, args.warmup, out=out_w, ws=ws)
        cur.copy_(out_w.C_bf16)
        del out_w
    out_k = cake.alloc_lloyd_outputs(X, C0, args.steps)
    barrier()
    launches0 = cake.cake_kmeans_kernel_launches()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(physical_gpu_index(local)) as clocks:
        barrier()
        e0.record(stream)
        cake.cake_kmeans_lloyd(X, cur, args.steps, out=out_k, ws=ws)
        e1.record(stream)
        barrier()
    del out_k
    launches = cake.cake_kmeans_kernel_launches() - launches0
    ms_total = e0.elapsed_time(e1)
    status = cake.cake_kmeans_device_status(ws)
    if status != cake.CAKE_OK:
        raise SystemExit(f"device status {status}: {cake.strerror(status)}")

    # ---------------- timed region 2: the same steps with events between the two kernels (roofline)
    cur.copy_(C0)
    idx, dist_buf = out.idx, out.dist
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    for _ in range(3):
        cake.cake_kmeans_assign(X, cur, out_idx=idx, out_dist=dist_buf, ws=ws)
        cake.cake_kmeans_update(X, idx, K, C_prev=cur, out_C=out.C, out_C_bf16=out.C_bf16, out_counts=out.counts, ws=ws)
    barrier()
    for s in range(args.steps):
        ev[s][0].record(stream)
        cake.cake_kmeans_assign(X, cur, out_idx=idx, out_dist=dist_buf, ws=ws)
        ev[s][1].record(stream)
        cake.cake_kmeans_update(X, idx, K, C_prev=cur, out_C=out.C, out_C_bf16=out.C_bf16, out_counts=out.counts, ws=ws)
        ev[s][2].record(stream)
        cur.copy_(out.C_bf16)
    barrier()
    assign_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in ev)
    update_ms = statistics.mean(e[1].elapsed_time(e[2]) for e in ev)

    # ---------------- timed region 3: end to end from pinned host memory
    e2e = None
    if not args.no_e2e:
        Xh, Ch = X.cpu().pin_memory(), C0.cpu().pin_memory()
        hout = cake.alloc_lloyd_outputs(Xh, Ch, 1, pin_host=True)
        scratch = torch.empty(cake.cake_kmeans_lloyd_host_device_bytes(B, N, D, K, 1), dtype=torch.uint8, device=dev)
        e2e_steps = max(3, min(args.steps, 20))
        for _ in range(2):
            cake.cake_kmeans_lloyd_host(Xh, Ch, 1, hout, scratch)
            Ch.copy_(hout.C_bf16)
        barrier()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(stream)
        for _ in range(e2e_steps):
            cake.cake_kmeans_lloyd_host(Xh, Ch, 1, hout, scratch)
            stream.synchronize()          # the caller reads the result (centroids, inertia) every step
            Ch.copy_(hout.C_bf16)
        f1.record(stream)
        barrier()
        e2e_ms = f0.elapsed_time(f1) / e2e_steps
        h2d = Xh.numel() * 2 + Ch.numel() * 2
        d2h = sum(t.numel() * t.element_size() for t in (hout.C, hout.C_bf16, hout.idx, hout.dist, hout.counts, hout.inertia))
        e2e = {"ms": e2e_ms, "h2d": h2d, "d2h": d2h}
        del scratch

    # ---------------- max over ranks
    ms_total, assign_ms, update_ms, e2e_ms = max_over_ranks(
        [ms_total, assign_ms, update_ms, e2e["ms"] if e2e else 0.0], dev, world)

    if rank == 0:
        whole = assemble_value(world, args.steps, ms_total)
        ms_step = whole["ms_per_step"]
        flop = 2.0 * B * N * K * D
        a_tflops = flop / (assign_ms * 1e-3) / 1e12
        u_gbs = algorithmic_update_bytes(w) / (update_ms * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": whole["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"{w.name}: N={N} D={D} K={K} B={B}, {w.components}-component Gaussian mixture, "
                                   f"sigma={w.sigma}, random-sample init, seed {w.seed}+rank",
                       "l2": f"X is {B * N * D * 2 / 2**20:.0f} MiB per step, larger than the 126 MB L2; no flush",
                       "step": "one Lloyd iteration; the K timed steps are one cake_kmeans_lloyd(iters=K) call that starts from the warm-up call's centroids",
                       "x_checksum": inputs.checksum(X.view(-1)[: 1 << 20])},
            "assign": {"ms": assign_ms, "tflops": a_tflops, "frac_of_measured_bf16_peak": a_tflops / peaks["bf16_tflops"],
                       "frac_of_measured_bf16_sustained": a_tflops / peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]),
                       "frac_of_nominal_2250": a_tflops / 2250.0},
            "update": {"ms": update_ms, "gbs": u_gbs, "frac_of_measured_hbm": u_gbs / peaks["hbm_gbs"],
                       "frac_of_nominal_8000": u_gbs / 8000.0, "algorithmic_bytes": algorithmic_update_bytes(w),
                       "traffic": NCU_DRAM_BYTES_PER_UPDATE_LAUNCH.get(w.name)},
            "roofline": {"bound": "tensor", "kernel": "assign_tc_kernel (+ half-norm prologue)", "achieved": a_tflops,
                         "peak": peaks["bf16_tflops"], "peak_source": peaks["source"] + " burst", "unit": "TFLOP/s",
                         "frac": a_tflops / peaks["bf16_tflops"], "traffic": None},
            "clocks": clocks.summary(),
            "gpu_launches": int(launches),
            "impl": "ours",
        }
        if e2e:
            line["e2e"] = {"value": world * 1000.0 / e2e_ms, "unit": UNIT, "h2d_bytes_per_step": e2e["h2d"],
                           "d2h_bytes_per_step": e2e["d2h"], "ms_per_step": e2e_ms}
        line["roofline"]["traffic"] = NCU_DRAM_BYTES_PER_ASSIGN_LAUNCH.get(w.name)
        line["roofline"]["algorithmic_bytes"] = B * (2 * N * D + 2 * K * D + 8 * N)
        if world == 1 and not args.no_cpu_baseline:
            Xb = inputs.to_bits(X if B == 1 else X[0])
            Cb = inputs.to_bits(C0 if B == 1 else C0[0])
            v, rows, dt, cores = oracle_sample_rate(w, Xb, Cb, 12.0, "")
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": f"{rows} of {N} rows of one problem (assign + update) in {dt:.1f} s, "
                                              f"time scaled by N/rows and B"}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
