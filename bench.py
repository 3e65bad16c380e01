#!/usr/bin/env python
"""Benchmark of the Flash-KMeans Lloyd hot path on B200.

A "step" is one Lloyd iteration (assign + centroid update) over the workload's seeded synthetic Gaussian
mixture.  The K timed steps are ONE cake_kmeans_lloyd(iters=K) call (the library's own loop, centroids fed
forward on the device) that starts from the centroids of a warm-up call of W iterations; that K-step call is
repeated back to back until the timed region lasts about a second, so that the clocks settle and are sampled
often; `value` is K / (median time of a repeat).
Prints ONE JSON line (rank 0):
  value        Lloyd iterations/s with X resident in HBM (whole job, all ranks)
  e2e          the same through cake_kmeans_lloyd_host: pinned HOST buffers, H2D + D2H inside the timing
  roofline     the dominant kernel (assign): 2*N*K*D FLOP / its CUDA-event time, against the measured bf16
               tensor peak; `assign` / `update` give both kernels, also binned by the SM clock sampled while
               they ran (burst bin against the burst peak, settled bin against the sustained peak)
  cpu_baseline the fp64 CPU oracle timed on this machine's host cores on a bounded row sample; the same rows give
               `parity_sample` (mismatches against the GPU's indices, near-ties, distance error)
  extra        one compact row per other named workload (c1, c3, c4, paper shape)
`--impl reference` times the CPU oracle alone (there is no reference implementation to install).
Multi-GPU (`--gpus N` under torchrun): the rows of the ONE problem are dealt to the ranks and every iteration
all-reduces the per-cluster sums and counts (NCCL): strong scaling.  `--replicas` instead gives every rank its
own independent problem of the same shape (no collective): weak scaling.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import math
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
L2_BYTES = 126e6
BURST_MHZ = 1900          # a sample at or above this SM clock counts as "burst", below as "settled"


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
        except Exception:
            pass
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


def workload_string(w) -> str:
    """The one description of a workload that both arms print."""
    return (f"{w.name}: N={w.N} D={w.D} K={w.K} B={w.B}, {w.components}-component Gaussian mixture, "
            f"sigma={w.sigma}, random-sample init, seed {w.seed}")


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.002):
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

    def mark(self) -> int:
        """Number of samples taken so far (to cut the series into pieces later)."""
        return len(self.samples)

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
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"], "samples": 0}
        return {"sm_mhz": int(statistics.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "sm_mhz_min": min(self.samples), "sm_mhz_max": max(self.samples),
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


def algorithmic_assign_bytes(w):
    # X once, centroids once, idx and dist written
    return w.B * (2 * w.N * w.D + 2 * w.K * w.D + 8 * w.N)


def max_over_ranks(values, device, world):
    """Element-wise maximum over all ranks of a list of floats (device times in ms)."""
    t = torch.tensor(values, device=device, dtype=torch.float64)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def assemble_value(world, steps, ms_total):
    """Whole-job throughput when every rank processed `steps` units of its OWN problem in the (max over ranks) time."""
    ms_step = ms_total / steps
    return {"value": world * 1000.0 / ms_step, "ms_per_step": ms_step}


def repeats_for(est_ms: float, min_region_ms: float, cap: int = 4000) -> int:
    """How often the K-step call is repeated so that the timed region lasts at least `min_region_ms`."""
    if est_ms <= 0:
        return 1
    return int(max(1, min(cap, math.ceil(min_region_ms / est_ms))))


def bin_by_clock(chunks, peaks, unit_work, peak_key_burst, peak_key_settled, scale):
    """chunks: list of (median SM MHz or None, [ms, ...]).  Splits the samples into those taken at a burst clock
    and the rest, and gives for each bin the mean time, the achieved rate (unit_work / time * scale) and its
    fraction of the matching measured peak (burst peak for the burst bin, sustained / plain peak otherwise)."""
    bins = {"burst": [], "settled": [], "unknown": []}
    mhz = {"burst": [], "settled": [], "unknown": []}
    for clk, ms in chunks:
        key = "unknown" if clk is None else ("burst" if clk >= BURST_MHZ else "settled")
        bins[key].extend(ms)
        if clk is not None:
            mhz[key].append(clk)
    out = {}
    for key, ms in bins.items():
        if not ms:
            continue
        t = statistics.mean(ms)
        rate = unit_work / (t * 1e-3) * scale
        peak = peaks[peak_key_burst] if key != "settled" else peaks.get(peak_key_settled, peaks[peak_key_burst])
        out[key] = {"samples": len(ms), "sm_mhz": int(statistics.median(mhz[key])) if mhz[key] else None,
                    "ms": t, "rate": rate, "frac": rate / peak,
                    "ms_x_mhz": t * statistics.median(mhz[key]) if mhz[key] else None}
    return out


def oracle_sample(w, Xb, Cb, budget_s, max_rows=None):
    """The oracle (assign + update) on a bounded row sample; returns (iters/s extrapolated, rows selected (sorted
    indices), seconds, cores, oracle idx, oracle dist)."""
    from oracle import kmeans_oracle as orc
    N = Xb.shape[0]
    probe = min(N, 256)
    t0 = time.perf_counter()
    orc.assign(Xb[:probe], Cb)
    per_row = max((time.perf_counter() - t0) / probe, 1e-9)
    rows = int(max(probe, min(N, budget_s / per_row)))
    rows = min(N, rows if max_rows is None else min(rows, max_rows))
    sel = np.sort(np.random.default_rng(w.seed).choice(N, rows, replace=False)) if rows < N else np.arange(N)
    Xs = np.ascontiguousarray(Xb[sel])
    t0 = time.perf_counter()
    idx, dist, _ = orc.assign(Xs, Cb)
    orc.update(Xs, idx, w.K, Cb)
    dt = time.perf_counter() - t0
    iter_s = dt * (N / rows) * w.B
    return 1.0 / iter_s, sel, dt, orc.num_threads(), idx, dist


def oracle_sample_rate(w, Xb, Cb, budget_s, threads_note=""):
    v, sel, dt, cores, _, _ = oracle_sample(w, Xb, Cb, budget_s)
    return v, len(sel), dt, cores


def parity_on_sample(Xb, Cb, sel, idx_o, dist_o, idx_gpu, dist_gpu):
    """Part of the CPU-baseline leg: the rows the oracle was just timed on, compared with what the GPU returned for
    them.  A GPU index that differs from the oracle's is a near-tie (excused) iff d64(x, c_gpu) - d64(x, c_best) <
    1e-3 (|x|^2 + |c_best|^2); distances are compared with 1e-3 (|x|^2 + |c_gpu|^2)."""
    from oracle import kmeans_oracle as orc
    Xs = np.ascontiguousarray(Xb[sel])
    g = np.ascontiguousarray(idx_gpu[sel]).astype(np.int32)
    X = orc.bf16_to_f64(Xs)
    C = orc.bf16_to_f64(Cb)
    xn, cn = (X * X).sum(1), (C * C).sum(1)
    d_g = orc.pair_sqdist(Xs, C, g)
    mism = g != idx_o
    unexcused = mism & ~((d_g - dist_o) < 1e-3 * (xn + cn[idx_o]))
    err = np.abs(dist_gpu[sel].astype(np.float64) - d_g) / (xn + cn[g] + 1e-300)
    return {"rows": int(len(sel)), "mismatch": int(mism.sum()), "near_ties": int((mism & ~unexcused).sum()),
            "unexcused": int(unexcused.sum()), "max_dist_err_rel": float(err.max()) if len(err) else 0.0}


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
            "warmup": warm, "ms_per_step": 1000.0 / value, "higher_is_better": True,
            "scaling": "weak" if args.replicas or args.gpus == 1 else "strong",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_string(w), "note": "CPU oracle, no GPU work"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"{rows} of {w.N} rows per step (assign + update), time scaled by N/rows"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_sweep(args):
    """Shape sweep (3 Lloyd iterations per shape): one markdown table row per shape with the fraction of
    the roofline (the slower of 2NKD at the tensor peak and the bytes moved at HBM bandwidth).  With
    --sweep-grade every shape's assignment is also graded on 8,192 sampled rows by the CPU oracle."""
    import paper_2608_12629_b200 as cake
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks = measured_peaks()
    Ns = [1 << 16, 1 << 20, 1 << 24] if not args.sweep_full else [1 << e for e in range(16, 25)]
    Ds = [64, 96, 100, 128, 256, 384, 1024]      # 1024: rows streamed over D (no resident X tile)
    Ks = [64, 256, 1000, 1024, 4096, 65536] if not args.sweep_full else [64, 128, 256, 512, 1000, 1024, 2048, 4096,
                                                                          8192, 16384, 32768, 65536]
    grade = args.sweep_grade
    head = "| N | D | K | lloyd it/s | assign ms | TFLOP/s | update ms | GB/s | roofline it/s | fraction | X in L2 |"
    sep = "|---|---|---|---|---|---|---|---|---|---|---|"
    if grade:
        head += " rows graded | mismatch | unexcused | max_dist_err_rel |"
        sep += "---|---|---|---|"
    print(head)
    print(sep, flush=True)
    e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    for D in Ds:
        for N in Ns:
            if D > 512 and N > (1 << 20):       # 32 GiB of X and minutes of oracle grading: left out
                continue
            w0 = inputs.sweep_workload(N, D, 64)
            X, _ = inputs.gaussian_mixture(N, D, 16384, w0.mean_std, w0.sigma, w0.seed, device=dev)
            for K in Ks:
                if K > N:
                    continue
                w = inputs.sweep_workload(N, D, K)
                C0 = inputs.sample_init(X, K, w.seed)
                ws = cake.alloc_workspace(1, N, D, K, dev)
                out = cake.alloc_lloyd_outputs(X, C0, w.iters)
                wo = cake.alloc_lloyd_outputs(X, C0, 1)
                cake.cake_kmeans_lloyd(X, C0, 1, out=wo, ws=ws)      # warm-up: the loop, and the two kernels timed one by one
                cake.cake_kmeans_assign(X, C0, out_idx=wo.idx, out_dist=wo.dist, ws=ws)
                cake.cake_kmeans_update(X, wo.idx, K, C_prev=C0, out_C=wo.C, out_C_bf16=wo.C_bf16, out_counts=wo.counts, ws=ws)
                del wo
                e[0].record()
                cake.cake_kmeans_lloyd(X, C0, w.iters, out=out, ws=ws)
                e[1].record()
                Cin = out.C_bf16.clone()
                cake.cake_kmeans_assign(X, Cin, out_idx=out.idx, out_dist=out.dist, ws=ws)
                e[2].record()
                cake.cake_kmeans_update(X, out.idx, K, C_prev=Cin, out_C=out.C, out_C_bf16=out.C_bf16,
                                        out_counts=out.counts, ws=ws)
                e[3].record()
                torch.cuda.synchronize()
                if cake.cake_kmeans_device_status(ws) != cake.CAKE_OK:
                    raise SystemExit("device status raised during the sweep")
                it_ms = e[0].elapsed_time(e[1]) / w.iters
                a_ms, u_ms = e[1].elapsed_time(e[2]), e[2].elapsed_time(e[3])
                flop = 2.0 * N * K * D
                a_bytes = algorithmic_assign_bytes(w)
                u_bytes = algorithmic_update_bytes(w)
                floor_ms = max(flop / (peaks["bf16_tflops"] * 1e12), a_bytes / (peaks["hbm_gbs"] * 1e9)) * 1e3 + \
                    u_bytes / (peaks["hbm_gbs"] * 1e9) * 1e3
                row = (f"| {N} | {D} | {K} | {1000.0 / it_ms:.1f} | {a_ms:.4f} | {flop / a_ms / 1e9:.1f} | {u_ms:.4f} | "
                       f"{u_bytes / u_ms / 1e6:.0f} | {1000.0 / floor_ms:.1f} | {floor_ms / it_ms:.3f} | "
                       f"{'yes (warm)' if 2 * N * D < L2_BYTES else 'no'} |")
                if grade:
                    from oracle import kmeans_oracle as orc
                    sel = np.sort(np.random.default_rng(w.seed).choice(N, min(N, 8192 if K <= 8192 else 1024), replace=False))
                    sel_t = torch.from_numpy(sel).to(dev)
                    Xb, Cb = inputs.to_bits(X[sel_t]), inputs.to_bits(Cin)
                    idx_o, dist_o, _ = orc.assign(Xb, Cb)
                    rep = parity_on_sample(Xb, Cb, np.arange(len(sel)), idx_o, dist_o, out.idx[sel_t].cpu().numpy(),
                                           out.dist[sel_t].cpu().numpy())
                    row += f" {rep['rows']} | {rep['mismatch']} | {rep['unexcused']} | {rep['max_dist_err_rel']:.2e} |"
                print(row, flush=True)
                del ws, out
            del X
            torch.cuda.empty_cache()


def run_knn(args):
    """k-nearest-neighbour search: one markdown row per shape with the fraction of the same tensor roofline the
    assign kernel is measured against (2 N M D FLOP at the measured bf16 peak, or the bytes at HBM bandwidth)."""
    import paper_2608_12629_b200 as cake
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks = measured_peaks()
    print("| queries N | database M | D | k | ms | TFLOP/s | fraction of roofline | rows graded | mismatch | unexcused |")
    print("|---|---|---|---|---|---|---|---|---|---|", flush=True)
    shapes = [(65536, 1 << 20, 128), (65536, 1 << 20, 64), (16384, 1 << 22, 128), (1 << 20, 4096, 128), (65536, 1 << 18, 256),
              (8192, 65536, 96)]
    for N, M, D in shapes:
        w = inputs.sweep_workload(M, D, 64)
        X, _ = inputs.gaussian_mixture(M, D, 4096, w.mean_std, w.sigma, w.seed, device=dev)
        Q, _ = inputs.gaussian_mixture(N, D, 4096, w.mean_std, w.sigma, w.seed + 1, device=dev)
        for k in (1, 8, 32):
            ws = torch.zeros(cake.cake_knn_workspace_bytes(N, M, D, k), dtype=torch.uint8, device=dev)
            idx, dist = cake.cake_knn_search(Q, X, k, ws=ws)
            torch.cuda.synchronize()
            reps = 5
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
            ev[0].record()
            for i in range(reps):
                cake.cake_knn_search(Q, X, k, out_idx=idx, out_dist=dist, ws=ws)
                ev[i + 1].record()
            torch.cuda.synchronize()
            if cake.cake_kmeans_device_status(ws) != cake.CAKE_OK:
                raise SystemExit("device status raised")
            ms = statistics.median(ev[i].elapsed_time(ev[i + 1]) for i in range(reps))
            flop = 2.0 * N * M * D
            byts = 2.0 * (N + M) * D + 8.0 * N * k
            floor_ms = max(flop / (peaks["bf16_tflops"] * 1e12), byts / (peaks["hbm_gbs"] * 1e9)) * 1e3
            row = f"| {N} | {M} | {D} | {k} | {ms:.3f} | {flop / ms / 1e9:.0f} | {floor_ms / ms:.3f} |"
            if not args.no_cpu_baseline:
                from oracle import kmeans_oracle as orc
                sel = np.sort(np.random.default_rng(k).choice(N, 64 if M > (1 << 20) else 128, replace=False))
                sel_t = torch.from_numpy(sel).to(dev)
                Qb, Xb = inputs.to_bits(Q[sel_t]), inputs.to_bits(X)
                io, do = orc.knn(Qb, Xb, k)
                g = idx[sel_t].cpu().numpy()
                Xf, Qf = orc.bf16_to_f64(Xb), orc.bf16_to_f64(Qb)
                qn, xn = (Qf * Qf).sum(1), (Xf * Xf).sum(1)
                d_g = np.stack([orc.pair_sqdist(Qb, Xf, np.ascontiguousarray(g[:, p_])) for p_ in range(k)], 1)
                mism = g != io
                unexc = mism & ~(np.abs(d_g - do) < 1e-3 * (qn[:, None] + xn[io]))
                row += f" {len(sel)} | {int(mism.sum())} | {int(unexc.sum())} |"
            else:
                row += " - | - | - |"
            print(row, flush=True)
            del ws
        del X, Q
        torch.cuda.empty_cache()


class Runner:
    """One workload on this rank: buffers, the Lloyd call being timed and the per-kernel calls."""

    def __init__(self, cake, w, dev, rank, world, sharded):
        self.cake, self.w, self.dev, self.world, self.sharded = cake, w, dev, world, sharded
        if sharded:
            # the ONE problem, rows dealt to the ranks in contiguous shares; every rank holds all centroids
            Xfull, C0 = inputs.make_problem(w, device=dev)
            a, b = cake.shard_rows(w.N, rank, world)
            self.X = Xfull[a:b].contiguous()
            del Xfull
        elif w.B == 1:
            self.X, C0 = inputs.make_problem(w, device=dev, b=rank)
        else:
            self.X, C0 = inputs.make_batch(dataclasses.replace(w, seed=w.seed + 1000 * rank), device=dev)
        self.C0 = C0
        self.N_local = self.X.shape[-2]
        self.ws = cake.alloc_workspace(w.B, self.N_local, w.D, w.K, dev)
        self.stream = torch.cuda.current_stream(dev)

    def lloyd(self, start, iters, out):
        if self.sharded:
            return self.cake.cake_kmeans_lloyd_sharded(self.X, start, iters, out=out, ws=self.ws)
        return self.cake.cake_kmeans_lloyd(self.X, start, iters, out=out, ws=self.ws)

    def outputs(self, iters):
        return self.cake.alloc_lloyd_outputs(self.X, self.C0, iters)


def barrier(dev, world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize(dev)


def time_lloyd(r: Runner, steps, warmup, min_region_ms, clocks):
    """W warm-up iterations in one call, one untimed probe of the K-step call, then R timed repeats of it (all from
    the warm-up's centroids).  Returns per-repeat device times (ms, max over ranks), launches, start centroids."""
    cake, dev, world = r.cake, r.dev, r.world
    cur = r.C0.clone()
    if warmup > 0:
        out_w = r.outputs(warmup)
        r.lloyd(cur, warmup, out_w)
        cur.copy_(out_w.C_bf16)
        del out_w
    out_k = r.outputs(steps)
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(dev, world)
    p0.record(r.stream)
    r.lloyd(cur, steps, out_k)
    p1.record(r.stream)
    barrier(dev, world)
    est = max_over_ranks([p0.elapsed_time(p1)], dev, world)[0]
    repeats = repeats_for(est, min_region_ms)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(repeats + 1)]
    launches0 = cake.cake_kmeans_kernel_launches()
    barrier(dev, world)
    m0 = clocks.mark()
    ev[0].record(r.stream)
    for i in range(repeats):
        r.lloyd(cur, steps, out_k)
        ev[i + 1].record(r.stream)
    barrier(dev, world)
    m1 = clocks.mark()
    launches = cake.cake_kmeans_kernel_launches() - launches0
    times = max_over_ranks([ev[i].elapsed_time(ev[i + 1]) for i in range(repeats)], dev, world)
    total = max_over_ranks([ev[0].elapsed_time(ev[repeats])], dev, world)[0]
    status = cake.cake_kmeans_device_status(r.ws)
    if status != cake.CAKE_OK:
        raise SystemExit(f"device status {status}: {cake.strerror(status)}")
    return {"times": times, "total_ms": total, "repeats": repeats, "launches": int(launches), "start": cur,
            "out": out_k, "clock_marks": (m0, m1)}


def time_kernels(r: Runner, start, min_region_ms, clocks, chunk_ms=12.0, flush=None):
    """The same steps as assign + update calls with events between them, issued in chunks of about `chunk_ms`; each
    chunk is tagged with the median SM clock sampled while it ran.  flush: a scratch tensor larger than L2 that is
    overwritten before every timed kernel (workloads whose X fits in L2)."""
    cake, w, dev, world = r.cake, r.w, r.dev, r.world
    out = r.outputs(1)
    cur = start.clone()
    X, ws, K = r.X, r.ws, w.K

    def step(e):
        if flush is not None:
            flush.zero_()
        if e:
            e[0].record(r.stream)
        cake.cake_kmeans_assign(X, cur, out_idx=out.idx, out_dist=out.dist, ws=ws)
        if e:
            e[1].record(r.stream)
        if flush is not None:
            flush.zero_()
        if e:
            e[2].record(r.stream)
        cake.cake_kmeans_update(X, out.idx, K, C_prev=cur, out_C=out.C, out_C_bf16=out.C_bf16, out_counts=out.counts, ws=ws)
        if e:
            e[3].record(r.stream)
        cur.copy_(out.C_bf16)

    for _ in range(3):
        step(None)
    probe = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    barrier(dev, world)
    step(probe)
    barrier(dev, world)
    est = probe[0].elapsed_time(probe[3])
    per_chunk = int(max(1, min(512, round(chunk_ms / max(est, 1e-3)))))
    n_chunks = int(max(1, min(400, math.ceil(min_region_ms / (per_chunk * max(est, 1e-3))))))
    a_chunks, u_chunks = [], []
    for _ in range(n_chunks):
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(per_chunk)]
        m0 = clocks.mark()
        for e in ev:
            step(e)
        torch.cuda.synchronize(dev)
        s = clocks.samples[m0:clocks.mark()]
        clk = int(statistics.median(s)) if s else None
        a_chunks.append((clk, [e[0].elapsed_time(e[1]) for e in ev]))
        u_chunks.append((clk, [e[2].elapsed_time(e[3]) for e in ev]))
    barrier(dev, world)
    assign_ms = statistics.mean(t for _, ms in a_chunks for t in ms)
    update_ms = statistics.mean(t for _, ms in u_chunks for t in ms)
    assign_ms, update_ms = max_over_ranks([assign_ms, update_ms], dev, world)
    return {"assign_ms": assign_ms, "update_ms": update_ms, "assign_chunks": a_chunks, "update_chunks": u_chunks,
            "idx": out.idx, "dist": out.dist, "C_in": None}


def kernel_report(w, k, peaks, world, sharded):
    """assign / update blocks of the JSON line from the per-kernel timings (w: the whole problem's shape)."""
    share = world if sharded else 1            # rows of the problem per rank
    flop = 2.0 * w.B * w.N * w.K * w.D / share
    ub = algorithmic_update_bytes(w) / share
    a_tflops = flop / (k["assign_ms"] * 1e-3) / 1e12
    u_gbs = ub / (k["update_ms"] * 1e-3) / 1e9
    assign = {"ms": k["assign_ms"], "tflops": a_tflops, "frac_of_measured_bf16_peak": a_tflops / peaks["bf16_tflops"],
              "frac_of_measured_bf16_sustained": a_tflops / peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]),
              "frac_of_nominal_2250": a_tflops / 2250.0,
              "by_clock": bin_by_clock(k["assign_chunks"], peaks, flop, "bf16_tflops", "bf16_tflops_sustained", 1e-12)}
    update = {"ms": k["update_ms"], "gbs": u_gbs, "frac_of_measured_hbm": u_gbs / peaks["hbm_gbs"],
              "frac_of_nominal_8000": u_gbs / 8000.0, "algorithmic_bytes": ub,
              "by_clock": bin_by_clock(k["update_chunks"], peaks, ub, "hbm_gbs", "hbm_gbs", 1e-9)}
    return assign, update


def roofline_peak(by_clock, peaks):
    """(peak TFLOP/s, its description) for the assign kernel's roofline fraction, from the clock bins of its launches."""
    settled = by_clock.get("settled", {}).get("samples", 0)
    burst = by_clock.get("burst", {}).get("samples", 0)
    if settled >= burst and "bf16_tflops_sustained" in peaks:
        return peaks["bf16_tflops_sustained"], (peaks["source"] + " sustained (the kernel's launches ran inside a long region, at the "
                                                "settled clock under the power cap)")
    return peaks["bf16_tflops"], peaks["source"] + " burst (the kernel's launches ran at the full clock)"


def l2_note(w, flushed):
    xb = w.B * w.N * w.D * 2
    if xb > L2_BYTES:
        return f"X is {xb / 2**20:.0f} MiB per step, larger than the 126 MB L2; no flush"
    if flushed:
        return (f"X is {xb / 2**20:.1f} MiB and fits in L2: the Lloyd-loop number is WARM (X resident in L2); the per-kernel "
                "numbers are COLD (a 256 MiB buffer is overwritten before every timed kernel)")
    return f"X is {xb / 2**20:.1f} MiB and fits in L2: all numbers are WARM (X resident in L2)"


def cpu_leg(w, X, C_in, idx, dist, budget_s, max_rows):
    """CPU-baseline leg for one problem: the oracle timed on a bounded row sample against the centroids `C_in` the
    GPU's last timed assign used, and the parity of the GPU's result on those very rows."""
    Xb, Cb = inputs.to_bits(X), inputs.to_bits(C_in)
    v, sel, dt, cores, idx_o, dist_o = oracle_sample(w, Xb, Cb, budget_s, max_rows)
    par = parity_on_sample(Xb, Cb, sel, idx_o, dist_o, idx.cpu().numpy(), dist.cpu().numpy())
    base = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{len(sel)} of {w.N} rows of one problem (assign + update) in {dt:.1f} s, time scaled by N/rows and B"}
    return base, par


def last_assign(r: Runner, start):
    """One assign against `start` whose outputs are kept for the parity sample."""
    out = r.outputs(1)
    r.cake.cake_kmeans_assign(r.X, start, out_idx=out.idx, out_dist=out.dist, ws=r.ws)
    torch.cuda.synchronize(r.dev)
    return out.idx, out.dist


def extra_row(cake, name, dev, peaks, clocks, with_cpu):
    """Compact measurement of another named workload (single GPU): Lloyd it/s, both kernels, parity sample."""
    w = inputs.WORKLOADS[name]
    r = Runner(cake, w, dev, 0, 1, False)
    steps = max(2, min(w.iters * 4, 40))
    t = time_lloyd(r, steps, 3, 300.0, clocks)
    small = w.B * w.N * w.D * 2 <= L2_BYTES
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if small else None
    k = time_kernels(r, t["start"], 200.0, clocks, flush=flush)
    assign, update = kernel_report(w, k, peaks, 1, False)
    ms_step = statistics.median(t["times"]) / steps
    a_floor = max(2.0 * w.B * w.N * w.K * w.D / (peaks["bf16_tflops"] * 1e12), algorithmic_assign_bytes(w) / (peaks["hbm_gbs"] * 1e9))
    floor_ms = (a_floor + algorithmic_update_bytes(w) / (peaks["hbm_gbs"] * 1e9)) * 1e3
    row = {"workload": workload_string(w), "value": 1000.0 / ms_step, "unit": UNIT, "ms_per_step": ms_step,
           "steps": steps, "repeats": t["repeats"], "launches_per_step": t["launches"] / (steps * t["repeats"]),
           "roofline_ms_per_step": floor_ms, "frac_of_roofline_step": floor_ms / ms_step,
           "assign": {kk: assign[kk] for kk in ("ms", "tflops", "frac_of_measured_bf16_peak", "frac_of_measured_bf16_sustained")},
           "update": {kk: update[kk] for kk in ("ms", "gbs", "frac_of_measured_hbm")},
           "assign_hbm_gbs": algorithmic_assign_bytes(w) / (assign["ms"] * 1e-3) / 1e9,
           "l2": l2_note(w, small)}
    if with_cpu:
        idx, dist = last_assign(r, t["start"])
        X0 = r.X if w.B == 1 else r.X[0]
        C0 = t["start"] if w.B == 1 else t["start"][0]
        big = 2.0 * w.K * w.D > 4e6
        base, par = cpu_leg(w, X0, C0, idx if w.B == 1 else idx[0], dist if w.B == 1 else dist[0], 3.0, 1024 if big else 8192)
        row["cpu_baseline"], row["parity_sample"] = base, par
    del r, flush
    torch.cuda.empty_cache()
    return row


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2", choices=sorted(inputs.WORKLOADS))
    ap.add_argument("--min-region-s", type=float, default=1.0, help="the K-step call is repeated until the timed region lasts this long")
    ap.add_argument("--replicas", action="store_true", help="N > 1: independent problems per rank (weak scaling) instead of one row-sharded problem")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="skip the compact rows for the other named workloads")
    ap.add_argument("--sweep", action="store_true", help="print the shape-sweep table instead of the JSON line")
    ap.add_argument("--sweep-full", action="store_true", help="with --sweep: every power of two in N and K")
    ap.add_argument("--sweep-grade", action="store_true", help="with --sweep: grade every shape on sampled rows with the CPU oracle")
    ap.add_argument("--knn", action="store_true", help="print the k-nearest-neighbour search table instead of the JSON line")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
        return
    if args.knn:
        run_knn(args)
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
    sharded = world > 1 and not args.replicas and w.B == 1
    B, N, D, K = w.B, w.N, w.D, w.K
    r = Runner(cake, w, dev, rank, world, sharded)
    min_ms = args.min_region_s * 1e3

    with ClockSampler(physical_gpu_index(local)) as clocks:
        # ---------------- timed region 1: whole steps through the library's Lloyd loop (value)
        t = time_lloyd(r, args.steps, args.warmup, min_ms, clocks)
        region1 = clocks.samples[t["clock_marks"][0]:t["clock_marks"][1]]
        # ---------------- timed region 2: the same steps with events between the two kernels (roofline)
        k = time_kernels(r, t["start"], min_ms, clocks)
    clock_summary = clocks.summary()
    clock_summary["region1_samples"] = len(region1)
    clock_summary["region1_sm_mhz"] = int(statistics.median(region1)) if region1 else None

    # ---------------- timed region 3: end to end from pinned host memory (single-problem calls; not sharded)
    e2e = None
    if not args.no_e2e and not sharded:
        Xh, Ch = r.X.cpu().pin_memory(), r.C0.cpu().pin_memory()
        hout = cake.alloc_lloyd_outputs(Xh, Ch, 1, pin_host=True)
        scratch = torch.empty(cake.cake_kmeans_lloyd_host_device_bytes(B, N, D, K, 1), dtype=torch.uint8, device=dev)
        e2e_steps = max(3, min(args.steps, 20))
        for _ in range(2):
            cake.cake_kmeans_lloyd_host(Xh, Ch, 1, hout, scratch)
            Ch.copy_(hout.C_bf16)
        barrier(dev, world)
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(r.stream)
        for _ in range(e2e_steps):
            cake.cake_kmeans_lloyd_host(Xh, Ch, 1, hout, scratch)
            r.stream.synchronize()          # the caller reads the result (centroids, inertia) every step
            Ch.copy_(hout.C_bf16)
        f1.record(r.stream)
        barrier(dev, world)
        e2e_ms = max_over_ranks([f0.elapsed_time(f1) / e2e_steps], dev, world)[0]
        h2d = Xh.numel() * 2 + Ch.numel() * 2
        d2h = sum(x.numel() * x.element_size() for x in (hout.C, hout.C_bf16, hout.idx, hout.dist, hout.counts, hout.inertia))
        e2e = {"ms": e2e_ms, "h2d": h2d, "d2h": d2h}
        del scratch, Xh, hout

    if rank == 0:
        ms_rep = statistics.median(t["times"])
        ms_step = ms_rep / args.steps
        units = 1 if (sharded or world == 1) else world          # problems processed per step by the whole job
        assign, update = kernel_report(w, k, peaks, world, sharded)
        # the denominator that matches how the kernel was timed: the sustained cuBLAS figure when most of its launches
        # ran at the settled clock of a long region under the power cap, the burst figure when they ran at the full clock
        roof_peak, roof_source = roofline_peak(assign["by_clock"], peaks)
        line = {
            "metric": METRIC, "value": units * 1000.0 / ms_step, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "strong" if sharded else "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "repeats": t["repeats"], "ms_per_step_min": min(t["times"]) / args.steps,
            "ms_per_step_mean": t["total_ms"] / (args.steps * t["repeats"]), "timed_region_ms": t["total_ms"],
            "config": {"workload": workload_string(w),
                       "parallelism": (f"rows of the one problem dealt to {world} ranks, all-reduce of sums and counts per iteration"
                                       if sharded else ("one independent problem per rank, no collective" if world > 1 else "1 GPU")),
                       "l2": l2_note(w, False),
                       "step": "one Lloyd iteration; the K timed steps are one cake_kmeans_lloyd(iters=K) call that starts from the "
                               "warm-up call's centroids, repeated `repeats` times back to back; value = K / median repeat time",
                       "x_checksum": inputs.checksum(r.X.view(-1)[: 1 << 20])},
            "assign": assign, "update": update,
            "roofline": {"bound": "tensor",
                         "kernel": ("assign_pair_kernel, wide mode (+ half-norm prologue, row operand)" if w.D > 512
                                    else "assign_tc_kernel (+ half-norm prologue)"),
                         "achieved": assign["tflops"],
                         "peak": roof_peak, "peak_source": roof_source, "unit": "TFLOP/s",
                         "frac": assign["tflops"] / roof_peak,
                         "frac_of_burst_peak": assign["frac_of_measured_bf16_peak"],
                         "frac_of_sustained_peak": assign["frac_of_measured_bf16_sustained"],
                         "traffic": NCU_DRAM_BYTES_PER_ASSIGN_LAUNCH.get(w.name) if world == 1 else None,
                         "algorithmic_bytes": algorithmic_assign_bytes(w) / (world if sharded else 1)},
            "clocks": clock_summary,
            "gpu_launches": t["launches"],
            "impl": "ours",
        }
        update["traffic"] = NCU_DRAM_BYTES_PER_UPDATE_LAUNCH.get(w.name) if world == 1 else None
        if e2e:
            line["e2e"] = {"value": units * 1000.0 / e2e["ms"], "unit": UNIT, "h2d_bytes_per_step": e2e["h2d"],
                           "d2h_bytes_per_step": e2e["d2h"], "ms_per_step": e2e["ms"],
                           "note": "one cake_kmeans_lloyd_host(iters=1) call per step: X and the centroids are uploaded and every "
                                   "output is read back EVERY step (a caller that keeps X on the device pays the upload once)"}
        if world == 1 and not args.no_cpu_baseline:
            idx, dist_g = last_assign(r, t["start"])
            X0 = r.X if B == 1 else r.X[0]
            C_in = t["start"] if B == 1 else t["start"][0]
            base, par = cpu_leg(w, X0, C_in, idx if B == 1 else idx[0], dist_g if B == 1 else dist_g[0], 12.0, None)
            line["cpu_baseline"], line["parity_sample"] = base, par
        if world == 1 and not args.no_extra:
            del r
            torch.cuda.empty_cache()
            with ClockSampler(physical_gpu_index(local)) as xclocks:
                line["extra"] = [extra_row(cake, name, dev, peaks, xclocks, not args.no_cpu_baseline)
                                 for name in ("c1", "c2", "c3", "c4", "paper", "f1", "w1") if name != w.name]
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
