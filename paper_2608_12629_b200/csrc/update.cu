// Centroid update: per-cluster sums and counts of the assigned points (paper Section 5,
// "Flash-KMeans clean-start workload": centroid_update), then the division into means.
//
// Three routes produce sums[B][K][D] (fp32) and counts[B][K]:
//   slab route : one kernel; every CTA counting-sorts its slab of rows by cluster in shared memory
//                and reduces the slab in that order (thread-block clusters combine the histograms of
//                2 or 4 CTAs over distributed shared memory when K is large against a slab).  The
//                automatic choice while a slab holds several rows per cluster.
//   sort route : global counting sort by cluster (histogram, exclusive scan, scatter of row numbers),
//                then one pass over X in that order.  K <= 8192: the sort works on per-slab
//                shared-memory histograms (no global atomics) and a segmented reduction follows in
//                which each warp sums a fixed-size run of the sorted order in registers and adds one
//                partial per cluster it touches.  Larger K (rows a multiple of 16 bytes): every
//                cluster is summed by one warp, which divides and writes the centroid itself; this
//                variant produces the means directly and needs no division pass.
//   smem route : every CTA keeps a private K x D table of partial sums in shared memory, streams a
//                slab of rows through it with shared-memory atomics and adds its table to the
//                global one at the end.  For K*D*4 bytes that fit in one SM's shared memory; slow
//                (shared-memory float atomics), on request only.
// All stream X exactly once with 16-byte (smem route: 4-byte) loads; HBM bandwidth is the bound.
#include <cooperative_groups.h>

#include "aug.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace cg = cooperative_groups;

namespace cake {
namespace {

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ cake_bf16 f32_to_bf16_rne(float f) {
    uint32_t u = __float_as_uint(f);
    if ((u & 0x7fffffffu) > 0x7f800000u) return static_cast<cake_bf16>((u >> 16) | 0x40u);
    u += 0x7fffu + ((u >> 16) & 1u);
    return static_cast<cake_bf16>(u >> 16);
}

// ======================================================================= smem route
// Table layout per cluster: the D/2 even columns first, then the D/2 odd ones, so that the 32 lanes
// of a warp (lane l holds columns 2l, 2l+1 of a 64-column group) hit 32 different banks.
constexpr int SMEM_THREADS = 512;
constexpr int SMEM_ROWS_PER_ITER = 8;  // rows in flight per warp

__global__ void __launch_bounds__(SMEM_THREADS)
update_smem_kernel(const cake_bf16* __restrict__ X, const int* __restrict__ idx, i64 N, int D, int K,
                   float* __restrict__ sums, int* __restrict__ counts, int* status) {
    extern __shared__ float tab[];                 // [K][D] permuted, then int cnt[K]
    int* cnt = reinterpret_cast<int*>(tab + static_cast<size_t>(K) * D);
    const int b = blockIdx.y;
    const int half = D >> 1;
    for (int e = threadIdx.x; e < K * D; e += blockDim.x) tab[e] = 0.f;
    for (int e = threadIdx.x; e < K; e += blockDim.x) cnt[e] = 0;
    __syncthreads();

    const uint32_t* Xw = reinterpret_cast<const uint32_t*>(X) + static_cast<size_t>(b) * N * half;
    const int* idx_b = idx + static_cast<size_t>(b) * N;
    const i64 per_cta = (N + gridDim.x - 1) / gridDim.x;
    const i64 r0 = per_cta * blockIdx.x;
    const i64 r1 = (r0 + per_cta < N) ? r0 + per_cta : N;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    bool bad = false;

    for (i64 base = r0 + static_cast<i64>(warp) * 32; base < r1; base += static_cast<i64>(nwarps) * 32) {
        const i64 mine = base + lane;
        int k_lane = -1;
        if (mine < r1) {
            k_lane = idx_b[mine];
            if (k_lane < 0 || k_lane >= K) { bad = true; k_lane = -1; }
            else atomicAdd(&cnt[k_lane], 1);
        }
        const int rows_here = (r1 - base < 32) ? static_cast<int>(r1 - base) : 32;
        for (int j0 = 0; j0 < rows_here; j0 += SMEM_ROWS_PER_ITER) {
            for (int c0 = 0; c0 < half; c0 += 32) {
                const int c = c0 + lane;
                uint32_t w[SMEM_ROWS_PER_ITER];
                int kk[SMEM_ROWS_PER_ITER];
#pragma unroll
                for (int u = 0; u < SMEM_ROWS_PER_ITER; ++u) {
                    kk[u] = __shfl_sync(0xffffffffu, k_lane, (j0 + u) & 31);
                    if (j0 + u >= rows_here) kk[u] = -1;
                    w[u] = 0;
                    if (kk[u] >= 0 && c < half) w[u] = __ldg(Xw + (base + j0 + u) * half + c);
                }
#pragma unroll
                for (int u = 0; u < SMEM_ROWS_PER_ITER; ++u) {
                    if (kk[u] >= 0 && c < half) {
                        float* row = tab + static_cast<size_t>(kk[u]) * D;
                        atomicAdd(row + c, bf16lo(w[u]));
                        atomicAdd(row + half + c, bf16hi(w[u]));
                    }
                }
            }
        }
    }
    if (bad) atomicCAS(status, CAKE_OK, CAKE_ERR_BAD_INDEX);
    __syncthreads();
    float* sums_b = sums + static_cast<size_t>(b) * K * D;
    for (int e = threadIdx.x; e < K * D; e += blockDim.x) {
        const float v = tab[e];
        if (v != 0.f) {
            const int k = e / D, pc = e - k * D;
            const int col = pc < half ? 2 * pc : 2 * (pc - half) + 1;
            atomicAdd(sums_b + static_cast<size_t>(k) * D + col, v);
        }
    }
    for (int e = threadIdx.x; e < K; e += blockDim.x)
        if (cnt[e]) atomicAdd(counts + static_cast<size_t>(b) * K + e, cnt[e]);
}

// ======================================================================= sort route
// Counting sort of the row numbers by cluster, then a segmented reduction over the sorted order.
//   sorted array : pairs[pos] = (row number, its cluster), pos in [0, n_valid)
// K <= BLK_MAX_K ("blocked"): per-slab shared-memory histograms, no global atomics, no zero-fill
// launches (hist_blocked zeroes `sums`, colscan writes `counts`).
// Larger K: global atomics (few rows per cluster, little contention); the histogram kernel zeroes `sums`.

// ---- large-K pieces
constexpr int HIST_THREADS = 512;

// counts[b][k] += 1 per row, and rank[b][i] = how many rows of the same cluster were counted before
// row i (-1 for an index outside [0, K)): the scatter then needs no second round of atomics.  Lanes of
// a warp that hit the same cluster take their ranks with a single atomic.
constexpr int HIST_PER_THREAD = 4;

__global__ void __launch_bounds__(HIST_THREADS)
hist_kernel(const int* __restrict__ idx, i64 N, int K, int* __restrict__ counts, int* __restrict__ rank,
            float4* __restrict__ sums4, i64 sums4_per_problem, int* status) {
    const int b = blockIdx.y;
    ptx::grid_dep_launch();    // the scan behind this kernel waits for its end by itself
    // this CTA's share of the fp32 sums starts at zero (the loads below are in flight meanwhile)
    {
        const i64 z0 = sums4_per_problem * blockIdx.x / gridDim.x, z1 = sums4_per_problem * (blockIdx.x + 1) / gridDim.x;
        float4* sb = sums4 + static_cast<size_t>(b) * sums4_per_problem;
        for (i64 e = z0 + threadIdx.x; e < z1; e += blockDim.x) sb[e] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    const int* idx_b = idx + static_cast<size_t>(b) * N;
    int* rank_b = rank + static_cast<size_t>(b) * N;
    int* counts_b = counts + static_cast<size_t>(b) * K;
    const int lane = threadIdx.x & 31;
    bool bad = false;
    const i64 span = static_cast<i64>(gridDim.x) * HIST_THREADS * HIST_PER_THREAD;
    const i64 n_round = (N + span - 1) / span * span;   // whole warps stay in the loop for the match
    for (i64 base = static_cast<i64>(blockIdx.x) * HIST_THREADS * HIST_PER_THREAD + threadIdx.x; base < n_round; base += span) {
        int k[HIST_PER_THREAD], r[HIST_PER_THREAD];
#pragma unroll
        for (int j = 0; j < HIST_PER_THREAD; ++j) {
            const i64 i = base + static_cast<i64>(j) * HIST_THREADS;
            k[j] = -1;
            if (i < N) {
                k[j] = idx_b[i];
                if (k[j] < 0 || k[j] >= K) { bad = true; k[j] = -1; }
            }
        }
#pragma unroll
        for (int j = 0; j < HIST_PER_THREAD; ++j) {
            const unsigned peers = __match_any_sync(0xffffffffu, k[j]);
            const int leader = __ffs(peers) - 1;
            r[j] = 0;
            if (k[j] >= 0 && lane == leader) r[j] = atomicAdd(counts_b + k[j], __popc(peers));
            r[j] = __shfl_sync(0xffffffffu, r[j], leader) + __popc(peers & ((1u << lane) - 1u));
        }
#pragma unroll
        for (int j = 0; j < HIST_PER_THREAD; ++j) {
            const i64 i = base + static_cast<i64>(j) * HIST_THREADS;
            if (i < N) rank_b[i] = k[j] >= 0 ? r[j] : -1;
        }
    }
    if (bad) atomicCAS(status, CAKE_OK, CAKE_ERR_BAD_INDEX);
}

// cursor[b][k] = sum_{j<k} counts[b][j]; nvalid[b] = total.  CTA (tile, problem) owns SCAN_TILE
// consecutive clusters; it first re-sums everything before its tile (coalesced, a few hundred KB at
// most), so the tiles need no communication and one launch does the whole scan.
constexpr int SCAN_TILE = 4096;
// A cluster with more rows than this is "heavy": the per-cluster mean kernel splits it over every warp
// whose window of the sorted order touches it (partials added into `sums`, the last one to arrive
// divides); lighter clusters are summed by the single warp in whose window they start.
constexpr int MEAN_HEAVY = 1024;

// heavy_sums (nullable): the scan also clears the sums row and the arrival counter of every heavy cluster.
__global__ void __launch_bounds__(1024)
scan_kernel(const int* __restrict__ counts, int K, int* __restrict__ cursor, int* __restrict__ nvalid,
            float* __restrict__ heavy_sums, int* __restrict__ heavy_done, int D) {
    __shared__ int warp_tot[32];
    __shared__ int pre_s;
    __shared__ int heavy_n;
    __shared__ int heavy_list[SCAN_TILE];
    ptx::grid_dep_wait();      // the histogram ahead of this kernel is complete
    ptx::grid_dep_launch();
    if (threadIdx.x == 0) heavy_n = 0;
    const int b = blockIdx.y, tile = blockIdx.x;
    const int* c = counts + static_cast<size_t>(b) * K;
    int* cur = cursor + static_cast<size_t>(b) * K;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // 1. everything before the tile
    int pre = 0;
    for (int i = threadIdx.x; i < tile * SCAN_TILE; i += 1024) pre += c[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) pre += __shfl_xor_sync(0xffffffffu, pre, o);
    if (lane == 0) warp_tot[warp] = pre;
    __syncthreads();
    if (threadIdx.x == 0) {
        int t = 0;
        for (int w = 0; w < 32; ++w) t += warp_tot[w];
        pre_s = t;
    }
    __syncthreads();
    pre = pre_s;
    __syncthreads();
    // 2. the tile: four consecutive clusters per thread
    const int k0 = tile * SCAN_TILE + threadIdx.x * 4;
    int v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = (k0 + j < K) ? c[k0 + j] : 0;
    const int local = v[0] + v[1] + v[2] + v[3];
    int incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int t = warp_tot[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int u = __shfl_up_sync(0xffffffffu, t, o);
            if (lane >= o) t += u;
        }
        warp_tot[lane] = t;  // inclusive over warps
    }
    __syncthreads();
    int run = pre + incl - local + (warp ? warp_tot[warp - 1] : 0);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        if (k0 + j < K) cur[k0 + j] = run;
        run += v[j];
    }
    if (tile == static_cast<int>(gridDim.x) - 1 && threadIdx.x == 0) nvalid[b] = pre + warp_tot[31];
    if (heavy_sums) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (v[j] > MEAN_HEAVY) heavy_list[atomicAdd(&heavy_n, 1)] = k0 + j;
        __syncthreads();
        const int nh = heavy_n;
        for (int h = 0; h < nh; ++h) {
            const size_t bk = static_cast<size_t>(b) * K + heavy_list[h];
            for (int d = threadIdx.x; d < D; d += 1024) heavy_sums[bk * D + d] = 0.f;
            if (threadIdx.x == 0) heavy_done[bk] = 0;
        }
    }
}

// row i goes to position offset[its cluster] + rank[i] of the sorted order
__global__ void __launch_bounds__(256)
scatter_kernel(const int* __restrict__ idx, const int* __restrict__ rank, i64 N, int K,
               const int* __restrict__ offset, int2* __restrict__ pairs) {
    const int b = blockIdx.y;
    ptx::grid_dep_wait();      // the scan (and with it the histogram) is complete
    ptx::grid_dep_launch();
    const int* idx_b = idx + static_cast<size_t>(b) * N;
    const int* rank_b = rank + static_cast<size_t>(b) * N;
    const int* off = offset + static_cast<size_t>(b) * K;
    int2* pairs_b = pairs + static_cast<size_t>(b) * N;
    const i64 span = static_cast<i64>(gridDim.x) * blockDim.x;
    for (i64 i = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; i < N; i += span) {
        const int r = rank_b[i];
        if (r < 0) continue;
        const int k = idx_b[i];
        pairs_b[__ldg(off + k) + r] = make_int2(static_cast<int>(i), k);
    }
}

// ---- blocked pieces (K <= BLK_MAX_K)
//   hist_blocked : CTA (slab, problem) histograms its slab of idx in shared memory and writes the
//                  K counters to part[problem][slab][*]; it also zeroes its share of `sums`.
//   colscan      : per cluster, exclusive prefix over the slabs (in place) and the total -> counts.
//   scatter_blocked : CTA (slab, problem) scans counts (redundantly per CTA) into cluster offsets,
//                  forms base[k] = offset[k] + part[slab][k] in shared memory and hands every row of
//                  its slab the next free position of its cluster.
constexpr int BLK_THREADS = 256;
constexpr int BLK_MAX_K = 8192;
constexpr int BLK_MAX_BLOCKS = 1024;
constexpr int BLK_MIN_SLAB = 8192;
constexpr int BLK_VEC = 4;            // idx values per load; slabs are multiples of it

__global__ void __launch_bounds__(BLK_THREADS)
hist_blocked_kernel(const int* __restrict__ idx, i64 N, int K, i64 slab, int* __restrict__ part,
                    float* __restrict__ sums, i64 sums_per_problem, int* status) {
    extern __shared__ int h[];
    const int b = blockIdx.y, blk = blockIdx.x, nblk = gridDim.x;
    for (int e = threadIdx.x; e < K; e += blockDim.x) h[e] = 0;
    __syncthreads();
    const int* idx_b = idx + static_cast<size_t>(b) * N;
    const i64 r0 = slab * blk, r1 = (r0 + slab < N) ? r0 + slab : N;
    bool bad = false;
    const bool vec_ok = (reinterpret_cast<uintptr_t>(idx_b + r0) & 15) == 0;
    i64 i = r0 + static_cast<i64>(threadIdx.x) * BLK_VEC;
    if (vec_ok) {
        for (; i + BLK_VEC <= r1; i += static_cast<i64>(blockDim.x) * BLK_VEC) {
            const int4 k4 = *reinterpret_cast<const int4*>(idx_b + i);
            const int ks[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (ks[u] < 0 || ks[u] >= K) bad = true;
                else atomicAdd(&h[ks[u]], 1);
            }
        }
    }
    // ragged tail (or everything, if the slab start is not 16-byte aligned)
    for (i64 j = vec_ok ? i : r0 + threadIdx.x; j < r1; j += vec_ok ? 1 : blockDim.x) {
        if (vec_ok && j >= i + BLK_VEC) break;
        const int k = idx_b[j];
        if (k < 0 || k >= K) bad = true;
        else atomicAdd(&h[k], 1);
    }
    if (bad) atomicCAS(status, CAKE_OK, CAKE_ERR_BAD_INDEX);
    // this CTA's share of the fp32 sums starts at zero
    const i64 z0 = sums_per_problem * blk / nblk, z1 = sums_per_problem * (blk + 1) / nblk;
    float* sums_b = sums + static_cast<size_t>(b) * sums_per_problem;
    for (i64 e = z0 + threadIdx.x; e < z1; e += blockDim.x) sums_b[e] = 0.f;
    __syncthreads();
    int* out = part + (static_cast<size_t>(b) * nblk + blk) * K;
    for (int e = threadIdx.x; e < K; e += blockDim.x) out[e] = h[e];
}

// CTA = 32 clusters (lanes) x 8 warps; warp w owns a contiguous range of slabs, walked 16 at a time.
__global__ void __launch_bounds__(256)
colscan_kernel(int* __restrict__ part, int nblk, int K, int* __restrict__ counts) {
    __shared__ int tot[8][32];
    const int b = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int k = blockIdx.x * 32 + lane;
    const int per = (nblk + 7) / 8;
    const int j0 = warp * per, j1 = (j0 + per < nblk) ? j0 + per : nblk;
    int* p = part + static_cast<size_t>(b) * nblk * K + k;
    // pass 1: this warp's total per cluster
    int sum = 0;
    for (int j = j0; j < j1; j += 16) {
        int v[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) v[u] = (k < K && j + u < j1) ? p[static_cast<size_t>(j + u) * K] : 0;
#pragma unroll
        for (int u = 0; u < 16; ++u) sum += v[u];
    }
    tot[warp][lane] = sum;
    __syncthreads();
    int run = 0, total = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
        if (w < warp) run += tot[w][lane];
        total += tot[w][lane];
    }
    // pass 2: exclusive prefix in place
    for (int j = j0; j < j1; j += 16) {
        int v[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) v[u] = (k < K && j + u < j1) ? p[static_cast<size_t>(j + u) * K] : 0;
#pragma unroll
        for (int u = 0; u < 16; ++u) {
            if (k < K && j + u < j1) p[static_cast<size_t>(j + u) * K] = run;
            run += v[u];
        }
    }
    if (warp == 0 && k < K) counts[static_cast<size_t>(b) * K + k] = total;
}

__global__ void __launch_bounds__(BLK_THREADS)
scatter_blocked_kernel(const int* __restrict__ idx, i64 N, int K, i64 slab, const int* __restrict__ part,
                       const int* __restrict__ counts, int* __restrict__ nvalid, int2* __restrict__ pairs) {
    extern __shared__ int base[];                 // [K]
    __shared__ int warp_tot[BLK_THREADS / 32];
    const int b = blockIdx.y, blk = blockIdx.x, nblk = gridDim.x;
    const int* c = counts + static_cast<size_t>(b) * K;
    const int* pre = part + (static_cast<size_t>(b) * nblk + blk) * K;
    // exclusive scan of counts: each thread owns `per` consecutive clusters
    const int per = (K + BLK_THREADS - 1) / BLK_THREADS;
    const int k0 = threadIdx.x * per, k1 = (k0 + per < K) ? k0 + per : K;
    int local = 0;
    for (int k = k0; k < k1; ++k) local += c[k];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    int before = 0, total = 0;
    for (int w = 0; w < BLK_THREADS / 32; ++w) {
        if (w < warp) before += warp_tot[w];
        total += warp_tot[w];
    }
    int run = before + incl - local;
    for (int k = k0; k < k1; ++k) {
        base[k] = run + pre[k];
        run += c[k];
    }
    if (blk == 0 && threadIdx.x == 0) nvalid[b] = total;
    __syncthreads();
    const int* idx_b = idx + static_cast<size_t>(b) * N;
    int2* pairs_b = pairs + static_cast<size_t>(b) * N;
    const i64 r0 = slab * blk, r1 = (r0 + slab < N) ? r0 + slab : N;
    const bool vec_ok = (reinterpret_cast<uintptr_t>(idx_b + r0) & 15) == 0;
    i64 i = r0 + static_cast<i64>(threadIdx.x) * BLK_VEC;
    if (vec_ok) {
        for (; i + BLK_VEC <= r1; i += static_cast<i64>(blockDim.x) * BLK_VEC) {
            const int4 k4 = *reinterpret_cast<const int4*>(idx_b + i);
            const int ks[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (ks[u] >= 0 && ks[u] < K)
                    pairs_b[atomicAdd(&base[ks[u]], 1)] = make_int2(static_cast<int>(i + u), ks[u]);
            }
        }
    }
    for (i64 j = vec_ok ? i : r0 + threadIdx.x; j < r1; j += vec_ok ? 1 : blockDim.x) {
        if (vec_ok && j >= i + BLK_VEC) break;
        const int k = idx_b[j];
        if (k >= 0 && k < K) pairs_b[atomicAdd(&base[k], 1)] = make_int2(static_cast<int>(j), k);
    }
}

// ---- segmented reduction over the sorted order.  Each warp owns SEG_ROWS consecutive sorted
// positions; it loads their row numbers and cluster ids once (two per lane) and hands them out by
// shuffles.  A row is read as 16-byte granules (8 bf16); LPR lanes share a row, 32/LPR rows are read
// per pass and several passes are in flight.  One vector atomic pair per granule per cluster touched.
constexpr int SEG_ROWS = 64;
constexpr int SEG_WARPS = 8;

template <int GPL>  // granules per lane (D <= 256*GPL)
__global__ void __launch_bounds__(SEG_WARPS * 32)
segreduce_kernel(const cake_bf16* __restrict__ X, const int2* __restrict__ pairs,
                 const int* __restrict__ nvalid, i64 N, int D, int K, int lpr, float* __restrict__ sums) {
    constexpr int SEG_UNROLL = GPL == 1 ? 8 : 4;   // passes in flight
    const int b = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const i64 w = static_cast<i64>(blockIdx.x) * SEG_WARPS + (threadIdx.x >> 5);
    const int n_valid = nvalid[b];
    const i64 p0 = w * SEG_ROWS;
    if (p0 >= n_valid) return;
    const int p1 = static_cast<int>((p0 + SEG_ROWS < n_valid) ? p0 + SEG_ROWS : n_valid);
    const int2* pairs_b = pairs + static_cast<size_t>(b) * N;
    const uint4* Xg = reinterpret_cast<const uint4*>(X) + static_cast<size_t>(b) * N * (D >> 3);
    float* sums_b = sums + static_cast<size_t>(b) * K * D;
    const int G = D >> 3;           // granules per row
    const int rpp = 32 / lpr;       // rows per pass
    const int sl = lane % lpr;      // granule slot inside the row
    const int rs = lane / lpr;      // row slot
    const bool in0 = p0 + lane < p1, in1 = p0 + 32 + lane < p1;
    const int2 pk0 = in0 ? __ldg(pairs_b + p0 + lane) : make_int2(0, -1);
    const int2 pk1 = in1 ? __ldg(pairs_b + p0 + 32 + lane) : make_int2(0, -1);
    const int pr0 = pk0.x, pr1 = pk1.x, ky0 = pk0.y, ky1 = pk1.y;

    int p = static_cast<int>(p0);
    while (p < p1) {
        // the run of equal keys that starts at p (the order is sorted, so it is contiguous)
        const int o0 = p - static_cast<int>(p0);
        const int k = o0 < 32 ? __shfl_sync(0xffffffffu, ky0, o0) : __shfl_sync(0xffffffffu, ky1, o0 - 32);
        const int e = p + __popc(__ballot_sync(0xffffffffu, ky0 == k)) + __popc(__ballot_sync(0xffffffffu, ky1 == k));
        float acc[GPL][8];
#pragma unroll
        for (int g = 0; g < GPL; ++g)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[g][j] = 0.f;
        for (int q = p; q < e; q += rpp * SEG_UNROLL) {
            uint4 v[SEG_UNROLL][GPL];
#pragma unroll
            for (int u = 0; u < SEG_UNROLL; ++u) {
                const int pos = q + u * rpp + rs;
                const bool on = pos < e;
                const int o = pos - static_cast<int>(p0);
                const int ra = __shfl_sync(0xffffffffu, pr0, o & 31);
                const int rb = __shfl_sync(0xffffffffu, pr1, o & 31);
                const int row = o < 32 ? ra : rb;
#pragma unroll
                for (int g = 0; g < GPL; ++g) {
                    const int gi = sl + g * lpr;
                    v[u][g] = make_uint4(0, 0, 0, 0);
                    if (on && gi < G) v[u][g] = __ldg(Xg + static_cast<size_t>(row) * G + gi);
                }
            }
#pragma unroll
            for (int u = 0; u < SEG_UNROLL; ++u)
#pragma unroll
                for (int g = 0; g < GPL; ++g) {
                    acc[g][0] += bf16lo(v[u][g].x); acc[g][1] += bf16hi(v[u][g].x);
                    acc[g][2] += bf16lo(v[u][g].y); acc[g][3] += bf16hi(v[u][g].y);
                    acc[g][4] += bf16lo(v[u][g].z); acc[g][5] += bf16hi(v[u][g].z);
                    acc[g][6] += bf16lo(v[u][g].w); acc[g][7] += bf16hi(v[u][g].w);
                }
        }
        // fold the row slots together, then one vector add per granule
#pragma unroll
        for (int g = 0; g < GPL; ++g)
#pragma unroll
            for (int j = 0; j < 8; ++j)
                for (int o = lpr; o < 32; o <<= 1) acc[g][j] += __shfl_xor_sync(0xffffffffu, acc[g][j], o);
        if (rs == 0) {
#pragma unroll
            for (int g = 0; g < GPL; ++g) {
                const int gi = sl + g * lpr;
                if (gi < G) {
                    float4* dst = reinterpret_cast<float4*>(sums_b + static_cast<size_t>(k) * D + gi * 8);
                    atomicAdd(dst, make_float4(acc[g][0], acc[g][1], acc[g][2], acc[g][3]));
                    atomicAdd(dst + 1, make_float4(acc[g][4], acc[g][5], acc[g][6], acc[g][7]));
                }
            }
        }
        p = e;
    }
}

// Scalar variant for D not a multiple of 8 (or very large D): one warp per run, lanes stride columns.
__global__ void __launch_bounds__(SEG_WARPS * 32)
segreduce_scalar_kernel(const cake_bf16* __restrict__ X, const int2* __restrict__ pairs,
                        const int* __restrict__ nvalid, i64 N, int D, int K, float* __restrict__ sums) {
    const int b = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const i64 w = static_cast<i64>(blockIdx.x) * SEG_WARPS + (threadIdx.x >> 5);
    const int n_valid = nvalid[b];
    const i64 p0 = w * SEG_ROWS;
    if (p0 >= n_valid) return;
    const int p1 = static_cast<int>((p0 + SEG_ROWS < n_valid) ? p0 + SEG_ROWS : n_valid);
    const int2* pairs_b = pairs + static_cast<size_t>(b) * N;
    const cake_bf16* Xb = X + static_cast<size_t>(b) * N * D;
    float* sums_b = sums + static_cast<size_t>(b) * K * D;
    int p = static_cast<int>(p0);
    while (p < p1) {
        const int k = pairs_b[p].y;
        int e = p + 1;
        while (e < p1 && pairs_b[e].y == k) ++e;
        for (int c = lane; c < D; c += 32) {
            float a = 0.f;
            for (int q = p; q < e; ++q)
                a += __uint_as_float(static_cast<uint32_t>(Xb[static_cast<size_t>(pairs_b[q].x) * D + c]) << 16);
            atomicAdd(sums_b + static_cast<size_t>(k) * D + c, a);
        }
        p = e;
    }
}

// ---- per-cluster means straight from the sorted order (K > 8192, D % 8 == 0): no partial sums in
// memory, no separate division pass.  The sorted positions are cut into windows of SEG_ROWS, one per
// warp (equal work whatever the cluster sizes).  A cluster belongs to the warp in whose window it
// starts: that warp follows it to its end (counts[k] rows, past the window if need be), sums it in
// registers, divides and writes the centroid.  Only a heavy cluster (more than MEAN_HEAVY rows) is
// shared: every warp adds the part inside its own window to `sums` (cleared by the scan) and counts its
// rows into `done`; the warp that completes the count divides.  Clusters without rows are dealt out
// evenly over all warps by cluster number and keep their previous centroid.
//
// The rows a warp has to read form one stream of sorted positions, cut into passes (one warp-wide
// load of 32/LPR rows) that never cross a run of equal clusters.  They are fetched with 16-byte
// asynchronous copies into a ring of the warp's own in shared memory (every lane later reads back the
// bytes it copied itself, so the copy groups of the thread are all the synchronisation there is; a
// lane without a row gets zeros): the loads run MEAN_AHEAD-1 batches ahead of the additions whatever
// the cluster boundaries, which keeps enough bytes in flight for random 2D-byte rows to arrive at the
// full HBM rate with few registers.  Few warps per CTA: streams differ in length, and a CTA holds its
// slots until its longest one ends.
constexpr int MEAN_WARPS = 2;
constexpr int MEAN_AHEAD = 3;          // batches in the ring (two in flight while one is added)
constexpr int MEAN_BATCH_GRANULES = 4; // 16-byte granules per lane and batch
// per warp: the ring (MEAN_AHEAD batches) and 128 row numbers
constexpr int MEAN_WARP_UINT4 = MEAN_AHEAD * MEAN_BATCH_GRANULES * 32 + 32;

// 16 bytes global -> shared, or 16 zero bytes when src_bytes == 0
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// two floats rounded to nearest-even bf16: lo in the low half, hi in the high half
__device__ __forceinline__ uint32_t bf16x2_rn(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
// two fp32 sums per instruction: acc.{lo,hi} += {bf16 in the low half, bf16 in the high half} of w
__device__ __forceinline__ void add_bf16x2(unsigned long long& acc, uint32_t w) {
    unsigned long long p;
    asm("mov.b64 %0, {%1, %2};" : "=l"(p) : "r"(w << 16), "r"(w & 0xFFFF0000u));
    asm("add.rn.f32x2 %0, %0, %1;" : "+l"(acc) : "l"(p));
}

template <int GPL, int LPR>   // granules per lane and row, lanes per row: D <= 8 * GPL * LPR
__global__ void __launch_bounds__(MEAN_WARPS * 32)
segmean_kernel(const cake_bf16* __restrict__ X, const int2* __restrict__ pairs, const int* __restrict__ nvalid,
               const int* __restrict__ counts, i64 N, int D, int K, const cake_bf16* __restrict__ C_prev,
               float* __restrict__ out_C, cake_bf16* __restrict__ out_C_bf16, float* sums, int* done) {
    constexpr int RPP = 32 / LPR;                  // rows per pass
    constexpr int U = MEAN_BATCH_GRANULES / GPL;   // passes per batch
    constexpr int R = U * MEAN_AHEAD;              // passes in the ring
    static_assert(U * RPP <= 32, "a batch must fit two blocks of the row table");
    extern __shared__ uint4 mean_ring[];           // [warp]{[R][GPL][32] ring, 128 row numbers}
    ptx::grid_dep_wait();      // the scatter (and with it scan and histogram) is complete
    const int b = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const i64 w = static_cast<i64>(blockIdx.x) * MEAN_WARPS + warp;
    const i64 n_warps = static_cast<i64>(gridDim.x) * MEAN_WARPS;
    const int G = D >> 3;           // granules per row
    const int sl = lane % LPR;      // granule slot inside the row
    const int rs = lane / LPR;      // row slot
    const int* counts_b = counts + static_cast<size_t>(b) * K;
    const size_t row0 = static_cast<size_t>(b) * K;     // first centroid row of this problem
    float4* out4 = reinterpret_cast<float4*>(out_C);
    uint4* outb = reinterpret_cast<uint4*>(out_C_bf16);
    bool gran_on[GPL];
#pragma unroll
    for (int g = 0; g < GPL; ++g) gran_on[g] = sl + g * LPR < G;

    // lanes (rs == 0) hold eight consecutive columns of granule sl + g*LPR: the centroid row k
    auto write_row = [&](int k, const float (&val)[GPL][8]) {
        if (rs != 0) return;
#pragma unroll
        for (int g = 0; g < GPL; ++g) {
            if (!gran_on[g]) continue;
            const size_t e = (row0 + k) * G + sl + g * LPR;
            out4[2 * e] = make_float4(val[g][0], val[g][1], val[g][2], val[g][3]);
            out4[2 * e + 1] = make_float4(val[g][4], val[g][5], val[g][6], val[g][7]);
            if (outb)
                outb[e] = make_uint4(bf16x2_rn(val[g][0], val[g][1]), bf16x2_rn(val[g][2], val[g][3]),
                                     bf16x2_rn(val[g][4], val[g][5]), bf16x2_rn(val[g][6], val[g][7]));
        }
    };

    // 1. clusters without rows: the previous centroid (or zero)
    for (i64 k = w; k < K; k += n_warps) {
        if (__ldg(counts_b + k) != 0) continue;
        float val[GPL][8];
#pragma unroll
        for (int g = 0; g < GPL; ++g) {
            uint4 pv = make_uint4(0, 0, 0, 0);
            if (C_prev && rs == 0 && gran_on[g])
                pv = __ldg(reinterpret_cast<const uint4*>(C_prev) + (row0 + k) * G + sl + g * LPR);
            val[g][0] = bf16lo(pv.x); val[g][1] = bf16hi(pv.x); val[g][2] = bf16lo(pv.y); val[g][3] = bf16hi(pv.y);
            val[g][4] = bf16lo(pv.z); val[g][5] = bf16hi(pv.z); val[g][6] = bf16lo(pv.w); val[g][7] = bf16hi(pv.w);
        }
        write_row(static_cast<int>(k), val);
    }

    // 2. this warp's window of the sorted order
    const int n_valid = nvalid[b];
    const i64 p0 = w * SEG_ROWS;
    if (p0 >= n_valid) return;
    const int nwin = static_cast<int>((p0 + SEG_ROWS < n_valid) ? SEG_ROWS : n_valid - p0);
    const int2* pairs_b = pairs + static_cast<size_t>(b) * N;
    const uint4* Xg = reinterpret_cast<const uint4*>(X) + static_cast<size_t>(b) * N * G;
    const bool in0 = lane < nwin, in1 = 32 + lane < nwin;
    const int2 pk0 = in0 ? __ldg(pairs_b + p0 + lane) : make_int2(0, -1);
    const int2 pk1 = in1 ? __ldg(pairs_b + p0 + 32 + lane) : make_int2(0, -1);
    const int k_before = p0 > 0 ? __ldg(&pairs_b[p0 - 1].y) : -1;   // cluster of the position ahead of the window
    const int ky0 = pk0.y, ky1 = pk1.y;
    const int cn0 = in0 ? __ldg(counts_b + ky0) : 0, cn1 = in1 ? __ldg(counts_b + ky1) : 0;
    auto key_at = [&](int o) { const int a = __shfl_sync(0xffffffffu, ky0, o & 31), c = __shfl_sync(0xffffffffu, ky1, o & 31); return o < 32 ? a : c; };
    auto cnt_at = [&](int o) { const int a = __shfl_sync(0xffffffffu, cn0, o & 31), c = __shfl_sync(0xffffffffu, cn1, o & 31); return o < 32 ? a : c; };

    // last[o]: position o closes a run of equal clusters inside the window (invalid positions carry -1)
    uint64_t last;
    {
        int nx0 = __shfl_down_sync(0xffffffffu, ky0, 1);
        const int first1 = __shfl_sync(0xffffffffu, ky1, 0);
        if (lane == 31) nx0 = first1;
        int nx1 = __shfl_down_sync(0xffffffffu, ky1, 1);
        if (lane == 31) nx1 = -2;
        const uint32_t l0 = __ballot_sync(0xffffffffu, in0 && nx0 != ky0), l1 = __ballot_sync(0xffffffffu, in1 && nx1 != ky1);
        last = (static_cast<uint64_t>(l1) << 32) | l0;
    }
    // the stream: everything in the window but a leading piece of a light cluster that started earlier,
    // plus what the last cluster (if light and started here) has beyond the window
    const int k_first = key_at(0), n_first = cnt_at(0);
    int ps = 0;
    if (k_first == k_before && n_first <= MEAN_HEAVY) ps = __ffsll(static_cast<long long>(last));   // end of the first run
    if (ps >= nwin) return;
    const int k_last = key_at(nwin - 1), n_last = cnt_at(nwin - 1);
    int ext = 0;
    {
        const uint64_t inner = last & ~(1ull << (nwin - 1));
        const int so = inner ? 64 - __clzll(static_cast<long long>(inner)) : 0;   // where the last run starts
        if (n_last <= MEAN_HEAVY && n_last > nwin - so) {
            ext = n_last - (nwin - so);      // then nwin == SEG_ROWS: the order goes on past the window
            last &= ~(1ull << (nwin - 1));
        }
    }
    const int S = nwin - ps + ext;                  // stream length
    // end (exclusive, as a stream index) of the run that holds stream index i
    auto run_end = [&](int i) {
        const int o = ps + i;
        if (o < SEG_ROWS) {
            const uint64_t m = last >> o;
            if (m) return i + __ffsll(static_cast<long long>(m));
        }
        return S;
    };

    // per warp: the ring, then a table of 128 row numbers indexed by position modulo 128 (the window's 64
    // first; blocks of 32 past the window replace entries the issuing side has long passed)
    uint4* ring = mean_ring + static_cast<size_t>(warp) * MEAN_WARP_UINT4;
    int* tab = reinterpret_cast<int*>(ring + R * GPL * 32);
    const uint32_t ring_a = static_cast<uint32_t>(__cvta_generic_to_shared(ring)) + lane * 16;
    tab[lane] = pk0.x;
    tab[32 + lane] = pk1.x;
    int ext_loaded = 0;    // blocks of 32 positions past the window already in the table
    int ext_next = -1;     // this lane's row number of the block after those (fetched one block early)
    if (ext > 0) ext_next = lane < ext ? __ldg(&pairs_b[p0 + SEG_ROWS + lane].x) : 0;
    __syncwarp();

    const char* Xlane[GPL];     // this lane's granules of row 0
#pragma unroll
    for (int g = 0; g < GPL; ++g) Xlane[g] = reinterpret_cast<const char*>(Xg + (gran_on[g] ? sl + g * LPR : 0));
    const uint32_t row_bytes = static_cast<uint32_t>(D) * 2u;

    int iq = 0, ie = run_end(0);          // issuing side: next position, end of its run
    uint32_t wr = ring_a;                 // where the next pass lands
    auto issue_batch = [&]() {
        // make sure the table covers the batch
        while (ps + iq + U * RPP > SEG_ROWS + 32 * ext_loaded && 32 * ext_loaded < ext) {
            tab[((2 + ext_loaded) & 3) * 32 + lane] = ext_next;
            ++ext_loaded;
            const int e = 32 * ext_loaded + lane;
            ext_next = e < ext ? __ldg(&pairs_b[p0 + SEG_ROWS + e].x) : 0;
            __syncwarp();
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            // a lane without a row (past the run, past the stream, past the row's granules) gets zeros
            const int pos = iq + rs;
            const bool on = pos < ie;
            const uint32_t row = static_cast<uint32_t>(tab[(ps + pos) & 127]);
            const uint64_t off = static_cast<uint64_t>(row) * row_bytes;
#pragma unroll
            for (int g = 0; g < GPL; ++g)
                cp_async16(wr + (u * GPL + g) * 512, Xlane[g] + off, on && gran_on[g] ? 16u : 0u);
            iq += RPP;
            if (iq >= ie) { iq = ie; ie = run_end(iq); }
        }
        wr += U * GPL * 512;
        if (wr == ring_a + R * GPL * 512) wr = ring_a;
    };

#pragma unroll
    for (int bt = 0; bt < MEAN_AHEAD - 1; ++bt) {
        issue_batch();
        cp_async_commit();
    }

    unsigned long long acc[GPL][4];   // four pairs of fp32 sums per granule
#pragma unroll
    for (int g = 0; g < GPL; ++g)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[g][j] = 0ull;

    // the run that ends at stream index i_close is complete (`piece` of its rows were read here): divide
    // and write, or (heavy) add the partial and count it
    auto flush = [&](int i_close, int piece) {
        const int o = ps + i_close;
        int k = key_at(o < nwin ? o : 0), n = cnt_at(o < nwin ? o : 0);
        if (o >= nwin) { k = k_last; n = n_last; }
        float val[GPL][8];
#pragma unroll
        for (int g = 0; g < GPL; ++g)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                asm("mov.b64 {%0, %1}, %2;" : "=f"(val[g][2 * j]), "=f"(val[g][2 * j + 1]) : "l"(acc[g][j]));
                acc[g][j] = 0ull;
            }
#pragma unroll
        for (int g = 0; g < GPL; ++g)
#pragma unroll
            for (int j = 0; j < 8; ++j)
#pragma unroll
                for (int x = LPR; x < 32; x <<= 1) val[g][j] += __shfl_xor_sync(0xffffffffu, val[g][j], x);
        const float fn = static_cast<float>(n);
        if (n <= MEAN_HEAVY) {
            const float inv = 1.0f / fn;     // one division per cluster; the products are within 1 ulp of sum / n
#pragma unroll
            for (int g = 0; g < GPL; ++g)
#pragma unroll
                for (int j = 0; j < 8; ++j) val[g][j] *= inv;
            write_row(k, val);
        } else {
            float* srow = sums + (row0 + k) * static_cast<size_t>(D);
            if (rs == 0) {
#pragma unroll
                for (int g = 0; g < GPL; ++g) {
                    if (!gran_on[g]) continue;
                    float4* dst = reinterpret_cast<float4*>(srow + (sl + g * LPR) * 8);
                    atomicAdd(dst, make_float4(val[g][0], val[g][1], val[g][2], val[g][3]));
                    atomicAdd(dst + 1, make_float4(val[g][4], val[g][5], val[g][6], val[g][7]));
                }
            }
            __threadfence();
            __syncwarp();
            int arrived = 0;
            if (lane == 0) arrived = atomicAdd(done + row0 + k, piece) + piece;
            arrived = __shfl_sync(0xffffffffu, arrived, 0);
            if (arrived == n) {   // every part is in: divide
                __threadfence();
#pragma unroll
                for (int g = 0; g < GPL; ++g) {
                    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), c = a;
                    if (rs == 0 && gran_on[g]) {
                        a = __ldcg(reinterpret_cast<const float4*>(srow + (sl + g * LPR) * 8));
                        c = __ldcg(reinterpret_cast<const float4*>(srow + (sl + g * LPR) * 8) + 1);
                    }
                    val[g][0] = a.x / fn; val[g][1] = a.y / fn; val[g][2] = a.z / fn; val[g][3] = a.w / fn;
                    val[g][4] = c.x / fn; val[g][5] = c.y / fn; val[g][6] = c.z / fn; val[g][7] = c.w / fn;
                }
                write_row(k, val);
            }
        }
    };

    int cq = 0, ce = run_end(0), run_start = 0;   // adding side: next position, end and start of its run
    const uint4* rd = ring + lane;
    int left = 0;                                 // passes of the current batch not yet added
    while (cq < S) {
        if (left == 0) {
            // keep the ring full, then wait for the next batch (all but the newest MEAN_AHEAD-1 groups)
            issue_batch();
            cp_async_commit();
            cp_async_wait<MEAN_AHEAD - 1>();
            left = U;
            if (rd == ring + lane + R * GPL * 32) rd = ring + lane;
        }
        // passes until the run or the batch ends
        int np = (ce - cq + RPP - 1) / RPP;
        if (np > left) np = left;
        left -= np;
        cq += np * RPP;
        for (; np > 0; --np) {
#pragma unroll
            for (int g = 0; g < GPL; ++g) {
                const uint4 v = rd[g * 32];
                add_bf16x2(acc[g][0], v.x); add_bf16x2(acc[g][1], v.y);
                add_bf16x2(acc[g][2], v.z); add_bf16x2(acc[g][3], v.w);
            }
            rd += GPL * 32;
        }
        if (cq >= ce) {
            flush(ce - 1, ce - run_start);
            cq = ce;
            run_start = ce;
            ce = run_end(cq);
        }
    }
    cp_async_wait<0>();
}

// ======================================================================= slab route
// One kernel sorts and reduces.  A CTA owns a slab of S consecutive rows: it keeps their cluster ids
// in registers, ranks every row inside its cluster with one shared-memory atomic, scans the
// histogram and writes the slab's rows in cluster order into shared memory; then lane groups walk
// that order, gather the rows and flush one vector atomic per run of equal clusters.  A run is S/K rows long, so when K
// is large against S, F CTAs form a thread-block cluster: their histograms are combined through
// distributed shared memory into one order over the F*S rows of the cluster, every CTA takes an
// equal contiguous share of it, and runs are F times longer (F times fewer atomics).
constexpr int SLAB_THREADS = 1024;
constexpr int SLAB_VPT = 16;                               // cluster ids per thread (registers)
constexpr int SLAB_MAX_ROWS = SLAB_THREADS * SLAB_VPT;     // rows per CTA
constexpr int SLAB_MAX_K = 8192;
constexpr int SLAB_AHEAD = 4;                              // rows in flight per lane group
constexpr int SLAB_MAX_F = 4;
constexpr int SLAB_GROW_RUN = 8;                           // clusters grow until a run has this many rows
constexpr int SLAB_MIN_RUN = 4;                            // rows per run below which the sort route is faster (K > 4096)

// sums and counts start at zero; the kernel behind it may begin at once (it waits before its first add)
__global__ void __launch_bounds__(256)
zero_sums_counts_kernel(float4* __restrict__ sums4, i64 n4, int* __restrict__ counts, i64 nc) {
    // the kernel ahead (assign) may still read or write what this one clears, and the kernel behind (the
    // slab sort) reads what the one ahead wrote: it may start only once this wait has returned
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    const i64 stride = static_cast<i64>(gridDim.x) * blockDim.x;
    const i64 t = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x;
    for (i64 e = t; e < n4; e += stride) sums4[e] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (i64 e = t; e < nc; e += stride) counts[e] = 0;
}

// WIDE: rows of more than 32 granules (D > 256), reduced in several column passes
template <int LPR, bool CLUSTER, bool WIDE = false>
__global__ void __launch_bounds__(SLAB_THREADS, 1)
slab_update_kernel(const cake_bf16* __restrict__ X, const int* __restrict__ idx, i64 N, int D, int K, int S,
                   int rowbits, float* __restrict__ sums, int* __restrict__ counts, int* status, i64 Nprob,
                   int Kidx) {
    extern __shared__ int sm[];
    int* h = sm;                                                   // [K] this CTA's rows per cluster
    int* off = sm + K;                                             // [K] first position of this CTA's rows of a cluster
    uint32_t* sorted = reinterpret_cast<uint32_t*>(sm + 2 * K);    // [S] this CTA's share of the order
    __shared__ int warp_tot[SLAB_THREADS / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // Nprob > 0 (never with thread-block clusters): the problems of a batch as one run of N = B * Nprob rows,
    // dealt to the CTAs without regard to where a problem ends (B problems seldom divide the SMs evenly).  A
    // slab is at most one problem long, so it holds rows of problem b and, from row `split` on, of problem
    // b + 1: those count as clusters Kidx .. 2 Kidx - 1 (K = 2 Kidx), which is where they lie in sums and
    // counts seen from problem b.  Otherwise Kidx = K, blockIdx.y is the problem and split is never reached.
    const bool flat = !CLUSTER && Nprob > 0;
    int b = blockIdx.y;
    unsigned F = 1, c = 0;
    if constexpr (CLUSTER) {
        F = cg::this_cluster().num_blocks();
        c = cg::this_cluster().block_rank();
    }
    const i64 super_row0 = static_cast<i64>(blockIdx.x / F) * F * S;   // first row of the cluster's rows
    const i64 r0 = super_row0 + static_cast<i64>(c) * S;
    const int rows = r0 >= N ? 0 : static_cast<int>(r0 + S <= N ? S : N - r0);
    int split = S;
    if (flat) {
        b = static_cast<int>(r0 / Nprob);
        const i64 left = static_cast<i64>(b + 1) * Nprob - r0;      // rows up to the end of problem b
        split = left < S ? static_cast<int>(left) : S;
    }
    const int* idx_b = idx + (flat ? 0 : static_cast<size_t>(b) * N) + (rows ? r0 : 0);
    int* counts_b = counts + static_cast<size_t>(b) * Kidx;

    for (int e = tid; e < K; e += SLAB_THREADS) h[e] = 0;
    __syncthreads();
    // ---- cluster ids into registers, rank inside (CTA, cluster) from the histogram atomic
    int kv[SLAB_VPT], rk[SLAB_VPT];
    const bool vec_ok = (reinterpret_cast<uintptr_t>(idx_b) & 15) == 0;
#pragma unroll
    for (int u = 0; u < SLAB_VPT / 4; ++u) {
        const int i = (u * SLAB_THREADS + tid) * 4;
        int4 k4 = make_int4(-1, -1, -1, -1);
        if (vec_ok && i + 4 <= rows) {
            k4 = *reinterpret_cast<const int4*>(idx_b + i);
        } else {
            if (i < rows) k4.x = idx_b[i];
            if (i + 1 < rows) k4.y = idx_b[i + 1];
            if (i + 2 < rows) k4.z = idx_b[i + 2];
            if (i + 3 < rows) k4.w = idx_b[i + 3];
        }
        kv[u * 4] = k4.x; kv[u * 4 + 1] = k4.y; kv[u * 4 + 2] = k4.z; kv[u * 4 + 3] = k4.w;
    }
    bool bad = false;
#pragma unroll
    for (int u = 0; u < SLAB_VPT; ++u) {
        const int i = ((u >> 2) * SLAB_THREADS + tid) * 4 + (u & 3);
        const bool ok = static_cast<unsigned>(kv[u]) < static_cast<unsigned>(Kidx);
        if (!ok && i < rows) bad = true;
        if (!ok || i >= rows) kv[u] = -1;
        else if (i >= split) kv[u] += Kidx;
        rk[u] = kv[u] >= 0 ? atomicAdd(&h[kv[u]], 1) : 0;
    }
    if (bad) atomicCAS(status, CAKE_OK, CAKE_ERR_BAD_INDEX);
    // nothing above touched what the zero-fill ahead of this kernel writes; from here on it must be done
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    if constexpr (CLUSTER) cg::this_cluster().sync();
    else __syncthreads();
    // ---- offsets: exclusive scan over clusters of the cluster-wide totals, plus the rows that CTAs of
    // lower rank hold of the same cluster
    int total;
    {
        const int per = (K + SLAB_THREADS - 1) / SLAB_THREADS;
        const int k0 = min(tid * per, K), k1 = min(k0 + per, K);
        int local = 0;
        for (int k = k0; k < k1; ++k) {
            if constexpr (CLUSTER) {
                for (unsigned j = 0; j < F; ++j) local += cg::this_cluster().map_shared_rank(h, j)[k];
            } else {
                local += h[k];
            }
        }
        int incl = local;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        int before = 0;
        total = 0;
        for (int w = 0; w < SLAB_THREADS / 32; ++w) {
            if (w < warp) before += warp_tot[w];
            total += warp_tot[w];
        }
        int run = before + incl - local;
        for (int k = k0; k < k1; ++k) {
            int tot = 0, lower = 0;
            if constexpr (CLUSTER) {
                for (unsigned j = 0; j < F; ++j) {
                    const int v = cg::this_cluster().map_shared_rank(h, j)[k];
                    tot += v;
                    if (j < c) lower += v;
                }
            } else {
                tot = h[k];
            }
            if (c == 0 && tot) atomicAdd(&counts_b[k], tot);
            off[k] = run + lower;
            run += tot;
        }
    }
    __syncthreads();
    // every CTA of the cluster takes `share` consecutive positions of the order
    const int share = CLUSTER ? ((total + static_cast<int>(F) - 1) / static_cast<int>(F) + 3) / 4 * 4 : total;
    const int mine = CLUSTER ? max(0, min(share, total - static_cast<int>(c) * share)) : total;
#pragma unroll
    for (int u = 0; u < SLAB_VPT; ++u) {
        if (kv[u] >= 0) {
            const int i = ((u >> 2) * SLAB_THREADS + tid) * 4 + (u & 3);
            const uint32_t rec = (static_cast<uint32_t>(kv[u]) << rowbits) | (c * static_cast<uint32_t>(S) + static_cast<uint32_t>(i));
            const int pos = off[kv[u]] + rk[u];
            if constexpr (CLUSTER) {
                const int j = pos / share;
                cg::this_cluster().map_shared_rank(sorted, j)[pos - j * share] = rec;
            } else {
                sorted[pos] = rec;
            }
        }
    }
    if constexpr (CLUSTER) cg::this_cluster().sync();
    else __syncthreads();

    // ---- segmented reduction: every lane group (LPR lanes, one 16-byte granule each) walks one
    // contiguous piece of this CTA's positions and flushes when the cluster changes
    constexpr int GROUPS = 32 / LPR;
    constexpr int NGROUPS = (SLAB_THREADS / 32) * GROUPS;
    const int G = D >> 3;
    const int sl = lane % LPR;
    const int gid = warp * GROUPS + lane / LPR;
    const uint4* Xg = reinterpret_cast<const uint4*>(X) + ((flat ? 0 : static_cast<size_t>(b) * N) + super_row0) * G;
    float* sums_b = sums + static_cast<size_t>(b) * Kidx * D;
    const uint32_t rowmask = (1u << rowbits) - 1u;
    const int seglen = max(SLAB_AHEAD, (mine + NGROUPS - 1) / NGROUPS);
    const int base = gid * seglen, end = min(base + seglen, mine);
    // rows wider than 32 granules (D > 256) are reduced in equal column blocks of at most 32 granules, one
    // pass over the records each
    const int n_pass = WIDE ? (G + LPR - 1) / LPR : 1, pass_w = WIDE ? (G + n_pass - 1) / n_pass : LPR;
    for (int pass = 0; pass < n_pass; ++pass) {
        const int sg = WIDE ? (sl < pass_w ? pass * pass_w + sl : G) : sl;   // this lane's granule (>= G: none)
        int cur = -1;
        float acc[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = 0.f;
        auto flush = [&]() {
            if (cur >= 0 && sg < G) {
                float4* dst = reinterpret_cast<float4*>(sums_b + static_cast<size_t>(cur) * D + sg * 8);
                atomicAdd(dst, make_float4(acc[0], acc[1], acc[2], acc[3]));
                atomicAdd(dst + 1, make_float4(acc[4], acc[5], acc[6], acc[7]));
            }
        };
        for (int q = base; q < end; q += SLAB_AHEAD) {
            uint4 v[SLAB_AHEAD];
            int kk[SLAB_AHEAD];
#pragma unroll
            for (int u = 0; u < SLAB_AHEAD; ++u) {
                kk[u] = -1;
                v[u] = make_uint4(0, 0, 0, 0);
                if (q + u < end) {
                    const uint32_t rec = sorted[q + u];
                    kk[u] = static_cast<int>(rec >> rowbits);
                    if (sg < G) v[u] = __ldg(Xg + static_cast<size_t>(rec & rowmask) * G + sg);
                }
            }
#pragma unroll
            for (int u = 0; u < SLAB_AHEAD; ++u) {
                if (kk[u] >= 0) {
                    if (kk[u] != cur) {
                        flush();
                        cur = kk[u];
#pragma unroll
                        for (int j = 0; j < 8; ++j) acc[j] = 0.f;
                    }
                    acc[0] += bf16lo(v[u].x); acc[1] += bf16hi(v[u].x);
                    acc[2] += bf16lo(v[u].y); acc[3] += bf16hi(v[u].y);
                    acc[4] += bf16lo(v[u].z); acc[5] += bf16hi(v[u].z);
                    acc[6] += bf16lo(v[u].w); acc[7] += bf16hi(v[u].w);
                }
            }
        }
        flush();
    }
}

// ======================================================================= division

__global__ void __launch_bounds__(256)
finalize_kernel(const float* __restrict__ sums, const int* __restrict__ counts,
                const cake_bf16* __restrict__ C_prev, i64 total, int D, int Ds, float* __restrict__ out_C,
                cake_bf16* __restrict__ out_C_bf16) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    for (i64 e = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; e < total;
         e += static_cast<i64>(gridDim.x) * blockDim.x) {
        const i64 row = e / D;  // b*K + k
        const int n = counts[row];
        float v;
        if (n > 0) v = sums[row * Ds + (e - row * D)] / static_cast<float>(n);
        else v = C_prev ? __uint_as_float(static_cast<uint32_t>(C_prev[e]) << 16) : 0.f;
        out_C[e] = v;
        if (out_C_bf16) out_C_bf16[e] = f32_to_bf16_rne(v);
    }
}

// D % 4 == 0: four columns per thread, 16-byte loads and stores
__global__ void __launch_bounds__(256)
finalize4_kernel(const float4* __restrict__ sums, const int* __restrict__ counts,
                 const uint2* __restrict__ C_prev, i64 total4, int D4, int Ds4, float4* __restrict__ out_C,
                 uint2* __restrict__ out_C_bf16) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    for (i64 e = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; e < total4;
         e += static_cast<i64>(gridDim.x) * blockDim.x) {
        const i64 row = e / D4;
        const int n = counts[row];
        float4 v;
        if (n > 0) {
            const float4 sv = sums[row * Ds4 + (e - row * D4)];
            const float fn = static_cast<float>(n);
            v = make_float4(sv.x / fn, sv.y / fn, sv.z / fn, sv.w / fn);
        } else if (C_prev) {
            const uint2 pv = C_prev[e];
            v = make_float4(bf16lo(pv.x), bf16hi(pv.x), bf16lo(pv.y), bf16hi(pv.y));
        } else {
            v = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        out_C[e] = v;
        if (out_C_bf16) {
            uint2 o;
            o.x = static_cast<uint32_t>(f32_to_bf16_rne(v.x)) | (static_cast<uint32_t>(f32_to_bf16_rne(v.y)) << 16);
            o.y = static_cast<uint32_t>(f32_to_bf16_rne(v.z)) | (static_cast<uint32_t>(f32_to_bf16_rne(v.w)) << 16);
            out_C_bf16[e] = o;
        }
    }
}

// D % 4 == 0, one warp per centroid row (lanes stride the row in quads of columns): the division as in
// finalize4_kernel and, on the way, what the tensor-core assign of these centroids needs as its
// prologue: ||c||^2 of the bf16-rounded row (summed as the assign prologue sums it), split into the
// k-step operand row, and cleared inertia entries.
__global__ void __launch_bounds__(256)
finalize_rows_kernel(const float4* __restrict__ sums, const int* __restrict__ counts,
                     const uint2* __restrict__ C_prev, i64 rows, int K, int D4, float4* __restrict__ out_C,
                     uint2* __restrict__ out_C_bf16, uint8_t* __restrict__ caug, int Kpad,
                     double* __restrict__ inertia, int inertia_stride, int B, uint2* __restrict__ cpad, int Dc4,
                     int Ds4) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    if (inertia && blockIdx.x == 0 && static_cast<int>(threadIdx.x) < B)
        inertia[static_cast<size_t>(threadIdx.x) * inertia_stride] = 0.0;
    const int lane = threadIdx.x & 31;
    const i64 n_warps = static_cast<i64>(gridDim.x) * (blockDim.x >> 5);
    for (i64 row = static_cast<i64>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); row < rows; row += n_warps) {
        if (cpad)   // the zero padding of the row's copy for the assign kernel
            for (int j = D4 + lane; j < Dc4; j += 32) cpad[row * Dc4 + j] = make_uint2(0u, 0u);
        const int n = counts[row];
        const float fn = static_cast<float>(n);
        float acc = 0.f;
        for (int j = lane; j < D4; j += 32) {
            const i64 e = row * D4 + j;
            float4 v;
            if (n > 0) {
                const float4 sv = sums[row * Ds4 + j];
                v = make_float4(sv.x / fn, sv.y / fn, sv.z / fn, sv.w / fn);
            } else if (C_prev) {
                const uint2 pv = C_prev[e];
                v = make_float4(bf16lo(pv.x), bf16hi(pv.x), bf16lo(pv.y), bf16hi(pv.y));
            } else {
                v = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            out_C[e] = v;
            uint2 o;
            o.x = static_cast<uint32_t>(f32_to_bf16_rne(v.x)) | (static_cast<uint32_t>(f32_to_bf16_rne(v.y)) << 16);
            o.y = static_cast<uint32_t>(f32_to_bf16_rne(v.z)) | (static_cast<uint32_t>(f32_to_bf16_rne(v.w)) << 16);
            out_C_bf16[e] = o;
            if (cpad) cpad[row * Dc4 + j] = o;
            acc = aug::add_squares(acc, o.x, o.y);
        }
        acc = aug::fold_lanes(acc);
        if (lane == 0) aug::write_row(caug, row / K, static_cast<int>(row % K), K, Kpad, acc);
    }
}

// Fused update, second half.  One CTA per centroid row k: the n_part partial rows [p][k][0..D) are added up (thread =
// (partial stripe, column quad)), then the first warp divides, applies the keep-previous rule, writes the fp32 and
// bf16 centroid and, if asked, the row of the next assign's half-norm operand, exactly as finalize_rows_kernel does.
__global__ void __launch_bounds__(256)
finalize_partials_kernel(const float* __restrict__ part_sums, const int* __restrict__ part_counts, int n_part, int n_cnt,
                         int pitch, const uint2* __restrict__ C_prev, int K, int D4, float4* __restrict__ out_C,
                         uint2* __restrict__ out_C_bf16, int* __restrict__ out_counts, uint8_t* __restrict__ caug, int Kpad,
                         double* __restrict__ inertia, uint2* __restrict__ cpad, int Dc4) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    __shared__ float4 red[256];
    __shared__ int cred[256];
    const int k = blockIdx.x;
    if (inertia && k == 0 && threadIdx.x == 0) inertia[0] = 0.0;
    const int t = threadIdx.x;
    const int stripes = 256 / D4;            // D4 <= 32: at least 8 stripes of partials
    const int col = t % D4, stripe = t / D4;
    // (the partials come from L2: all loads of a thread are requested before the first is added -- counts first -- so
    // that the kernel pays one L2 latency per batch and not one per partial; same order of additions)
    int cnt = t < n_cnt ? part_counts[static_cast<size_t>(t) * 128 + k] : 0;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (stripe < stripes) {
        constexpr int BATCH = 10;
        const float* base = part_sums + static_cast<size_t>(k) * pitch + col * 4;
        const size_t pstep = static_cast<size_t>(128) * pitch;
        for (int p0 = stripe; p0 < n_part; p0 += BATCH * stripes) {
            float4 v[BATCH];
#pragma unroll
            for (int u = 0; u < BATCH; ++u) {
                const int p = p0 + u * stripes;
                v[u] = p < n_part ? *reinterpret_cast<const float4*>(base + static_cast<size_t>(p) * pstep) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < BATCH; ++u) { acc.x += v[u].x; acc.y += v[u].y; acc.z += v[u].z; acc.w += v[u].w; }
        }
    }
    for (int p = t + 256; p < n_cnt; p += 256) cnt += part_counts[static_cast<size_t>(p) * 128 + k];
    red[t] = acc;
    cred[t] = cnt;
    __syncthreads();
    for (int o = 128; o >= 32; o >>= 1) {
        if (t < o) cred[t] += cred[t + o];
        __syncthreads();
    }
    if (t >= 32) return;
    int n = cred[t];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) n += __shfl_xor_sync(0xffffffffu, n, o);
    if (t == 0) out_counts[k] = n;
    const float fn = static_cast<float>(n);
    float nacc = 0.f;
    if (cpad)
        for (int j = D4 + t; j < Dc4; j += 32) cpad[static_cast<size_t>(k) * Dc4 + j] = make_uint2(0u, 0u);
    if (t < D4) {
        float4 sv = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int sidx = 0; sidx < stripes; ++sidx) {
            const float4 v = red[sidx * D4 + t];
            sv.x += v.x; sv.y += v.y; sv.z += v.z; sv.w += v.w;
        }
        const size_t e = static_cast<size_t>(k) * D4 + t;
        float4 v;
        if (n > 0) {
            v = make_float4(sv.x / fn, sv.y / fn, sv.z / fn, sv.w / fn);
        } else if (C_prev) {
            const uint2 pv = C_prev[e];
            v = make_float4(bf16lo(pv.x), bf16hi(pv.x), bf16lo(pv.y), bf16hi(pv.y));
        } else {
            v = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        out_C[e] = v;
        uint2 o;
        o.x = static_cast<uint32_t>(f32_to_bf16_rne(v.x)) | (static_cast<uint32_t>(f32_to_bf16_rne(v.y)) << 16);
        o.y = static_cast<uint32_t>(f32_to_bf16_rne(v.z)) | (static_cast<uint32_t>(f32_to_bf16_rne(v.w)) << 16);
        if (out_C_bf16) out_C_bf16[e] = o;
        if (cpad) cpad[static_cast<size_t>(k) * Dc4 + t] = o;
        nacc = aug::add_squares(nacc, o.x, o.y);
    }
    if (caug) {
        nacc = aug::fold_lanes(nacc);
        if (t == 0) aug::write_row(caug, 0, k, K, Kpad, nacc);
    }
}

}  // namespace

// ======================================================================= host side
// Launch that may start while the kernel ahead of it in the stream drains (programmatic dependent
// launch): the kernel itself waits (griddepcontrol.wait) before it touches what that kernel wrote.
template <typename... KArgs, typename... Args>
cudaError_t launch_early(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
bool update_smem_supports(int D, int K, int smem_optin) {
    if (D % 2 != 0) return false;
    const i64 need = static_cast<i64>(K) * D * 4 + static_cast<i64>(K) * 4;
    return need <= smem_optin;
}

int launch_update_smem(const cake_bf16* X, const int* idx, int B, i64 N, int D, int K, float* sums,
                       int* counts, int* status, cudaStream_t s) {
    DeviceInfo di;
    int rc = current_device_info(&di);
    if (rc != CAKE_OK) return rc;
    if (!update_smem_supports(D, K, di.smem_optin)) return CAKE_ERR_UNSUPPORTED;
    const size_t kd = static_cast<size_t>(B) * K * D;
    if (cudaMemsetAsync(sums, 0, kd * sizeof(float), s) != cudaSuccess) return CAKE_ERR_CUDA;
    if (cudaMemsetAsync(counts, 0, static_cast<size_t>(B) * K * sizeof(int), s) != cudaSuccess)
        return CAKE_ERR_CUDA;
    if (N == 0) return CAKE_OK;
    const size_t smem = static_cast<size_t>(K) * D * 4 + static_cast<size_t>(K) * 4;
    static int attr_done_for_device = -1;
    if (attr_done_for_device != di.device) {
        if (cudaFuncSetAttribute(update_smem_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 di.smem_optin) != cudaSuccess)
            return CAKE_ERR_CUDA;
        attr_done_for_device = di.device;
    }
    // CTAs per SM limited by shared memory (228 KiB per SM, 1 KiB reserved per CTA) and threads
    int per_sm = static_cast<int>((228 * 1024) / (smem + 1024));
    if (per_sm > 2048 / SMEM_THREADS) per_sm = 2048 / SMEM_THREADS;
    if (per_sm < 1) per_sm = 1;
    i64 ctas = (static_cast<i64>(di.sm_count) * per_sm + B - 1) / B;
    const i64 max_useful = (N + 255) / 256;  // at least 256 rows per CTA
    if (ctas > max_useful) ctas = max_useful;
    if (ctas < 1) ctas = 1;
    dim3 grid(static_cast<unsigned>(ctas), static_cast<unsigned>(B));
    update_smem_kernel<<<grid, SMEM_THREADS, smem, s>>>(X, idx, N, D, K, sums, counts, status);
    note_launches(1);
    return cudaGetLastError() == cudaSuccess ? CAKE_OK : CAKE_ERR_CUDA;
}

namespace {
struct SortPlan {
    bool blocked;
    int nblk;
    i64 slab;
};
SortPlan sort_plan(i64 N, int K) {
    SortPlan pl;
    pl.blocked = K <= BLK_MAX_K;
    i64 nblk = (N + BLK_MIN_SLAB - 1) / BLK_MIN_SLAB;
    if (nblk > BLK_MAX_BLOCKS) nblk = BLK_MAX_BLOCKS;
    if (nblk < 1) nblk = 1;
    pl.nblk = static_cast<int>(nblk);
    pl.slab = ((N + nblk - 1) / nblk + BLK_VEC - 1) / BLK_VEC * BLK_VEC;
    return pl;
}
}  // namespace

size_t update_sort_part_bytes(i64 B, i64 N, int K) {
    const SortPlan pl = sort_plan(N, K);
    return pl.blocked ? static_cast<size_t>(B) * pl.nblk * K * sizeof(int) : 0;
}

size_t update_sort_rank_bytes(i64 B, i64 N, int K) {
    return sort_plan(N, K).blocked ? 0 : static_cast<size_t>(B) * N * sizeof(int);
}

int launch_update_sort(const cake_bf16* X, const int* idx, int B, i64 N, int D, int K,
                       const UpdateScratch& scr, int* counts, const cake_bf16* C_prev, float* out_C,
                       cake_bf16* out_C_bf16, bool* divided, int* status, cudaStream_t s) {
    DeviceInfo di;
    int rc = current_device_info(&di);
    if (rc != CAKE_OK) return rc;
    *divided = false;
    const size_t kd = static_cast<size_t>(B) * K * D;
    const SortPlan pl = sort_plan(N, K);
    // large K, rows of whole 16-byte granules: the last kernel writes the means itself (no partial sums)
    // (only where the caller wants centroids: without out_C the sums themselves are the result)
    const bool means = out_C && N > 0 && !pl.blocked && D % 8 == 0 && D >= 24 && D <= 1024;
    const bool zero_in_hist = N > 0 && !pl.blocked && !means && (static_cast<i64>(K) * D) % 4 == 0;
    if (N == 0 || !pl.blocked) {
        if (!means && !zero_in_hist && cudaMemsetAsync(scr.sums, 0, kd * sizeof(float), s) != cudaSuccess)
            return CAKE_ERR_CUDA;
        if (cudaMemsetAsync(counts, 0, static_cast<size_t>(B) * K * sizeof(int), s) != cudaSuccess)
            return CAKE_ERR_CUDA;
    }
    if (N == 0) return CAKE_OK;
    if (pl.blocked) {
        const dim3 grid(static_cast<unsigned>(pl.nblk), static_cast<unsigned>(B));
        const size_t smem = static_cast<size_t>(K) * sizeof(int);
        hist_blocked_kernel<<<grid, BLK_THREADS, smem, s>>>(idx, N, K, pl.slab, scr.part, scr.sums,
                                                            static_cast<i64>(K) * D, status);
        colscan_kernel<<<dim3((K + 31) / 32, B), 256, 0, s>>>(scr.part, pl.nblk, K, counts);
        scatter_blocked_kernel<<<grid, BLK_THREADS, smem, s>>>(idx, N, K, pl.slab, scr.part, counts, scr.nvalid,
                                                               scr.pairs);
    } else {
        {
            i64 ctas = (N + HIST_THREADS * HIST_PER_THREAD - 1) / (HIST_THREADS * HIST_PER_THREAD);
            const i64 cap = (static_cast<i64>(di.sm_count) * 4 + B - 1) / B;
            if (ctas > cap) ctas = cap;
            if (ctas < 1) ctas = 1;
            hist_kernel<<<dim3(static_cast<unsigned>(ctas), B), HIST_THREADS, 0, s>>>(
                idx, N, K, counts, scr.rank, reinterpret_cast<float4*>(scr.sums),
                zero_in_hist ? static_cast<i64>(K) * D / 4 : 0, status);
        }
        if (launch_early(scan_kernel, dim3((K + SCAN_TILE - 1) / SCAN_TILE, B), dim3(1024), 0, s, counts, K, scr.cursor,
                         scr.nvalid, means ? scr.sums : nullptr, scr.done, D) != cudaSuccess)
            return CAKE_ERR_CUDA;
        {
            i64 ctas = (N + 256 * 4 - 1) / (256 * 4);
            const i64 cap = (static_cast<i64>(di.sm_count) * 8 + B - 1) / B;
            if (ctas > cap) ctas = cap;
            if (ctas < 1) ctas = 1;
            if (launch_early(scatter_kernel, dim3(static_cast<unsigned>(ctas), B), dim3(256), 0, s, idx, scr.rank, N, K,
                             scr.cursor, scr.pairs) != cudaSuccess)
                return CAKE_ERR_CUDA;
        }
    }
    if (means) {
        // one warp per window of the sorted order, and enough warps to deal out the empty clusters
        i64 warps = (N + SEG_ROWS - 1) / SEG_ROWS;
        if (warps < K / 4) warps = K / 4;
        dim3 grid(static_cast<unsigned>((warps + MEAN_WARPS - 1) / MEAN_WARPS), B);
        const int G = D / 8;
        int lpr = 4;
        while (lpr < G && lpr < 32) lpr <<= 1;
        const int gpl = (G + lpr - 1) / lpr;
        // per warp: MEAN_AHEAD batches of MEAN_BATCH_GRANULES granules per lane (6 KiB) and the row table
        const size_t mean_smem = static_cast<size_t>(MEAN_WARPS) * MEAN_WARP_UINT4 * sizeof(uint4);
        using MeanKernel = void (*)(const cake_bf16*, const int2*, const int*, const int*, i64, int, int,
                                    const cake_bf16*, float*, cake_bf16*, float*, int*);
        MeanKernel kernel = gpl > 2 ? segmean_kernel<4, 32> : gpl == 2 ? segmean_kernel<2, 32>
                          : lpr == 32 ? segmean_kernel<1, 32> : lpr == 16 ? segmean_kernel<1, 16>
                          : lpr == 8 ? segmean_kernel<1, 8> : segmean_kernel<1, 4>;
        if (launch_early(kernel, grid, dim3(MEAN_WARPS * 32), mean_smem, s, X, scr.pairs, scr.nvalid, counts, N, D, K, C_prev,
                         out_C, out_C_bf16, scr.sums, scr.done) != cudaSuccess)
            return CAKE_ERR_CUDA;
        *divided = true;
    } else {
        const i64 warps = (N + SEG_ROWS - 1) / SEG_ROWS;
        const unsigned ctas = static_cast<unsigned>((warps + SEG_WARPS - 1) / SEG_WARPS);
        dim3 grid(ctas, B);
        if (D % 8 == 0 && D <= 1024) {
            const int G = D / 8;
            int lpr = 1;
            while (lpr < G && lpr < 32) lpr <<= 1;
            const int gpl = (G + lpr - 1) / lpr;
            if (gpl == 1)
                segreduce_kernel<1><<<grid, SEG_WARPS * 32, 0, s>>>(X, scr.pairs, scr.nvalid, N, D, K, lpr, scr.sums);
            else if (gpl == 2)
                segreduce_kernel<2><<<grid, SEG_WARPS * 32, 0, s>>>(X, scr.pairs, scr.nvalid, N, D, K, lpr, scr.sums);
            else
                segreduce_kernel<4><<<grid, SEG_WARPS * 32, 0, s>>>(X, scr.pairs, scr.nvalid, N, D, K, lpr, scr.sums);
        } else {
            segreduce_scalar_kernel<<<grid, SEG_WARPS * 32, 0, s>>>(X, scr.pairs, scr.nvalid, N, D, K, scr.sums);
        }
    }
    note_launches(4);  // histogram, scan, scatter, segmented reduction
    return cudaGetLastError() == cudaSuccess ? CAKE_OK : CAKE_ERR_CUDA;
}

// ---- slab route, host side
namespace {
struct SlabPlan {
    int S;         // rows per CTA (multiple of 4)
    int n_ctas;    // CTAs per problem (multiple of F)
    int F;         // CTAs per thread-block cluster
    int rowbits;   // bits of a row number inside a cluster's F*S rows
    bool flat;     // slabs dealt over the rows of all problems (n_ctas is then the total)
};

using SlabKernel = void (*)(const cake_bf16*, const int*, i64, int, int, int, int, float*, int*, int*, i64, int);

SlabKernel slab_kernel_for(int lpr, bool cluster, bool wide) {
    if (wide) return cluster ? slab_update_kernel<32, true, true> : slab_update_kernel<32, false, true>;
    switch (lpr) {
        case 4: return cluster ? slab_update_kernel<4, true> : slab_update_kernel<4, false>;
        case 8: return cluster ? slab_update_kernel<8, true> : slab_update_kernel<8, false>;
        case 16: return cluster ? slab_update_kernel<16, true> : slab_update_kernel<16, false>;
        default: return cluster ? slab_update_kernel<32, true> : slab_update_kernel<32, false>;
    }
}

int slab_lpr(int D) {
    int lpr = 4;
    while (lpr < D / 8 && lpr < 32) lpr <<= 1;
    return lpr;
}

size_t slab_smem_bytes(int K, int S) { return (static_cast<size_t>(2) * K + S) * sizeof(int); }

// CTAs of `kernel` that can be resident at once when launched as clusters of F (F = 1: one per SM)
int slab_slots(const DeviceInfo& di, SlabKernel kernel, int F, size_t smem) {
    if (cudaFuncSetAttribute(reinterpret_cast<const void*>(kernel), cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(slab_smem_bytes(SLAB_MAX_K, SLAB_MAX_ROWS))) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    if (F == 1) return di.sm_count;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(F) * di.sm_count);
    cfg.blockDim = dim3(SLAB_THREADS);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = static_cast<unsigned>(F);
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, reinterpret_cast<const void*>(kernel), &cfg) != cudaSuccess || n < 1) {
        cudaGetLastError();
        return 0;
    }
    return n * F;
}

// Rows per CTA so that the CTAs of all problems fill whole waves of the resident slots.
void slab_rows_for(int slots, int B, i64 N, int F, int* S, int* n_ctas) {
    for (int w = 1;; ++w) {
        i64 per_problem = static_cast<i64>(w) * slots / B / F * F;
        if (per_problem < F) per_problem = F;
        i64 rows = (N + per_problem - 1) / per_problem;
        if (rows < 1024) rows = 1024;                       // smaller slabs only add atomics (measured: 512 loses)
        rows = (rows + 3) / 4 * 4;
        if (rows <= SLAB_MAX_ROWS) {
            *S = static_cast<int>(rows);
            const i64 n = (N + rows - 1) / rows;
            *n_ctas = static_cast<int>((n + F - 1) / F * F);
            return;
        }
    }
}
}  // namespace

bool update_slab_supports(int D, int K) { return D % 8 == 0 && D >= 8 && D <= 1024 && K <= SLAB_MAX_K; }

static int slab_make_plan(const DeviceInfo& di, int B, i64 N, int D, int K, int force_f, SlabPlan* out) {
    const int lpr = slab_lpr(D);
    SlabPlan best = {};
    for (int F = 1; F <= SLAB_MAX_F; F <<= 1) {
        if (force_f && F != force_f) continue;
        SlabPlan pl;
        pl.F = F;
        const int slots = slab_slots(di, slab_kernel_for(lpr, F > 1, D > 256), F, slab_smem_bytes(K, SLAB_MAX_ROWS));
        if (slots < F) continue;
        slab_rows_for(slots, B, N, F, &pl.S, &pl.n_ctas);
        pl.rowbits = 1;
        while ((static_cast<i64>(1) << pl.rowbits) < static_cast<i64>(pl.S) * F) ++pl.rowbits;
        best = pl;
        // runs of SLAB_GROW_RUN rows keep the atomics cheap (measured); larger clusters only cost
        if (static_cast<i64>(pl.S) * F >= static_cast<i64>(SLAB_GROW_RUN) * K || pl.n_ctas <= F) break;
    }
    if (best.F == 0) return CAKE_ERR_UNSUPPORTED;
    best.flat = false;
    // A batch whose problems leave SMs idle (32 problems on 148 SMs: 4 CTAs each, 20 SMs without work): deal
    // the rows of all problems to the CTAs instead.  Needs no thread-block clusters, a slab no longer than a
    // problem, and twice K counters in shared memory.
    if (B > 1 && best.F == 1 && !force_f && 2 * static_cast<i64>(K) <= SLAB_MAX_K) {
        const i64 total = static_cast<i64>(B) * N;
        const int slots = di.sm_count;
        for (int w = 1; w <= 64; ++w) {
            i64 rows = (total + static_cast<i64>(w) * slots - 1) / (static_cast<i64>(w) * slots);
            if (rows < 1024) rows = 1024;
            rows = (rows + 3) / 4 * 4;
            if (rows > SLAB_MAX_ROWS) continue;
            const i64 n = (total + rows - 1) / rows;
            const i64 waves = (n + slots - 1) / slots, waves_now = (static_cast<i64>(best.n_ctas) * B + slots - 1) / slots;
            // taken when it runs as many rows per run and fewer or equally many, fuller waves
            if (rows <= N && rows >= static_cast<i64>(SLAB_GROW_RUN) * K && waves * rows < waves_now * best.S) {
                best.flat = true;
                best.S = static_cast<int>(rows);
                best.n_ctas = static_cast<int>(n);
                best.rowbits = 1;
                while ((static_cast<i64>(1) << best.rowbits) < rows) ++best.rowbits;
            }
            break;
        }
    }
    *out = best;
    return CAKE_OK;
}

bool update_slab_preferred(int B, i64 N, int D, int K) {
    DeviceInfo di;
    SlabPlan pl;
    if (N < 1 || !update_slab_supports(D, K) || current_device_info(&di) != CAKE_OK) return false;
    if (slab_make_plan(di, B, N, D, K, 0, &pl) != CAKE_OK) return false;
    // measured against the sort route: up to 4,096 clusters the slab route wins from 1.5 rows per run on
    // (equal at 1.7, 17-45 % faster at 2-3.5); above, its per-CTA scan of K counters needs 4 rows per run
    const i64 rows = static_cast<i64>(pl.S) * pl.F;
    const i64 have = rows < N ? rows : N;
    return K <= 4096 ? 2 * have >= 3 * static_cast<i64>(K) : have >= static_cast<i64>(SLAB_MIN_RUN) * K;
}

int launch_update_slab(const cake_bf16* X, const int* idx, int B, i64 N, int D, int K, float* sums, int* counts,
                       int* status, int force_f, cudaStream_t s) {
    DeviceInfo di;
    int rc = current_device_info(&di);
    if (rc != CAKE_OK) return rc;
    if (!update_slab_supports(D, K)) return CAKE_ERR_UNSUPPORTED;
    {
        // D % 8 == 0, so the sums are whole float4s
        const i64 n4 = static_cast<i64>(B) * K * D / 4, nc = static_cast<i64>(B) * K;
        i64 ctas = (n4 + 256 * 4 - 1) / (256 * 4);
        if (ctas > di.sm_count * 4) ctas = di.sm_count * 4;
        cudaLaunchAttribute zat[1];
        zat[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        zat[0].val.programmaticStreamSerializationAllowed = 1;
        cudaLaunchConfig_t zcfg = {};
        zcfg.gridDim = dim3(static_cast<unsigned>(ctas));
        zcfg.blockDim = dim3(256);
        zcfg.stream = s;
        zcfg.attrs = zat;
        zcfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&zcfg, zero_sums_counts_kernel, reinterpret_cast<float4*>(sums), n4, counts, nc) != cudaSuccess) {
            cudaGetLastError();
            return CAKE_ERR_CUDA;
        }
        note_launches(1);
    }
    if (N == 0) return CAKE_OK;
    SlabPlan pl;
    rc = slab_make_plan(di, B, N, D, K, force_f, &pl);
    if (rc != CAKE_OK) return rc;
    const int lpr = slab_lpr(D);
    SlabKernel kernel = slab_kernel_for(lpr, pl.F > 1, D > 256);
    const int Kh = pl.flat ? 2 * K : K;                      // counters per CTA
    const i64 Nk = pl.flat ? static_cast<i64>(B) * N : N;    // rows the grid's x dimension is dealt over
    const size_t smem = slab_smem_bytes(Kh, pl.S);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(pl.n_ctas), pl.flat ? 1u : static_cast<unsigned>(B));
    cfg.blockDim = dim3(SLAB_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    // may start while the zero-fill still runs (it waits for it before its first add)
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    at[1].id = cudaLaunchAttributeClusterDimension;
    at[1].val.clusterDim.x = static_cast<unsigned>(pl.F);
    at[1].val.clusterDim.y = 1;
    at[1].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = pl.F > 1 ? 2 : 1;
    if (cudaLaunchKernelEx(&cfg, kernel, X, idx, Nk, D, Kh, pl.S, pl.rowbits, sums, counts, status,
                           pl.flat ? N : static_cast<i64>(0), K) != cudaSuccess) {
        cudaGetLastError();
        return CAKE_ERR_CUDA;
    }
    note_launches(1);
    return CAKE_OK;
}

cudaError_t launch_finalize(const float* sums, const int* counts, const cake_bf16* C_prev, int B, int K,
                            int D, float* out_C, cake_bf16* out_C_bf16, bool early, const NextAssign* next,
                            bool* prepared, cudaStream_t s, int sums_columns) {
    const i64 total = static_cast<i64>(B) * K * D;
    const int Ds = sums_columns ? sums_columns : D;   // columns of a row of sums (a multiple of 4 when D is)
    if (prepared) *prepared = false;
    if (next && out_C_bf16 && D % 4 == 0 && B <= 256) {
        const i64 rows = static_cast<i64>(B) * K;
        i64 ctas = (rows + 7) / 8;
        if (ctas > 148 * 8) ctas = 148 * 8;
        if (ctas < 1) ctas = 1;
        cudaError_t e = launch_early(finalize_rows_kernel, dim3(static_cast<unsigned>(ctas)), dim3(256), 0, s,
                                     reinterpret_cast<const float4*>(sums), counts, reinterpret_cast<const uint2*>(C_prev), rows,
                                     K, D / 4, reinterpret_cast<float4*>(out_C), reinterpret_cast<uint2*>(out_C_bf16),
                                     static_cast<uint8_t*>(next->caug), padded_k(K), next->inertia,
                                     next->inertia_stride, B, reinterpret_cast<uint2*>(next->cpad), next->cpad_columns / 4,
                                     Ds / 4);
        note_launches(1);
        if (e == cudaSuccess && prepared) *prepared = true;
        return e;
    }
    // early: the launch may overlap the tail of the kernel ahead (the kernels wait for it themselves)
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(256);
    cfg.stream = s;
    cfg.attrs = at;
    cfg.numAttrs = early ? 1 : 0;
    if (D % 4 == 0) {
        i64 ctas = (total / 4 + 255) / 256;
        if (ctas > 148 * 16) ctas = 148 * 16;
        if (ctas < 1) ctas = 1;
        cfg.gridDim = dim3(static_cast<unsigned>(ctas));
        note_launches(1);
        return cudaLaunchKernelEx(&cfg, finalize4_kernel, reinterpret_cast<const float4*>(sums), counts,
                                  reinterpret_cast<const uint2*>(C_prev), total / 4, D / 4, Ds / 4,
                                  reinterpret_cast<float4*>(out_C), reinterpret_cast<uint2*>(out_C_bf16));
    }
    i64 ctas = (total + 256 * 4 - 1) / (256 * 4);
    if (ctas > 148 * 16) ctas = 148 * 16;
    if (ctas < 1) ctas = 1;
    cfg.gridDim = dim3(static_cast<unsigned>(ctas));
    note_launches(1);
    return cudaLaunchKernelEx(&cfg, finalize_kernel, sums, counts, C_prev, total, D, Ds, out_C, out_C_bf16);
}

cudaError_t launch_finalize_partials(const float* part_sums, const int* part_counts, int n_ctas, const cake_bf16* C_prev,
                                     int K, int D, float* out_C, cake_bf16* out_C_bf16, int* out_counts,
                                     const NextAssign* next, bool* prepared, cudaStream_t s) {
    if (prepared) *prepared = false;
    const bool prep = next && out_C_bf16;
    const int Kpad = padded_k(K);
    // (the operand's padding rows K..Kpad-1 were written by the first iteration's prologue and never change)
    cudaError_t e = launch_early(finalize_partials_kernel, dim3(static_cast<unsigned>(K)), dim3(256), 0, s, part_sums, part_counts,
                                 n_ctas, n_ctas, (D + 15) & ~15, reinterpret_cast<const uint2*>(C_prev), K, D / 4,
                                 reinterpret_cast<float4*>(out_C), reinterpret_cast<uint2*>(out_C_bf16), out_counts,
                                 prep ? static_cast<uint8_t*>(next->caug) : static_cast<uint8_t*>(nullptr), Kpad,
                                 prep ? next->inertia : static_cast<double*>(nullptr),
                                 prep ? reinterpret_cast<uint2*>(next->cpad) : static_cast<uint2*>(nullptr),
                                 prep ? next->cpad_columns / 4 : 0);
    note_launches(1);
    if (e == cudaSuccess && prep && prepared) *prepared = true;
    return e;
}

}  // namespace cake
