// Lloyd iterations of a SMALL problem in one kernel launch (paper Section 5, "Flash-KMeans clean-start workload": the
// assignment and update steps of every iteration; Appendix F lists a single-pass "gap-fused" route for the iteration).
//
// One problem, at most 128 clusters, D <= 128 (a multiple of 8), and few enough rows that every CTA can keep its row tiles in
// shared memory for the whole call (at most four 128-row tiles per SM).  Such problems are bound by launch and set-up
// latency, not by arithmetic: the two-kernel iteration of the general path costs about 14 us there, of which the
// tensor pipe works for less than one.  Here one cooperative launch runs all iterations:
//   once      : the CTA's X tiles come in by TMA and stay; each row's ||x||^2/2 + m operand is computed once.
//   iteration : centroids -> shared memory (plain loads, the half-norm operand computed on the way); per tile the
//               distance MMAs (tcgen05, accumulator in tensor memory), the arg-min over packed keys (same arithmetic
//               and tie rule as assign_tc.cu), the tile's one-hot operand and sums += onehot^T X on the tensor core;
//               the CTA's partial sums and counts go to global memory; grid barrier; every cluster is divided by
//               one CTA (keep-previous rule for empty clusters) and written as the next iteration's centroids; grid
//               barrier.
// 128 threads per CTA: thread r is row r of every tile, lane r of tensor memory, and cluster r of the sums.  Every
// wait is bounded; a time-out sets the workspace's status word and lets all loops run out.

#include "aug.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace cake {
namespace {

constexpr int BLOCK_M = 128;
constexpr int KCHUNK = 64;
constexpr int UMMA_K = 16;
constexpr int THREADS = 128;
constexpr int MAX_R = 4;                                  // row tiles a CTA keeps
constexpr uint32_t X_CHUNK_BYTES = BLOCK_M * 128;         // 16 KiB: 128 rows x 64 columns, 128-byte swizzle
constexpr uint32_t C_CHUNK_BYTES = 128 * 128;             // 16 KiB: up to 128 centroids x 64 columns
constexpr uint32_t AUG_BYTES = 128 * 16;                  // 2 KiB: one 16-byte row per X row / centroid
constexpr uint32_t ZERO_BYTES = 4096;
constexpr uint32_t OH_BYTES = 2 * X_CHUNK_BYTES;          // one-hot operand: [128 clusters][128 rows] bf16
constexpr uint32_t COL_MASK = 0x7Fu;
constexpr uint32_t F32_INF = 0x7f800000u;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t SUMS_COL = 256;                        // tensor-memory columns of the per-cluster sums
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;

struct Params {
    const cake_bf16* C0;      // [K][D] initial centroids
    i64 N;
    int D, K, iters;
    int nchunks;              // ceil(D / 64): columns D .. 64 nchunks - 1 of the tiles are zeros
    int ncol;                 // D rounded up to 16: columns of the sums (the update MMA's N), pitch of the partial sums
    int c_rows;               // K rounded up to 32: columns of an accumulator
    int tiles;                // ceil(N / 128)
    float* part_sums;         // [grid][128][ncol] per-CTA partial sums
    int* part_counts;         // [grid][128]
    cake_bf16* cbuf;          // [K][D] the centroids between iterations
    float* out_C;             // [K][D] fp32, may be null
    cake_bf16* out_C_bf16;    // [K][D], may be null
    int* out_idx;             // [N]
    float* out_dist;          // [N], may be null
    int* out_counts;          // [K]
    double* inertia;          // [iters], zeroed by the host, may be null
    unsigned* gbar;           // grid barrier counter, zeroed by the host
    int* status;
};

struct Ctrl {
    uint64_t bar_x, bar_mma[2], bar_upd;
    uint32_t tmem_base;
    int abort_flag;
    int cnt[128];             // rows per cluster (this CTA, this iteration)
    float4 red[THREADS];      // finalize: partial rows per stripe
    int cred[THREADS];
    double dred[4];           // the warps' shares of the iteration's inertia
};
static_assert(sizeof(Ctrl) <= 4096, "control block");

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t f32_to_bf16_rne(float f) { return aug::bf16_rne_bits(f); }

// bounded wait on an mbarrier phase; after a time-out every later wait returns at once
__device__ __forceinline__ void wait_bar(uint64_t* bar, uint32_t parity, Ctrl* ctrl, int* status) {
    const uint32_t addr = ptx::smem_u32(bar);
    if (ptx::mbar_try_wait(addr, parity)) return;
    const uint64_t t0 = ptx::globaltimer_ns();
    while (!ptx::mbar_try_wait_hint(addr, parity, 20000)) {
        if (*reinterpret_cast<volatile int*>(&ctrl->abort_flag)) return;
        if (ptx::globaltimer_ns() - t0 > WAIT_LIMIT_NS) {
            *reinterpret_cast<volatile int*>(&ctrl->abort_flag) = 1;
            atomicCAS(status, CAKE_OK, CAKE_ERR_TIMEOUT);
            return;
        }
    }
}

// All CTAs of the (cooperative) launch meet; `round` counts the barriers so far.  Bounded like every other wait.
__device__ __forceinline__ void grid_barrier(unsigned* counter, unsigned round, Ctrl* ctrl, int* status) {
    __syncthreads();
    if (threadIdx.x == 0) {
        // arrive with release (the CTA's writes, ordered before this thread by the barrier above, become visible with
        // it), poll with acquire: no full fences
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(counter) : "memory");
        const unsigned want = (round + 1u) * gridDim.x;
        uint64_t t0 = 0;
        for (unsigned n = 0;; ++n) {
            unsigned v;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
            if (v >= want) break;
            if ((n & 255u) != 255u) continue;
            if (*reinterpret_cast<volatile int*>(&ctrl->abort_flag)) break;
            const uint64_t now = ptx::globaltimer_ns();
            if (t0 == 0) t0 = now;
            if (now - t0 > WAIT_LIMIT_NS) {
                *reinterpret_cast<volatile int*>(&ctrl->abort_flag) = 1;
                atomicCAS(status, CAKE_OK, CAKE_ERR_TIMEOUT);
                break;
            }
        }
    }
    __syncthreads();
}

// key = the accumulator with its low 7 bits replaced by the column; minimum over 32 columns (see assign_tc.cu)
__device__ __forceinline__ float packed_min32(const uint32_t (&r)[32], int col_base, float run, uint32_t kmask) {
    float v[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(ptx::and_or(r[j], kmask, static_cast<uint32_t>(col_base + j)));
    float t[11];
#pragma unroll
    for (int q = 0; q < 10; ++q) t[q] = ptx::fmin3(v[3 * q], v[3 * q + 1], v[3 * q + 2]);
    t[10] = fminf(v[30], v[31]);
    const float u0 = ptx::fmin3(t[0], t[1], t[2]);
    const float u1 = ptx::fmin3(t[3], t[4], t[5]);
    const float u2 = ptx::fmin3(t[6], t[7], t[8]);
    const float u3 = fminf(t[9], t[10]);
    return fminf(run, fminf(ptx::fmin3(u0, u1, u2), u3));
}

__global__ void __launch_bounds__(THREADS, 1)
lloyd_small_kernel(const __grid_constant__ CUtensorMap tmap_x, const Params p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = ptx::smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    uint8_t* smem = smem_raw + pad;
    const uint32_t smem_base = raw_addr + pad;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int R = (p.tiles + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);      // most tiles any CTA has
    const int nt_mine = (p.tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
    const uint32_t xtile_bytes = static_cast<uint32_t>(p.nchunks) * X_CHUNK_BYTES;
    const uint32_t c_off = static_cast<uint32_t>(R) * xtile_bytes;
    const uint32_t auga_off = c_off + static_cast<uint32_t>(p.nchunks) * C_CHUNK_BYTES;
    const uint32_t augb_off = auga_off + static_cast<uint32_t>(R) * AUG_BYTES;
    const uint32_t zero_off = augb_off + AUG_BYTES;
    const uint32_t oh_off = (zero_off + ZERO_BYTES + 1023u) & ~1023u;
    const uint32_t ctrl_off = oh_off + OH_BYTES;
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem + ctrl_off);

    if (tid == 0) {
        ptx::mbar_init(ptx::smem_u32(&ctrl->bar_x), 1);
        ptx::mbar_init(ptx::smem_u32(&ctrl->bar_mma[0]), 1);
        ptx::mbar_init(ptx::smem_u32(&ctrl->bar_mma[1]), 1);
        ptx::mbar_init(ptx::smem_u32(&ctrl->bar_upd), 1);
        ctrl->abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_x);
    }
    // zeros: columns 8..15 of the operands of the extra k-step, and the one-hot operand (kept up to date element by element)
    for (uint32_t o = tid * 16; o < ZERO_BYTES; o += THREADS * 16) *reinterpret_cast<uint4*>(smem + zero_off + o) = make_uint4(0, 0, 0, 0);
    for (uint32_t o = tid * 16; o < OH_BYTES; o += THREADS * 16) *reinterpret_cast<uint4*>(smem + oh_off + o) = make_uint4(0, 0, 0, 0);
    // (the centroid tile too: the granules behind column D of its last chunk are never written and must read as zeros)
    for (uint32_t o = tid * 16; o < static_cast<uint32_t>(p.nchunks) * C_CHUNK_BYTES; o += THREADS * 16)
        *reinterpret_cast<uint4*>(smem + c_off + o) = make_uint4(0, 0, 0, 0);
    ptx::fence_proxy_async_smem();
    if (warp == 0) {
        ptx::tmem_alloc(ptx::smem_u32(&ctrl->tmem_base), TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&ctrl->tmem_base);

    // ---- once: this CTA's X tiles (rows behind N arrive as zeros), and every row's operand of the extra k-step
    if (tid == 0) {
        const uint32_t bar = ptx::smem_u32(&ctrl->bar_x);
        ptx::mbar_arrive_expect_tx(bar, static_cast<uint32_t>(nt_mine) * xtile_bytes);
        for (int j = 0; j < nt_mine; ++j)
            for (int c = 0; c < p.nchunks; ++c)
                ptx::tma_load_3d(smem_base + j * xtile_bytes + c * X_CHUNK_BYTES, &tmap_x, bar, c * KCHUNK,
                                 (static_cast<int>(blockIdx.x) + j * static_cast<int>(gridDim.x)) * BLOCK_M, 0);
    }
    wait_bar(&ctrl->bar_x, 0u, ctrl, p.status);
    float rowM[MAX_R];
#pragma unroll
    for (int j = 0; j < MAX_R; ++j) {
        rowM[j] = 0.f;
        if (j < nt_mine) {
            // ||x||^2 from the swizzled tile (16-byte granule g of row r sits at position g ^ (r & 7)); margin
            // m = 2^(e-11) for ||x||^2 in [2^e, 2^(e+1)), at least 2^-100; operand [hi mid lo 1 1 1 0 0] (see assign_tc.cu)
            const uint8_t* xrow = smem + j * xtile_bytes + tid * 128;
            float xn0 = 0.f, xn1 = 0.f, xn2 = 0.f, xn3 = 0.f;
            for (int c = 0; c < p.nchunks; ++c) {
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    const uint4 w = *reinterpret_cast<const uint4*>(xrow + c * X_CHUNK_BYTES + ((g ^ (tid & 7)) << 4));
                    float a = bf16lo(w.x); xn0 = fmaf(a, a, xn0); a = bf16hi(w.x); xn1 = fmaf(a, a, xn1);
                    a = bf16lo(w.y); xn2 = fmaf(a, a, xn2); a = bf16hi(w.y); xn3 = fmaf(a, a, xn3);
                    a = bf16lo(w.z); xn0 = fmaf(a, a, xn0); a = bf16hi(w.z); xn1 = fmaf(a, a, xn1);
                    a = bf16lo(w.w); xn2 = fmaf(a, a, xn2); a = bf16hi(w.w); xn3 = fmaf(a, a, xn3);
                }
            }
            const float xn = (xn0 + xn1) + (xn2 + xn3);
            const uint32_t xe = __float_as_uint(xn) >> 23;
            const uint32_t mbits = (xe > 38u ? xe - 11u : 27u) << 23;
            uint32_t hi, mid, lo;
            aug::split3(fmaf(0.5f, xn, __uint_as_float(mbits)), hi, mid, lo);
            const uint32_t one = 0x3F80u;
            *reinterpret_cast<uint4*>(smem + auga_off + j * AUG_BYTES + tid * 16) =
                make_uint4(hi | (mid << 16), lo | (one << 16), one | (one << 16), 0u);
            rowM[j] = __uint_as_float(mbits);
        }
    }

    const uint32_t kmask = ~COL_MASK | (static_cast<uint32_t>(p.K) >> 31);   // in a register (see assign_tc.cu)
    const int ng = p.c_rows >> 5;
    const int gpr = p.D >> 3;                                  // 16-byte granules per row
    constexpr uint32_t KSTEP = (UMMA_K * 2) >> 4;
    const uint32_t idesc_aug = ptx::umma_idesc_bf16(BLOCK_M, p.c_rows);
    const uint32_t idesc_main = idesc_aug | ptx::UMMA_IDESC_NEGATE_B;   // accumulates -x.c
    const uint32_t idesc_upd = ptx::umma_idesc_bf16(BLOCK_M, p.ncol) | ptx::UMMA_IDESC_B_MN_MAJOR;
    uint32_t ph0 = 0, ph1 = 0, upd_n = 0;                      // completed uses of the barriers
    unsigned gb = 0;
    int prev_oh = -1;                                          // the cluster whose one-hot entry this row has set

    // thread 0: the MMAs of tile j of this CTA: D[acc j & 1] = m + ||x||^2/2 - x.c + ||c||^2/2
    auto issue_assign = [&](int j) {
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(j & 1) * 128u;
        for (int c = 0; c < p.nchunks; ++c) {
            const uint32_t a_lo = ptx::umma_desc_lo_sw128(smem_base + j * xtile_bytes + c * X_CHUNK_BYTES);
            const uint32_t b_lo = ptx::umma_desc_lo_sw128(smem_base + c_off + c * C_CHUNK_BYTES);
#pragma unroll
            for (uint32_t ks = 0; ks < KCHUNK / UMMA_K; ++ks) {
                if (c == 0 && ks == 0)
                    ptx::umma_bf16_lohi<false>(d_tmem, a_lo, ptx::UMMA_DESC_HI_SW128, b_lo, ptx::UMMA_DESC_HI_SW128, idesc_main);
                else
                    ptx::umma_bf16_lohi<true>(d_tmem, a_lo + ks * KSTEP, ptx::UMMA_DESC_HI_SW128, b_lo + ks * KSTEP,
                                              ptx::UMMA_DESC_HI_SW128, idesc_main);
            }
        }
        ptx::umma_bf16_lohi<true>(d_tmem, ptx::umma_desc_lo_aug(smem_base + auga_off + j * AUG_BYTES, smem_base + zero_off),
                                  ptx::UMMA_DESC_HI_AUG, ptx::umma_desc_lo_aug(smem_base + augb_off, smem_base + zero_off),
                                  ptx::UMMA_DESC_HI_AUG, idesc_aug);
        ptx::umma_commit(ptx::smem_u32(&ctrl->bar_mma[j & 1]));
    };

    for (int it = 0; it < p.iters; ++it) {
        const cake_bf16* src = it == 0 ? p.C0 : p.cbuf;
        // ---- this iteration's centroids into shared memory, K-major with the 128-byte swizzle the MMA reads (rows K ..
        // c_rows - 1 are zeros).  Loads that bypass L1: after the first iteration other CTAs wrote these rows in this launch.
        // (eight loads of a thread are requested before the first is stored: one L2 latency per batch, not per load)
        constexpr int CBATCH = 8;
        for (int e0 = tid; e0 < p.c_rows * gpr; e0 += THREADS * CBATCH) {
            uint4 v[CBATCH];
#pragma unroll
            for (int u = 0; u < CBATCH; ++u) {
                const int e = e0 + u * THREADS;
                const int k = e / gpr, g = e - k * gpr;
                v[u] = make_uint4(0, 0, 0, 0);
                if (e < p.c_rows * gpr && k < p.K) v[u] = __ldcg(reinterpret_cast<const uint4*>(src + static_cast<size_t>(k) * p.D) + g);
            }
#pragma unroll
            for (int u = 0; u < CBATCH; ++u) {
                const int e = e0 + u * THREADS;
                const int k = e / gpr, g = e - k * gpr;
                if (e < p.c_rows * gpr)
                    *reinterpret_cast<uint4*>(smem + c_off + (g >> 3) * C_CHUNK_BYTES + k * 128 + (((g & 7) ^ (k & 7)) << 4)) = v[u];
            }
        }
        ctrl->cnt[tid] = 0;
        __syncthreads();
        {   // the centroid-side operand of the extra k-step, row `tid`: [1 1 1 h_hi h_mid h_lo 0 0], h = ||c||^2 / 2
            uint32_t hi = 0x7B80u, mid = 0, lo = 0;   // rows behind K: 2^120, never the minimum
            if (tid < p.K) {
                // ||c||^2 added up in the order of the other writers of this operand (aug.cuh: one partial per column
                // quad, folded pairwise at distances 16, 8, 4, 2, 1), so that the same centroid gives the same bits
                const uint8_t* crow = smem + c_off + tid * 128;
                float q[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) q[i] = 0.f;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    if (c < p.nchunks) {
#pragma unroll
                        for (int g = 0; g < 8; ++g) {
                            const uint4 w = *reinterpret_cast<const uint4*>(crow + c * C_CHUNK_BYTES + ((g ^ (tid & 7)) << 4));
                            q[c * 16 + 2 * g] = aug::add_squares(0.f, w.x, w.y);
                            q[c * 16 + 2 * g + 1] = aug::add_squares(0.f, w.z, w.w);
                        }
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                    for (int i = 0; i < o; ++i) q[i] = q[i] + q[i + o];
                aug::split3(0.5f * q[0], hi, mid, lo);
            }
            const uint32_t one = 0x3F80u;
            *reinterpret_cast<uint4*>(smem + augb_off + tid * 16) = make_uint4(one | (one << 16), one | (hi << 16), mid | (lo << 16), 0u);
        }
        ptx::fence_proxy_async_smem();
        ptx::tc_fence_before();
        __syncthreads();

        // ---- the CTA's tiles
        if (tid == 0) {
            ptx::tc_fence_after();
            issue_assign(0);
        }
        double dsum = 0.0;
        for (int j = 0; j < nt_mine; ++j) {
            // the next tile's distances meanwhile (its accumulator was read before the barrier that ended tile j - 1)
            if (tid == 0 && j + 1 < nt_mine) {
                ptx::tc_fence_after();
                issue_assign(j + 1);
            }
            const uint32_t acc = static_cast<uint32_t>(j & 1);
            wait_bar(&ctrl->bar_mma[acc], (acc ? ph1 : ph0) & 1u, ctrl, p.status);
            if (acc) ++ph1; else ++ph0;
            ptx::tc_fence_after();
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(warp * 32) << 16) + acc * 128u;
            float best;
            {
                uint32_t ra[32], rb[32], rc[32], rd[32];
                ptx::tmem_ld_x32(taddr, ra);
                if (ng > 1) ptx::tmem_ld_x32(taddr + 32, rb);
                if (ng > 2) ptx::tmem_ld_x32(taddr + 64, rc);
                if (ng > 3) ptx::tmem_ld_x32(taddr + 96, rd);
                ptx::tmem_ld_wait(ra);
                ptx::reg_dep(rb);
                ptx::reg_dep(rc);
                ptx::reg_dep(rd);
                best = packed_min32(ra, 0, __uint_as_float(F32_INF), kmask);
                if (ng > 1) best = packed_min32(rb, 32, best, kmask);
                if (ng > 2) best = packed_min32(rc, 64, best, kmask);
                if (ng > 3) best = packed_min32(rd, 96, best, kmask);
            }
            ptx::tc_fence_before();
            const uint32_t kb = __float_as_uint(best);
            const float bval = __uint_as_float(kb & ~COL_MASK);
            const int bidx = static_cast<int>(kb & COL_MASK);
            const i64 row = (static_cast<i64>(blockIdx.x) + static_cast<i64>(j) * gridDim.x) * BLOCK_M + tid;
            const bool valid = row < p.N;
            if (valid) {
                const float dist = fmaxf(0.f, 2.f * (bval - rowM[j]));   // the accumulator is m + d/2
                p.out_idx[row] = bidx;
                if (p.out_dist) p.out_dist[row] = dist;
                dsum += static_cast<double>(dist);
            }
            // the tile's one-hot operand: element [cluster][row] of a 128 x 128 bf16 tile, K-major with the 128-byte swizzle,
            // two 64-row chunks; the MMAs that read the previous tile's operand must have completed
            if (upd_n > 0u) wait_bar(&ctrl->bar_upd, (upd_n - 1u) & 1u, ctrl, p.status);
            {
                uint8_t* oh = smem + oh_off + (tid >> 6) * X_CHUNK_BYTES + ((tid & 7) << 1);
                const int g8 = (tid & 63) >> 3;
                if (prev_oh >= 0) *reinterpret_cast<uint16_t*>(oh + prev_oh * 128 + ((g8 ^ (prev_oh & 7)) << 4)) = 0;
                const int now = valid ? bidx : -1;
                if (now >= 0) {
                    *reinterpret_cast<uint16_t*>(oh + now * 128 + ((g8 ^ (now & 7)) << 4)) = 0x3F80;
                    atomicAdd(&ctrl->cnt[now], 1);
                }
                prev_oh = now;
            }
            ptx::fence_proxy_async_smem();
            __syncthreads();
            if (tid == 0) {
                // sums (clusters on the lanes, D columns) += onehot^T X: A = one-hot, K-major (the rows of the tile are the
                // contraction); B = the X tile as it lies in shared memory, read MN-major (64-column atoms X_CHUNK_BYTES apart)
                ptx::tc_fence_after();
                const uint32_t a0 = ptx::umma_desc_lo_sw128(smem_base + oh_off);
                const uint32_t b0 = (((smem_base + j * xtile_bytes) & 0x3FFFFu) >> 4) | ((X_CHUNK_BYTES >> 4) << 16);
#pragma unroll
                for (uint32_t ks = 0; ks < BLOCK_M / UMMA_K; ++ks) {
                    const uint32_t a_lo = a0 + (ks >> 2) * (X_CHUNK_BYTES >> 4) + (ks & 3u) * KSTEP;
                    const uint32_t b_lo = b0 + ks * ((UMMA_K * 128u) >> 4);
                    if (ks == 0 && j == 0)
                        ptx::umma_bf16_lohi<false>(tmem_base + SUMS_COL, a_lo, ptx::UMMA_DESC_HI_SW128, b_lo, ptx::UMMA_DESC_HI_SW128, idesc_upd);
                    else
                        ptx::umma_bf16_lohi<true>(tmem_base + SUMS_COL, a_lo, ptx::UMMA_DESC_HI_SW128, b_lo, ptx::UMMA_DESC_HI_SW128, idesc_upd);
                }
                ptx::umma_commit(ptx::smem_u32(&ctrl->bar_upd));
            }
            ++upd_n;
        }

        // ---- this CTA's partial sums (thread = cluster) and counts, and its share of the inertia
        wait_bar(&ctrl->bar_upd, (upd_n - 1u) & 1u, ctrl, p.status);
        ptx::tc_fence_after();
        {
            float* dst = p.part_sums + (static_cast<size_t>(blockIdx.x) * 128 + tid) * p.ncol;
            for (int c0 = 0; c0 < p.ncol; c0 += 16) {
                uint32_t v[16];
                ptx::tmem_ld_x16(tmem_base + (static_cast<uint32_t>(warp * 32) << 16) + SUMS_COL + c0, v);
#pragma unroll
                for (int q = 0; q < 16; q += 4) *reinterpret_cast<uint4*>(dst + c0 + q) = make_uint4(v[q], v[q + 1], v[q + 2], v[q + 3]);
            }
            p.part_counts[static_cast<size_t>(blockIdx.x) * 128 + tid] = ctrl->cnt[tid];
        }
        ptx::tc_fence_before();
        if (p.inertia) {   // one fp64 atomic per CTA and iteration
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, o);
            if (lane == 0) ctrl->dred[warp] = dsum;
            __syncthreads();
            if (tid == 0) atomicAdd(p.inertia + it, (ctrl->dred[0] + ctrl->dred[1]) + (ctrl->dred[2] + ctrl->dred[3]));
        }
        grid_barrier(p.gbar, gb++, ctrl, p.status);

        // ---- division: cluster k by CTA k mod grid.  Thread = (stripe of partials, column quad), the threads behind the
        // last whole stripe idle; the first warp adds the stripes up, divides (an empty cluster keeps its previous centroid) and writes fp32 and bf16 (RNE) centroids.
        const int D4 = p.D >> 2, stripes = THREADS / D4;
        const int n_part = static_cast<int>(gridDim.x);
        for (int k = blockIdx.x; k < p.K; k += gridDim.x) {
            const int col = tid % D4, stripe = tid / D4;
            // (all loads of a stripe are requested before the first is added: the loop is a chain of L2 latencies otherwise)
            // (the counts are requested first: their loads are in flight together with the sums')
            int cn0 = tid < n_part ? __ldcg(p.part_counts + static_cast<size_t>(tid) * 128 + k) : 0;
            int cn1 = tid + THREADS < n_part ? __ldcg(p.part_counts + static_cast<size_t>(tid + THREADS) * 128 + k) : 0;
            float4 acc4 = make_float4(0.f, 0.f, 0.f, 0.f);
            const float4* prow = reinterpret_cast<const float4*>(p.part_sums + static_cast<size_t>(k) * p.ncol) + col;
            const size_t pstep = static_cast<size_t>(128) * p.ncol / 4;
            constexpr int BATCH = 20;   // (148 partials over 8 stripes: one batch)
            for (int q0 = stripe; stripe < stripes && q0 < n_part; q0 += BATCH * stripes) {
                float4 v[BATCH];
#pragma unroll
                for (int u = 0; u < BATCH; ++u) {
                    const int q = q0 + u * stripes;
                    v[u] = q < n_part ? __ldcg(prow + static_cast<size_t>(q) * pstep) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int u = 0; u < BATCH; ++u) { acc4.x += v[u].x; acc4.y += v[u].y; acc4.z += v[u].z; acc4.w += v[u].w; }
            }
            int cn = cn0 + cn1;
            for (int q = tid + 2 * THREADS; q < n_part; q += THREADS) cn += __ldcg(p.part_counts + static_cast<size_t>(q) * 128 + k);
            ctrl->red[tid] = acc4;
            ctrl->cred[tid] = cn;
            __syncthreads();
            if (warp == 0) {
                int n = ctrl->cred[lane] + ctrl->cred[lane + 32] + ctrl->cred[lane + 64] + ctrl->cred[lane + 96];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) n += __shfl_xor_sync(0xffffffffu, n, o);
                if (lane == 0) p.out_counts[k] = n;
                if (lane < D4) {
                    float4 sv = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (int sidx = 0; sidx < stripes; ++sidx) {
                        const float4 v = ctrl->red[sidx * D4 + lane];
                        sv.x += v.x; sv.y += v.y; sv.z += v.z; sv.w += v.w;
                    }
                    const size_t e = static_cast<size_t>(k) * D4 + lane;
                    float4 v;
                    if (n > 0) {
                        const float fn = static_cast<float>(n);
                        v = make_float4(sv.x / fn, sv.y / fn, sv.z / fn, sv.w / fn);
                    } else {
                        const uint2 pv = __ldcg(reinterpret_cast<const uint2*>(src) + e);
                        v = make_float4(bf16lo(pv.x), bf16hi(pv.x), bf16lo(pv.y), bf16hi(pv.y));
                    }
                    uint2 o;
                    o.x = f32_to_bf16_rne(v.x) | (f32_to_bf16_rne(v.y) << 16);
                    o.y = f32_to_bf16_rne(v.z) | (f32_to_bf16_rne(v.w) << 16);
                    if (p.out_C) reinterpret_cast<float4*>(p.out_C)[e] = v;
                    reinterpret_cast<uint2*>(p.cbuf)[e] = o;
                    if (p.out_C_bf16) reinterpret_cast<uint2*>(p.out_C_bf16)[e] = o;
                }
            }
            __syncthreads();
        }
        if (it + 1 < p.iters) grid_barrier(p.gbar, gb++, ctrl, p.status);
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace

// ======================================================================= host side
namespace {
size_t small_smem_bytes(int R, int nchunks) {
    const size_t x = static_cast<size_t>(R) * nchunks * X_CHUNK_BYTES;
    const size_t rest = static_cast<size_t>(nchunks) * C_CHUNK_BYTES + static_cast<size_t>(R) * AUG_BYTES + AUG_BYTES + ZERO_BYTES;
    return 1024 + ((x + rest + 1023) & ~static_cast<size_t>(1023)) + OH_BYTES + 4096;
}
}  // namespace

// One problem of at most 128 clusters, D <= 128 (a multiple of 8), whose row tiles fit four to an SM.
bool lloyd_small_supports(const DeviceInfo& di, i64 N, int D, int K) {
    if (di.cc_major != 10 || N < 1 || K < 1 || K > 128 || D < 8 || D > 128 || D % 8 != 0) return false;
    const i64 tiles = (N + BLOCK_M - 1) / BLOCK_M;
    if (tiles > static_cast<i64>(MAX_R) * di.sm_count) return false;
    const int grid = static_cast<int>(tiles < di.sm_count ? tiles : di.sm_count);
    const int R = static_cast<int>((tiles + grid - 1) / grid);
    return small_smem_bytes(R, (D + KCHUNK - 1) / KCHUNK) <= static_cast<size_t>(di.smem_optin);
}

// part_sums [grid][128][round_up(D, 16)] fp32, part_counts [grid][128] int, cbuf [K][D] bf16 and gbar (one word) are scratch; inertia
// (nullable) has one entry per iteration.  Everything is enqueued on `s`: two small clears and one cooperative launch.
int launch_lloyd_small(const cake_bf16* X, const cake_bf16* C0, i64 N, int D, int K, int iters, float* part_sums,
                       int* part_counts, cake_bf16* cbuf, unsigned* gbar, float* out_C, cake_bf16* out_C_bf16, int* out_idx,
                       float* out_dist, int* out_counts, double* inertia, int* status, const DeviceInfo& di, cudaStream_t s) {
    if (!lloyd_small_supports(di, N, D, K) || iters < 1) return CAKE_ERR_UNSUPPORTED;
    Params p;
    p.C0 = C0; p.N = N; p.D = D; p.K = K; p.iters = iters;
    p.nchunks = (D + KCHUNK - 1) / KCHUNK;
    p.ncol = static_cast<int>(round_up(D, 16));
    p.c_rows = static_cast<int>(round_up(K, 32));
    p.tiles = static_cast<int>((N + BLOCK_M - 1) / BLOCK_M);
    p.part_sums = part_sums; p.part_counts = part_counts; p.cbuf = cbuf;
    p.out_C = out_C; p.out_C_bf16 = out_C_bf16; p.out_idx = out_idx; p.out_dist = out_dist; p.out_counts = out_counts;
    p.inertia = inertia; p.gbar = gbar; p.status = status;
    const int grid = p.tiles < di.sm_count ? p.tiles : di.sm_count;
    const int R = (p.tiles + grid - 1) / grid;
    const size_t smem = small_smem_bytes(R, p.nchunks);
    CUtensorMap tx;
    int rc = make_tmap_bf16_rows(&tx, X, D, N, 1, BLOCK_M);
    if (rc != CAKE_OK) return rc;
    static bool attr_done[64] = {false};   // per device; benign race: the attribute call is idempotent
    const bool known = di.device >= 0 && di.device < 64;
    if (!known || !attr_done[di.device]) {
        if (cudaFuncSetAttribute(lloyd_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess)
            return CAKE_ERR_CUDA;
        if (known) attr_done[di.device] = true;
    }
    // every host-side check has passed: from here on work is enqueued
    if (cudaMemsetAsync(gbar, 0, sizeof(unsigned), s) != cudaSuccess) return CAKE_ERR_CUDA;
    if (inertia && cudaMemsetAsync(inertia, 0, static_cast<size_t>(iters) * sizeof(double), s) != cudaSuccess) return CAKE_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeCooperative;   // all CTAs resident at once: they meet at grid barriers
    at[0].val.cooperative = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, lloyd_small_kernel, tx, p) != cudaSuccess) {
        cudaGetLastError();
        return CAKE_ERR_CUDA;
    }
    note_launches(1);
    return CAKE_OK;
}

}  // namespace cake
