// Fused nearest-centroid assignment on the sm_100a tensor cores.
//
// Operation (paper Section 5, "Flash-KMeans clean-start workload"): for every point the squared
// Euclidean distance to all K centroids and the arg-min.  Evaluated as
//     argmin_k ( ||c_k||^2 - 2 x.c_k ),   dist = max(0, ||x||^2 + min_k(...)),
// with S = X.C^T produced tile by tile in tensor memory and consumed on the spot, so the N x K
// matrix never exists in HBM.
//
// One persistent CTA per SM, 10 warps, three roles:
//   warp 8  producer : TMA loads.  A 128-row X tile (whole D) into one of the X buffers, then the
//                      centroid tiles of 256 rows, 64 columns (128 bytes, 128B-swizzled) at a time
//                      through an mbarrier ring.
//   warp 9  MMA      : one thread issues tcgen05.mma (M=128, N=256, K=16, bf16 -> fp32) into one
//                      of two 256-column TMEM accumulators; tcgen05.commit releases ring slots and
//                      publishes finished accumulators.
//   warps 0-7 epilogue: warp w reads TMEM lanes 32*(w%4).. (one X row per thread) and columns
//                      128*(w/4).. of the tile with tcgen05.ld, forms ||c||^2 - 2s, keeps a running
//                      (best, index) per row across all centroid tiles; the two column halves are
//                      merged through shared memory at the end of the row tile.
// Every wait is bounded: on expiry the CTA raises CAKE_ERR_TIMEOUT in the status word, all roles
// leave their loops, TMEM is freed and the kernel returns.
#include "internal.h"
#include "ptx.cuh"

namespace cake {
namespace {

constexpr int BLOCK_M = 128;
constexpr int BLOCK_N = kAssignBlockN;  // 256
constexpr int KCHUNK = 64;              // bf16 columns per swizzled 128-byte row
constexpr int UMMA_K = 16;
constexpr int NUM_EPI_WARPS = 8;
constexpr int PRODUCER_WARP = 8;
constexpr int MMA_WARP = 9;
constexpr int NUM_THREADS = 320;
constexpr uint32_t X_CHUNK_BYTES = BLOCK_M * 128;  // 16 KiB
constexpr uint32_t C_STAGE_BYTES = BLOCK_N * 128;  // 32 KiB
constexpr int MAX_STAGES = 6;
constexpr int TMEM_COLS = 512;
constexpr uint32_t CTRL_BYTES = 4096;  // barriers, TMEM pointer, abort flag, merge scratch
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;

struct Params {
    int B;
    i64 N;
    int D, K;
    int nchunks;      // ceil(D / 64)
    int ksteps_last;  // UMMA k-steps in the last chunk
    int m_tiles;      // ceil(N / 128)
    int n_tiles;      // ceil(K / 256)
    i64 total_tiles;  // B * m_tiles
    int n_stages;     // ring depth
    int n_xbuf;       // 1 or 2 X buffers
    int Kpad;
    const float* cn;  // [B][Kpad]
    int* out_idx;
    float* out_dist;
    int* status;
};

struct Ctrl {  // lives in shared memory
    uint64_t x_full[2], x_empty[2];
    uint64_t ring_full[MAX_STAGES], ring_empty[MAX_STAGES];
    uint64_t tmem_full[2], tmem_empty[2];
    uint64_t merge_full[2], merge_empty[2];
    uint32_t tmem_base;
    int abort_flag;
    float merge_best[2][BLOCK_M];
    int merge_idx[2][BLOCK_M];
};
static_assert(sizeof(Ctrl) <= CTRL_BYTES, "control block too large");

// Bounded wait on an mbarrier phase. Returns false if the CTA is aborting.
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, Ctrl* ctrl, int* status) {
    const uint32_t addr = ptx::smem_u32(bar);
    if (ptx::mbar_try_wait(addr, parity)) return true;
    const uint64_t t0 = ptx::globaltimer_ns();
    for (uint32_t it = 1;; ++it) {
        if (ptx::mbar_try_wait(addr, parity)) return true;
        if ((it & 63u) == 0) {
            if (*reinterpret_cast<volatile int*>(&ctrl->abort_flag)) return false;
            if (ptx::globaltimer_ns() - t0 > WAIT_LIMIT_NS) {
                *reinterpret_cast<volatile int*>(&ctrl->abort_flag) = 1;
                atomicCAS(status, CAKE_OK, CAKE_ERR_TIMEOUT);
                return false;
            }
        }
    }
}

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// One group of 32 accumulator columns of this thread's row: v_j = cn_j - 2 s_j, chunk minimum by a
// min tree, and only if it beats the running best is the position looked up (first match, so the
// lowest column wins exact ties; later tiles need a strictly smaller value).
__device__ __forceinline__ void scan32(const uint32_t (&r)[32], const float4* __restrict__ cn4,
                                       int col_base, float& best, int& bidx) {
    float v[32];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const float4 c = __ldg(cn4 + q);
        v[4 * q + 0] = fmaf(-2.f, __uint_as_float(r[4 * q + 0]), c.x);
        v[4 * q + 1] = fmaf(-2.f, __uint_as_float(r[4 * q + 1]), c.y);
        v[4 * q + 2] = fmaf(-2.f, __uint_as_float(r[4 * q + 2]), c.z);
        v[4 * q + 3] = fmaf(-2.f, __uint_as_float(r[4 * q + 3]), c.w);
    }
    float t[11];
#pragma unroll
    for (int q = 0; q < 10; ++q) t[q] = ptx::fmin3(v[3 * q], v[3 * q + 1], v[3 * q + 2]);
    t[10] = fminf(v[30], v[31]);
    const float u0 = ptx::fmin3(t[0], t[1], t[2]);
    const float u1 = ptx::fmin3(t[3], t[4], t[5]);
    const float u2 = ptx::fmin3(t[6], t[7], t[8]);
    const float u3 = fminf(t[9], t[10]);
    const float m = fminf(ptx::fmin3(u0, u1, u2), u3);
    if (m < best) {
        best = m;
        int loc = 31;
#pragma unroll
        for (int j = 30; j >= 0; --j)
            if (v[j] == m) loc = j;
        bidx = col_base + loc;
    }
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
assign_tc_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_c,
                 const Params p) {
    extern __shared__ uint8_t smem_raw[];
    // 128B-swizzled tiles need 1024-byte alignment
    const uint32_t raw_addr = ptx::smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    uint8_t* smem = smem_raw + pad;
    const uint32_t smem_base = raw_addr + pad;
    const uint32_t xbuf_bytes = static_cast<uint32_t>(p.nchunks) * X_CHUNK_BYTES;
    const uint32_t x_base = smem_base;
    const uint32_t ring_base = x_base + static_cast<uint32_t>(p.n_xbuf) * xbuf_bytes;
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem + static_cast<size_t>(p.n_xbuf) * xbuf_bytes +
                                         static_cast<size_t>(p.n_stages) * C_STAGE_BYTES);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(ptx::smem_u32(&ctrl->x_full[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctrl->x_empty[i]), 1 + 4);  // MMA commit + 4 norm warps
            ptx::mbar_init(ptx::smem_u32(&ctrl->tmem_full[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctrl->tmem_empty[i]), NUM_EPI_WARPS);
            ptx::mbar_init(ptx::smem_u32(&ctrl->merge_full[i]), 4);
            ptx::mbar_init(ptx::smem_u32(&ctrl->merge_empty[i]), 4);
        }
        for (int i = 0; i < MAX_STAGES; ++i) {
            ptx::mbar_init(ptx::smem_u32(&ctrl->ring_full[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctrl->ring_empty[i]), 1);
        }
        ctrl->abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == MMA_WARP) {
        ptx::tmem_alloc(ptx::smem_u32(&ctrl->tmem_base), TMEM_COLS);
        ptx::tmem_relinquish();
    }
    if (warp == PRODUCER_WARP && lane == 0) {
        ptx::prefetch_tensormap(&tmap_x);
        ptx::prefetch_tensormap(&tmap_c);
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&ctrl->tmem_base);

    if (warp == PRODUCER_WARP) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t ring_it = 0, tile_it = 0;
            bool ok = true;
            for (i64 tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x, ++tile_it) {
                const int b = static_cast<int>(tile / p.m_tiles);
                const int mt = static_cast<int>(tile % p.m_tiles);
                const uint32_t xb = tile_it % p.n_xbuf, xph = (tile_it / p.n_xbuf) & 1u;
                ok = wait_bar(&ctrl->x_empty[xb], xph ^ 1u, ctrl, p.status);
                if (!ok) break;
                const uint32_t xfull = ptx::smem_u32(&ctrl->x_full[xb]);
                ptx::mbar_arrive_expect_tx(xfull, xbuf_bytes);
                for (int c = 0; c < p.nchunks; ++c)
                    ptx::tma_load_3d(x_base + xb * xbuf_bytes + c * X_CHUNK_BYTES, &tmap_x, xfull,
                                     c * KCHUNK, mt * BLOCK_M, b);
                for (int nt = 0; ok && nt < p.n_tiles; ++nt) {
                    for (int c = 0; c < p.nchunks; ++c, ++ring_it) {
                        const uint32_t s = ring_it % p.n_stages, ph = (ring_it / p.n_stages) & 1u;
                        ok = wait_bar(&ctrl->ring_empty[s], ph ^ 1u, ctrl, p.status);
                        if (!ok) break;
                        const uint32_t full = ptx::smem_u32(&ctrl->ring_full[s]);
                        ptx::mbar_arrive_expect_tx(full, C_STAGE_BYTES);
                        ptx::tma_load_3d(ring_base + s * C_STAGE_BYTES, &tmap_c, full, c * KCHUNK,
                                         nt * BLOCK_N, b);
                    }
                }
            }
            if (!ok) {
                // aborting: give our loads in flight a bounded time to land before the CTA's
                // shared memory is given up
                const uint64_t t0 = ptx::globaltimer_ns();
                const uint32_t pending = ring_it < static_cast<uint32_t>(p.n_stages)
                                             ? ring_it : static_cast<uint32_t>(p.n_stages);
                for (uint32_t k = 1; k <= pending; ++k) {
                    const uint32_t it_s = ring_it - k;
                    const uint32_t st = it_s % p.n_stages, ph = (it_s / p.n_stages) & 1u;
                    while (!ptx::mbar_try_wait(ptx::smem_u32(&ctrl->ring_full[st]), ph) &&
                           ptx::globaltimer_ns() - t0 < 100000000ull) {
                    }
                }
            }
        }
    } else if (warp == MMA_WARP) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::umma_idesc_bf16(BLOCK_M, BLOCK_N);
            uint32_t ring_it = 0, tile_it = 0, acc_it = 0;
            bool ok = true;
            for (i64 tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x, ++tile_it) {
                const uint32_t xb = tile_it % p.n_xbuf, xph = (tile_it / p.n_xbuf) & 1u;
                ok = wait_bar(&ctrl->x_full[xb], xph, ctrl, p.status);
                if (!ok) break;
                ptx::tc_fence_after();
                for (int nt = 0; ok && nt < p.n_tiles; ++nt, ++acc_it) {
                    const uint32_t as = acc_it & 1u, aph = (acc_it >> 1) & 1u;
                    ok = wait_bar(&ctrl->tmem_empty[as], aph ^ 1u, ctrl, p.status);
                    if (!ok) break;
                    ptx::tc_fence_after();
                    const uint32_t d_tmem = tmem_base + as * BLOCK_N;
                    for (int c = 0; c < p.nchunks; ++c, ++ring_it) {
                        const uint32_t s = ring_it % p.n_stages, ph = (ring_it / p.n_stages) & 1u;
                        ok = wait_bar(&ctrl->ring_full[s], ph, ctrl, p.status);
                        if (!ok) break;
                        ptx::tc_fence_after();
                        const uint32_t a_addr = x_base + xb * xbuf_bytes + c * X_CHUNK_BYTES;
                        const uint32_t b_addr = ring_base + s * C_STAGE_BYTES;
                        const int nk = (c == p.nchunks - 1) ? p.ksteps_last : KCHUNK / UMMA_K;
                        for (int ks = 0; ks < nk; ++ks) {
                            ptx::umma_bf16(d_tmem, ptx::umma_desc_sw128(a_addr + ks * UMMA_K * 2),
                                           ptx::umma_desc_sw128(b_addr + ks * UMMA_K * 2), idesc,
                                           (c | ks) != 0 ? 1u : 0u);
                        }
                        ptx::umma_commit(ptx::smem_u32(&ctrl->ring_empty[s]));
                    }
                    if (ok) ptx::umma_commit(ptx::smem_u32(&ctrl->tmem_full[as]));
                }
                if (ok) ptx::umma_commit(ptx::smem_u32(&ctrl->x_empty[xb]));
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        const int wg = warp >> 2;            // column half of every tile
        const int q = warp & 3;              // TMEM lane quarter this warp may read
        const int r = q * 32 + lane;         // row inside the X tile
        uint32_t tile_it = 0, acc_it = 0;
        bool ok = true;
        for (i64 tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x, ++tile_it) {
            const int b = static_cast<int>(tile / p.m_tiles);
            const int mt = static_cast<int>(tile % p.m_tiles);
            const uint32_t xb = tile_it % p.n_xbuf, xph = (tile_it / p.n_xbuf) & 1u;
            float xn = 0.f;
            if (wg == 0) {
                // ||x||^2 of this thread's row from the swizzled X tile (16-byte granule g of row r
                // sits at position g ^ (r & 7); the order of the granules does not matter for a sum)
                ok = wait_bar(&ctrl->x_full[xb], xph, ctrl, p.status);
                if (!ok) break;
                const uint8_t* xrow = smem + xb * xbuf_bytes + r * 128;
                for (int c = 0; c < p.nchunks; ++c) {
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        const uint4 w = *reinterpret_cast<const uint4*>(xrow + c * X_CHUNK_BYTES +
                                                                        ((g ^ (r & 7)) << 4));
                        float a;
                        a = bf16lo(w.x); xn = fmaf(a, a, xn); a = bf16hi(w.x); xn = fmaf(a, a, xn);
                        a = bf16lo(w.y); xn = fmaf(a, a, xn); a = bf16hi(w.y); xn = fmaf(a, a, xn);
                        a = bf16lo(w.z); xn = fmaf(a, a, xn); a = bf16hi(w.z); xn = fmaf(a, a, xn);
                        a = bf16lo(w.w); xn = fmaf(a, a, xn); a = bf16hi(w.w); xn = fmaf(a, a, xn);
                    }
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->x_empty[xb]));
            }
            float best = __int_as_float(0x7f800000);
            int bidx = 0;
            const float* cn_b = p.cn + static_cast<size_t>(b) * p.Kpad + wg * (BLOCK_N / 2);
            for (int nt = 0; nt < p.n_tiles; ++nt, ++acc_it) {
                const uint32_t as = acc_it & 1u, aph = (acc_it >> 1) & 1u;
                ok = wait_bar(&ctrl->tmem_full[as], aph, ctrl, p.status);
                if (!ok) break;
                ptx::tc_fence_after();
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                       as * BLOCK_N + wg * (BLOCK_N / 2);
                const int col0 = nt * BLOCK_N + wg * (BLOCK_N / 2);
                const float4* cn4 = reinterpret_cast<const float4*>(cn_b + nt * BLOCK_N);
#pragma unroll 1
                for (int h = 0; h < 2; ++h) {
                    uint32_t r0[32], r1[32];
                    ptx::tmem_ld_x32(taddr + h * 64, r0);
                    ptx::tmem_ld_x32(taddr + h * 64 + 32, r1);
                    ptx::tmem_ld_wait(r0);
                    ptx::reg_dep(r1);
                    scan32(r0, cn4 + h * 16, col0 + h * 64, best, bidx);
                    scan32(r1, cn4 + h * 16 + 8, col0 + h * 64 + 32, best, bidx);
                }
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->tmem_empty[as]));
            }
            if (!ok) break;
            // merge the two column halves: the upper half hands its (best, index) to the lower one
            const uint32_t mb = tile_it & 1u, mph = (tile_it >> 1) & 1u;
            if (wg == 1) {
                ok = wait_bar(&ctrl->merge_empty[mb], mph ^ 1u, ctrl, p.status);
                if (!ok) break;
                ctrl->merge_best[mb][r] = best;
                ctrl->merge_idx[mb][r] = bidx;
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->merge_full[mb]));
            } else {
                ok = wait_bar(&ctrl->merge_full[mb], mph, ctrl, p.status);
                if (!ok) break;
                const float ob = ctrl->merge_best[mb][r];
                const int oi = ctrl->merge_idx[mb][r];
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->merge_empty[mb]));
                if (ob < best || (ob == best && oi < bidx)) {
                    best = ob;
                    bidx = oi;
                }
                const i64 row = static_cast<i64>(mt) * BLOCK_M + r;
                if (row < p.N) {
                    const size_t o = static_cast<size_t>(b) * static_cast<size_t>(p.N) + row;
                    p.out_idx[o] = bidx;
                    if (p.out_dist) p.out_dist[o] = fmaxf(0.f, xn + best);
                }
            }
        }
    }

    // ---------------------------------------------------------------- teardown
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == MMA_WARP) {
        __syncwarp();
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link-time libcuda dependency)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            f = nullptr;
        return reinterpret_cast<EncodeTiledFn>(f);
    }();
    return fn;
}

// bf16 tensor [batch][rows][D] viewed as (D, rows, batch); box = 64 columns x box_rows rows.
int make_tmap(CUtensorMap* m, const void* base, int D, i64 rows, int batch, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return CAKE_ERR_CUDA;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(rows),
                          static_cast<cuuint64_t>(batch)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(D) * 2,
                             static_cast<cuuint64_t>(D) * 2 * static_cast<cuuint64_t>(rows)};
    cuuint32_t box[3] = {KCHUNK, static_cast<cuuint32_t>(box_rows), 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box,
                    estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? CAKE_OK : CAKE_ERR_CUDA;
}

}  // namespace

bool assign_tc_supports(int D) { return D >= 8 && D % 8 == 0 && D <= 256; }

int launch_assign_tc(const cake_bf16* X, const cake_bf16* C, int B, i64 N, int D, int K, const float* cn,
                     int Kpad, int* out_idx, float* out_dist, int* status, cudaStream_t s) {
    if (!assign_tc_supports(D)) return CAKE_ERR_UNSUPPORTED;
    DeviceInfo di;
    int rc = current_device_info(&di);
    if (rc != CAKE_OK) return rc;
    if (di.cc_major != 10) return CAKE_ERR_DEVICE;

    Params p;
    p.B = B; p.N = N; p.D = D; p.K = K;
    p.nchunks = (D + KCHUNK - 1) / KCHUNK;
    p.ksteps_last = (D - (p.nchunks - 1) * KCHUNK + UMMA_K - 1) / UMMA_K;
    p.m_tiles = static_cast<int>((N + BLOCK_M - 1) / BLOCK_M);
    p.n_tiles = (K + BLOCK_N - 1) / BLOCK_N;
    p.total_tiles = static_cast<i64>(B) * p.m_tiles;
    p.Kpad = Kpad; p.cn = cn; p.out_idx = out_idx; p.out_dist = out_dist; p.status = status;
    if (p.total_tiles == 0) return CAKE_OK;

    const i64 budget = static_cast<i64>(di.smem_optin) - 1024 - CTRL_BYTES;
    const i64 xbuf = static_cast<i64>(p.nchunks) * X_CHUNK_BYTES;
    p.n_xbuf = 2;
    i64 stages = (budget - 2 * xbuf) / C_STAGE_BYTES;
    if (stages < 3 || (p.nchunks >= 4 && p.n_tiles >= 8)) {
        p.n_xbuf = 1;
        stages = (budget - xbuf) / C_STAGE_BYTES;
    }
    if (stages < 2) return CAKE_ERR_UNSUPPORTED;
    p.n_stages = static_cast<int>(stages > MAX_STAGES ? MAX_STAGES : stages);
    const size_t smem_bytes = 1024 + static_cast<size_t>(p.n_xbuf) * xbuf +
                              static_cast<size_t>(p.n_stages) * C_STAGE_BYTES + CTRL_BYTES;

    CUtensorMap tx, tc;
    rc = make_tmap(&tx, X, D, N, B, BLOCK_M);
    if (rc != CAKE_OK) return rc;
    rc = make_tmap(&tc, C, D, K, B, BLOCK_N);
    if (rc != CAKE_OK) return rc;

    static int attr_done_for_device = -1;  // benign race: the attribute call is idempotent
    if (attr_done_for_device != di.device) {
        if (cudaFuncSetAttribute(assign_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 di.smem_optin) != cudaSuccess)
            return CAKE_ERR_CUDA;
        attr_done_for_device = di.device;
    }
    const i64 grid = p.total_tiles < di.sm_count ? p.total_tiles : di.sm_count;
    assign_tc_kernel<<<static_cast<unsigned>(grid), NUM_THREADS, smem_bytes, s>>>(tx, tc, p);
    note_launches(1);
    return cudaGetLastError() == cudaSuccess ? CAKE_OK : CAKE_ERR_CUDA;
}

}  // namespace cake
