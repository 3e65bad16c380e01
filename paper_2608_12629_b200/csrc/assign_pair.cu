// Fused nearest-centroid assignment on the sm_100a tensor cores, CTA-pair version: an alternative to assign_tc.cu
// that the caller selects (flags = CAKE_ASSIGN_TCGEN05_PAIR); the default route stays the single-CTA kernel.
//
// Same operation, same arithmetic, same epilogue and bit-identical results as assign_tc.cu (paper Section 5,
// "Flash-KMeans clean-start workload"; see that file for the accumulators m + d/2 and the packed keys).  What
// differs is how the tensor cores are fed.  Two CTAs of a thread-block cluster share every tile:
// tcgen05.mma.cta_group::2 with M = 256, N = 256.  A pair owns 256 consecutive rows of X (128 per CTA); of every
// 256-centroid tile each CTA loads only ITS 128 rows (16 KiB per 64-column chunk instead of 32).  Per MMA a CTA's
// shared memory then serves 4 KiB of X and 4 KiB of centroids where the single-CTA kernel serves 4 + 8 KiB, and
// one issuing thread's instruction feeds two tensor cores.
//
// Measured (B200, N = 1M): the issuing threads of rank 0 wait for a free accumulator about half of the time; the
// tile time is set by the epilogue, whose 1.5 ALU-pipe instructions per distance (key + 3-input minimum) take
// about as long as the tile's MMAs at D = 128.  So the pair ties the single-CTA kernel at D = 128, K = 1024
// (0.248 against 0.250 ms) and stays 2-25 % behind it elsewhere (D = 128 K = 4096: 0.866 against 0.853 ms;
// D = 256 K = 4096: 1.23 against 0.89 ms, where only one X buffer fits).  Three things were worth 40 % on the
// way: arrivals on the other CTA's barriers with CTA-scope release (a cluster-scope release cost about 1,100
// clocks each), one sub-ring of stages per issuer (no passing over other issuers' slots), a whole centroid tile
// per stage (one wait and one commit per tile).
//
// Roles per CTA (16 warps, as in the single-CTA kernel):
//   warp 8  producer : its own X tile (plain TMA, own barrier) and its half of every centroid chunk,
//                      plus its half of the tile's half-norm operand with the last chunk; the byte
//                      counts of both CTAs go to rank 0's barrier, which alone is waited on.  No multicast loads.
//   warps 9-11 MMA   : rank 0 only; tiles round robin, each issuer with its own stages of the ring; commits are
//                      multicast to both CTAs.
//   warps 12-15 norms: own rows; they tell their own epilogue (local barrier) and rank 0's issuers.
//   warps 0-7 epilogue: own rows out of the CTA's own tensor memory; accumulators are released to
//                      rank 0's issuers by both CTAs.
// Every wait inside the tile loops is bounded as in the single-CTA kernel; the two cluster-wide
// barriers (after set-up, before the tensor memory is freed) are reached by every thread on every
// path, also after a time-out.
#include "aug.cuh"
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
constexpr int MMA_WARP = 9;             // warps 9, 10 and 11: the MMA issuers
constexpr int NUM_ISSUERS = 3;
constexpr int AUX_WARP0 = 12;           // warps 12..15: row norms
constexpr int NUM_WARPS = 16;
constexpr int EPI_REGS = 192;           // registers per thread after reallocation: epilogue warpgroups
constexpr int AUX_REGS = 56;            // ... and the producer / MMA / norm warpgroups
constexpr int NUM_THREADS = NUM_WARPS * 32;
constexpr uint32_t X_CHUNK_BYTES = BLOCK_M * 128;        // 16 KiB
constexpr uint32_t C_HALF_BYTES = (BLOCK_N / 2) * 128;   // 16 KiB: this CTA's 128 rows of a centroid chunk
constexpr uint32_t AUG_B_HALF = (BLOCK_N / 2) * 16;      // 2 KiB: its rows of the half-norm operand
// a ring stage holds `cps` chunks and, behind them, room for the operand
// Operands of the extra k-step: only columns 0..7 are non-zero, so each buffer holds just those
// (one 16-byte row per X row / centroid) and every descriptor points its second 8-column core
// matrices at one shared block of zeros.
constexpr uint32_t AUG_A_BYTES = BLOCK_M * 16;           // 2 KiB
constexpr uint32_t AUG_ZERO_BYTES = BLOCK_N * 16;        // 4 KiB of zeros
constexpr int MAX_STAGES = 12;
constexpr int MAX_XBUF = 4;
constexpr int TMEM_COLS = 512;
constexpr uint32_t CTRL_BYTES = 6144;  // barriers, TMEM pointer, abort flag, merge scratch, row exponents
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;
constexpr uint32_t WAIT_SLICE_NS = 20000;   // longest single sleep inside a wait
constexpr uint32_t COL_MASK = 0x7Fu;   // packed policy: 7 bits address the 128 columns of a half tile
constexpr uint32_t F32_INF = 0x7f800000u;

struct Params {
    int B;
    i64 N;
    int D, K;
    int nchunks;      // ceil(D / 64)
    int ksteps_last;  // UMMA k-steps in the last chunk
    int m_tiles;      // ceil(N / 256): row tiles of a CTA pair
    int n_tiles;      // ceil(K / 256)
    i64 total_tiles;  // B * m_tiles
    int Kpad;         // K rounded up to 256
    int n_stages;     // ring depth: NUM_ISSUERS sub-rings of `spi` stages, one sub-ring per issuer
    int spi;          // stages per issuer
    int cps;          // 64-column chunks per stage
    int n_xbuf;       // 1 or 2 X buffers
    int* out_idx;
    float* out_dist;
    const float* row_m;   // wide mode: every row's margin m, [B][Npad]
    i64 Npad;             // ... rows per problem there (N rounded up to a multiple of 256)
    double* inertia;      // optional: inertia[b * inertia_stride] += sum of the problem's distances
    int inertia_stride;
    int* status;
};

struct Ctrl {  // lives in shared memory
    uint64_t x_full[MAX_XBUF], x_empty[MAX_XBUF];
    uint64_t ring_full[MAX_STAGES], ring_empty[MAX_STAGES];
    uint64_t tmem_full[2];
    // release of accumulator a, one barrier per issuer that may take it next: each barrier has a
    // single waiter that sees every one of its phases
    uint64_t tmem_empty[2][NUM_ISSUERS];
    uint64_t auga_full[MAX_XBUF];    // rank 0: the X-side operands of both CTAs are written (8 warps)
    uint64_t auga_local[MAX_XBUF];   // this CTA's row exponents are written (4 warps)
    uint64_t merge_full[2], merge_empty[2];
    uint32_t tmem_base;
    int abort_flag;
    float merge_best[2][BLOCK_M];
    int merge_idx[2][BLOCK_M];
    float row_m[MAX_XBUF][BLOCK_M];   // each row's margin m
#ifdef CAKE_ASSIGN_TRACE
    int trace_n[NUM_WARPS];
#endif
};
static_assert(sizeof(Ctrl) <= CTRL_BYTES, "control block too large");

#ifdef CAKE_ASSIGN_TRACE
// Profiling build only (-DCAKE_ASSIGN_TRACE): CTA 0 logs every barrier wait of its warp leaders as
// {barrier slot in Ctrl, start clock, end clock} per warp; read back with cake_debug_read_trace.
constexpr int TRACE_CAP = 4096;   // records per warp
__device__ long long g_trace[NUM_WARPS * TRACE_CAP * 3];
__device__ __forceinline__ bool wait_bar_impl(uint64_t* bar, uint32_t parity, Ctrl* ctrl, int* status);
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, Ctrl* ctrl, int* status) {
    const bool log = blockIdx.x == 0 && (threadIdx.x & 31) == 0;
    const long long t0 = clock64();
    const bool ok = wait_bar_impl(bar, parity, ctrl, status);
    const long long t1 = clock64();
    if (log) {
        const int w = threadIdx.x >> 5;
        const int n = ctrl->trace_n[w]++;
        if (n < TRACE_CAP) {
            long long* r = g_trace + (static_cast<size_t>(w) * TRACE_CAP + n) * 3;
            r[0] = bar - reinterpret_cast<uint64_t*>(ctrl);
            r[1] = t0;
            r[2] = t1;
        }
    }
    return ok;
}
// a bare time stamp with a caller-chosen tag (>= 100)
__device__ __forceinline__ void trace_mark(Ctrl* ctrl, int tag) {
    if (blockIdx.x == 0 && (threadIdx.x & 31) == 0) {
        const int w = threadIdx.x >> 5;
        const int n = ctrl->trace_n[w]++;
        if (n < TRACE_CAP) {
            long long* r = g_trace + (static_cast<size_t>(w) * TRACE_CAP + n) * 3;
            r[0] = tag;
            r[1] = r[2] = clock64();
        }
    }
}
#define wait_bar_body wait_bar_impl
#else
#define wait_bar_body wait_bar
#define trace_mark(ctrl, tag) ((void)0)
#endif

// Bounded wait on an mbarrier phase. Returns false if the CTA is aborting.  After a first quick
// poll the thread sleeps in the barrier unit (it wakes when the phase completes or after
// WAIT_SLICE_NS), so a waiting warp issues next to nothing and leaves the issue slots and the ALU
// pipe to the warps that have work.
__device__ __forceinline__ bool wait_bar_body(uint64_t* bar, uint32_t parity, Ctrl* ctrl, int* status) {
    const uint32_t addr = ptx::smem_u32(bar);
    if (ptx::mbar_try_wait(addr, parity)) return true;
    const uint64_t t0 = ptx::globaltimer_ns();
    for (;;) {
        if (ptx::mbar_try_wait_hint(addr, parity, WAIT_SLICE_NS)) return true;
        if (*reinterpret_cast<volatile int*>(&ctrl->abort_flag)) return false;
        if (ptx::globaltimer_ns() - t0 > WAIT_LIMIT_NS) {
            *reinterpret_cast<volatile int*>(&ctrl->abort_flag) = 1;
            atomicCAS(status, CAKE_OK, CAKE_ERR_TIMEOUT);
            return false;
        }
    }
}

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

using aug::split3;

// min over 32 floats with 3-input min instructions
__device__ __forceinline__ float min32(const float (&v)[32]) {
    float t[11];
#pragma unroll
    for (int q = 0; q < 10; ++q) t[q] = ptx::fmin3(v[3 * q], v[3 * q + 1], v[3 * q + 2]);
    t[10] = fminf(v[30], v[31]);
    const float u0 = ptx::fmin3(t[0], t[1], t[2]);
    const float u1 = ptx::fmin3(t[3], t[4], t[5]);
    const float u2 = ptx::fmin3(t[6], t[7], t[8]);
    const float u3 = fminf(t[9], t[10]);
    return fminf(ptx::fmin3(u0, u1, u2), u3);
}

// packed policy: key = the accumulator with its low 7 bits replaced by the column (0..127 inside the half
// tile): one logic instruction (mask in a register, column immediate); see assign_tc.cu
__device__ __forceinline__ float packed_min32(const uint32_t (&r)[32], int col_base, float run, uint32_t kmask) {
    float v[32];
#pragma unroll
    for (int j = 0; j < 32; ++j)
        v[j] = __uint_as_float(ptx::and_or(r[j], kmask, static_cast<uint32_t>(col_base + j)));
    return fminf(run, min32(v));
}

// exact policy: full-precision group minimum; position looked up (lowest column first) only on a hit.
__device__ __forceinline__ void exact_scan32(const uint32_t (&r)[32], int col_base, float& best, int& bidx) {
    float v[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
    const float m = min32(v);
    if (m < best) {
        best = m;
        int c[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) c[j] = (v[j] == m) ? j : 32;
#pragma unroll
        for (int s = 16; s > 0; s >>= 1)
#pragma unroll
            for (int j = 0; j < s; ++j) c[j] = min(c[j], c[j + s]);
        bidx = col_base + c[0];
    }
}

// BULK: the epilogue requests a whole 128-column slice at once, hands the accumulator back as soon as it has
// landed and reduces from registers; otherwise the four 32-column groups go through two register buffers.
// WIDE (rows of more than 512 columns, which no CTA can keep resident): X is streamed like the centroids, a chunk
// of each per ring stage, and the X-side operand of the extra k-step and the row margins come from global memory
// (row_aug_kernel wrote them); the norm warps idle.
template <bool PACKED, bool BULK, bool WIDE = false>
__global__ void __launch_bounds__(NUM_THREADS, 1)
assign_pair_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_c,
                  const __grid_constant__ CUtensorMap tmap_aug, const __grid_constant__ CUtensorMap tmap_xaug, const Params p) {
    extern __shared__ uint8_t smem_raw[];
    // 128B-swizzled tiles need 1024-byte alignment
    const uint32_t raw_addr = ptx::smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    uint8_t* smem = smem_raw + pad;
    const uint32_t smem_base = raw_addr + pad;
    const uint32_t xbuf_bytes = WIDE ? 0u : static_cast<uint32_t>(p.nchunks) * X_CHUNK_BYTES;
    const uint32_t x_base = smem_base;
    const uint32_t ring_off = static_cast<uint32_t>(p.n_xbuf) * xbuf_bytes;
    const uint32_t ring_base = smem_base + ring_off;
    // a chunk of a stage: this CTA's half of the centroid chunk, in the wide mode behind its X chunk
    // Wide rows: one issuer with the whole ring.  A tile is tens of stages long there, the issuers would work one
    // after the other anyway, and a load takes longer than the MMAs of the two or three stages a sub-ring holds.
    constexpr int NISS = WIDE ? 1 : NUM_ISSUERS;
    constexpr uint32_t CHUNK_STRIDE = WIDE ? X_CHUNK_BYTES + C_HALF_BYTES : C_HALF_BYTES;
    constexpr uint32_t C_IN_CHUNK = WIDE ? X_CHUNK_BYTES : 0u;
    const uint32_t stage_bytes = static_cast<uint32_t>(p.cps) * CHUNK_STRIDE + AUG_B_HALF;
    const uint32_t auga_off = ring_off + static_cast<uint32_t>(p.n_stages) * stage_bytes;
    const uint32_t zero_off = auga_off + static_cast<uint32_t>(p.n_xbuf) * AUG_A_BYTES;
    const uint32_t ctrl_off = zero_off + AUG_ZERO_BYTES;
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem + ctrl_off);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();          // 0 issues the MMAs
    const i64 pair = blockIdx.x >> 1;                        // this pair's first row tile
    const i64 n_pairs = gridDim.x >> 1;
    // the same barrier in rank 0's shared memory (rank 0: its own)
    auto at_rank0 = [](const void* bar) { return ptx::smem_u32(bar) & ~ptx::CLUSTER_PEER_BIT; };

    if (threadIdx.x == 0) {
        for (int i = 0; i < MAX_XBUF; ++i) {
            ptx::mbar_init(ptx::smem_u32(&ctrl->x_full[i]), 1);
            // MMA issuers, norm warps, one epilogue warpgroup (wide: the issuers alone)
            ptx::mbar_init(ptx::smem_u32(&ctrl->x_empty[i]), WIDE ? NISS : NISS + 4 + 4);
            ptx::mbar_init(ptx::smem_u32(&ctrl->auga_full[i]), WIDE ? 1 : 8);   // norm warps of both CTAs (wide: rank 0's producer)
            ptx::mbar_init(ptx::smem_u32(&ctrl->auga_local[i]), 4);
        }
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(ptx::smem_u32(&ctrl->tmem_full[i]), 1);
            for (int j = 0; j < NUM_ISSUERS; ++j)
                ptx::mbar_init(ptx::smem_u32(&ctrl->tmem_empty[i][j]), 2 * NUM_EPI_WARPS);   // both CTAs' epilogues
            ptx::mbar_init(ptx::smem_u32(&ctrl->merge_full[i]), 4);
            ptx::mbar_init(ptx::smem_u32(&ctrl->merge_empty[i]), 4);
        }
        for (int i = 0; i < MAX_STAGES; ++i) {
            ptx::mbar_init(ptx::smem_u32(&ctrl->ring_full[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctrl->ring_empty[i]), 1);   // the commit of the sub-ring's issuer
        }
        ctrl->abort_flag = 0;
#ifdef CAKE_ASSIGN_TRACE
        for (int i = 0; i < NUM_WARPS; ++i) ctrl->trace_n[i] = 0;
#endif
        ptx::fence_mbar_init();
    }
    // columns 8..15 of both operands of the extra k-step: one block of zeros for the whole kernel
    for (uint32_t o = threadIdx.x * 16; o < AUG_ZERO_BYTES; o += NUM_THREADS * 16)
        *reinterpret_cast<uint4*>(smem + zero_off + o) = make_uint4(0, 0, 0, 0);
    ptx::fence_proxy_async_smem();
    if (warp == MMA_WARP) {
        ptx::tmem_alloc_pair(ptx::smem_u32(&ctrl->tmem_base), TMEM_COLS);
        ptx::tmem_relinquish_pair();
    }
    if (warp == PRODUCER_WARP && lane == 0) {
        ptx::prefetch_tensormap(&tmap_x);
        ptx::prefetch_tensormap(&tmap_c);
        ptx::prefetch_tensormap(&tmap_aug);
        if (WIDE) ptx::prefetch_tensormap(&tmap_xaug);
    }
    ptx::tc_fence_before();
    __syncthreads();
    // no CTA may signal the other's barriers, or issue MMAs into its tensor memory, before both are set up
    ptx::cluster_sync_all();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&ctrl->tmem_base);
    // everything above touched no global memory: it may overlap the prologue kernel's tail
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();

    // The epilogue keeps a whole 128-column accumulator slice in registers; the other roles need few.
    // Registers move between warpgroups accordingly (warps 0-7 grow, warps 8-15 shrink).
    if (warp >= NUM_EPI_WARPS) {
    ptx::setmaxnreg_dec<AUX_REGS>();
    if (warp == PRODUCER_WARP) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            // each issuer has its own sub-ring of `spi` stages; (sr, sp)[i] = next slot and phase of issuer i's
            const uint32_t spi = static_cast<uint32_t>(p.spi);
            uint32_t sr0 = 0, sr1 = 0, sr2 = 0, sp0 = 0, sp1 = 0, sp2 = 0;
            uint32_t turn = 0;
            bool ok = true;
            // X tiles run ahead of the MMAs by up to n_xbuf row tiles: `x_next` is the next row tile
            // whose X has not been requested yet, (ixb, ixph) the buffer and phase it will use
            i64 x_next = pair;
            uint32_t ixb = 0, ixph = 0;
            auto issue_x = [&]() {
                const int tb = static_cast<int>(x_next / p.m_tiles);
                const int tmt = static_cast<int>(x_next % p.m_tiles);
                if (WIDE) {
                    // the row tile's X-side operand of the extra k-step (this CTA's 128 rows of it); both CTAs' bytes
                    // are counted on rank 0's barrier, where the issuers wait
                    if (rank == 0) ptx::mbar_arrive_expect_tx(ptx::smem_u32(&ctrl->auga_full[ixb]), 2u * AUG_A_BYTES);
                    ptx::tma_load_2d_pair(smem_base + auga_off + ixb * AUG_A_BYTES, &tmap_xaug, at_rank0(&ctrl->auga_full[ixb]), 0,
                                          static_cast<int>(tb * p.Npad + tmt * (2 * BLOCK_M) + static_cast<int>(rank) * BLOCK_M));
                } else {
                    const uint32_t xfull = ptx::smem_u32(&ctrl->x_full[ixb]);
                    ptx::mbar_arrive_expect_tx(xfull, xbuf_bytes);
                    for (int c = 0; c < p.nchunks; ++c)
                        ptx::tma_load_3d(x_base + ixb * xbuf_bytes + c * X_CHUNK_BYTES, &tmap_x, xfull,
                                         c * KCHUNK, tmt * (2 * BLOCK_M) + static_cast<int>(rank) * BLOCK_M, tb);
                }
                x_next += n_pairs;
                if (++ixb == static_cast<uint32_t>(p.n_xbuf)) { ixb = 0; ixph ^= 1u; }
            };
            // request X tiles for as long as a buffer is free, without ever blocking
            auto prefetch_x = [&]() {
                while (x_next < p.total_tiles &&
                       ptx::mbar_test_wait(ptx::smem_u32(&ctrl->x_empty[ixb]), ixph ^ 1u))
                    issue_x();
            };
            for (i64 tile = pair; ok && tile < p.total_tiles; tile += n_pairs) {
                const int b = static_cast<int>(tile / p.m_tiles);
                const int xrow = static_cast<int>(tile % p.m_tiles) * (2 * BLOCK_M) + static_cast<int>(rank) * BLOCK_M;
                prefetch_x();
                if (x_next <= tile) {   // this tile's own X is still outstanding: its buffer must free up
                    ok = wait_bar(&ctrl->x_empty[ixb], ixph ^ 1u, ctrl, p.status);
                    if (!ok) break;
                    issue_x();
                }
                for (int nt = 0; ok && nt < p.n_tiles; ++nt, turn = (turn + 1 == NISS) ? 0 : turn + 1) {
                    const int crow = nt * BLOCK_N + static_cast<int>(rank) * (BLOCK_N / 2);   // this CTA's centroid rows
                    uint32_t rs = turn == 0 ? sr0 : (turn == 1 ? sr1 : sr2);
                    uint32_t rph = turn == 0 ? sp0 : (turn == 1 ? sp1 : sp2);
                    for (int c = 0; c < p.nchunks; c += p.cps) {
                        prefetch_x();
                        const uint32_t slot = turn * spi + rs;
                        // this CTA's copy of the barrier: the MMA commits are multicast to both
                        ok = wait_bar(&ctrl->ring_empty[slot], rph ^ 1u, ctrl, p.status);
                        if (!ok) break;
                        const int nc = min(p.cps, p.nchunks - c);
                        const bool last = c + nc == p.nchunks;
                        // both CTAs' bytes are counted on rank 0's barrier, which rank 0 arms
                        if (rank == 0)
                            ptx::mbar_arrive_expect_tx(ptx::smem_u32(&ctrl->ring_full[slot]),
                                                       2u * (static_cast<uint32_t>(nc) * CHUNK_STRIDE + (last ? AUG_B_HALF : 0u)));
                        const uint32_t full0 = at_rank0(&ctrl->ring_full[slot]);
                        const uint32_t stage = ring_base + slot * stage_bytes;
                        for (int j = 0; j < nc; ++j) {
                            if (WIDE) ptx::tma_load_3d_pair(stage + j * CHUNK_STRIDE, &tmap_x, full0, (c + j) * KCHUNK, xrow, b);
                            ptx::tma_load_3d_pair(stage + j * CHUNK_STRIDE + C_IN_CHUNK, &tmap_c, full0, (c + j) * KCHUNK, crow, b);
                        }
                        if (last)   // the tile's half-norm operand rides with its last chunks
                            ptx::tma_load_2d_pair(stage + static_cast<uint32_t>(p.cps) * CHUNK_STRIDE, &tmap_aug, full0, 0,
                                                  b * p.Kpad + crow);
                        if (++rs == spi) { rs = 0; rph ^= 1u; }
                    }
                    if (turn == 0) { sr0 = rs; sp0 = rph; } else if (turn == 1) { sr1 = rs; sp1 = rph; } else { sr2 = rs; sp2 = rph; }
                }
            }
            if (!ok) {
                // aborting: give our loads in flight a bounded time to land before the CTA's shared memory is given up
                const uint64_t t0 = ptx::globaltimer_ns();
                while (ptx::globaltimer_ns() - t0 < 1000000ull) {
                }
            }
        }
    } else if (warp >= MMA_WARP && warp < MMA_WARP + NISS) {
        // ------------------------------------------------------------ MMA issuers (rank 0 only)
        // Three warps, one issuing thread each; centroid tiles go round robin over them (tile t to
        // issuer t mod 3, into accumulator t mod 2) because one thread's own instruction stream is too
        // slow to keep the tensor pipe fed.  Every MMA spans both CTAs; every commit reaches the
        // barrier at the same offset in both.
        if (rank == 0 && lane == 0) {
            const uint32_t iss = static_cast<uint32_t>(warp - MMA_WARP);
            constexpr uint32_t idesc_aug = ptx::umma_idesc_bf16(2 * BLOCK_M, BLOCK_N);
            constexpr uint32_t idesc_main = idesc_aug | ptx::UMMA_IDESC_NEGATE_B;   // accumulates -x.c
            constexpr uint32_t KSTEP = (UMMA_K * 2) >> 4;   // descriptor units per k-step
            constexpr uint16_t BOTH = 3;                    // commit to rank 0 and rank 1
            const uint32_t spi = static_cast<uint32_t>(p.spi);
            const uint32_t slot0 = iss * spi;               // this issuer's sub-ring
            uint32_t s = 0, ph = 0;                         // position in it and its phase
            uint32_t xb = 0, xph = 0;                       // X buffer and its phase
            uint32_t acc_it = 0;
            uint32_t turn = 0;                              // acc_it mod NUM_ISSUERS
            uint32_t rel0 = 0, rel1 = 0;                    // releases of accumulator 0 / 1 this issuer has consumed
            bool ok = true;
            for (i64 tile = pair; ok && tile < p.total_tiles; tile += n_pairs) {
                // The norm warps of both CTAs have written their operand of the extra k-step, which
                // they do after their X tile has landed: both X tiles are in place.  Every issuer sees
                // every phase, also in row tiles it has no centroid tile in.
                ok = wait_bar(&ctrl->auga_full[xb], xph, ctrl, p.status);
                if (!ok) break;
                const uint32_t a_lo_tile = ptx::umma_desc_lo_sw128(x_base + xb * xbuf_bytes);
                const uint32_t auga_lo = ptx::umma_desc_lo_aug(smem_base + auga_off + xb * AUG_A_BYTES,
                                                               smem_base + zero_off);
                for (int nt = 0; ok && nt < p.n_tiles; ++nt, ++acc_it, turn = (turn + 1 == NISS) ? 0 : turn + 1) {
                    if (turn != iss) continue;   // another issuer's tile, in that issuer's sub-ring
                    const uint32_t acc = acc_it & 1u;
                    const uint32_t d_tmem = tmem_base + acc * BLOCK_N;
                    // the accumulator was last used by tile acc_it - 2, whose release (by the epilogues of
                    // both CTAs) is addressed to this issuer; the first two tiles find theirs free
                    if (acc_it >= 2u) {
                        const uint32_t rel = acc ? rel1 : rel0;
                        ok = wait_bar(&ctrl->tmem_empty[acc][iss], rel & 1u, ctrl, p.status);
                        if (!ok) break;
                        if (acc) ++rel1; else ++rel0;
                    }
                    ptx::tc_fence_after();
                    uint32_t a_lo = a_lo_tile;
                    for (int c0 = 0; c0 < p.nchunks; c0 += p.cps) {
                        ok = wait_bar(&ctrl->ring_full[slot0 + s], ph, ctrl, p.status);
                        if (!ok) break;
                        ptx::tc_fence_after();
                        const uint32_t stage = ring_base + (slot0 + s) * stage_bytes;
                        const int nc = min(p.cps, p.nchunks - c0);
                        for (int j = 0; j < nc; ++j, a_lo += X_CHUNK_BYTES >> 4) {
                            if (WIDE) a_lo = ptx::umma_desc_lo_sw128(stage + j * CHUNK_STRIDE);   // the X chunk of this stage
                            const uint32_t b_lo = ptx::umma_desc_lo_sw128(stage + j * CHUNK_STRIDE + C_IN_CHUNK);
                            const bool last = c0 + j == p.nchunks - 1;
                            const int nk = last ? p.ksteps_last : KCHUNK / UMMA_K;
                            if (c0 + j == 0)
                                ptx::umma_pair_bf16_lohi<false>(d_tmem, a_lo, ptx::UMMA_DESC_HI_SW128, b_lo,
                                                                ptx::UMMA_DESC_HI_SW128, idesc_main);
                            else
                                ptx::umma_pair_bf16_lohi<true>(d_tmem, a_lo, ptx::UMMA_DESC_HI_SW128, b_lo,
                                                               ptx::UMMA_DESC_HI_SW128, idesc_main);
                            if (nk == KCHUNK / UMMA_K) {
#pragma unroll
                                for (uint32_t ks = 1; ks < KCHUNK / UMMA_K; ++ks)
                                    ptx::umma_pair_bf16_lohi<true>(d_tmem, a_lo + ks * KSTEP, ptx::UMMA_DESC_HI_SW128,
                                                                   b_lo + ks * KSTEP, ptx::UMMA_DESC_HI_SW128, idesc_main);
                            } else {
                                for (int ks = 1; ks < nk; ++ks)
                                    ptx::umma_pair_bf16_lohi<true>(d_tmem, a_lo + ks * KSTEP, ptx::UMMA_DESC_HI_SW128,
                                                                   b_lo + ks * KSTEP, ptx::UMMA_DESC_HI_SW128, idesc_main);
                            }
                            // the extra k-step: + ||x||^2/2 + m + ||c||^2/2; its centroid side came with this stage
                            if (last)
                                ptx::umma_pair_bf16_lohi<true>(d_tmem, auga_lo, ptx::UMMA_DESC_HI_AUG,
                                                               ptx::umma_desc_lo_aug(stage + static_cast<uint32_t>(p.cps) * CHUNK_STRIDE,
                                                                                     smem_base + zero_off),
                                                               ptx::UMMA_DESC_HI_AUG, idesc_aug);
                        }
                        ptx::umma_pair_commit(ptx::smem_u32(&ctrl->ring_empty[slot0 + s]), BOTH);
                        if (++s == spi) { s = 0; ph ^= 1u; }
                    }
                    if (!ok) break;
                    ptx::umma_pair_commit(ptx::smem_u32(&ctrl->tmem_full[acc]), BOTH);
                }
                // this issuer's MMAs on the X buffers (of both CTAs) are done when this commit fires (it
                // fires at once if the issuer had no tile in this row tile)
                if (ok) ptx::umma_pair_commit(ptx::smem_u32(&ctrl->x_empty[xb]), BOTH);
                if (++xb == static_cast<uint32_t>(p.n_xbuf)) { xb = 0; xph ^= 1u; }
            }
        }
    } else if (!WIDE && warp >= AUX_WARP0) {
        // ------------------------------------------------------------ norm warps
        // One thread per X row: ||x||^2/2 + m from the swizzled X tile (16-byte granule g of row r sits
        // at position g ^ (r & 7); the order of the granules does not matter for a sum), split into
        // three bf16 terms and written as the X-side operand of the extra k-step.  These warps run a row tile ahead of the MMA warps, so the operand is
        // ready when the first centroid tile needs it.
        const int r = (warp - AUX_WARP0) * 32 + lane;
        uint32_t xb = 0, xph = 0;
        bool ok = true;
        for (i64 tile = pair; ok && tile < p.total_tiles; tile += n_pairs) {
            ok = wait_bar(&ctrl->x_full[xb], xph, ctrl, p.status);
            if (!ok) break;
            const uint8_t* xrow = smem + xb * xbuf_bytes + r * 128;
            float xn0 = 0.f, xn1 = 0.f, xn2 = 0.f, xn3 = 0.f;
            for (int c = 0; c < p.nchunks; ++c) {
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    const uint4 w = *reinterpret_cast<const uint4*>(xrow + c * X_CHUNK_BYTES +
                                                                    ((g ^ (r & 7)) << 4));
                    float a;
                    a = bf16lo(w.x); xn0 = fmaf(a, a, xn0); a = bf16hi(w.x); xn1 = fmaf(a, a, xn1);
                    a = bf16lo(w.y); xn2 = fmaf(a, a, xn2); a = bf16hi(w.y); xn3 = fmaf(a, a, xn3);
                    a = bf16lo(w.z); xn0 = fmaf(a, a, xn0); a = bf16hi(w.z); xn1 = fmaf(a, a, xn1);
                    a = bf16lo(w.w); xn2 = fmaf(a, a, xn2); a = bf16hi(w.w); xn3 = fmaf(a, a, xn3);
                }
            }
            const float xn = (xn0 + xn1) + (xn2 + xn3);
            // margin m = 2^(e-11) for ||x||^2 in [2^e, 2^(e+1)), at least 2^-100 (see assign_tc.cu)
            const uint32_t xe = __float_as_uint(xn) >> 23;
            const uint32_t mbits = (xe > 38u ? xe - 11u : 27u) << 23;
            uint32_t hi, mid, lo;
            split3(fmaf(0.5f, xn, __uint_as_float(mbits)), hi, mid, lo);
            ctrl->row_m[xb][r] = __uint_as_float(mbits);
            const uint32_t one = 0x3F80u;
            *reinterpret_cast<uint4*>(smem + auga_off + xb * AUG_A_BYTES + r * 16) =
                make_uint4(hi | (mid << 16), lo | (one << 16), one | (one << 16), 0u);
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                ptx::mbar_arrive(ptx::smem_u32(&ctrl->auga_local[xb]));           // this CTA's epilogue
                ptx::mbar_arrive_cluster(at_rank0(&ctrl->auga_full[xb]));         // the issuers
                ptx::mbar_arrive(ptx::smem_u32(&ctrl->x_empty[xb]));
            }
            if (++xb == static_cast<uint32_t>(p.n_xbuf)) { xb = 0; xph ^= 1u; }
        }
    }
    } else {
        // ------------------------------------------------------------ epilogue warps
        ptx::setmaxnreg_inc<EPI_REGS>();
        const int wg = warp >> 2;            // column half of every tile
        const int q = warp & 3;              // TMEM lane quarter this warp may read
        const int r = q * 32 + lane;         // row inside the X tile
        uint32_t tile_it = 0, acc_it = 0;
        uint32_t next_iss = 2 % NISS;   // (acc_it + 2) mod the number of issuers
        uint32_t exb = 0, exph = 0;          // X buffer (slot of the row margins) and its phase
        const uint32_t kmask = ~COL_MASK | (static_cast<uint32_t>(p.K) >> 31);   // in a register (see assign_tc.cu)
        bool ok = true;
        double dsum = 0.0;                   // this thread's share of the current problem's inertia
        int dsum_b = -1;
        // one fp64 atomic per warp and problem
        auto flush_inertia = [&]() {
            if (wg == 0 && p.inertia && dsum_b >= 0) {
                double t = dsum;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
                if (lane == 0) atomicAdd(p.inertia + static_cast<size_t>(dsum_b) * p.inertia_stride, t);
            }
            dsum = 0.0;
        };
        // (problem, row tile) of the current tile, stepped instead of divided
        int b = static_cast<int>(pair / p.m_tiles);
        int mt = static_cast<int>(pair % p.m_tiles);
        auto next_tile = [&]() {
            mt += static_cast<int>(n_pairs);
            while (mt >= p.m_tiles) { mt -= p.m_tiles; ++b; }
        };
        for (i64 tile = pair; ok && tile < p.total_tiles; tile += n_pairs, ++tile_it, next_tile()) {
            if (b != dsum_b) {
                flush_inertia();
                dsum_b = b;
            }
            float best = __uint_as_float(F32_INF);   // packed: a key; exact: a value
            int bsel = 0;                            // packed: tile number; exact: global column
            float rowM = 0.f;                        // this row's margin m (wg 0 only)
            for (int nt = 0; nt < p.n_tiles; ++nt, ++acc_it) {
                const uint32_t as = acc_it & 1u, aph = (acc_it >> 1) & 1u;
                ok = wait_bar(&ctrl->tmem_full[as], aph, ctrl, p.status);
                if (!ok) break;
                ptx::tc_fence_after();
                if (nt == 0 && wg == 0) {
                    if (WIDE) {
                        rowM = p.row_m[static_cast<i64>(b) * p.Npad + static_cast<i64>(mt) * (2 * BLOCK_M) + rank * BLOCK_M + r];
                    } else {
                        // written by the norm warps before they completed auga_local; read now, while the X
                        // buffer (and with it this slot) cannot have been handed to a later row tile
                        ok = wait_bar(&ctrl->auga_local[exb], exph, ctrl, p.status);
                        if (!ok) break;
                        rowM = ctrl->row_m[exb][r];
                        // the slot of the margins goes back with the X buffer: this warpgroup has read it
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->x_empty[exb]));
                    }
                }
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                       as * BLOCK_N + wg * (BLOCK_N / 2);
                if (!BULK) {
                    // the load of group g + 1 is in flight while group g is reduced; the accumulator goes back to the
                    // issuers (rank 0's, from both CTAs) when the last group has landed
                    uint32_t ra[32], rb[32];
                    ptx::tmem_ld_x32(taddr, ra);
                    ptx::tmem_ld_wait(ra);
                    ptx::tmem_ld_x32_before(taddr + 32, rb, ra);
                    if (PACKED) {
                        float tmin = packed_min32(ra, 0, __uint_as_float(F32_INF), kmask);
                        ptx::tmem_ld_wait_after(rb, tmin);
                        ptx::tmem_ld_x32_before(taddr + 64, ra, rb);
                        tmin = packed_min32(rb, 32, tmin, kmask);
                        ptx::tmem_ld_wait_after(ra, tmin);
                        ptx::tmem_ld_x32_before(taddr + 96, rb, ra);
                        tmin = packed_min32(ra, 64, tmin, kmask);
                        ptx::tmem_ld_wait_after(rb, tmin);
                        ptx::tc_fence_before();
                        __syncwarp();
                        // to the issuer of tile acc_it + 2, which takes this accumulator next
                        if (lane == 0) ptx::mbar_arrive_cluster(at_rank0(&ctrl->tmem_empty[as][next_iss]));
                        trace_mark(ctrl, 100);
                        tmin = packed_min32(rb, 96, tmin, kmask);
                        // across tiles only the (truncated) value decides: an equal value keeps the earlier tile
                        if (__uint_as_float(__float_as_uint(tmin) & ~COL_MASK) <
                            __uint_as_float(__float_as_uint(best) & ~COL_MASK)) {
                            best = tmin;
                            bsel = nt;
                        }
                    } else {
                        const int col0 = nt * BLOCK_N + wg * (BLOCK_N / 2);
                        exact_scan32(ra, col0, best, bsel);
                        ptx::tmem_ld_wait_after(rb, best);
                        ptx::tmem_ld_x32_before(taddr + 64, ra, rb);
                        exact_scan32(rb, col0 + 32, best, bsel);
                        ptx::tmem_ld_wait_after(ra, best);
                        ptx::tmem_ld_x32_before(taddr + 96, rb, ra);
                        exact_scan32(ra, col0 + 64, best, bsel);
                        ptx::tmem_ld_wait_after(rb, best);
                        ptx::tc_fence_before();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive_cluster(at_rank0(&ctrl->tmem_empty[as][next_iss]));
                        trace_mark(ctrl, 100);
                        exact_scan32(rb, col0 + 96, best, bsel);
                    }
                } else {
                    uint32_t ra[32], rb[32], rc[32], rd[32];
                    ptx::tmem_ld_x32(taddr, ra);
                    ptx::tmem_ld_x32(taddr + 32, rb);
                    ptx::tmem_ld_x32(taddr + 64, rc);
                    ptx::tmem_ld_x32(taddr + 96, rd);
                    ptx::tmem_ld_wait(ra);
                    ptx::reg_dep(rb);
                    ptx::reg_dep(rc);
                    ptx::reg_dep(rd);
                    ptx::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive_cluster(at_rank0(&ctrl->tmem_empty[as][next_iss]));
                    trace_mark(ctrl, 100);
                    if (PACKED) {
                        float tmin = packed_min32(ra, 0, __uint_as_float(F32_INF), kmask);
                        tmin = packed_min32(rb, 32, tmin, kmask);
                        tmin = packed_min32(rc, 64, tmin, kmask);
                        tmin = packed_min32(rd, 96, tmin, kmask);
                        if (__uint_as_float(__float_as_uint(tmin) & ~COL_MASK) <
                            __uint_as_float(__float_as_uint(best) & ~COL_MASK)) {
                            best = tmin;
                            bsel = nt;
                        }
                    } else {
                        const int col0 = nt * BLOCK_N + wg * (BLOCK_N / 2);
                        exact_scan32(ra, col0, best, bsel);
                        exact_scan32(rb, col0 + 32, best, bsel);
                        exact_scan32(rc, col0 + 64, best, bsel);
                        exact_scan32(rd, col0 + 96, best, bsel);
                    }
                }
                next_iss = (next_iss + 1 == NISS) ? 0 : next_iss + 1;
            }
            if (!ok) break;
            trace_mark(ctrl, 102);
            if (++exb == static_cast<uint32_t>(p.n_xbuf)) { exb = 0; exph ^= 1u; }
            // (value, index) of this half; the value is a key with its column bits cleared (packed) or
            // the accumulator itself (exact)
            float bval;
            int bidx;
            if (PACKED) {
                const uint32_t kb = __float_as_uint(best);
                bval = __uint_as_float(kb & ~COL_MASK);
                bidx = bsel * BLOCK_N + wg * (BLOCK_N / 2) + static_cast<int>(kb & COL_MASK);
            } else {
                bval = best;
                bidx = bsel;
            }
            // merge the two column halves: the upper half hands its (value, index) to the lower one
            const uint32_t mb = tile_it & 1u, mph = (tile_it >> 1) & 1u;
            if (wg == 1) {
                ok = wait_bar(&ctrl->merge_empty[mb], mph ^ 1u, ctrl, p.status);
                if (!ok) break;
                ctrl->merge_best[mb][r] = bval;
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
                if (ob < bval || (ob == bval && oi < bidx)) {
                    bval = ob;
                    bidx = oi;
                }
                const i64 row = static_cast<i64>(mt) * (2 * BLOCK_M) + static_cast<i64>(rank) * BLOCK_M + r;
                if (row < p.N) {
                    const size_t o = static_cast<size_t>(b) * static_cast<size_t>(p.N) + row;
                    const float dist = fmaxf(0.f, 2.f * (bval - rowM));   // the accumulator is m + d/2
                    p.out_idx[o] = bidx;
                    if (p.out_dist) p.out_dist[o] = dist;
                    dsum += static_cast<double>(dist);
                }
            }
            trace_mark(ctrl, 103);
        }
        if (ok) flush_inertia();
    }

    // ---------------------------------------------------------------- teardown
    // Neither CTA may leave, or give up its tensor memory, while the other's MMAs, loads or arrivals
    // can still touch it: every thread of the pair meets here (also after a time-out: all loops above
    // are bounded).
    ptx::tc_fence_before();
    __syncthreads();
    ptx::cluster_sync_all();
    if (warp == MMA_WARP) {
        __syncwarp();
        ptx::tc_fence_after();
        ptx::tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

}  // namespace

#ifdef CAKE_ASSIGN_TRACE
// Profiling build only: copies warp `w`'s trace records of the pair kernel's CTA 0 (3 x int64 each, up to `cap`) to `host`.
extern "C" __attribute__((visibility("default"))) int cake_debug_read_trace_pair(int w, long long* host, int cap) {
    cudaDeviceSynchronize();
    if (w < 0 || w >= NUM_WARPS) return 0;
    const int n = cap < TRACE_CAP ? cap : TRACE_CAP;
    cudaMemcpyFromSymbol(host, g_trace, static_cast<size_t>(n) * 3 * sizeof(long long),
                         static_cast<size_t>(w) * TRACE_CAP * 3 * sizeof(long long));
    return n;
}
#endif

// ======================================================================= rows of more than 512 columns
namespace {
// One warp per row of X: ||x||^2 in fp32, the margin m and the X-side operand of the extra k-step
// ([hi mid lo 1 1 1 0 0] in bf16, hi + mid + lo = ||x||^2/2 + m), as the norm warps of the kernels with a resident X
// tile compute them in shared memory.  Rows N .. Npad-1 of a problem (the last row tile's tail) get zeros.
__global__ void __launch_bounds__(256)
row_aug_kernel(const cake_bf16* __restrict__ X, i64 N, int D, i64 Npad, i64 rows_total, uint4* __restrict__ aug,
               float* __restrict__ row_m) {
    const int lane = threadIdx.x & 31;
    const i64 row = static_cast<i64>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= rows_total) return;
    const i64 b = row / Npad, i = row - b * Npad;
    if (i >= N) {
        if (lane == 0) {
            aug[row] = make_uint4(0, 0, 0, 0);
            row_m[row] = 0.f;
        }
        return;
    }
    const uint4* x = reinterpret_cast<const uint4*>(X + (static_cast<size_t>(b) * N + i) * D);
    float xn0 = 0.f, xn1 = 0.f, xn2 = 0.f, xn3 = 0.f;
    for (int g = lane; g < D / 8; g += 32) {
        const uint4 w = __ldg(x + g);
        float a = bf16lo(w.x); xn0 = fmaf(a, a, xn0); a = bf16hi(w.x); xn1 = fmaf(a, a, xn1);
        a = bf16lo(w.y); xn2 = fmaf(a, a, xn2); a = bf16hi(w.y); xn3 = fmaf(a, a, xn3);
        a = bf16lo(w.z); xn0 = fmaf(a, a, xn0); a = bf16hi(w.z); xn1 = fmaf(a, a, xn1);
        a = bf16lo(w.w); xn2 = fmaf(a, a, xn2); a = bf16hi(w.w); xn3 = fmaf(a, a, xn3);
    }
    float xn = (xn0 + xn1) + (xn2 + xn3);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) xn += __shfl_xor_sync(0xffffffffu, xn, o);
    if (lane == 0) {
        // margin m = 2^(e-11) for ||x||^2 in [2^e, 2^(e+1)), at least 2^-100 (see assign_tc.cu)
        const uint32_t xe = __float_as_uint(xn) >> 23;
        const uint32_t mbits = (xe > 38u ? xe - 11u : 27u) << 23;
        uint32_t hi, mid, lo;
        split3(fmaf(0.5f, xn, __uint_as_float(mbits)), hi, mid, lo);
        const uint32_t one = 0x3F80u;
        aug[row] = make_uint4(hi | (mid << 16), lo | (one << 16), one | (one << 16), 0u);
        row_m[row] = __uint_as_float(mbits);
    }
}

}  // namespace

size_t assign_wide_aug_bytes(i64 B, i64 N) { return static_cast<size_t>(B) * round_up(N, 2 * BLOCK_M) * 16; }
size_t assign_wide_margin_bytes(i64 B, i64 N) { return static_cast<size_t>(B) * round_up(N, 2 * BLOCK_M) * 4; }

cudaError_t launch_row_aug(const cake_bf16* X, int B, i64 N, int D, void* xaug, float* xrowm, cudaStream_t s) {
    const i64 Npad = round_up(N, 2 * BLOCK_M);
    const i64 rows = static_cast<i64>(B) * Npad;
    if (rows == 0) return cudaSuccess;
    row_aug_kernel<<<static_cast<unsigned>((rows + 7) / 8), 256, 0, s>>>(X, N, D, Npad, rows, static_cast<uint4*>(xaug), xrowm);
    note_launches(1);
    return cudaGetLastError();
}

// ======================================================================= host side
namespace {
struct PairPlan {
    int n_xbuf, spi, cps;
    size_t smem_bytes;
};

// Shared memory: n_xbuf X buffers and NUM_ISSUERS sub-rings of spi stages of cps chunks.  Preferred: a whole
// centroid tile per stage (one wait and one commit per tile on the issuing thread), then more than one stage per
// issuer; few centroid tiles per row tile want more X buffers instead.  Wide rows: no X buffer (two 2 KiB operands
// of the extra k-step instead), a stage holds one chunk of X and of the centroids.
bool plan_pair(const DeviceInfo& di, int nchunks, int n_tiles, bool wide, PairPlan* out) {
    const i64 fixed = 1024 + CTRL_BYTES + AUG_ZERO_BYTES;
    const i64 budget = static_cast<i64>(di.smem_optin) - fixed;
    if (wide) {
        const i64 stage = X_CHUNK_BYTES + C_HALF_BYTES + AUG_B_HALF;
        i64 spi = (budget - 2 * AUG_A_BYTES) / stage;   // one issuer: the whole ring is its sub-ring
        if (spi < 2) return false;
        if (spi > MAX_STAGES) spi = MAX_STAGES;
        out->n_xbuf = 2;
        out->spi = static_cast<int>(spi);
        out->cps = 1;
        out->smem_bytes = static_cast<size_t>(fixed + 2 * AUG_A_BYTES + spi * stage);
        return true;
    }
    const i64 xbuf = static_cast<i64>(nchunks) * X_CHUNK_BYTES + AUG_A_BYTES;
    const int want_xbuf = n_tiles <= 2 ? MAX_XBUF : 2;
    for (int n_xbuf = want_xbuf; n_xbuf >= 1; --n_xbuf) {
        const int cand[3] = {nchunks, (nchunks + 1) / 2, 1};
        for (int ci = 0; ci < 3; ++ci) {
            const int cps = cand[ci];
            if (ci > 0 && cps == cand[ci - 1]) continue;
            const i64 stage = static_cast<i64>(cps) * C_HALF_BYTES + AUG_B_HALF;
            i64 spi = (budget - n_xbuf * xbuf) / (NUM_ISSUERS * stage);
            if (spi < 1) continue;
            const i64 per_tile = (nchunks + cps - 1) / cps;
            if (spi > 2 * per_tile) spi = 2 * per_tile;       // two tiles per issuer are plenty
            if (spi * NUM_ISSUERS > MAX_STAGES) spi = MAX_STAGES / NUM_ISSUERS;
            // with a single X buffer left, take what fits; otherwise insist on a whole tile per issuer
            if (spi * cps < nchunks && n_xbuf > 1) continue;
            out->n_xbuf = n_xbuf;
            out->spi = static_cast<int>(spi);
            out->cps = cps;
            out->smem_bytes = static_cast<size_t>(fixed + n_xbuf * xbuf + spi * NUM_ISSUERS * stage);
            return true;
        }
    }
    return false;
}
}  // namespace

// whether the pair kernel has a shared-memory layout for these sizes (the caller checks before it enqueues anything)
bool assign_pair_supports(const DeviceInfo& di, int Dk, int K) {
    PairPlan pl;
    return plan_pair(di, (Dk + KCHUNK - 1) / KCHUNK, (K + BLOCK_N - 1) / BLOCK_N, Dk > kAssignResidentMaxD, &pl);
}

// X and C as for launch_assign_tc (C may be the zero-padded copy: Dc columns, a multiple of 64); the half-norm
// operand `caug` must have been written (the caller ran the prologue).  Dk > 512 selects the wide mode: xaug and
// xrowm as launch_row_aug wrote them for this X.
int launch_assign_pair(const cake_bf16* X, const cake_bf16* C, int B, i64 N, int Dk, int Dc, int K, const void* caug,
                       bool exact, int* out_idx, float* out_dist, double* inertia, int inertia_stride, int* status,
                       const DeviceInfo& di, cudaStream_t s, const void* xaug, const float* xrowm) {
    const bool wide = Dk > kAssignResidentMaxD;
    if (wide && (!xaug || !xrowm)) return CAKE_ERR_NULL;
    Params p;
    p.B = B; p.N = N; p.D = Dk; p.K = K;
    p.nchunks = (Dk + KCHUNK - 1) / KCHUNK;
    p.ksteps_last = (Dk - (p.nchunks - 1) * KCHUNK + UMMA_K - 1) / UMMA_K;
    p.m_tiles = static_cast<int>((N + 2 * BLOCK_M - 1) / (2 * BLOCK_M));
    p.n_tiles = (K + BLOCK_N - 1) / BLOCK_N;
    p.total_tiles = static_cast<i64>(B) * p.m_tiles;
    p.Kpad = padded_k(K);
    p.out_idx = out_idx; p.out_dist = out_dist; p.status = status;
    p.inertia = inertia; p.inertia_stride = inertia_stride;
    p.row_m = xrowm;
    p.Npad = round_up(N, 2 * BLOCK_M);
    if (p.total_tiles == 0) return CAKE_OK;

    PairPlan pl;
    if (!plan_pair(di, p.nchunks, p.n_tiles, wide, &pl)) return CAKE_ERR_UNSUPPORTED;
    p.n_xbuf = pl.n_xbuf;
    p.spi = pl.spi;
    p.cps = pl.cps;
    p.n_stages = pl.spi * (wide ? 1 : NUM_ISSUERS);

    CUtensorMap tx, tc, ta, txa;
    int rc = make_tmap_bf16_rows(&tx, X, Dk, N, B, BLOCK_M);
    if (rc != CAKE_OK) return rc;
    rc = make_tmap_bf16_rows(&tc, C, Dc, K, B, BLOCK_N / 2);
    if (rc != CAKE_OK) return rc;
    rc = make_tmap_rows16(&ta, caug, static_cast<i64>(B) * p.Kpad, BLOCK_N / 2);
    if (rc != CAKE_OK) return rc;
    if (wide) {
        rc = make_tmap_rows16(&txa, xaug, static_cast<i64>(B) * p.Npad, BLOCK_M);
        if (rc != CAKE_OK) return rc;
    } else {
        txa = ta;   // not read
    }

    using Kernel = void (*)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, const Params);
    static const Kernel kernels[6] = {assign_pair_kernel<true, false>,  assign_pair_kernel<false, false>,
                                      assign_pair_kernel<true, true>,   assign_pair_kernel<false, true>,
                                      assign_pair_kernel<true, false, true>, assign_pair_kernel<false, false, true>};
    static bool attr_done[64] = {false};   // per device; benign race: the attribute calls are idempotent
    const bool known = di.device >= 0 && di.device < 64;
    if (!known || !attr_done[di.device]) {
        for (Kernel k : kernels)
            if (cudaFuncSetAttribute(reinterpret_cast<const void*>(k), cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess)
                return CAKE_ERR_CUDA;
        if (known) attr_done[di.device] = true;
    }
    // one CTA per SM, in pairs; no more pairs than row tiles
    i64 pairs = di.sm_count / 2;
    if (pairs > p.total_tiles) pairs = p.total_tiles;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(2 * pairs));
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = pl.smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 2;
    const bool bulk = !wide && p.n_tiles >= 8;   // measured: 2-4 % at K >= 2048, nothing or a small loss below
    const Kernel kernel = kernels[(wide ? 4 : bulk ? 2 : 0) + (exact ? 1 : 0)];
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, tx, tc, ta, txa, p);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return CAKE_ERR_CUDA;
    }
    note_launches(1);
    return CAKE_OK;
}

}  // namespace cake
