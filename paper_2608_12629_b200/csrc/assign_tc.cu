// Fused nearest-centroid assignment on the sm_100a tensor cores.
//
// Operation (paper Section 5, "Flash-KMeans clean-start workload"): for every point the squared
// Euclidean distance to all K centroids and the arg-min.  The whole expansion
//     m + d(x,c)/2 = m + ||x||^2/2 - x.c + ||c||^2/2
// is accumulated in tensor memory in fp32: the D-long contraction -x.c runs with the B operand
// negated, and one extra 16-wide k-step adds the two half-norms (the X side carries
// [xh xm xl 1 1 1 0..], the centroid side [1 1 1 ch cm cl 0..], each half-norm split into three bf16
// terms so that nothing of its fp32 value is lost).  m is a per-row margin, a power of two between
// 2^-12 and 2^-11 of ||x||^2, added to ||x||^2/2 before the split: it keeps every accumulator of the
// row positive when the true distance is zero and rounding noise is not (a point that is its own
// centroid), so that accumulators order like their bit patterns.  Every accumulator is a plain fp32
// number whose error follows ||x||^2 + ||c_k||^2 of ITS OWN centroid: one centroid of huge norm
// does not touch the resolution of the others.  Padded centroid rows carry a half-norm of 2^120
// and lose to every real one.  The epilogue only has to find a row minimum; the N x K matrix never
// exists outside tensor memory.
//
// One persistent CTA per SM, 16 warps, four roles:
//   warp 8  producer : TMA.  A 128-row X tile (whole D) into one of the X buffers per row tile (up to
//                      four row tiles ahead); per centroid tile of 256 rows, D/64 chunks of 64 columns
//                      (128-byte swizzle) through an mbarrier ring.  A ring stage holds one chunk, or two
//                      when the chunk count is even (one wait and one commit for both), and has room
//                      for the tile's 4 KiB block of split half-norms, which arrives (bulk copy) on the
//                      barrier of the tile's last stage.
//   warps 9-11 MMA   : one thread each issues tcgen05.mma (M=128, N=256, K=16, bf16 -> fp32); centroid
//                      tiles go round robin over the three (tile t: issuer t mod 3, accumulator t mod 2
//                      of two 256-column TMEM accumulators); tcgen05.commit frees ring slots and
//                      publishes finished accumulators.
//                      With one or two centroid tiles per row tile a second instantiation makes
//                      warp 11 a producer for the X tiles alone and keeps two issuers.  With a single
//                      centroid tile (K <= 256) that fits beside an even number of X buffers, the tile
//                      stays in shared memory (loaded once per problem) and row tiles alternate between
//                      the two issuers and between the two epilogue warpgroups (see the kernel); two
//                      centroid tiles (K <= 512, D <= 128) stay resident too, one per issuer.
//   warps 0-7 epilogue: warp w reads TMEM lanes 32*(w%4).. (one X row per thread) and columns
//                      128*(w/4).. of every tile with tcgen05.ld and keeps a running minimum per row.
//                      The two column halves are merged through shared memory per row tile.
//   warps 12-15 norms : one thread per X row forms ||x||^2/2 from the shared-memory X tile and writes
//                      the X-side operand of the extra k-step, one row tile ahead of the MMA warps.
// Barrier discipline: every mbarrier has waiters that see each of its phases, and whoever refills a
// buffer waits for every reader of it (a parity wait that falls two phases behind never returns).
// Two epilogue policies (ties to the lowest index):
//   packed : key = the accumulator's bits with the low 7 replaced by the column (one logic
//            instruction); a plain 3-input float minimum over the keys finds value and position at
//            once, no branch.  Values are compared with 17 significant bits, i.e. to 2^-16 of the
//            half-distance itself: far inside the tolerance of 1e-3 (||x||^2 + ||c||^2), whatever the
//            norms of the other centroids.
//   exact  : minimum of the full fp32 values; the position is looked up only when a 32-column group
//            beats the running best.
// Every wait is bounded: on expiry the CTA raises CAKE_ERR_TIMEOUT in the status word, all roles
// leave their loops, TMEM is freed and the kernel returns.
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
constexpr int MMA_WARP = 9;             // warps 9, 10 (and 11): the MMA issuers
constexpr int MAX_ISSUERS = 3;
constexpr int XLOAD_WARP = 11;          // or warp 11 loads the X tiles (then two issuers)
constexpr int AUX_WARP0 = 12;           // warps 12..15: row norms
constexpr int NUM_WARPS = 16;
constexpr int EPI_REGS = 192;           // registers per thread after reallocation: epilogue warpgroups
constexpr int AUX_REGS = 56;            // ... and the producer / MMA / norm warpgroups
constexpr int NUM_THREADS = NUM_WARPS * 32;
constexpr uint32_t X_CHUNK_BYTES = BLOCK_M * 128;        // 16 KiB
constexpr uint32_t C_CHUNK_BYTES = BLOCK_N * 128;        // 32 KiB: 256 centroid rows x 64 columns
// Operands of the extra k-step: only columns 0..7 are non-zero, so each buffer holds just those
// (one 16-byte row per X row / centroid) and every descriptor points its second 8-column core
// matrices at one shared block of zeros.
constexpr uint32_t AUG_A_BYTES = BLOCK_M * 16;           // 2 KiB
constexpr uint32_t AUG_B_BYTES = kAssignAugTileBytes;    // 4 KiB
// a ring stage: one or two centroid chunks plus room for the tile's half-norm block, which rides with the
// last chunk (Params::cps, Params::stage_bytes)
constexpr uint32_t AUG_ZERO_BYTES = BLOCK_N * 16;        // 4 KiB of zeros
constexpr uint32_t OH_BYTES = 128 * 128 * 2;             // FUSE: the one-hot operand, 128 clusters x 128 rows of a tile, bf16
constexpr int MAX_STAGES = 6;
constexpr int MAX_XBUF = 6;                              // (more than four only in the fused mode)
constexpr int MAX_XBUF_PLAIN = 4;
#ifndef GATE_MIN_TILES
#define GATE_MIN_TILES 64                                 // centroid tiles per row tile from which the gated epilogue is used
#endif
constexpr int MAX_XCHUNKS = 8;                           // 64-column chunks of an X tile (D <= 512)
constexpr int TMEM_COLS = 512;
constexpr uint32_t CTRL_BYTES = 6144;  // barriers, TMEM pointer, abort flag, merge scratch, row margins
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;
constexpr uint32_t WAIT_SLICE_NS = 20000;   // longest single sleep inside a wait
constexpr uint32_t COL_MASK = 0x7Fu;   // packed policy: 7 bits address the 128 columns of a half tile
constexpr uint32_t F32_INF = 0x7f800000u;

// Kept as small as it gets (112 bytes; with the two tensor maps 368 bytes of kernel parameters): a larger parameter
// block measurably slows the many-tile kernel down although not one instruction of it reads the extra members -- 24 more
// bytes cost 5-10 % (D = 64, K = 16,384: 1.22 -> 1.34 ms; D = 128, K = 4,096: 0.87 -> 0.94 ms), whatever their position.
// Hence the narrow integer types.
struct Params {
    i64 N;
    i64 total_tiles;      // B * m_tiles
    const uint8_t* caug;  // [B][n_tiles][4 KiB] centroid-side operand of the extra k-step
    int* out_idx;
    float* out_dist;
    double* inertia;      // optional: inertia[b * inertia_stride] += sum of the problem's distances
    int* status;
    float* fuse_sums;     // FUSE: [gridDim.x][128][round_up(D, 16)] partial sums per CTA; fuse_counts [gridDim.x][128]
    int* fuse_counts;
    int B, K;
    int m_tiles;          // ceil(N / 128)
    int n_tiles;          // ceil(K / 256)
    uint32_t stage_bytes; // cps * 32 KiB + 4 KiB; resident centroids: bytes of one chunk of the tile (rows * 128),
                          // the tile's chunks lie one behind the other, its 4 KiB half-norm block after them
    int inertia_stride;
    uint16_t D;
    uint16_t alt_epi;     // one centroid tile per row tile: the two epilogue warpgroups take whole row tiles in turn;
                          // the value is the number of accumulator columns in use (32..128, or 256)
    uint8_t nchunks;      // ceil(D / 64)
    uint8_t ksteps_last;  // UMMA k-steps in the last chunk
    uint8_t n_stages;     // ring depth (stages)
    uint8_t cps;          // centroid chunks per ring stage: 2 when nchunks is even (half the barrier traffic), else 1
    uint8_t n_xbuf;       // X buffers (1..6)
    uint8_t res_c;        // 1: alt_epi and the centroid tile stays in shared memory (loaded once per problem): the two
                          // issuers share no ring and each works on its own row tiles only; 2: two resident
                          // tiles, issuer i computes tile i of every row tile (shared epilogue)
    uint8_t knn_k;        // TOPK instantiations (unused otherwise); out_idx / out_dist are then [N][2][TOPK]: one sorted
                          // list per column half, merged by a small kernel afterwards
    uint8_t fuse_oh2;     // FUSE: 1 = one one-hot buffer per epilogue warpgroup (else both share one)
};
static_assert(sizeof(Params) == 112, "kernel parameter block grew");

struct Ctrl {  // lives in shared memory
    uint64_t x_full[MAX_XBUF], x_empty[MAX_XBUF];
    // split X buffer (a single buffer whose 64-column chunks are filled and handed back one by one): chunk
    // c < nchunks - 1 has these barriers, the last chunk x_full[0] / x_empty[0]
    uint64_t xc_full[MAX_XCHUNKS], xc_empty[MAX_XCHUNKS];
    uint64_t ring_full[MAX_STAGES], ring_empty[MAX_STAGES];
    uint64_t tmem_full[2];
    // release of accumulator a, one barrier per issuer that may take it next: each barrier has a
    // single waiter that sees every one of its phases
    uint64_t tmem_empty[2][MAX_ISSUERS];
    uint64_t auga_full[MAX_XBUF];
    uint64_t merge_full[2], merge_empty[2];
    // FUSE: the one-hot operand of row tile t is written (by the epilogue warpgroup t % 2) / has been read by the MMAs
    // that add tile t to the sums (barrier t % 2); upd_done: the last such MMAs have completed
    uint64_t oh_full[2], oh_empty[2], upd_done[2];   // (upd_done[0] only)
    uint64_t turn[MAX_ISSUERS];   // resident-centroid mode: issuer i may issue its next tile's MMAs (the other one has issued its own)
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

#ifdef CAKE_ASSIGN_ACC
// Profiling build only (-DCAKE_ASSIGN_ACC): clocks spent in sections of CTA 0's issuing threads, added up in registers
__device__ long long g_acc[32];
#define ACC_DECL(v) long long v = 0
#define ACC_T(v) const long long v = clock64()
#define ACC_SUM(v, d) v += (d)
#define ACC_SET(v, d) v = (d)
#define ACC_DUMP(slot, v) do { if (blockIdx.x == 0) g_acc[slot] = v; } while (0)
#else
#define ACC_DECL(v) ((void)0)
#define ACC_T(v) ((void)0)
#define ACC_SUM(v, d) ((void)0)
#define ACC_SET(v, d) ((void)0)
#define ACC_DUMP(slot, v) ((void)0)
#endif
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
// tile).  Accumulators are positive finite floats (margin m), so the keys are too, and float order ==
// (value truncated to 17 significant bits, column) order.
__device__ __forceinline__ float packed_min32(const uint32_t (&r)[32], int col_base, float run, uint32_t kmask) {
    float v[32];
#pragma unroll
    for (int j = 0; j < 32; ++j)
        v[j] = __uint_as_float(ptx::and_or(r[j], kmask, static_cast<uint32_t>(col_base + j)));
    return fminf(run, min32(v));
}

// GATE: the group's smallest accumulator first, with 3-input minima on the raw values (half an instruction per column);
// the keys are built and reduced (another 1.1 per column) only if some row of the warp can still improve on `thr`, the
// truncated value of its best key before this tile.  Same result as without the gate: a group whose smallest truncated
// value is not below thr cannot replace the best (across tiles an equal value keeps the earlier tile), and leaving it
// out of the tile's minimum changes nothing else, since what remains is then not below thr either.  After t tiles a
// group still passes with probability about 1 - exp(-8 / t) on unordered centroids: worth it from 64 tiles on.
template <bool GATE>
__device__ __forceinline__ float group_min32(const uint32_t (&r)[32], int col_base, float run, float thr, uint32_t kmask) {
    if (GATE) {
        float v[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
        const float g = min32(v);
        const bool want = __uint_as_float(__float_as_uint(g) & kmask) < thr;
        if (!__any_sync(0xffffffffu, want)) return run;
    }
    return packed_min32(r, col_base, run, kmask);
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

// Top-k epilogue (k-nearest-neighbour search): a row's list of its KMAX smallest values so far, in registers, sorted
// ascending; candidates come in ascending column order, so one that equals an entry goes behind it (strict <) and
// equal distances end up ordered by column.  x = +inf is a no-op (lanes without a candidate in a warp-wide step).
template <int KMAX>
__device__ __forceinline__ void topk_insert_sorted(float (&lv)[KMAX], int (&li)[KMAX], float x, int col) {
#pragma unroll
    for (int s = KMAX - 1; s >= 1; --s) {
        const bool shift = x < lv[s - 1];          // the entry above moves down one place
        const bool here = !shift && x < lv[s];     // x lands here
        lv[s] = shift ? lv[s - 1] : (here ? x : lv[s]);
        li[s] = shift ? li[s - 1] : (here ? col : li[s]);
    }
    if (x < lv[0]) {
        lv[0] = x;
        li[0] = col;
    }
}

// XLOAD: warp 11 loads the X tiles and two warps issue MMAs (few centroid tiles per row tile);
// otherwise the centroid producer also loads X and three warps issue MMAs.
// Row tiles of a CTA.  Interleaved over the CTAs (blockIdx.x, blockIdx.x + gridDim.x, ...), except for a batch
// of problems with resident centroids: there the CTA takes as many row tiles as interleaving would give it,
// but consecutive ones, so that it meets few problems (every change of problem reloads the resident tile:
// 32 problems of 512 row tiles on 148 CTAs change problem every 3.5 tiles when interleaved).
// first_tile: (problem, row tile) of the CTA's first tile; tile_step: distance to its next one.
template <bool CONSEC>
__device__ __forceinline__ void first_tile(const Params& p, int& tb, int& tmt) {
    if (CONSEC) {
        const i64 q = p.total_tiles / gridDim.x, r = p.total_tiles - q * gridDim.x;
        const i64 first = blockIdx.x * q + (static_cast<i64>(blockIdx.x) < r ? static_cast<i64>(blockIdx.x) : r);
        tb = static_cast<int>(first / p.m_tiles);
        tmt = static_cast<int>(first - static_cast<i64>(tb) * p.m_tiles);
    } else {
        tb = static_cast<int>(blockIdx.x / static_cast<unsigned>(p.m_tiles));
        tmt = static_cast<int>(blockIdx.x % static_cast<unsigned>(p.m_tiles));
    }
}
template <bool CONSEC>
__device__ __forceinline__ int tile_step() { return CONSEC ? 1 : static_cast<int>(gridDim.x); }

// CONSEC: consecutive row tiles per CTA (a batch of problems with resident centroids: see first_tile)
// XSPLIT: one X buffer (all that fits beside the centroid ring when D > 256) whose chunks are loaded, consumed
// and handed back one by one, so that the next row tile's first chunks arrive while this one's last are in use
// BULK: the many-tile epilogue loads a whole 128-column slice, releases the accumulator and then reduces; otherwise
// it reduces each 32-column group while the next one is being loaded (a template parameter and not a run-time
// choice: with both epilogues in one kernel every shape measured 3-8 % slower)
// TOPK (0, 8 or 32): instead of the arg-min each epilogue thread keeps the TOPK smallest accumulators of its row and
// column half (k-nearest-neighbour search: the "centroids" are the database rows); many-tile structure, packed gate.
// FUSE (resident mode with at most 128 centroids and D <= 128, one problem): the kernel also adds every row tile to
// per-cluster sums while the tile is still in shared memory -- on the tensor core, as sums += onehot^T X with the
// assignment written as a one-hot bf16 operand -- so that the centroid update needs no second pass over X.
// NARROW: the resident single-tile mode with at most 128 centroids (or D <= 64), packed policy, whole X buffers: the
// epilogue for at most 128 centroids (two register buffers) in an instantiation of its own.  The shared code for such tiles (four buffers, a run-time branch
// beside the 256-column epilogue) spills 64 registers and ran 25-35 % slower at 64 < K <= 128; it remains for the
// exact policy, the split X buffer and the fused update (where it is the only branch and does not spill).
template <bool PACKED, bool XLOAD, bool CONSEC = false, bool XSPLIT = false, bool BULK = false, int TOPK = 0, bool FUSE = false,
          bool NARROW = false, bool GATE = false>
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
    const uint32_t ring_off = static_cast<uint32_t>(p.n_xbuf) * xbuf_bytes;
    const uint32_t ring_base = smem_base + ring_off;
    // bytes of one resident centroid tile (chunks, then its half-norm block)
    const uint32_t res_tile_bytes = static_cast<uint32_t>(p.nchunks) * p.stage_bytes + AUG_B_BYTES;
    // FUSE: the one-hot operand sits behind the resident tile (a multiple of 4 KiB: 1024-byte aligned as the swizzle needs)
    const uint32_t oh_off = ring_off + res_tile_bytes;
    const uint32_t auga_off = ring_off + ((XLOAD && p.res_c) ? static_cast<uint32_t>(p.res_c) * res_tile_bytes
                                                             : static_cast<uint32_t>(p.n_stages) * p.stage_bytes) +
                              (FUSE ? OH_BYTES * (p.fuse_oh2 ? 2u : 1u) : 0u);
    const uint32_t zero_off = auga_off + static_cast<uint32_t>(p.n_xbuf) * AUG_A_BYTES;
    const uint32_t ctrl_off = zero_off + AUG_ZERO_BYTES;
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem + ctrl_off);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    constexpr int NUM_ISSUERS = XLOAD ? 2 : MAX_ISSUERS;

    if (threadIdx.x == 0) {
        for (int i = 0; i < MAX_XBUF; ++i) {
            ptx::mbar_init(ptx::smem_u32(&ctrl->x_full[i]), 1);
            // MMA issuers + 4 norm warps + the 4 epilogue warps that read the row margins
            // (TOPK: the upper column half reads the margins as well)
            // (one resident tile, whole X buffers: the epilogue's arrival comes after the accumulator is complete and stands
            // for the MMAs as well; FUSE: the thread that issues the update commits)
            ptx::mbar_init(ptx::smem_u32(&ctrl->x_empty[i]),
                           ((XLOAD && p.res_c == 1) ? ((XSPLIT || FUSE) ? 1 : 0) : NUM_ISSUERS) + 4 + 4 + (TOPK ? 4 : 0));
            ptx::mbar_init(ptx::smem_u32(&ctrl->auga_full[i]), 4);
        }
        for (int i = 0; i < MAX_XCHUNKS; ++i) {
            ptx::mbar_init(ptx::smem_u32(&ctrl->xc_full[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctrl->xc_empty[i]), ((XLOAD && p.res_c == 1) ? 1 : NUM_ISSUERS) + 4);   // MMA issuers + 4 norm warps
        }
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(ptx::smem_u32(&ctrl->tmem_full[i]), 1);
            for (int j = 0; j < MAX_ISSUERS; ++j)
                ptx::mbar_init(ptx::smem_u32(&ctrl->tmem_empty[i][j]), (XLOAD && p.alt_epi) ? NUM_EPI_WARPS / 2 : NUM_EPI_WARPS);
            ptx::mbar_init(ptx::smem_u32(&ctrl->merge_full[i]), 4);
            ptx::mbar_init(ptx::smem_u32(&ctrl->merge_empty[i]), 4);
        }
        for (int i = 0; i < MAX_ISSUERS; ++i) ptx::mbar_init(ptx::smem_u32(&ctrl->turn[i]), 1);
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(ptx::smem_u32(&ctrl->oh_full[i]), NUM_EPI_WARPS / 2);
            ptx::mbar_init(ptx::smem_u32(&ctrl->oh_empty[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctrl->upd_done[i]), 1);
        }
        for (int i = 0; i < MAX_STAGES; ++i) {
            ptx::mbar_init(ptx::smem_u32(&ctrl->ring_full[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctrl->ring_empty[i]), NUM_ISSUERS);   // the consuming issuer and those passing over
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
    // FUSE: the one-hot operand starts as zeros and is kept up to date element by element (a thread clears the one it
    // set for its row in an earlier tile: fuse_last) ; fuse_cnt counts the rows of every cluster
    int* fuse_last = reinterpret_cast<int*>(ctrl->merge_best[0]);    // [2][128]: per one-hot buffer
    int* fuse_cnt = ctrl->merge_idx[0];
    if (FUSE) {
        for (uint32_t o = threadIdx.x * 16; o < OH_BYTES * (p.fuse_oh2 ? 2u : 1u); o += NUM_THREADS * 16)
            *reinterpret_cast<uint4*>(smem + oh_off + o) = make_uint4(0, 0, 0, 0);
        if (threadIdx.x < BLOCK_M) {
            fuse_last[threadIdx.x] = -1;
            fuse_last[BLOCK_M + threadIdx.x] = -1;
            fuse_cnt[threadIdx.x] = 0;
        }
    }
    ptx::fence_proxy_async_smem();
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
    // everything above touched no global memory: it may overlap the prologue kernel's tail
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();

    // The epilogue keeps a whole 128-column accumulator slice in registers; the other roles need few.
    // Registers move between warpgroups accordingly (warps 0-7 grow, warps 8-15 shrink).
    if (warp >= NUM_EPI_WARPS) {
    // (FUSE: the issuing threads carry the update's descriptors as well: eight registers more for them, eight fewer
    // for the epilogue warps; the sum stays the same)
    ptx::setmaxnreg_dec<FUSE ? AUX_REGS + 8 : AUX_REGS>();
    if (warp == PRODUCER_WARP) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t ring_it = 0, acc_it = 0;
            uint32_t rs = 0, rph = 0;   // ring stage and its phase
            bool ok = true;
            // X tiles run ahead of the MMAs by up to n_xbuf row tiles: `x_next` is the next row tile
            // whose X has not been requested yet, (ixb, ixph) the buffer and phase it will use
            i64 x_next = blockIdx.x;
            uint32_t ixb = 0, ixph = 0;
            auto issue_x = [&]() {
                const int tb = static_cast<int>(x_next / p.m_tiles);
                const int tmt = static_cast<int>(x_next % p.m_tiles);
                const uint32_t xfull = ptx::smem_u32(&ctrl->x_full[ixb]);
                ptx::mbar_arrive_expect_tx(xfull, xbuf_bytes);
                for (int c = 0; c < p.nchunks; ++c)
                    ptx::tma_load_3d(x_base + ixb * xbuf_bytes + c * X_CHUNK_BYTES, &tmap_x, xfull,
                                     c * KCHUNK, tmt * BLOCK_M, tb);
                x_next += gridDim.x;
                if (++ixb == static_cast<uint32_t>(p.n_xbuf)) { ixb = 0; ixph ^= 1u; }
            };
            // request X tiles for as long as a buffer is free, without ever blocking
            auto prefetch_x = [&]() {
                while (x_next < p.total_tiles &&
                       ptx::mbar_test_wait(ptx::smem_u32(&ctrl->x_empty[ixb]), ixph ^ 1u))
                    issue_x();
            };
            if (XLOAD && p.res_c) {
                // resident centroids: the whole tile (all chunks and the half-norm block) once per problem
                // this CTA meets; "stage 0" of the ring stands for the whole buffer
                int cur_b = -1;
                uint32_t pc = 0;
                int tb, tmt;
                first_tile<CONSEC>(p, tb, tmt);
                const int tmt_step = tile_step<CONSEC>();
                for (i64 tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x) {
                    if (tb != cur_b) {
                        ok = wait_bar(&ctrl->ring_empty[0], (pc & 1u) ^ 1u, ctrl, p.status);
                        if (!ok) break;
                        const uint32_t full = ptx::smem_u32(&ctrl->ring_full[0]);
                        // (res_c = 2: two centroid tiles, one behind the other)
                        ptx::mbar_arrive_expect_tx(full, static_cast<uint32_t>(p.res_c) *
                                                             res_tile_bytes);
                        for (int j = 0; j < p.res_c; ++j) {
                            const uint32_t tbase = ring_base + j * res_tile_bytes;
                            for (int c = 0; c < p.nchunks; ++c)
                                ptx::tma_load_3d(tbase + c * p.stage_bytes, &tmap_c, full, c * KCHUNK, j * BLOCK_N, tb);
                            ptx::bulk_load(tbase + res_tile_bytes - AUG_B_BYTES,
                                           p.caug + (static_cast<size_t>(tb) * p.res_c + j) * AUG_B_BYTES, AUG_B_BYTES, full);
                        }
                        cur_b = tb;
                        ++pc;
                    }
                    tmt += tmt_step;
                    while (tmt >= p.m_tiles) { tmt -= p.m_tiles; ++tb; }
                }
                if (!ok || pc == 0) {
                } else {
                    // leave only when the last load has landed (bounded)
                    const uint64_t t0 = ptx::globaltimer_ns();
                    while (!ptx::mbar_try_wait(ptx::smem_u32(&ctrl->ring_full[0]), (pc - 1u) & 1u) &&
                           ptx::globaltimer_ns() - t0 < 100000000ull) {
                    }
                }
                if (FUSE && ok) {
                    // The centroids are in (one problem): this thread now issues the MMAs of the update, tile by tile:
                    // sums (128 clusters on the TMEM lanes x D, columns 128..) += onehot^T X once the tile's epilogue has
                    // written the one-hot operand.  A = one-hot, K-major (the rows of the tile are the contraction);
                    // B = the X tile as it lies in its buffer, read MN-major: 64-column atoms X_CHUNK_BYTES apart, 8-row
                    // groups 1024 B apart.  The two MMA issuers of the assign spend all their time on their own
                    // instruction streams; eight more MMAs per tile there halved the kernel's speed.
                    constexpr uint32_t KSTEP = (UMMA_K * 2) >> 4;
                    const uint32_t idesc_upd = ptx::umma_idesc_bf16(BLOCK_M, (p.D + 15) & ~15) | ptx::UMMA_IDESC_B_MN_MAJOR;
                    const uint32_t d_sums = tmem_base + BLOCK_N / 2;
                    const uint32_t nxb = static_cast<uint32_t>(p.n_xbuf);
                    uint32_t t_it = 0;
                    for (i64 tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x, ++t_it) {
                        const uint32_t g = t_it & 1u;
                        ok = wait_bar(&ctrl->oh_full[g], (t_it >> 1) & 1u, ctrl, p.status);
                        if (!ok) break;
                        ptx::tc_fence_after();
                        const uint32_t uxb = t_it % nxb;
                        const uint32_t a0 = ptx::umma_desc_lo_sw128(smem_base + oh_off + (p.fuse_oh2 ? g * OH_BYTES : 0u));
                        const uint32_t b0 = (((x_base + uxb * xbuf_bytes) & 0x3FFFFu) >> 4) | ((X_CHUNK_BYTES >> 4) << 16);
#pragma unroll
                        for (uint32_t ks = 0; ks < BLOCK_M / UMMA_K; ++ks) {
                            const uint32_t a_lo = a0 + (ks >> 2) * (X_CHUNK_BYTES >> 4) + (ks & 3u) * KSTEP;
                            const uint32_t b_lo = b0 + ks * ((UMMA_K * 128u) >> 4);
                            if (ks == 0 && t_it == 0)
                                ptx::umma_bf16_lohi<false>(d_sums, a_lo, ptx::UMMA_DESC_HI_SW128, b_lo, ptx::UMMA_DESC_HI_SW128, idesc_upd);
                            else
                                ptx::umma_bf16_lohi<true>(d_sums, a_lo, ptx::UMMA_DESC_HI_SW128, b_lo, ptx::UMMA_DESC_HI_SW128, idesc_upd);
                        }
                        ptx::umma_commit(ptx::smem_u32(&ctrl->oh_empty[g]));
                        ptx::umma_commit(ptx::smem_u32(&ctrl->x_empty[uxb]));
                    }
                    if (ok) ptx::umma_commit(ptx::smem_u32(&ctrl->upd_done[0]));
                }
            } else {
            for (i64 tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x) {
                const int b = static_cast<int>(tile / p.m_tiles);
                if (!XLOAD) prefetch_x();
                if (!XLOAD && x_next <= tile) {   // this tile's own X is still outstanding: its buffer must free up
                    ok = wait_bar(&ctrl->x_empty[ixb], ixph ^ 1u, ctrl, p.status);
                    if (!ok) break;
                    issue_x();
                }
                const uint8_t* caug_b = p.caug + static_cast<size_t>(b) * p.n_tiles * AUG_B_BYTES;
                for (int nt = 0; ok && nt < p.n_tiles; ++nt, ++acc_it) {
                    for (int c = 0; c < p.nchunks; c += p.cps, ++ring_it) {
                        if (!XLOAD) prefetch_x();
                        ok = wait_bar(&ctrl->ring_empty[rs], rph ^ 1u, ctrl, p.status);
                        if (!ok) break;
                        const uint32_t full = ptx::smem_u32(&ctrl->ring_full[rs]);
                        const uint32_t stage = ring_base + rs * p.stage_bytes;
                        const bool last = c + p.cps == p.nchunks;
                        ptx::mbar_arrive_expect_tx(full, static_cast<uint32_t>(p.cps) * C_CHUNK_BYTES + (last ? AUG_B_BYTES : 0u));
                        for (int j = 0; j < p.cps; ++j)
                            ptx::tma_load_3d(stage + j * C_CHUNK_BYTES, &tmap_c, full, (c + j) * KCHUNK, nt * BLOCK_N, b);
                        if (last)   // the tile's half-norm block rides with its last chunk
                            ptx::bulk_load(stage + static_cast<uint32_t>(p.cps) * C_CHUNK_BYTES,
                                           caug_b + static_cast<size_t>(nt) * AUG_B_BYTES, AUG_B_BYTES, full);
                        if (++rs == static_cast<uint32_t>(p.n_stages)) { rs = 0; rph ^= 1u; }
                    }
                    if (!ok) break;
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
        }
    } else if (XLOAD && warp == XLOAD_WARP) {
        // ------------------------------------------------------------ X producer (few centroid tiles per row tile)
        // A 128-row X tile per row tile, into the next X buffer the moment that buffer is free (up to
        // n_xbuf row tiles ahead of the MMAs).  With one or two centroid tiles per row tile the kernel
        // is as fast as X arrives, and behind the centroid stream's barriers in one thread it arrives
        // late: here the X loads have a thread of their own, at the price of the third MMA issuer.
        if (lane == 0) {
            uint32_t ixb = 0, ixph = 0;
            int tb, tmt;
            first_tile<CONSEC>(p, tb, tmt);
                const int tmt_step = tile_step<CONSEC>();
            bool ok = true;
            for (i64 tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x) {
                if (XSPLIT) {
                    // chunk by chunk, each as soon as the previous row tile is done with it
                    for (int c = 0; ok && c < p.nchunks; ++c) {
                        const bool lastc = c == p.nchunks - 1;
                        ok = wait_bar(lastc ? &ctrl->x_empty[0] : &ctrl->xc_empty[c], ixph ^ 1u, ctrl, p.status);
                        if (!ok) break;
                        const uint32_t full = ptx::smem_u32(lastc ? &ctrl->x_full[0] : &ctrl->xc_full[c]);
                        ptx::mbar_arrive_expect_tx(full, X_CHUNK_BYTES);
                        ptx::tma_load_3d(x_base + c * X_CHUNK_BYTES, &tmap_x, full, c * KCHUNK, tmt * BLOCK_M, tb);
                    }
                    if (!ok) break;
                } else {
                ok = wait_bar(&ctrl->x_empty[ixb], ixph ^ 1u, ctrl, p.status);
                if (!ok) break;
                const uint32_t xfull = ptx::smem_u32(&ctrl->x_full[ixb]);
                ptx::mbar_arrive_expect_tx(xfull, xbuf_bytes);
                for (int c = 0; c < p.nchunks; ++c)
                    ptx::tma_load_3d(x_base + ixb * xbuf_bytes + c * X_CHUNK_BYTES, &tmap_x, xfull,
                                     c * KCHUNK, tmt * BLOCK_M, tb);
                }
                if (++ixb == static_cast<uint32_t>(p.n_xbuf)) { ixb = 0; ixph ^= 1u; }
                tmt += tmt_step;
                while (tmt >= p.m_tiles) { tmt -= p.m_tiles; ++tb; }
            }
            if (!ok) {   // aborting: a bounded time for the X loads in flight to land
                const uint64_t t0 = ptx::globaltimer_ns();
                while (ptx::globaltimer_ns() - t0 < 20000ull) {
                }
            }
        }
    } else if (warp >= MMA_WARP && warp < MMA_WARP + NUM_ISSUERS) {
        // ------------------------------------------------------------ MMA issuers
        // Three warps (two when warp 11 loads X), one issuing thread each; centroid tiles go round robin
        // over them (tile t to issuer t mod 3, into accumulator t mod 2).  One thread cannot keep the tensor pipe fed: per
        // tile it spends about three times the pipe's 9 x 128 clocks on its own instruction stream
        // (waits, descriptor arithmetic, commits, and MMA issue that blocks at the pipe's pace), so
        // three of them take turns.  No two ever hold the same accumulator or ring slot at a time.
        if (lane == 0) {
            const uint32_t iss = static_cast<uint32_t>(warp - MMA_WARP);
            constexpr uint32_t idesc_aug = ptx::umma_idesc_bf16(BLOCK_M, BLOCK_N);
            constexpr uint32_t idesc_main = idesc_aug | ptx::UMMA_IDESC_NEGATE_B;   // accumulates -x.c
            // descriptors are (low, high) words with the high word constant; stage / phase counters
            // are stepped instead of divided; full 64-column chunks issue four MMAs back to back
            constexpr uint32_t KSTEP = (UMMA_K * 2) >> 4;   // descriptor units per k-step
            const uint32_t nstg = static_cast<uint32_t>(p.n_stages);
            uint32_t s = 0, ph = 0;                         // ring position of the next chunk (all tiles)
            uint32_t xb = 0, xph = 0;                       // X buffer and its phase
            uint32_t acc_it = 0;
            constexpr uint32_t n_iss = NUM_ISSUERS;
            uint32_t turn = 0;                              // acc_it mod n_iss
            uint32_t rel0 = 0, rel1 = 0;                    // releases of accumulator 0 / 1 this issuer has consumed
            bool ok = true;
            if (XLOAD && p.res_c) {
                // Resident centroids, one tile per row tile: issuer i takes the row tiles with
                // tile_it % 2 == i, and with them accumulator i and the X buffers of its parity (their
                // number is even): every barrier it waits on has phases only it consumes.  The two meet
                // only when the problem changes: each hands the centroid buffer back once its own MMAs
                // on it are done, and waits for the next problem's centroids.
                int cur_b = -1;
                uint32_t pc = 0, tile_it = 0;
                int tb, tmt;
                ACC_DECL(acc_main); ACC_DECL(acc_tail); ACC_DECL(acc_n); ACC_DECL(acc_all);
                ACC_DECL(acc_top); ACC_DECL(acc_xf); ACC_DECL(acc_pre); ACC_DECL(t_prev);
                ACC_T(t_loop0);
                first_tile<CONSEC>(p, tb, tmt);
                const int tmt_step = tile_step<CONSEC>();
                const uint32_t nxb = static_cast<uint32_t>(p.n_xbuf);
                const uint32_t idesc_aug_n = ptx::umma_idesc_bf16(BLOCK_M, p.alt_epi ? p.alt_epi : BLOCK_N);
                const uint32_t idesc_main_n = idesc_aug_n | ptx::UMMA_IDESC_NEGATE_B;
                if (!XSPLIT && !FUSE && p.res_c == 1) {
                    // One resident tile, whole X buffers (the fused update keeps the general loop below: it measured 3 % faster
                    // there): this loop is the thread's whole life and every row tile passes
                    // through it, so it does as little as it can.  Buffer, phases and descriptors are stepped (no
                    // divisions); one wait covers X and its half-norm operand (the norm warps arrive on it after they
                    // have seen the X tile); the X buffer is handed back by the epilogue warpgroup once the accumulator
                    // is complete, not by a commit of this thread.
                    const uint32_t n_my = static_cast<uint32_t>((p.total_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x);
                    const uint32_t d_tmem = tmem_base + iss * BLOCK_N;
                    const uint32_t b0 = ptx::umma_desc_lo_sw128(ring_base);
                    const uint32_t b_step = p.stage_bytes >> 4;
                    const uint32_t augb_lo = ptx::umma_desc_lo_aug(ring_base + res_tile_bytes - AUG_B_BYTES, smem_base + zero_off);
                    const int turn_c = (p.nchunks - 1) >> 1;   // the turn goes on after the first half of the MMAs
                    uint32_t rxb = iss, rxph = 0, k_own = 0;   // this issuer's X buffer and phase, its own tiles so far
                    for (; ok && tile_it < n_my; ++tile_it) {
                        const int b_now = tb;
                        tmt += tmt_step;
                        while (tmt >= p.m_tiles) { tmt -= p.m_tiles; ++tb; }
                        if (b_now != cur_b) {
                            if (cur_b >= 0) ptx::umma_commit(ptx::smem_u32(&ctrl->ring_empty[0]));
                            ok = wait_bar(&ctrl->ring_full[0], pc & 1u, ctrl, p.status);
                            if (!ok) break;
                            cur_b = b_now;
                            ++pc;
                        }
                        if ((tile_it & 1u) != iss) continue;
                        ACC_T(t_0);
                        ACC_SUM(acc_top, t_prev ? t_0 - t_prev : 0);
                        ok = wait_bar(&ctrl->auga_full[rxb], rxph, ctrl, p.status);
                        if (!ok) break;
                        ACC_T(t_1);
                        if (k_own > 0u) {
                            ok = wait_bar(&ctrl->tmem_empty[iss][iss], (k_own - 1u) & 1u, ctrl, p.status);
                            if (!ok) break;
                        }
                        // (the issuers take turns, see below: issuer 0 waits for issuer 1's previous tile, issuer 1 for
                        // issuer 0's current one)
                        if (iss == 1u || k_own > 0u) {
                            ok = wait_bar(&ctrl->turn[iss], (iss == 1u ? k_own : k_own - 1u) & 1u, ctrl, p.status);
                            if (!ok) break;
                        }
                        ptx::tc_fence_after();
                        ACC_T(t_a);
                        uint32_t a_lo = ptx::umma_desc_lo_sw128(x_base + rxb * xbuf_bytes), b_lo = b0;
                        for (int c = 0; c < p.nchunks; ++c, a_lo += X_CHUNK_BYTES >> 4, b_lo += b_step) {
                            if (c == 0)
                                ptx::umma_bf16_lohi<false>(d_tmem, a_lo, ptx::UMMA_DESC_HI_SW128, b_lo, ptx::UMMA_DESC_HI_SW128, idesc_main_n);
                            else
                                ptx::umma_bf16_lohi<true>(d_tmem, a_lo, ptx::UMMA_DESC_HI_SW128, b_lo, ptx::UMMA_DESC_HI_SW128, idesc_main_n);
                            if (c < p.nchunks - 1 || p.ksteps_last == KCHUNK / UMMA_K) {   // a whole chunk: straight-line code
#pragma unroll
                                for (int ks = 1; ks < KCHUNK / UMMA_K; ++ks)
                                    ptx::umma_bf16_lohi<true>(d_tmem, a_lo + ks * KSTEP, ptx::UMMA_DESC_HI_SW128,
                                                              b_lo + ks * KSTEP, ptx::UMMA_DESC_HI_SW128, idesc_main_n);
                            } else {
                                for (int ks = 1; ks < p.ksteps_last; ++ks)
                                    ptx::umma_bf16_lohi<true>(d_tmem, a_lo + ks * KSTEP, ptx::UMMA_DESC_HI_SW128,
                                                              b_lo + ks * KSTEP, ptx::UMMA_DESC_HI_SW128, idesc_main_n);
                            }
                            if (c == turn_c) ptx::mbar_arrive(ptx::smem_u32(&ctrl->turn[iss ^ 1u]));
                        }
                        ACC_T(t_b);
                        ptx::umma_bf16_lohi<true>(d_tmem,
                                                  ptx::umma_desc_lo_aug(smem_base + auga_off + rxb * AUG_A_BYTES, smem_base + zero_off),
                                                  ptx::UMMA_DESC_HI_AUG, augb_lo, ptx::UMMA_DESC_HI_AUG, idesc_aug_n);
                        ptx::umma_commit(ptx::smem_u32(&ctrl->tmem_full[iss]));
                        ACC_T(t_c);
                        ACC_SUM(acc_main, t_b - t_a); ACC_SUM(acc_tail, t_c - t_b); ACC_SUM(acc_n, 1);
                        ACC_SUM(acc_xf, t_1 - t_0); ACC_SUM(acc_pre, t_a - t_1);
                        ACC_SET(t_prev, t_c);
                        ++k_own;
                        rxb += 2u;
                        if (rxb >= nxb) { rxb -= nxb; rxph ^= 1u; }
                    }
                } else
                for (i64 tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x, ++tile_it) {
                    const int b_now = tb;
                    tmt += tmt_step;
                    while (tmt >= p.m_tiles) { tmt -= p.m_tiles; ++tb; }
                    if (b_now != cur_b) {
                        if (cur_b >= 0) ptx::umma_commit(ptx::smem_u32(&ctrl->ring_empty[0]));
                        ok = wait_bar(&ctrl->ring_full[0], pc & 1u, ctrl, p.status);
                        if (!ok) break;
                        cur_b = b_now;
                        ++pc;
                    }
                    // two resident tiles: issuer i computes centroid tile i of EVERY row tile into accumulator i
                    // (the shared epilogue reads both and merges)
                    const bool both = p.res_c == 2;
                    if (!both && (tile_it & 1u) != iss) continue;
                    const uint32_t rxb = tile_it % nxb, rxph = (tile_it / nxb) & 1u;
                    // (split X buffer: both issuers share the one buffer, so an issuer sees only every other
                    // phase of its barriers and may look at them only once it has the turn: the other issuer
                    // has then seen all of the previous row tile's phases complete)
                    if (!XSPLIT) ok = wait_bar(&ctrl->x_full[rxb], rxph, ctrl, p.status);
                    if (!ok) break;
                    const uint32_t use = both ? tile_it : tile_it >> 1;   // how often this accumulator has been used before
                    if (use > 0u) {
                        ok = wait_bar(&ctrl->tmem_empty[iss][iss], (use - 1u) & 1u, ctrl, p.status);
                        if (!ok) break;
                    }
                    // The two issuers hand the tensor pipe to each other tile by tile.  Left alone they fall
                    // into step (X tiles arrive in pairs), their MMAs interleave instruction by instruction,
                    // both accumulators complete together and both epilogue warpgroups then work while
                    // the pipe idles.  In turns, one tile's MMAs run while the other tile is being reduced.
                    // (order of the groups of MMAs: one tile: t0 t1 t2 ..., issuers alternating; two tiles: t0/A t0/B
                    // t1/A t1/B ...; issuer 0 waits for issuer 1's previous group, issuer 1 for issuer 0's current one)
                    if (both ? (iss == 1u || tile_it > 0u) : tile_it > 0u) {
                        const uint32_t tph = both ? (iss == 0u ? tile_it - 1u : tile_it) : (tile_it - 1u) >> 1;
                        ok = wait_bar(&ctrl->turn[iss], tph & 1u, ctrl, p.status);
                        if (!ok) break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t d_tmem = tmem_base + iss * BLOCK_N;
                    const uint32_t c_base = ring_base + (both ? iss * res_tile_bytes : 0u);   // this issuer's centroid tile
                    uint32_t a_lo = ptx::umma_desc_lo_sw128(x_base + rxb * xbuf_bytes);
                    for (int c = 0; c < p.nchunks; ++c, a_lo += X_CHUNK_BYTES >> 4) {
                        if (XSPLIT) {
                            ok = wait_bar(c == p.nchunks - 1 ? &ctrl->x_full[0] : &ctrl->xc_full[c], rxph, ctrl, p.status);
                            if (!ok) break;
                        }
                        const uint32_t b_lo = ptx::umma_desc_lo_sw128(c_base + c * p.stage_bytes);
                        const int nk = (c == p.nchunks - 1) ? p.ksteps_last : KCHUNK / UMMA_K;
                        if (c == 0)
                            ptx::umma_bf16_lohi<false>(d_tmem, a_lo, ptx::UMMA_DESC_HI_SW128, b_lo,
                                                       ptx::UMMA_DESC_HI_SW128, idesc_main_n);
                        else
                            ptx::umma_bf16_lohi<true>(d_tmem, a_lo, ptx::UMMA_DESC_HI_SW128, b_lo,
                                                      ptx::UMMA_DESC_HI_SW128, idesc_main_n);
                        if (nk == KCHUNK / UMMA_K) {   // a whole chunk: straight-line code
#pragma unroll
                            for (int ks = 1; ks < KCHUNK / UMMA_K; ++ks)
                                ptx::umma_bf16_lohi<true>(d_tmem, a_lo + ks * KSTEP, ptx::UMMA_DESC_HI_SW128,
                                                          b_lo + ks * KSTEP, ptx::UMMA_DESC_HI_SW128, idesc_main_n);
                        } else {
                            for (int ks = 1; ks < nk; ++ks)
                                ptx::umma_bf16_lohi<true>(d_tmem, a_lo + ks * KSTEP, ptx::UMMA_DESC_HI_SW128,
                                                          b_lo + ks * KSTEP, ptx::UMMA_DESC_HI_SW128, idesc_main_n);
                        }
                        if (XSPLIT && c < p.nchunks - 1) ptx::umma_commit(ptx::smem_u32(&ctrl->xc_empty[c]));
                    }
                    if (!ok) break;
                    ptx::mbar_arrive(ptx::smem_u32(&ctrl->turn[iss ^ 1u]));
                    ok = wait_bar(&ctrl->auga_full[rxb], rxph, ctrl, p.status);
                    if (!ok) break;
                    ptx::umma_bf16_lohi<true>(d_tmem,
                                              ptx::umma_desc_lo_aug(smem_base + auga_off + rxb * AUG_A_BYTES, smem_base + zero_off),
                                              ptx::UMMA_DESC_HI_AUG,
                                              ptx::umma_desc_lo_aug(c_base + res_tile_bytes - AUG_B_BYTES,
                                                                    smem_base + zero_off),
                                              ptx::UMMA_DESC_HI_AUG, idesc_aug_n);
                    ptx::umma_commit(ptx::smem_u32(&ctrl->tmem_full[iss]));
                    // (FUSE: the X buffer is also an operand of the update, whose MMAs come after these: the thread that
                    // issues those hands the buffer back)
                    if (!FUSE) ptx::umma_commit(ptx::smem_u32(&ctrl->x_empty[rxb]));
                }
                ACC_T(t_loop1);
                ACC_SUM(acc_all, t_loop1 - t_loop0);
                ACC_DUMP(iss * 8 + 0, acc_main); ACC_DUMP(iss * 8 + 1, acc_tail); ACC_DUMP(iss * 8 + 2, acc_n); ACC_DUMP(iss * 8 + 3, acc_all);
                ACC_DUMP(iss * 8 + 4, acc_top); ACC_DUMP(iss * 8 + 5, acc_xf); ACC_DUMP(iss * 8 + 6, acc_pre);
            } else
            for (i64 tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x) {
                // every phase of the shared barriers is observed, also in row / centroid tiles this
                // issuer has no work in: a parity wait must never fall two phases behind
                if (!XSPLIT) ok = wait_bar(&ctrl->x_full[xb], xph, ctrl, p.status);   // (split: chunk by chunk, below)
                if (!ok) break;
                bool have_aug = false;
                bool owned = false;   // this issuer had a centroid tile of this row tile (at most one when XSPLIT)
                const uint32_t a_lo_tile = ptx::umma_desc_lo_sw128(x_base + xb * xbuf_bytes);
                const uint32_t auga_lo = ptx::umma_desc_lo_aug(smem_base + auga_off + xb * AUG_A_BYTES,
                                                               smem_base + zero_off);
                for (int nt = 0; ok && nt < p.n_tiles; ++nt, ++acc_it, turn = (turn + 1 == n_iss) ? 0 : turn + 1) {
                    if (turn != iss) {
                        // Another issuer's tile: pass over its ring slots, but see each of them filled
                        // and only then let the slot be refilled.  That keeps the issuers in tile order
                        // and this one at most one phase behind any slot (a parity wait that falls two
                        // phases behind waits for ever).
                        for (int c = 0; ok && c < p.nchunks; c += p.cps) {
                            ok = wait_bar(&ctrl->ring_full[s], ph, ctrl, p.status);
                            if (ok) ptx::mbar_arrive(ptx::smem_u32(&ctrl->ring_empty[s]));
                            if (++s == nstg) { s = 0; ph ^= 1u; }
                        }
                        continue;
                    }
                    const uint32_t acc = acc_it & 1u;
                    const uint32_t d_tmem = tmem_base + acc * BLOCK_N;
                    // the accumulator was last used by tile acc_it - 2, whose release is addressed to
                    // this issuer (the first two tiles find their accumulators free)
                    if (acc_it >= 2u) {
                        const uint32_t rel = acc ? rel1 : rel0;
                        ok = wait_bar(&ctrl->tmem_empty[acc][iss], rel & 1u, ctrl, p.status);
                        if (!ok) break;
                        if (acc) ++rel1; else ++rel0;
                    }
                    ptx::tc_fence_after();
                    owned = true;
                    uint32_t a_lo = a_lo_tile;
                    for (int c0 = 0; c0 < p.nchunks; c0 += p.cps) {
                        if (XSPLIT) {   // (one chunk per stage in this mode) this chunk of X has landed
                            ok = wait_bar(c0 == p.nchunks - 1 ? &ctrl->x_full[0] : &ctrl->xc_full[c0], xph, ctrl, p.status);
                            if (!ok) break;
                        }
                        ok = wait_bar(&ctrl->ring_full[s], ph, ctrl, p.status);
                        if (!ok) break;
                        const uint32_t stage = ring_base + s * p.stage_bytes;
                        for (int j = 0; j < p.cps; ++j, a_lo += X_CHUNK_BYTES >> 4) {
                            const int c = c0 + j;
                            const uint32_t b_lo = ptx::umma_desc_lo_sw128(stage + j * C_CHUNK_BYTES);
                            const int nk = (c == p.nchunks - 1) ? p.ksteps_last : KCHUNK / UMMA_K;
                            if (c == 0)
                                ptx::umma_bf16_lohi<false>(d_tmem, a_lo, ptx::UMMA_DESC_HI_SW128, b_lo,
                                                           ptx::UMMA_DESC_HI_SW128, idesc_main);
                            else
                                ptx::umma_bf16_lohi<true>(d_tmem, a_lo, ptx::UMMA_DESC_HI_SW128, b_lo,
                                                          ptx::UMMA_DESC_HI_SW128, idesc_main);
                            if (nk == KCHUNK / UMMA_K) {
#pragma unroll
                                for (uint32_t ks = 1; ks < KCHUNK / UMMA_K; ++ks)
                                    ptx::umma_bf16_lohi<true>(d_tmem, a_lo + ks * KSTEP, ptx::UMMA_DESC_HI_SW128,
                                                              b_lo + ks * KSTEP, ptx::UMMA_DESC_HI_SW128, idesc_main);
                            } else {
                                for (int ks = 1; ks < nk; ++ks)
                                    ptx::umma_bf16_lohi<true>(d_tmem, a_lo + ks * KSTEP, ptx::UMMA_DESC_HI_SW128,
                                                              b_lo + ks * KSTEP, ptx::UMMA_DESC_HI_SW128, idesc_main);
                            }
                        }
                        if (c0 + p.cps == p.nchunks) {
                            // the extra k-step: + ||x||^2/2 + ||c||^2/2 + M + m; its centroid side came with this stage
                            if (!have_aug) {
                                ok = wait_bar(&ctrl->auga_full[xb], xph, ctrl, p.status);
                                if (!ok) break;
                                have_aug = true;
                            }
                            ptx::umma_bf16_lohi<true>(d_tmem, auga_lo, ptx::UMMA_DESC_HI_AUG,
                                                      ptx::umma_desc_lo_aug(stage + static_cast<uint32_t>(p.cps) * C_CHUNK_BYTES,
                                                                            smem_base + zero_off),
                                                      ptx::UMMA_DESC_HI_AUG, idesc_aug);
                        }
                        ptx::umma_commit(ptx::smem_u32(&ctrl->ring_empty[s]));
                        // split X buffer: this issuer's only tile of the row tile is done with the chunk
                        if (XSPLIT && c0 < p.nchunks - 1) ptx::umma_commit(ptx::smem_u32(&ctrl->xc_empty[c0]));
                        if (++s == nstg) { s = 0; ph ^= 1u; }
                    }
                    if (!ok) break;
                    ptx::umma_commit(ptx::smem_u32(&ctrl->tmem_full[acc]));
                }
                if (XSPLIT && ok && !owned) {
                    // no tile of this row tile: see every chunk filled (a parity wait must not fall two phases
                    // behind) and hand it back at once
                    for (int c = 0; ok && c < p.nchunks - 1; ++c) {
                        ok = wait_bar(&ctrl->xc_full[c], xph, ctrl, p.status);
                        if (ok) ptx::mbar_arrive(ptx::smem_u32(&ctrl->xc_empty[c]));
                    }
                    if (ok) ok = wait_bar(&ctrl->x_full[0], xph, ctrl, p.status);
                }
                if (ok && !have_aug) ok = wait_bar(&ctrl->auga_full[xb], xph, ctrl, p.status);
                // this issuer's MMAs on the X buffer are done when this commit fires (it fires at once
                // if the issuer had no tile in this row tile)
                if (ok) ptx::umma_commit(ptx::smem_u32(&ctrl->x_empty[xb]));
                if (++xb == static_cast<uint32_t>(p.n_xbuf)) { xb = 0; xph ^= 1u; }
            }
        }
    } else if (warp >= AUX_WARP0) {
        // ------------------------------------------------------------ norm warps
        // One thread per X row: ||x||^2/2 from the swizzled X tile (16-byte granule g of row r sits
        // at position g ^ (r & 7); the order of the granules does not matter for a sum), split into
        // three bf16 terms and written, with the row's offset M and margin m, as the X-side operand of
        // the extra k-step.  These warps run a row tile ahead of the MMA warps, so the operand is
        // ready when the first centroid tile needs it.
        const int r = (warp - AUX_WARP0) * 32 + lane;
        uint32_t xb = 0, xph = 0;
        bool ok = true;
        for (i64 tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x) {
            if (!XSPLIT) ok = wait_bar(&ctrl->x_full[xb], xph, ctrl, p.status);
            if (!ok) break;
            const uint8_t* xrow = smem + xb * xbuf_bytes + r * 128;
            float xn0 = 0.f, xn1 = 0.f, xn2 = 0.f, xn3 = 0.f;
            for (int c = 0; c < p.nchunks; ++c) {
                if (XSPLIT) {
                    // chunk by chunk: the one before is handed back once the whole warp has read it
                    if (c > 0) {
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->xc_empty[c - 1]));
                    }
                    ok = wait_bar(c == p.nchunks - 1 ? &ctrl->x_full[0] : &ctrl->xc_full[c], xph, ctrl, p.status);
                    if (!ok) break;
                }
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
            if (!ok) break;
            const float xn = (xn0 + xn1) + (xn2 + xn3);
            // margin m = 2^(e-11) for ||x||^2 in [2^e, 2^(e+1)), at least 2^-100: above the rounding noise of a
            // zero distance (D * 2^-24 of ||x||^2 at worst), and a power of two so that it disturbs no exact sum
            const uint32_t xe = __float_as_uint(xn) >> 23;
            const uint32_t mbits = (xe > 38u ? xe - 11u : 27u) << 23;
            uint32_t hi, mid, lo;
            split3(fmaf(0.5f, xn, __uint_as_float(mbits)), hi, mid, lo);
            ctrl->row_m[xb][r] = __uint_as_float(mbits);
            // interleaved (no-swizzle) K-major layout, columns 0..7 only: one 16-byte row per X row
            const uint32_t one = 0x3F80u;
            *reinterpret_cast<uint4*>(smem + auga_off + xb * AUG_A_BYTES + r * 16) =
                make_uint4(hi | (mid << 16), lo | (one << 16), one | (one << 16), 0u);
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                ptx::mbar_arrive(ptx::smem_u32(&ctrl->auga_full[xb]));
                ptx::mbar_arrive(ptx::smem_u32(&ctrl->x_empty[xb]));
            }
            if (++xb == static_cast<uint32_t>(p.n_xbuf)) { xb = 0; xph ^= 1u; }
        }
    }
    } else {
        // ------------------------------------------------------------ epilogue warps
        ptx::setmaxnreg_inc<FUSE ? EPI_REGS - 8 : EPI_REGS>();
        const int wg = warp >> 2;            // column half of every tile
        const int q = warp & 3;              // TMEM lane quarter this warp may read
        const int r = q * 32 + lane;         // row inside the X tile
        uint32_t tile_it = 0, acc_it = 0;
        constexpr uint32_t n_iss = NUM_ISSUERS;
        uint32_t next_iss = 2 % n_iss;         // (acc_it + 2) mod n_iss
        uint32_t exb = 0, exph = 0;          // X buffer (slot of the row margins) and its phase
        // all ones but the 7 column bits; formed from a run-time value (K < 2^31) so that it stays in a register
        // and each key is ONE logic instruction (register, register, immediate column)
        const uint32_t kmask = ~COL_MASK | (static_cast<uint32_t>(p.K) >> 31);
        bool ok = true;
        double dsum = 0.0;                   // this thread's share of the current problem's inertia
        int dsum_b = -1;
        // one fp64 atomic per warp and problem
        auto flush_inertia = [&]() {
            if ((wg == 0 || (XLOAD && p.alt_epi)) && p.inertia && dsum_b >= 0) {
                double t = dsum;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
                if (lane == 0) atomicAdd(p.inertia + static_cast<size_t>(dsum_b) * p.inertia_stride, t);
            }
            dsum = 0.0;
        };
        // (problem, row tile) of the current tile, stepped instead of divided
        int b, mt;
        first_tile<CONSEC>(p, b, mt);
        const int mt_step = tile_step<CONSEC>();
        auto next_tile = [&]() {
            mt += mt_step;
            while (mt >= p.m_tiles) { mt -= p.m_tiles; ++b; }
        };
        // One centroid tile per row tile: accumulator, X buffer and warpgroup all alternate with the row
        // tile.  Warpgroup g takes the row tiles with tile_it % 2 == g and reads all 256 columns of their
        // accumulator (two passes of 128), so nothing is merged through shared memory and neither
        // warpgroup ever waits for the other; with an even number of X buffers each warpgroup sees every
        // phase of the barriers of "its" buffers.
        // (this warpgroup's X buffer is stepped, not divided out of the tile count: the loop is the warpgroup's critical
        // path; with a single buffer -- XSPLIT -- it is not used)
        uint32_t axb = static_cast<uint32_t>(wg) % static_cast<uint32_t>(p.n_xbuf);
        ACC_DECL(ea_n); ACC_DECL(ea_w1); ACC_DECL(ea_w2); ACC_DECL(ea_red); ACC_DECL(ea_st);
        ACC_DECL(ea_w3); ACC_DECL(ea_oh); ACC_DECL(ea_top); ACC_DECL(ea_prev);
        // (the loop walks this warpgroup's own tiles only: every other one of the CTA's)
        if (XLOAD && p.alt_epi) {
        const uint32_t n_alt = static_cast<uint32_t>((p.total_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x);
        if (wg == 1) next_tile();
        for (tile_it = static_cast<uint32_t>(wg); ok && tile_it < n_alt; tile_it += 2u, next_tile(), next_tile()) {
            ACC_T(e_0);
            ACC_SUM(ea_top, ea_prev ? e_0 - ea_prev : 0);
            if (b != dsum_b) {
                flush_inertia();
                dsum_b = b;
            }
            // the row margins are there long before the accumulator is: fetch them while waiting for it
            // (the X buffer is not refilled before the issuer's MMAs on it have completed either)
            ACC_T(e_1);
            const uint32_t as = tile_it & 1u, aph = (tile_it >> 1) & 1u;
            ok = wait_bar(&ctrl->tmem_full[as], aph, ctrl, p.status);
            if (!ok) break;
            ACC_T(e_2);
            // The row margins: written by the norm warps before they completed auga_full, which the issuer waited for
            // before the tile's last MMA, so they are there once the accumulator is complete (no wait of this warp's own).
            // The X buffer, and with it this slot, is handed to a later row tile only after this warp's arrival (the
            // norm warps could otherwise get two row tiles of the buffer ahead and overwrite the margins); the MMAs
            // that read the buffer are complete as well, so outside FUSE and XSPLIT (where the update's or the
            // issuers' commits do that) the arrival also stands for them.
            const uint32_t mxb = XSPLIT ? 0u : axb;
            const float rowM = ctrl->row_m[mxb][r];
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->x_empty[mxb]));
            ptx::tc_fence_after();
            float best = __uint_as_float(F32_INF);
            int bsel = 0;
            if (NARROW && p.alt_epi <= BLOCK_N / 2) {
                // at most 128 centroids: only the 32-column groups that hold some were written; they go through two
                // register buffers, the load of the next group in flight while one is reduced
                const int ng = p.alt_epi >> 5;
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + as * BLOCK_N;
                uint32_t ra[32], rb[32];
                ptx::tmem_ld_x32(taddr, ra);
                ptx::tmem_ld_wait(ra);
                if (ng > 1) ptx::tmem_ld_x32_before(taddr + 32, rb, ra);
                if (PACKED) best = packed_min32(ra, 0, __uint_as_float(F32_INF), kmask);
                else exact_scan32(ra, 0, best, bsel);
                if (ng > 1) {
                    ptx::tmem_ld_wait_after(rb, best);
                    if (ng > 2) ptx::tmem_ld_x32_before(taddr + 64, ra, rb);
                    if (PACKED) best = packed_min32(rb, 32, best, kmask);
                    else exact_scan32(rb, 32, best, bsel);
                    if (ng > 2) {
                        ptx::tmem_ld_wait_after(ra, best);
                        if (ng > 3) ptx::tmem_ld_x32_before(taddr + 96, rb, ra);
                        if (PACKED) best = packed_min32(ra, 64, best, kmask);
                        else exact_scan32(ra, 64, best, bsel);
                        if (ng > 3) {
                            ptx::tmem_ld_wait_after(rb, best);
                            if (PACKED) best = packed_min32(rb, 96, best, kmask);
                            else exact_scan32(rb, 96, best, bsel);
                        }
                    }
                }
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->tmem_empty[as][(tile_it + 2u) % n_iss]));
                if (PACKED) bsel = 0;
            } else if (FUSE || (!NARROW && p.alt_epi <= BLOCK_N / 2)) {   // (FUSE: at most 128 centroids by construction; else: the exact policy, split X buffer)
                // at most 128 centroids: only the 32-column groups that hold some were written
                const int ng = p.alt_epi >> 5;
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + as * BLOCK_N;
                uint32_t ra[32], rb[32], rc[32], rd[32];
                ptx::tmem_ld_x32(taddr, ra);
                if (ng > 1) ptx::tmem_ld_x32(taddr + 32, rb);
                if (ng > 2) ptx::tmem_ld_x32(taddr + 64, rc);
                if (ng > 3) ptx::tmem_ld_x32(taddr + 96, rd);
                ptx::tmem_ld_wait(ra);
                ptx::reg_dep(rb);
                ptx::reg_dep(rc);
                ptx::reg_dep(rd);
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->tmem_empty[as][(tile_it + 2u) % n_iss]));
                if (PACKED) {
                    best = packed_min32(ra, 0, __uint_as_float(F32_INF), kmask);
                    if (ng > 1) best = packed_min32(rb, 32, best, kmask);
                    if (ng > 2) best = packed_min32(rc, 64, best, kmask);
                    if (ng > 3) best = packed_min32(rd, 96, best, kmask);
                    bsel = 0;
                } else {
                    exact_scan32(ra, 0, best, bsel);
                    if (ng > 1) exact_scan32(rb, 32, best, bsel);
                    if (ng > 2) exact_scan32(rc, 64, best, bsel);
                    if (ng > 3) exact_scan32(rd, 96, best, bsel);
                }
            } else {
                // lower 128 columns into registers; then every 32-column group is reduced and its
                // registers take the matching group of the upper half at once: the accumulator goes
                // back to its issuer after one and a half passes instead of two
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + as * BLOCK_N;
                uint32_t ra[32], rb[32], rc[32], rd[32];
                ptx::tmem_ld_x32(taddr, ra);
                ptx::tmem_ld_x32(taddr + 32, rb);
                ptx::tmem_ld_x32(taddr + 64, rc);
                ptx::tmem_ld_x32(taddr + 96, rd);
                ptx::tmem_ld_wait(ra);
                ptx::reg_dep(rb);
                ptx::reg_dep(rc);
                ptx::reg_dep(rd);
                float lo_min = 0.f;
                if (PACKED) {
                    lo_min = packed_min32(ra, 0, __uint_as_float(F32_INF), kmask);
                    ptx::tmem_ld_x32(taddr + 128, ra);
                    lo_min = packed_min32(rb, 32, lo_min, kmask);
                    ptx::tmem_ld_x32(taddr + 160, rb);
                    lo_min = packed_min32(rc, 64, lo_min, kmask);
                    ptx::tmem_ld_x32(taddr + 192, rc);
                    lo_min = packed_min32(rd, 96, lo_min, kmask);
                    ptx::tmem_ld_x32(taddr + 224, rd);
                } else {
                    exact_scan32(ra, 0, best, bsel);
                    ptx::tmem_ld_x32(taddr + 128, ra);
                    exact_scan32(rb, 32, best, bsel);
                    ptx::tmem_ld_x32(taddr + 160, rb);
                    exact_scan32(rc, 64, best, bsel);
                    ptx::tmem_ld_x32(taddr + 192, rc);
                    exact_scan32(rd, 96, best, bsel);
                    ptx::tmem_ld_x32(taddr + 224, rd);
                }
                ptx::tmem_ld_wait(ra);
                ptx::reg_dep(rb);
                ptx::reg_dep(rc);
                ptx::reg_dep(rd);
                ptx::tc_fence_before();
                __syncwarp();
                // to the issuer of row tile tile_it + 2, which takes this accumulator next
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->tmem_empty[as][(tile_it + 2u) % n_iss]));
                if (PACKED) {
                    float hi_min = packed_min32(ra, 0, __uint_as_float(F32_INF), kmask);
                    hi_min = packed_min32(rb, 32, hi_min, kmask);
                    hi_min = packed_min32(rc, 64, hi_min, kmask);
                    hi_min = packed_min32(rd, 96, hi_min, kmask);
                    // across the halves only the (truncated) value decides: an equal value keeps the lower half
                    best = lo_min;
                    bsel = 0;
                    if (__uint_as_float(__float_as_uint(hi_min) & ~COL_MASK) <
                        __uint_as_float(__float_as_uint(lo_min) & ~COL_MASK)) {
                        best = hi_min;
                        bsel = 1;
                    }
                } else {
                    exact_scan32(ra, 128, best, bsel);
                    exact_scan32(rb, 160, best, bsel);
                    exact_scan32(rc, 192, best, bsel);
                    exact_scan32(rd, 224, best, bsel);
                }
            }
            float bval;
            int bidx;
            if (PACKED) {
                const uint32_t kb = __float_as_uint(best);
                bval = __uint_as_float(kb & ~COL_MASK);
                bidx = bsel * (BLOCK_N / 2) + static_cast<int>(kb & COL_MASK);
            } else {
                bval = best;
                bidx = bsel;
            }
            ACC_T(e_3);
            const i64 row = static_cast<i64>(mt) * BLOCK_M + r;
            if (row < p.N) {
                const size_t o = static_cast<size_t>(b) * static_cast<size_t>(p.N) + row;
                const float dist = fmaxf(0.f, 2.f * (bval - rowM));   // the accumulator is m + d/2
                p.out_idx[o] = bidx;
                if (p.out_dist) p.out_dist[o] = dist;
                dsum += static_cast<double>(dist);
            }
            if (!XSPLIT) {
                axb += 2u;
                if (axb >= static_cast<uint32_t>(p.n_xbuf)) axb -= static_cast<uint32_t>(p.n_xbuf);
            }
            ACC_T(e_4);
            ACC_SUM(ea_n, 1); ACC_SUM(ea_w1, e_1 - e_0); ACC_SUM(ea_w2, e_2 - e_1); ACC_SUM(ea_red, e_3 - e_2); ACC_SUM(ea_st, e_4 - e_3);
            ACC_SET(ea_prev, e_4);
            if (FUSE) {
                // The one-hot operand of this tile: element [cluster][row] of a 128 x 128 bf16 tile, K-major with the
                // 128-byte swizzle, two 64-row chunks.  The buffer is shared by both warpgroups (they alternate tiles):
                // the MMAs that read the previous tile's operand must have completed.
                // (one buffer per warpgroup: the MMAs on this warpgroup's previous tile)
                if (p.fuse_oh2 ? tile_it > 1u : tile_it > 0u) {
                    const uint32_t pt = p.fuse_oh2 ? tile_it - 2u : tile_it - 1u;
                    ok = wait_bar(&ctrl->oh_empty[pt & 1u], (pt >> 1) & 1u, ctrl, p.status);
                    if (!ok) break;
                }
                ACC_T(e_5);
                const uint32_t ohb = p.fuse_oh2 ? static_cast<uint32_t>(wg) : 0u;
                uint8_t* oh = smem + oh_off + ohb * OH_BYTES + (r >> 6) * X_CHUNK_BYTES + ((r & 7) << 1);
                const int g8 = (r & 63) >> 3;          // 16-byte granule of the row inside its chunk
                int* last = fuse_last + ohb * BLOCK_M;
                const int prev = last[r];
                if (prev >= 0) *reinterpret_cast<uint16_t*>(oh + prev * 128 + ((g8 ^ (prev & 7)) << 4)) = 0;
                int now = -1;
                if (row < p.N) {
                    now = bidx;
                    *reinterpret_cast<uint16_t*>(oh + now * 128 + ((g8 ^ (now & 7)) << 4)) = 0x3F80;
                    atomicAdd(fuse_cnt + now, 1);
                }
                last[r] = now;
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->oh_full[wg]));
                ACC_T(e_6);
                ACC_SUM(ea_w3, e_5 - e_4); ACC_SUM(ea_oh, e_6 - e_5);
                ACC_SET(ea_prev, e_6);
            }
        }
        }
        if (XLOAD && lane == 0 && (warp == 0 || warp == 4)) {
            ACC_DUMP(16 + wg * 8 + 0, ea_n); ACC_DUMP(16 + wg * 8 + 1, ea_top); ACC_DUMP(16 + wg * 8 + 2, ea_w1); ACC_DUMP(16 + wg * 8 + 3, ea_w2);
            ACC_DUMP(16 + wg * 8 + 4, ea_red); ACC_DUMP(16 + wg * 8 + 5, ea_st); ACC_DUMP(16 + wg * 8 + 6, ea_w3); ACC_DUMP(16 + wg * 8 + 7, ea_oh);
        }
        if (FUSE && ok && wg == 0) {
            // every tile has been added: the sums (clusters on the TMEM lanes, D columns) go out as this CTA's partial
            ok = wait_bar(&ctrl->upd_done[0], 0u, ctrl, p.status);
            if (ok) {
                ptx::tc_fence_after();
                const int ncol = (p.D + 15) & ~15;
                float* dst = p.fuse_sums + (static_cast<size_t>(blockIdx.x) * BLOCK_M + r) * ncol;
                for (int c0 = 0; c0 < ncol; c0 += 16) {
                    uint32_t v[16];
                    ptx::tmem_ld_x16(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + BLOCK_N / 2 + c0, v);
#pragma unroll
                    for (int j = 0; j < 16; j += 4)
                        *reinterpret_cast<uint4*>(dst + c0 + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                }
            }
        }
        // ---- TOPK: the row's sorted list (registers) of the smallest accumulators seen so far in this column half;
        // its last entry is the threshold a candidate has to beat (+inf until the list is full)
        constexpr int KL = TOPK ? TOPK : 1;
        float lv[KL] = {};
        int li[KL] = {};
        float stash[TOPK ? 32 : 1];                      // a group's values, parked in local memory while it is walked
        // One 32-column group.  Its smallest (truncated) value is compared with the threshold first; if any row of the
        // warp may have a candidate, the group is walked: every lane marks its candidates, then all lanes insert their
        // next candidate together, step by step (one copy of the insertion code, no lane waits for another lane's column).
        auto topk_group = [&](const uint32_t (&rg)[32], int col0) {
            const float gmin = packed_min32(rg, 0, __uint_as_float(F32_INF), kmask);
            const bool want = __uint_as_float(__float_as_uint(gmin) & ~COL_MASK) < lv[KL - 1];
            if (__any_sync(0xffffffffu, want)) {
                uint32_t m = 0;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float v = __uint_as_float(rg[j]);
                    stash[j] = v;
                    m |= (v < lv[KL - 1] && col0 + j < p.K) ? (1u << j) : 0u;   // (columns behind the last row: padding)
                }
                while (__any_sync(0xffffffffu, m != 0u)) {
                    const int j = m ? __ffs(static_cast<int>(m)) - 1 : 0;
                    const float x = m ? stash[j] : __uint_as_float(F32_INF);
                    m &= m - 1u;
                    topk_insert_sorted<KL>(lv, li, x, col0 + j);
                }
            }
        };
        ACC_DECL(mt_n); ACC_DECL(mt_wait); ACC_DECL(mt_row0); ACC_DECL(mt_hold); ACC_DECL(mt_red); ACC_DECL(mt_end); ACC_DECL(mt_top); ACC_DECL(mt_prev);
        for (i64 tile = blockIdx.x; !(XLOAD && p.alt_epi) && ok && tile < p.total_tiles; tile += gridDim.x, ++tile_it, next_tile()) {
            ACC_T(m_0);
            ACC_SUM(mt_top, mt_prev ? m_0 - mt_prev : 0);
            ACC_SUM(mt_n, 1);
            if (TOPK) {
#pragma unroll
                for (int s = 0; s < KL; ++s) {
                    lv[s] = __uint_as_float(F32_INF);
                    li[s] = -1;
                }
            }
            if (b != dsum_b) {
                flush_inertia();
                dsum_b = b;
            }
            float best = __uint_as_float(F32_INF);   // packed: a key; exact: a value
            int bsel = 0;                            // packed: tile number; exact: global column
            float rowM = 0.f;                        // this row's margin m (wg 0 only)
            for (int nt = 0; nt < p.n_tiles; ++nt, ++acc_it) {
                const uint32_t as = acc_it & 1u, aph = (acc_it >> 1) & 1u;
                ACC_T(m_1);
                ok = wait_bar(&ctrl->tmem_full[as], aph, ctrl, p.status);
                if (!ok) break;
                ACC_T(m_2);
                ACC_SUM(mt_wait, m_2 - m_1);
                ptx::tc_fence_after();
                if (nt == 0 && (wg == 0 || TOPK)) {
                    // Written by the norm warps before they completed auga_full.  The X buffer -- and with
                    // it this slot and the next phase of this barrier -- is handed to a later row tile
                    // only after these warps have arrived on x_empty: without that, with one centroid
                    // tile per row tile, the norm warps can get two row tiles of this buffer ahead,
                    // overwrite the margins and leave this parity wait behind for good.
                    ok = wait_bar(&ctrl->auga_full[exb], exph, ctrl, p.status);
                    if (!ok) break;
                    rowM = ctrl->row_m[exb][r];
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->x_empty[exb]));
                }
                ACC_T(m_3);
                ACC_SUM(mt_row0, m_3 - m_2);
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                       as * BLOCK_N + wg * (BLOCK_N / 2);
                if (TOPK) {
                    // two sites of the group code (ra, rb), run twice: the list lives in registers and its insertion
                    // is long, so the code is kept small
                    const int col0 = nt * BLOCK_N + wg * (BLOCK_N / 2);
                    uint32_t ra[32], rb[32];
                    ptx::tmem_ld_x32(taddr, ra);
                    ptx::tmem_ld_wait(ra);
#pragma unroll 1
                    for (int h = 0; h < 2; ++h) {
                        ptx::tmem_ld_x32_before(taddr + 64 * h + 32, rb, ra);
                        topk_group(ra, col0 + 64 * h);
                        ptx::tmem_ld_wait_after(rb, lv[KL - 1]);
                        if (h == 0) {
                            ptx::tmem_ld_x32_before(taddr + 64, ra, rb);
                        } else {
                            ptx::tc_fence_before();
                            __syncwarp();
                            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->tmem_empty[as][next_iss]));
                        }
                        topk_group(rb, col0 + 64 * h + 32);
                        if (h == 0) ptx::tmem_ld_wait_after(ra, lv[KL - 1]);
                    }
                } else if (!BULK) {
                    // The four 32-column groups go through two register buffers: the load of group g + 1 is in
                    // flight while group g is reduced (a warp that first loads everything and then reduces
                    // leaves the TMEM path idle half of the time and the ALU pipe the other half: both warps
                    // of a scheduler wait for the same accumulator and run in step).  The accumulator goes
                    // back to its MMA issuer when the last group has landed.
                    uint32_t ra[32], rb[32];
                    ptx::tmem_ld_x32(taddr, ra);
                    ptx::tmem_ld_wait(ra);
                    ptx::tmem_ld_x32_before(taddr + 32, rb, ra);
                    if (PACKED) {
                        const float thr = __uint_as_float(__float_as_uint(best) & ~COL_MASK);
                        float tmin = group_min32<GATE>(ra, 0, __uint_as_float(F32_INF), thr, kmask);
                        ptx::tmem_ld_wait_after(rb, tmin);
                        ptx::tmem_ld_x32_before(taddr + 64, ra, rb);
                        tmin = group_min32<GATE>(rb, 32, tmin, thr, kmask);
                        ptx::tmem_ld_wait_after(ra, tmin);
                        ptx::tmem_ld_x32_before(taddr + 96, rb, ra);
                        tmin = group_min32<GATE>(ra, 64, tmin, thr, kmask);
                        ptx::tmem_ld_wait_after(rb, tmin);
                        ptx::tc_fence_before();
                        __syncwarp();
                        // to the issuer of tile acc_it + 2, which takes this accumulator next
                        if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->tmem_empty[as][next_iss]));
                        trace_mark(ctrl, 100);
                        ACC_T(m_4); ACC_SUM(mt_hold, m_4 - m_3); ACC_SET(mt_prev, m_4);
                        tmin = group_min32<GATE>(rb, 96, tmin, thr, kmask);
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
                        if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->tmem_empty[as][next_iss]));
                        trace_mark(ctrl, 100);
                        ACC_T(m_4); ACC_SUM(mt_hold, m_4 - m_3); ACC_SET(mt_prev, m_4);
                        exact_scan32(rb, col0 + 96, best, bsel);
                    }
                } else {
                    // (D = 128 with many centroid tiles per row tile measured 3-6 % faster when the accumulator is
                    // handed back at once: all four groups are requested together, the accumulator is released as
                    // soon as they have landed, and the reduction runs on registers afterwards)
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
                    if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->tmem_empty[as][next_iss]));
                    trace_mark(ctrl, 100);
                    ACC_T(m_4); ACC_SUM(mt_hold, m_4 - m_3); ACC_SET(mt_prev, m_4);
                    if (PACKED) {
                        const float thr = __uint_as_float(__float_as_uint(best) & ~COL_MASK);
                        float tmin = group_min32<GATE>(ra, 0, __uint_as_float(F32_INF), thr, kmask);
                        tmin = group_min32<GATE>(rb, 32, tmin, thr, kmask);
                        tmin = group_min32<GATE>(rc, 64, tmin, thr, kmask);
                        tmin = group_min32<GATE>(rd, 96, tmin, thr, kmask);
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
                next_iss = (next_iss + 1 == n_iss) ? 0 : next_iss + 1;
                ACC_T(m_5);
                ACC_SUM(mt_red, mt_prev ? m_5 - mt_prev : 0);
                ACC_SET(mt_prev, m_5);
            }
            if (!ok) break;
            trace_mark(ctrl, 102);
            if (++exb == static_cast<uint32_t>(p.n_xbuf)) { exb = 0; exph ^= 1u; }
            if (TOPK) {
                // the list is sorted by (value, column): write it out, out_idx / out_dist [row][half][TOPK]; the two
                // halves are merged by a small kernel afterwards.  Unused places: index -1, distance +inf.
                const i64 row = static_cast<i64>(mt) * BLOCK_M + r;
                if (row < p.N) {
                    const size_t o = ((static_cast<size_t>(b) * static_cast<size_t>(p.N) + row) * 2 + wg) * KL;
#pragma unroll
                    for (int s = 0; s < KL; ++s) {
                        p.out_idx[o + s] = li[s];
                        p.out_dist[o + s] = fmaxf(0.f, 2.f * (lv[s] - rowM));
                    }
                }
                continue;
            }
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
                const i64 row = static_cast<i64>(mt) * BLOCK_M + r;
                if (row < p.N) {
                    const size_t o = static_cast<size_t>(b) * static_cast<size_t>(p.N) + row;
                    const float dist = fmaxf(0.f, 2.f * (bval - rowM));   // the accumulator is m + d/2
                    p.out_idx[o] = bidx;
                    if (p.out_dist) p.out_dist[o] = dist;
                    dsum += static_cast<double>(dist);
                }
            }
            trace_mark(ctrl, 103);
            ACC_T(m_6);
            ACC_SUM(mt_end, mt_prev ? m_6 - mt_prev : 0);
            ACC_SET(mt_prev, m_6);
        }
        if (!(XLOAD && p.alt_epi) && lane == 0 && (warp == 0 || warp == 4)) {
            ACC_DUMP(16 + wg * 8 + 0, mt_n); ACC_DUMP(16 + wg * 8 + 1, mt_top); ACC_DUMP(16 + wg * 8 + 2, mt_wait); ACC_DUMP(16 + wg * 8 + 3, mt_row0);
            ACC_DUMP(16 + wg * 8 + 4, mt_hold); ACC_DUMP(16 + wg * 8 + 5, mt_red); ACC_DUMP(16 + wg * 8 + 6, mt_end);
        }
        if (ok) flush_inertia();
    }

    // ---------------------------------------------------------------- teardown
    ptx::tc_fence_before();
    __syncthreads();
    if (FUSE && threadIdx.x < BLOCK_M) p.fuse_counts[static_cast<size_t>(blockIdx.x) * BLOCK_M + threadIdx.x] = fuse_cnt[threadIdx.x];
    if (warp == MMA_WARP) {
        __syncwarp();
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// Prologue: the centroid-side operand of the extra k-step.  One warp per padded centroid row k:
// h = ||c_k||^2 / 2 split into three bf16 terms, written as the 16-byte row [1 1 1 h_hi h_mid h_lo 0 0]
// (columns 0..7 of the operand in the interleaved K-major layout the MMA reads: 256 rows x 16 B = 4 KiB
// per tile; columns 8..15 are zeros the kernel supplies itself).  Rows k >= K carry h = 2^120 and can
// never win.  With `inertia` the kernel also zeroes inertia[b * inertia_stride] for the B <= 256
// problems (what the assign kernel adds to).
__global__ void __launch_bounds__(256)
centroid_aug_kernel(const cake_bf16* __restrict__ C, int K, int D, int Kpad, i64 total_rows,
                    uint8_t* __restrict__ caug, double* __restrict__ inertia,
                    int inertia_stride, int B, cake_bf16* __restrict__ cpad, int Dc) {
    ptx::grid_dep_wait();      // C may come from the kernel ahead (the previous iteration's division)
    ptx::grid_dep_launch();
    // the assign kernel adds the distances up here: start from zero
    if (inertia && blockIdx.x == 0 && static_cast<int>(threadIdx.x) < B)
        inertia[static_cast<size_t>(threadIdx.x) * inertia_stride] = 0.0;
    const i64 w = (static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (w >= total_rows) return;
    const i64 b = w / Kpad;
    const int k = static_cast<int>(w - b * Kpad);
    float acc = 0.f;
    if (k < K) {
        const cake_bf16* row = C + (static_cast<size_t>(b) * K + k) * D;
        if (D % 4 == 0) {   // rows are 8-byte aligned: four columns per load
            const uint2* row4 = reinterpret_cast<const uint2*>(row);
            for (int j = lane; j < D / 4; j += 32) {
                const uint2 q = __ldg(row4 + j);
                acc = aug::add_squares(acc, q.x, q.y);
            }
        } else {
            for (int d = lane; d < D; d += 32) {
                const float v = __uint_as_float(static_cast<uint32_t>(row[d]) << 16);
                acc = fmaf(v, v, acc);
            }
        }
        acc = aug::fold_lanes(acc);
        if (cpad) aug::copy_row_padded(row, D, cpad + (static_cast<size_t>(b) * K + k) * Dc, Dc, lane);
    }
    if (lane == 0) aug::write_row(caug, b, k, K, Kpad, acc);
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

int make_tmap_bf16_rows(CUtensorMap* m, const void* base, int D, i64 rows, int batch, int box_rows) {
    return make_tmap(m, base, D, rows, batch, box_rows);
}

// bytes viewed as rows of 16 (the half-norm operand: one 16-byte row per centroid); box = box_rows rows, no swizzle
int make_tmap_rows16(CUtensorMap* m, const void* base, i64 rows, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return CAKE_ERR_CUDA;
    cuuint64_t dims[2] = {16, static_cast<cuuint64_t>(rows)};
    cuuint64_t strides[1] = {16};
    cuuint32_t box[2] = {16, static_cast<cuuint32_t>(box_rows)};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? CAKE_OK : CAKE_ERR_CUDA;
}

#ifdef CAKE_ASSIGN_ACC
extern "C" __attribute__((visibility("default"))) int cake_debug_read_acc(long long* host) {
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(host, g_acc, sizeof(long long) * 32);
    return 32;
}
#endif
#ifdef CAKE_ASSIGN_TRACE
// Profiling build only: copies warp `w`'s trace records (3 x int64 each, up to `cap`) to `host`.
extern "C" __attribute__((visibility("default"))) int cake_debug_read_trace(int w, long long* host, int cap) {
    cudaDeviceSynchronize();
    if (w < 0 || w >= NUM_WARPS) return 0;
    const int n = cap < TRACE_CAP ? cap : TRACE_CAP;
    cudaMemcpyFromSymbol(host, g_trace, static_cast<size_t>(n) * 3 * sizeof(long long),
                         static_cast<size_t>(w) * TRACE_CAP * 3 * sizeof(long long));
    return n;
}
#endif

bool assign_tc_supports(int D) { return D >= 8 && D % 8 == 0 && D <= 512; }

size_t assign_tc_aug_bytes(i64 B, int K) {
    return static_cast<size_t>(B) * (padded_k(K) / BLOCK_N) * AUG_B_BYTES;
}

// The prologue of a tensor-core assign: the centroids' half-norm operand into caug (and the zero-padded copy of C
// into cpad, and zeros into the inertia entries when asked), with programmatic dependent launch allowed.
static int launch_centroid_prologue(const cake_bf16* C, int B, int D, int K, void* caug, cake_bf16* cpad, int Dc,
                                    double* inertia, int inertia_stride, bool zero_inertia, cudaStream_t s) {
    const int Kpad = padded_k(K);
    const i64 rows = static_cast<i64>(B) * Kpad;
    const i64 ctas = (rows * 32 + 255) / 256;
    if (zero_inertia && inertia && B > 256) {   // more problems than the prologue's first CTA has threads
        if (cudaMemset2DAsync(inertia, static_cast<size_t>(inertia_stride) * sizeof(double), 0, sizeof(double),
                              static_cast<size_t>(B), s) != cudaSuccess)
            return CAKE_ERR_CUDA;
    }
    cudaLaunchAttribute pdl[1];
    pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(ctas));
    cfg.blockDim = dim3(256);
    cfg.stream = s;
    cfg.attrs = pdl;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, centroid_aug_kernel, C, K, D, Kpad, rows, static_cast<uint8_t*>(caug),
                           (zero_inertia && B <= 256) ? inertia : static_cast<double*>(nullptr), inertia_stride,
                           B, cpad, Dc) != cudaSuccess) {
        cudaGetLastError();
        return CAKE_ERR_CUDA;
    }
    note_launches(1);
    return CAKE_OK;
}

int launch_assign_tc(const cake_bf16* X, const cake_bf16* C, int B, i64 N, int D, int K, void* caug,
                     bool exact, int* out_idx, float* out_dist, double* inertia,
                     int inertia_stride, bool zero_inertia, bool aug_ready, int* status, cudaStream_t s, int Dx,
                     cake_bf16* cpad, int knn_k, float* fuse_sums, int* fuse_counts, int* fuse_ctas, bool pair,
                     void* xaug, float* xrowm, bool xaug_ready) {
    // D: columns of a row of C; Dk: columns of a row of X and length of the contraction (D, or D rounded up to
    // a multiple of 8 with zeros in the copy of X); Dc: columns of a row of the centroid operand the kernel
    // streams (C itself, or its zero-padded copy of a multiple of 64 columns, written by the prologue)
    const int Dk = Dx ? Dx : D;
    const int Dc = cpad ? static_cast<int>(round_up(Dk, KCHUNK)) : D;
    const bool wide = assign_wide_supports(Dk);
    if ((!assign_tc_supports(Dk) && !wide) || Dk < D || (!cpad && Dk != D)) return CAKE_ERR_UNSUPPORTED;
    DeviceInfo di;
    int rc = current_device_info(&di);
    if (rc != CAKE_OK) return rc;
    if (di.cc_major != 10) return CAKE_ERR_DEVICE;
    if (wide) {
        // rows too long for a resident X tile: the CTA-pair kernel streams X beside the centroids
        if (knn_k != 0 || Dc % KCHUNK != 0 || !xaug || !xrowm || !assign_pair_supports(di, Dk, K)) return CAKE_ERR_UNSUPPORTED;
        if (fuse_ctas) *fuse_ctas = 0;
        if (N == 0) return CAKE_OK;
        if (!aug_ready) {
            rc = launch_centroid_prologue(C, B, D, K, caug, cpad, Dc, inertia, inertia_stride, zero_inertia, s);
            if (rc != CAKE_OK) return rc;
        }
        if (!xaug_ready && launch_row_aug(X, B, N, Dk, xaug, xrowm, s) != cudaSuccess) return CAKE_ERR_CUDA;
        return launch_assign_pair(X, cpad ? cpad : C, B, N, Dk, Dc, K, caug, exact, out_idx, out_dist, inertia, inertia_stride,
                                  status, di, s, xaug, xrowm);
    }

    Params p;
    p.B = B; p.N = N; p.D = Dk; p.K = K;
    p.nchunks = (Dk + KCHUNK - 1) / KCHUNK;
    p.ksteps_last = (Dk - (p.nchunks - 1) * KCHUNK + UMMA_K - 1) / UMMA_K;
    p.m_tiles = static_cast<int>((N + BLOCK_M - 1) / BLOCK_M);
    p.n_tiles = (K + BLOCK_N - 1) / BLOCK_N;
    p.total_tiles = static_cast<i64>(B) * p.m_tiles;
    p.caug = static_cast<const uint8_t*>(caug);
    p.out_idx = out_idx; p.out_dist = out_dist; p.status = status;
    p.inertia = inertia; p.inertia_stride = inertia_stride;
    p.knn_k = knn_k;
    p.fuse_sums = fuse_sums;
    p.fuse_counts = fuse_counts;
    if (fuse_ctas) *fuse_ctas = 0;
    if ((knn_k != 0 && knn_k != 8 && knn_k != 32) || (knn_k > 0 && (B != 1 || !out_dist || inertia))) return CAKE_ERR_UNSUPPORTED;
    if (p.total_tiles == 0) return CAKE_OK;

    const int Kpad = padded_k(K);
    // Every launch of a step may start while its predecessor drains (each kernel waits for the
    // predecessor itself before it touches global memory).
    cudaLaunchAttribute pdl[1];
    pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl[0].val.programmaticStreamSerializationAllowed = 1;
    // Shared memory: X buffers (each with its 4 KiB norm operand), the centroid ring, fixed parts.
    // Few centroid tiles per row tile make row tiles short, so X has to run further ahead: up to four
    // X buffers then, two otherwise; a single one only if the ring would drop below three stages.
    const i64 fixed = 1024 + CTRL_BYTES + AUG_ZERO_BYTES;
    const i64 budget = static_cast<i64>(di.smem_optin) - fixed;
    const i64 xbuf = static_cast<i64>(p.nchunks) * X_CHUNK_BYTES + AUG_A_BYTES;
    int want_xbuf = p.n_tiles <= 2 ? MAX_XBUF_PLAIN : 2;
    if ((p.nchunks >= 4 && p.n_tiles >= 8) || (p.nchunks == 3 && p.n_tiles >= 16)) want_xbuf = 1;   // measured
    // two chunks per ring stage when the chunk count is even (one wait and one commit per stage), unless the
    // ring would then hold a single stage, X is the bound (few centroid tiles: X buffers matter more) or the
    // last chunk is a partial one (short tiles: waiting for both chunks costs more than the barriers saved)
    i64 stages = 0;
    for (p.cps = (p.nchunks % 2 == 0 && (Dk % KCHUNK == 0 || cpad) && p.n_tiles > 2) ? 2 : 1; p.cps >= 1; --p.cps) {
        p.stage_bytes = static_cast<uint32_t>(p.cps) * C_CHUNK_BYTES + AUG_B_BYTES;
        const int spt = p.nchunks / p.cps;                       // stages per centroid tile
        const i64 min_stages = p.cps == 1 ? (p.n_tiles <= 2 ? 2 : 3) : (p.n_tiles <= 2 ? 2 : 2 * spt);
        for (p.n_xbuf = want_xbuf; p.n_xbuf >= 1; --p.n_xbuf) {
            stages = (budget - p.n_xbuf * xbuf) / p.stage_bytes;
            if (stages >= min_stages || p.n_xbuf == 1) break;
        }
        if (stages >= 2) break;
    }
    if (stages < 2) return CAKE_ERR_UNSUPPORTED;
    p.n_stages = static_cast<int>(stages > MAX_STAGES ? MAX_STAGES : stages);

    CUtensorMap tx, tc;
    rc = make_tmap(&tx, X, Dk, N, B, BLOCK_M);
    if (rc != CAKE_OK) return rc;

    // one or two centroid tiles per row tile: the kernel is as fast as X arrives, X gets its own producer
    // (the top-k epilogue exists in the many-tile structure only)
    const bool xload = p.n_tiles <= 2 && knn_k == 0;
    p.alt_epi = 0;   // without resident centroids (D = 256) the shared epilogue measured faster
    p.res_c = 0;
    int c_rows = BLOCK_N;   // rows of a centroid chunk in shared memory (the TMA box)
    if (p.n_tiles == 1 && xload) {
        // a single centroid tile: keep it in shared memory if an even number of X buffers fits beside it
        // (of the tile only the rows that hold centroids, in steps of 32, when there are at most 128)
        c_rows = K <= BLOCK_N / 2 ? static_cast<int>(round_up(K, 32)) : BLOCK_N;
        const i64 c_bytes = static_cast<i64>(p.nchunks) * c_rows * 128 + AUG_B_BYTES;
        for (int nx = MAX_XBUF_PLAIN; nx >= 2; nx -= 2) {
            if (p.nchunks <= MAX_STAGES && c_bytes + nx * xbuf <= budget) {
                p.res_c = 1;
                // its value: the accumulator columns the MMAs write and the epilogue reads (K <= 128: only
                // the 32-column groups that hold centroids; the tensor pipe and the epilogue do less)
                p.alt_epi = c_rows;
                p.cps = 1;
                p.stage_bytes = static_cast<uint32_t>(c_rows) * 128u;
                p.n_stages = p.nchunks;
                p.n_xbuf = nx;
                break;
            }
        }
        // D > 256: one X buffer beside the resident tile, filled and handed back chunk by chunk
        // (the ring's stage count only sizes the buffer here: the resident tile has one barrier pair)
        if (!p.res_c && p.nchunks <= MAX_XCHUNKS && c_bytes + xbuf <= budget) {
            p.res_c = 1;
            p.alt_epi = c_rows;
            p.cps = 1;
            p.stage_bytes = static_cast<uint32_t>(c_rows) * 128u;
            p.n_stages = p.nchunks;
            p.n_xbuf = 1;
        }
    }
    if (p.n_tiles == 2 && xload) {
        // two centroid tiles: both stay in shared memory if at least two X buffers fit beside them (D <= 128)
        const i64 c_bytes = 2 * (static_cast<i64>(p.nchunks) * C_CHUNK_BYTES + AUG_B_BYTES);
        for (int nx = MAX_XBUF_PLAIN; nx >= 2; --nx) {
            if (2 * p.nchunks <= MAX_STAGES && c_bytes + nx * xbuf <= budget) {
                p.res_c = 2;
                p.cps = 1;
                p.stage_bytes = C_CHUNK_BYTES;
                p.n_stages = 2 * p.nchunks;
                p.n_xbuf = nx;
                break;
            }
        }
    }
    // fused update: the resident single-tile mode with at most 128 centroids, D <= 128, one problem, and room for the
    // one-hot operand beside FOUR X buffers (an X buffer is held until its tile has been added to the sums, which is
    // issued behind the MMAs of the issuer's next tile: with two buffers that would wait on itself)
    // More X buffers than the plain kernel where they fit (a buffer is held longer), and one one-hot operand per
    // epilogue warpgroup where two fit (with a shared one the updates of consecutive tiles wait for each other).
    bool fuse = false;
    p.fuse_oh2 = 0;
    if (fuse_sums && fuse_counts && B == 1 && p.res_c == 1 && K <= BLOCK_N / 2 && Dk <= 128 && !exact && knn_k == 0 && p.n_xbuf == 4 &&
        di.sm_count <= kFuseMaxCtas) {
        const i64 c_bytes = static_cast<i64>(p.nchunks) * c_rows * 128 + AUG_B_BYTES;
        for (int oh = 2; oh >= 1 && !fuse; --oh)
            for (int nx = MAX_XBUF; nx >= 4 && !fuse; nx -= 2)
                if (c_bytes + nx * xbuf + oh * static_cast<i64>(OH_BYTES) <= budget) {
                    fuse = true;
                    p.fuse_oh2 = oh == 2 ? 1 : 0;
                    p.n_xbuf = nx;
                }
    }
    if (p.res_c != 1) c_rows = BLOCK_N;
    rc = make_tmap(&tc, cpad ? cpad : C, Dc, K, B, c_rows);
    if (rc != CAKE_OK) return rc;
    const size_t ring_bytes = p.res_c ? static_cast<size_t>(p.res_c) * (static_cast<size_t>(p.nchunks) * p.stage_bytes + AUG_B_BYTES)
                                      : static_cast<size_t>(p.n_stages) * p.stage_bytes;
    const size_t smem_bytes = static_cast<size_t>(fixed) + static_cast<size_t>(p.n_xbuf) * xbuf + ring_bytes +
                              (fuse ? OH_BYTES * (p.fuse_oh2 ? 2u : 1u) : 0u);
    using Kernel = void (*)(const CUtensorMap, const CUtensorMap, const Params);
    const bool consec = xload && p.res_c && B > 1;
    // a single X buffer (D > 256) is filled and handed back chunk by chunk
    const bool xsplit = xload && p.res_c != 2 && p.n_xbuf == 1 && p.cps == 1 && p.nchunks <= MAX_XCHUNKS;
    Kernel kernel;
    // D = 128 (two chunks) with many centroid tiles per row tile measured 3-6 % faster when the accumulator is handed
    // back before the reduction; every other shape gains from reducing while loading (D = 64 up to 8 %)
    const bool bulk = p.nchunks == 2 && p.n_tiles >= 8;
    if (fuse)
        kernel = assign_tc_kernel<true, true, false, false, false, 0, true>;
    else if (knn_k > 0)
        kernel = knn_k == 8 ? assign_tc_kernel<true, false, false, false, false, 8> : assign_tc_kernel<true, false, false, false, false, 32>;
    else if (!xload && !exact && p.n_tiles >= GATE_MIN_TILES)   // (see group_min32)
        kernel = bulk ? assign_tc_kernel<true, false, false, false, true, 0, false, false, true>
                      : assign_tc_kernel<true, false, false, false, false, 0, false, false, true>;
    else if (!xload)
        kernel = exact ? (bulk ? assign_tc_kernel<false, false, false, false, true> : assign_tc_kernel<false, false>)
                       : (bulk ? assign_tc_kernel<true, false, false, false, true> : assign_tc_kernel<true, false>);
    else if (exact)
        kernel = consec ? (xsplit ? assign_tc_kernel<false, true, true, true> : assign_tc_kernel<false, true, true, false>)
                        : (xsplit ? assign_tc_kernel<false, true, false, true> : assign_tc_kernel<false, true, false, false>);
    // (with the split X buffer the shared code measured faster; the 256-column epilogue of the instantiation without the
    // spilling branch measured 13 % faster at D = 64 and 1.5-3 % slower at D = 128)
    else if (p.res_c == 1 && !xsplit && (p.alt_epi <= BLOCK_N / 2 || p.nchunks == 1))
        kernel = consec ? assign_tc_kernel<true, true, true, false, false, 0, false, true>
                        : assign_tc_kernel<true, true, false, false, false, 0, false, true>;
    else
        kernel = consec ? (xsplit ? assign_tc_kernel<true, true, true, true> : assign_tc_kernel<true, true, true, false>)
                        : (xsplit ? assign_tc_kernel<true, true, false, true> : assign_tc_kernel<true, true, false, false>);
    static bool attr_done[64] = {false};   // per device; benign race: the attribute calls are idempotent
    const bool attr_known = di.device >= 0 && di.device < 64;
    if (!attr_known || !attr_done[di.device]) {
        if (cudaFuncSetAttribute(assign_tc_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess ||
            cudaFuncSetAttribute(assign_tc_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess ||
            cudaFuncSetAttribute(assign_tc_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess ||
            cudaFuncSetAttribute(assign_tc_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess ||
            cudaFuncSetAttribute(assign_tc_kernel<true, false, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess ||
            cudaFuncSetAttribute(assign_tc_kernel<true, true, false, false, false, 0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess ||
            cudaFuncSetAttribute(assign_tc_kernel<true, false, false, false, false, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess ||
            cudaFuncSetAttribute(assign_tc_kernel<true, false, false, false, false, 32>, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess ||
            cudaFuncSetAttribute(assign_tc_kernel<false, false, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess ||
            cudaFuncSetAttribute(assign_tc_kernel<true, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess ||
            cudaFuncSetAttribute(assign_tc_kernel<false, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess ||
            cudaFuncSetAttribute(assign_tc_kernel<true, true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess ||
            cudaFuncSetAttribute(assign_tc_kernel<false, true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess ||
            cudaFuncSetAttribute(assign_tc_kernel<true, true, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess ||
            cudaFuncSetAttribute(assign_tc_kernel<false, true, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess ||
            cudaFuncSetAttribute(assign_tc_kernel<true, true, true, false, false, 0, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess ||
            cudaFuncSetAttribute(assign_tc_kernel<true, true, false, false, false, 0, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess ||
            cudaFuncSetAttribute(assign_tc_kernel<true, false, false, false, true, 0, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess ||
            cudaFuncSetAttribute(assign_tc_kernel<true, false, false, false, false, 0, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, di.smem_optin) != cudaSuccess)
            return CAKE_ERR_CUDA;
        if (attr_known) attr_done[di.device] = true;
    }
    // CTA pairs (on request): many centroid tiles per row tile, the centroid operand in rows of a multiple of 64 columns
    if (pair && (xload || knn_k != 0 || fuse || Dc % KCHUNK != 0 || !assign_pair_supports(di, Dk, K))) return CAKE_ERR_UNSUPPORTED;
    // every host-side check has passed: from here on work is enqueued
    if (!aug_ready) {
        rc = launch_centroid_prologue(C, B, D, K, caug, cpad, Dc, inertia, inertia_stride, zero_inertia, s);
        if (rc != CAKE_OK) return rc;
    }

    if (pair)
        return launch_assign_pair(X, cpad ? cpad : C, B, N, Dk, Dc, K, caug, exact, out_idx, out_dist, inertia, inertia_stride,
                                  status, di, s);
    const unsigned grid = static_cast<unsigned>(p.total_tiles < di.sm_count ? p.total_tiles : di.sm_count);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = s;
    cfg.attrs = pdl;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kernel, tx, tc, p) != cudaSuccess) {
        cudaGetLastError();
        return CAKE_ERR_CUDA;
    }
    note_launches(1);
    if (fuse && fuse_ctas) *fuse_ctas = static_cast<int>(grid);
    return CAKE_OK;
}

}  // namespace cake
