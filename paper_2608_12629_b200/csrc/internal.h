// Host-side declarations shared by the translation units of the library (not a public header).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/cake_kmeans.h"

namespace cake {

typedef long long i64;

struct DeviceInfo {
    int device;
    int sm_count;
    int smem_optin;   // max dynamic shared memory per block (opt-in), bytes
    int cc_major;
};
// Properties of the current device (cached per device). Returns CAKE_OK / CAKE_ERR_DEVICE / CAKE_ERR_CUDA.
int current_device_info(DeviceInfo* out);

// Number of kernels this library has launched since it was loaded (all devices, all streams).
void note_launches(int n);
unsigned long long launches_so_far();

inline i64 round_up(i64 a, i64 b) { return (a + b - 1) / b * b; }

// Centroid tiles of the tensor-core assign kernel are 256 wide; K is padded to that (padding rows
// carry a half-norm of 2^120).  Per tile the kernel's prologue writes a 4 KiB operand block.
constexpr int kAssignBlockN = 256;
constexpr unsigned kAssignAugTileBytes = kAssignBlockN * 16;
inline int padded_k(int K) { return (int)round_up(K, kAssignBlockN); }

// ---- assign
bool assign_tc_supports(int D);
// Rows of up to kAssignResidentMaxD columns keep a whole X tile resident in shared memory (assign_tc.cu, and
// assign_pair.cu on request); longer rows (D % 8 == 0, up to kAssignWideMaxD) stream X chunk by chunk beside the
// centroids in the CTA-pair kernel's wide mode, which needs two per-row arrays written by launch_row_aug.
constexpr int kAssignResidentMaxD = 512;
constexpr int kAssignWideMaxD = 8192;
inline bool assign_wide_supports(int D) { return D % 8 == 0 && D > kAssignResidentMaxD && D <= kAssignWideMaxD; }
size_t assign_wide_aug_bytes(i64 B, i64 N);      // X-side operand of the extra k-step, 16 bytes per row
size_t assign_wide_margin_bytes(i64 B, i64 N);   // the rows' margins m, 4 bytes per row
cudaError_t launch_row_aug(const cake_bf16* X, int B, i64 N, int D, void* xaug, float* xrowm, cudaStream_t s);
// bytes of scratch (`caug`) the tensor-core assign needs for B problems of K centroids
size_t assign_tc_aug_bytes(i64 B, int K);
// prologue (half-norm operand into caug) + the assign kernel; exact selects the exact epilogue;
// inertia (nullable): inertia[b * inertia_stride] += sum_i dist[b][i], fp64.  zero_inertia: the prologue
// starts the inertia entries from zero (otherwise the caller has).
// aug_ready: caug and (if asked for) the cleared inertia entries are already what the prologue
// would write for these centroids (the division kernel of the update ahead wrote them): no prologue.
// cpad (nullable): [B][K][round_up(Dx or D, 64)] scratch; the prologue copies C there, rows padded with
// zeros, and the kernel streams that copy (rows whose pitch is a multiple of 128 bytes stream faster).
// Dx (0 = D): columns of a row of X when X is a copy padded with zeros to a multiple of 8 columns
// (needs cpad).  aug_ready then also means that cpad holds the copy.
// knn_k (0 = arg-min, else 8 or 32): k-nearest-neighbour search, B = 1; out_idx / out_dist are then [N][2][knn_k]
// scratch, one list of the knn_k smallest distances per row and 128-column half of the tiles, each sorted by
// (distance, column), unused places -1 / +inf; launch_knn_merge merges the two.
int launch_assign_tc(const cake_bf16* X, const cake_bf16* C, int B, i64 N, int D, int K, void* caug,
                     bool exact, int* out_idx, float* out_dist, double* inertia,
                     int inertia_stride, bool zero_inertia, bool aug_ready, int* status, cudaStream_t s,
                     int Dx = 0, cake_bf16* cpad = nullptr, int knn_k = 0, float* fuse_sums = nullptr,
                     int* fuse_counts = nullptr, int* fuse_ctas = nullptr, bool pair = false, void* xaug = nullptr, float* xrowm = nullptr,
                     bool xaug_ready = false);
// pair: the CTA-pair kernel (tcgen05.mma.cta_group::2; assign_pair.cu) instead of the single-CTA one; needs more than
// two centroid tiles per row tile.  Rows of more than kAssignResidentMaxD columns always take that kernel, in its
// wide mode: xaug / xrowm are the scratch arrays of launch_row_aug (run here unless xaug_ready).
bool assign_pair_supports(const DeviceInfo& di, int Dk, int K);
int launch_assign_pair(const cake_bf16* X, const cake_bf16* C, int B, i64 N, int Dk, int Dc, int K, const void* caug,
                       bool exact, int* out_idx, float* out_dist, double* inertia, int inertia_stride, int* status,
                       const DeviceInfo& di, cudaStream_t s, const void* xaug = nullptr, const float* xrowm = nullptr);
// tensor maps: bf16 [batch][rows][D] viewed as (D, rows, batch), box 64 columns x box_rows rows, 128-byte swizzle;
// and bytes viewed as [rows][16], box 16 x box_rows, no swizzle
int make_tmap_bf16_rows(CUtensorMap* m, const void* base, int D, i64 rows, int batch, int box_rows);
int make_tmap_rows16(CUtensorMap* m, const void* base, i64 rows, int box_rows);
// Fused update (fuse_sums / fuse_counts / fuse_ctas all given, one problem, K <= 128, D <= 128 and room in shared
// memory): the assign kernel also adds the rows of every tile to per-cluster sums on the tensor core.  On return
// *fuse_ctas = n > 0 says that it did: fuse_sums then holds n partial sums of [128][round_up(D, 16)] floats (one per
// CTA) and fuse_counts n partial counts of [128]; launch_finalize_partials adds them up and divides.
// *fuse_ctas = 0: the kernel ran without (the shape does not qualify) and the update has to be done separately.
constexpr int kFuseMaxCtas = 160;
constexpr int kFuseMaxK = 128, kFuseMaxD = 128;
inline bool fuse_shape_ok(i64 B, int D, int K) { return B == 1 && K <= kFuseMaxK && D <= kFuseMaxD && D % 8 == 0; }

int launch_assign_simt(const cake_bf16* X, const cake_bf16* C, int B, i64 N, int D, int K,
                       int* out_idx, float* out_dist, cudaStream_t s);
// D that is not a multiple of 8 (rows are then no multiple of 16 bytes, which TMA needs): the automatic
// route copies X into rows of padded_d(D) columns, zeros in the padding (distances and norms do not
// change), and runs the tensor-core kernel on the copy.
inline int padded_d(int D) { return (int)round_up(D, 8); }
inline bool assign_pad_supports(int D) {
    return D % 8 != 0 && (assign_tc_supports(padded_d(D)) || assign_wide_supports(padded_d(D)));
}
// columns of a row of the centroid copy the tensor-core kernel streams when D is not a multiple of 64 (else 0)
inline int assign_cpad_columns(int D) {
    return (D % 64 != 0 && (assign_tc_supports(padded_d(D)) || assign_wide_supports(padded_d(D)))) ? (int)round_up(D, 64) : 0;
}
// dst[r][0..Dpad) = src[r][0..D) followed by zeros, for r < rows (Dpad % 8 == 0, dst 16-byte aligned)
cudaError_t launch_pad_rows(const cake_bf16* src, i64 rows, int D, int Dpad, cake_bf16* dst, cudaStream_t s);

// ---- update
struct UpdateScratch {
    float* sums;      // [B][K][D]
    int* nvalid;      // [B]        rows with a valid index (sort path)
    int* cursor;      // [B][K]     first sorted position of every cluster (sort path, K > 8192)
    int2* pairs;      // [B][N]     (row number, cluster) in cluster order (sort path)
    int* part;        // [B][slabs][K] per-slab histograms (sort path, K <= 8192)
    int* done;        // [B][K]     rows of a heavy cluster already added to sums (sort path, K > 8192)
    int* rank;        // [B][N]     rank of every row inside its cluster (sort path, K > 8192)
};
// bytes of the per-slab histogram scratch of the sort route (0 when it uses global atomics instead)
size_t update_sort_part_bytes(i64 B, i64 N, int K);
// bytes of the per-row rank scratch of the sort route (0 when it sorts slab by slab in shared memory)
size_t update_sort_rank_bytes(i64 B, i64 N, int K);
bool update_smem_supports(int D, int K, int smem_optin);
int launch_update_smem(const cake_bf16* X, const int* idx, int B, i64 N, int D, int K, float* sums,
                       int* counts, int* status, cudaStream_t s);
// *divided = true when the route wrote out_C / out_C_bf16 itself (means, keep-previous rule and all);
// otherwise sums and counts are ready for launch_finalize.
int launch_update_sort(const cake_bf16* X, const int* idx, int B, i64 N, int D, int K,
                       const UpdateScratch& scr, int* counts, const cake_bf16* C_prev, float* out_C,
                       cake_bf16* out_C_bf16, bool* divided, int* status, cudaStream_t s);
// slab route (one kernel sorts and reduces slab by slab): D % 8 == 0, D <= 1024, K <= 8192.
// force_f = 0 lets the launcher choose the thread-block cluster size, else 1, 2 or 4.
bool update_slab_supports(int D, int K);
// true when its runs of equal clusters are long enough to beat the sort route (measured threshold)
bool update_slab_preferred(int B, i64 N, int D, int K);
int launch_update_slab(const cake_bf16* X, const int* idx, int B, i64 N, int D, int K, float* sums,
                       int* counts, int* status, int force_f, cudaStream_t s);
// out_C = counts>0 ? sums/counts : C_prev (or 0); optional bf16 copy.  early: launched so that it may
// start before the kernel ahead of it in the stream has drained (it waits for that kernel itself)
// next (nullable): also prepare the tensor-core assign of the centroids being written (its half-norm
// operand, cleared inertia entries), so that that assign needs no prologue.  Needs
// D % 4 == 0 and out_C_bf16; *prepared tells whether it was done.
// sums_columns (0 = D): columns of a row of sums, when they were added up from the padded copy of X.
struct NextAssign {
    void* caug;             // as for launch_assign_tc
    double* inertia;        // nullable: inertia[b * inertia_stride] = 0 for b < B (B <= 256)
    int inertia_stride;
    cake_bf16* cpad;        // nullable: as for launch_assign_tc, rows of cpad_columns columns
    int cpad_columns;
};
cudaError_t launch_finalize(const float* sums, const int* counts, const cake_bf16* C_prev, int B,
                            int K, int D, float* out_C, cake_bf16* out_C_bf16, bool early,
                            const NextAssign* next, bool* prepared, cudaStream_t s, int sums_columns = 0);
// The division of the fused update: partial sums / counts of launch_assign_tc's fused mode are added up, then as
// launch_finalize (one problem; `next` as there; out_counts receives the total counts).
cudaError_t launch_finalize_partials(const float* part_sums, const int* part_counts, int n_ctas, const cake_bf16* C_prev,
                                     int K, int D, float* out_C, cake_bf16* out_C_bf16, int* out_counts,
                                     const NextAssign* next, bool* prepared, cudaStream_t s);

// ---- all Lloyd iterations of a small problem in one cooperative launch (lloyd_small.cu): one problem, K <= 128,
// D <= 128 (D % 8 == 0), at most four 128-row tiles per SM.  part_sums [SMs][128][round_up(D, 16)], part_counts [SMs][128], cbuf [K][D] and
// gbar (one word) are scratch; inertia (nullable) gets one entry per iteration.
bool lloyd_small_supports(const DeviceInfo& di, i64 N, int D, int K);
int launch_lloyd_small(const cake_bf16* X, const cake_bf16* C0, i64 N, int D, int K, int iters, float* part_sums,
                       int* part_counts, cake_bf16* cbuf, unsigned* gbar, float* out_C, cake_bf16* out_C_bf16, int* out_idx,
                       float* out_dist, int* out_counts, double* inertia, int* status, const DeviceInfo& di, cudaStream_t s);

// ---- inertia: acc[b] += sum_i dist[b][i] (fp64 atomics); acc stride given in elements
cudaError_t launch_inertia(const float* dist, int B, i64 N, double* acc, int acc_stride,
                           cudaStream_t s);

// ---- k nearest neighbours: out[row][0..k) = the k smallest of the two sorted lists half[row][0..2)[0..kl), k <= kl
cudaError_t launch_knn_merge(const int* half_idx, const float* half_dist, i64 N, int kl, int k, int* out_idx,
                             float* out_dist, cudaStream_t s);

// ---- k-means++ seeding: running minimum of the distances and its slab sums; the draw itself
constexpr int kPlusPlusMaxSlabs = 1024;
// mind = first ? dist : min(mind, dist); part[slab] = sum of the slab's mind (fp64); part holds kPlusPlusMaxSlabs doubles
cudaError_t launch_pp_accumulate(const float* dist, float* mind, i64 N, bool first, double* part, cudaStream_t s);
// row k of the seeding: floor(u[0] N) for k = 0, else the first row whose running sum of mind exceeds u[k] * sum(mind)
// (a uniform row if the sum is zero); copies X[row] to out_row and records the row in rows_out[k] (nullable)
cudaError_t launch_pp_pick(const cake_bf16* X, const float* mind, const double* part, i64 N, int D, const float* u, int k,
                           cake_bf16* out_row, int* rows_out, cudaStream_t s);

// ---- bounded-wait self test
cudaError_t launch_bounded_wait_selftest(int* status, int limit_ms, cudaStream_t s);

}  // namespace cake
