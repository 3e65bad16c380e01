/*
 * cake_kmeans.h -- C ABI of the B200 (sm_100a) Flash-KMeans Lloyd hot path.
 *
 * The operations are the two kernels of the paper's Section 5, paragraph "Flash-KMeans
 * clean-start workload", and the Lloyd iteration they make up:
 *   assign           squared Euclidean distance from every point to all K centroids, arg-min
 *                    (bf16 inputs, fp32 accumulation; the N x K distance matrix is never stored);
 *   centroid_update  per-cluster sums and counts of the assigned points (then, in this library,
 *                    the division into means, with empty clusters keeping their previous centroid);
 *   lloyd            iters x (assign, update).
 *
 * Conventions shared by every entry point
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer on the current device.
 *     The caller owns all buffers; the library allocates nothing and frees nothing.
 *   - cake_bf16 is a raw bfloat16 bit pattern.  Matrices are row-major and contiguous:
 *     X[B][N][D], C[B][K][D], idx[B][N], counts[B][K].  The un-batched calls are B = 1.
 *     Base pointers must be 16-byte aligned.  Inputs must be finite.
 *   - `ws` is caller-provided scratch of at least cake_kmeans_workspace_bytes(...) bytes
 *     (for D % 8 != 0 that includes room for a zero-padded copy of X), 256-byte aligned.  Its first word is a sticky device status (see cake_kmeans_device_status);
 *     the caller zeroes the first 256 bytes once, before the first call that uses the buffer.
 *     Calls that run concurrently must use distinct workspaces.
 *   - Work is enqueued on `stream` (a cudaStream_t; NULL = the legacy default stream) and the
 *     call returns without synchronising.  The return value reports what the host could check:
 *     CAKE_OK or a negative CAKE_ERR_* code; on error nothing was enqueued.
 *   - N = 0 is valid and does nothing (update then treats every cluster as empty).
 *   - Ties in the arg-min go to the lowest centroid index.  Indices and counts are int32.
 *   - `flags` selects a code path for testing; 0 lets the library choose.
 */
#ifndef CAKE_KMEANS_H_
#define CAKE_KMEANS_H_

#include <stddef.h>

#if defined(__GNUC__)
#define CAKE_API __attribute__((visibility("default")))
#else
#define CAKE_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* cake_stream_t;
typedef unsigned short cake_bf16;

enum {
    CAKE_OK = 0,
    CAKE_ERR_NULL = -1,        /* a required pointer is NULL                                   */
    CAKE_ERR_SHAPE = -2,       /* B < 1, N < 0, D < 1, K < 1, iters < 0, or sizes over int32    */
    CAKE_ERR_ALIGN = -3,       /* a base pointer is not 16-byte aligned (ws: 256)              */
    CAKE_ERR_UNSUPPORTED = -4, /* the requested path cannot run this shape                     */
    CAKE_ERR_WORKSPACE = -5,   /* ws_bytes too small                                           */
    CAKE_ERR_CUDA = -6,        /* a CUDA runtime / driver call failed                          */
    CAKE_ERR_BAD_INDEX = -7,   /* device status: an idx value was outside [0,K) and was skipped */
    CAKE_ERR_TIMEOUT = -8,     /* device status: a bounded in-kernel wait expired              */
    CAKE_ERR_DEVICE = -9       /* no CUDA device, or not compute capability 10.x               */
};

enum {
    CAKE_ASSIGN_AUTO = 0,      /* the tensor-core pipeline for D <= 8192 (for D % 8 != 0 on a zero-padded
                                  copy of X kept in the workspace: same results), else the fallback  */
    CAKE_ASSIGN_TCGEN05 = 1,   /* TMA + tcgen05.mma + TMEM pipeline; needs D % 8 == 0, D <= 8192.  Up to D = 512
                                  a CTA keeps its 128-row X tile in shared memory; longer rows are streamed chunk
                                  by chunk beside the centroids by pairs of CTAs (two more scratch arrays in the
                                  workspace, 20 bytes per row, written once per call).
                                  Each distance is an fp32 number whose error follows |x|^2 + |c|^2 of
                                  its own centroid (other centroids' norms do not matter); distances are
                                  compared with 17 significant bits (2^-16 of the distance), equal ones
                                  go to the lower index; out_dist carries the same 17 bits.  Squared
                                  norms must stay below 2^120                                      */
    CAKE_ASSIGN_SIMT = 2,      /* plain CUDA-core fallback, any D                               */
    CAKE_ASSIGN_TCGEN05_EXACT = 3, /* same pipeline, all 24 bits compared and returned (slower epilogue) */
    CAKE_ASSIGN_TCGEN05_PAIR = 4,  /* the arithmetic and results of CAKE_ASSIGN_TCGEN05 on pairs of CTAs
                                      (tcgen05.mma.cta_group::2: two SMs share every 256 x 256 tile and each loads half
                                      of the centroid tile).  Never chosen automatically: measured equal to the single-CTA
                                      kernel at D = 128, K = 1024 and behind it elsewhere.  D % 8 == 0; D <= 512 needs K > 512
                                      (longer rows take the pair kernel under every tensor-core flag).                 */
    CAKE_ASSIGN_TCGEN05_PAIR_EXACT = 5, /* ... with the epilogue of CAKE_ASSIGN_TCGEN05_EXACT                        */
    CAKE_ASSIGN_MASK = 0xF,
    CAKE_UPDATE_AUTO = 0,
    CAKE_UPDATE_SMEM = 1 << 4, /* shared-memory partial sums; needs K*D*4 + K*4 bytes of smem   */
    CAKE_UPDATE_SORT = 2 << 4, /* counting sort by cluster, then one pass over X in that order (a
                                  segmented reduction; for K > 8192 and D % 8 == 0 every cluster is
                                  summed and divided by one warp), any K                         */
    CAKE_UPDATE_SLAB = 3 << 4, /* one kernel sorts and reduces slab by slab (thread-block clusters
                                  when K is large against the slab); D % 8 == 0, D <= 1024, K <= 8192 */
    CAKE_UPDATE_SLAB_F1 = 4 << 4, /* the same with the cluster size forced to 1, 2 or 4 CTAs      */
    CAKE_UPDATE_SLAB_F2 = 5 << 4,
    CAKE_UPDATE_SLAB_F4 = 6 << 4,
    CAKE_UPDATE_MASK = 0xF << 4,
    CAKE_LLOYD_NO_FUSE = 1 << 8, /* lloyd: keep assign and update as two passes over X also where one problem of
                                   K <= 128, D <= 128 (D % 8 == 0) would take the single-pass iteration, in which
                                   the assign kernel adds each row tile to per-cluster sums on the tensor core
                                   (sums += onehot^T X) while the tile is in shared memory                      */
    CAKE_LLOYD_NO_RESIDENT = 1 << 9 /* lloyd: do not take the one-launch form of the single-pass iteration, which a
                                   problem of D <= 128 (D % 8 == 0) and at most four 128-row tiles per SM runs in: all
                                   iterations in one cooperative kernel whose CTAs keep their rows in shared memory and
                                   meet at grid barriers (same arithmetic; fp32 partial sums added in another order) */
};

/* Library version (major*10000 + minor*100 + patch).  No paper counterpart. */
CAKE_API int cake_version(void);

/*
 * Number of CUDA kernels this library has launched since it was loaded (memsets and copies are
 * not counted).  For accounting in benchmarks.  No paper counterpart.
 */
CAKE_API unsigned long long cake_kmeans_kernel_launches(void);

/* Static, human-readable text for a CAKE_* code.  Never NULL.  No paper counterpart. */
CAKE_API const char* cake_strerror(int code);

/*
 * Bytes of device scratch that any of the calls below needs for B problems of N points,
 * D features and K clusters (one figure covers assign, update and lloyd).
 *   out_bytes  host pointer, receives the size.
 * Returns CAKE_OK, CAKE_ERR_NULL or CAKE_ERR_SHAPE.  Touches no device.
 */
CAKE_API int cake_kmeans_workspace_bytes(long long B, long long N, int D, int K, size_t* out_bytes);

/*
 * assign (Section 5, "Flash-KMeans clean-start workload": squared Euclidean distances to all K
 * centroids and the arg-min).  Computed as ||x||^2 - 2 x.c + ||c||^2, accumulated in fp32 on the
 * tensor cores.
 *   X        [B][N][D] bf16, in
 *   C        [B][K][D] bf16, in
 *   out_idx  [B][N] int32, out: arg-min_k, lowest k on ties
 *   out_dist [B][N] fp32, out, may be NULL: max(0, squared distance to the chosen centroid)
 */
CAKE_API int cake_kmeans_assign(const cake_bf16* X, const cake_bf16* C, long long N, int D, int K,
                       int* out_idx, float* out_dist, void* ws, size_t ws_bytes,
                       cake_stream_t stream, unsigned flags);
CAKE_API int cake_kmeans_assign_batched(const cake_bf16* X, const cake_bf16* C, long long B, long long N,
                               int D, int K, int* out_idx, float* out_dist, void* ws,
                               size_t ws_bytes, cake_stream_t stream, unsigned flags);

/*
 * assign without any workspace, for callers that cannot allocate device memory (code running
 * inside another framework's allocator callback, or in a process whose device memory is already
 * fully carved up, has no cudaMalloc to give this library a scratch buffer).  The paper has no
 * counterpart: this is the un-batched cake_kmeans_assign with its scratch (the centroid half-norm
 * operand and the status word) held in a fixed 262,400-byte array inside the library image, which every GPU that
 * loads the library keeps until the process exits.
 *   X, C, out_idx, out_dist: as cake_kmeans_assign (one problem).
 *   K must be <= 16384; a larger K returns CAKE_ERR_UNSUPPORTED and nothing is enqueued.
 * The call allocates nothing and frees nothing.  The first call on each device resolves the
 * array's device address (one-time set-up with that device current); make that first call
 * outside any stream capture.  All calls on a device share the one array, which keeps the
 * previous call's contents: the call itself clears what must start at zero, but two calls whose
 * work overlaps on the GPU (different streams, no ordering between them) race on it -- order them.
 * For D % 64 != 0 the centroid rows are streamed as they are (the workspace calls stream a zero-padded
 * copy, which this call has no room for): same results, up to twice the time.
 *
 * cake_kmeans_assign_static_status reads the array's sticky device status word (CAKE_OK, or
 * CAKE_ERR_TIMEOUT if a bounded in-kernel wait of an earlier static call expired): it synchronises
 * `stream`, copies the word to *host_out (host pointer) and clears it.  Allocates nothing either.
 */
CAKE_API int cake_kmeans_assign_static(const cake_bf16* X, const cake_bf16* C, long long N, int D, int K,
                                       int* out_idx, float* out_dist, cake_stream_t stream);
CAKE_API int cake_kmeans_assign_static_status(cake_stream_t stream, int* host_out);

/*
 * centroid_update (same paragraph: per-cluster sums and counts), followed by the division.
 *   X          [B][N][D] bf16, in
 *   idx        [B][N] int32, in; values outside [0,K) are skipped and raise the device status
 *              CAKE_ERR_BAD_INDEX
 *   C_prev     [B][K][D] bf16, in, may be NULL: centroid kept by an empty cluster (zeros if NULL)
 *   out_C      [B][K][D] fp32, out: sums / counts in fp32
 *   out_C_bf16 [B][K][D] bf16, out, may be NULL: out_C rounded to nearest even
 *   out_counts [B][K] int32, out
 * fp32 summation order is unspecified (results agree to fp32 rounding between calls).
 */
CAKE_API int cake_kmeans_update(const cake_bf16* X, const int* idx, long long N, int D, int K,
                       const cake_bf16* C_prev, float* out_C, cake_bf16* out_C_bf16,
                       int* out_counts, void* ws, size_t ws_bytes, cake_stream_t stream,
                       unsigned flags);
CAKE_API int cake_kmeans_update_batched(const cake_bf16* X, const int* idx, long long B, long long N, int D,
                               int K, const cake_bf16* C_prev, float* out_C,
                               cake_bf16* out_C_bf16, int* out_counts, void* ws, size_t ws_bytes,
                               cake_stream_t stream, unsigned flags);

/*
 * centroid_update in two halves, for rows of X that are spread over several devices (the paper
 * describes one device; the per-cluster sums and counts of the same paragraph are what has to cross
 * devices).  Each device adds up its own rows, the caller adds the sums and counts of all devices (an
 * all-reduce), and every device divides.
 *   update_partial: out_sums[B][K][D] fp32 and out_counts[B][K] int32 of the rows given (overwritten,
 *                   not accumulated); other arguments as for update.  flags: 0, CAKE_UPDATE_SLAB or
 *                   CAKE_UPDATE_SORT.
 *   update_finish:  out_C = sums / counts where counts > 0, else C_prev (zeros if NULL); out_C_bf16
 *                   (may be NULL) its rounding.  No workspace.
 */
CAKE_API int cake_kmeans_update_partial_batched(const cake_bf16* X, const int* idx, long long B, long long N,
                               int D, int K, float* out_sums, int* out_counts, void* ws,
                               size_t ws_bytes, cake_stream_t stream, unsigned flags);
/* out_inertia[b * inertia_stride] = sum_i dist[b][i] in fp64 (overwritten), the inertia of an assignment:
 * what lloyd reports per iteration, for callers that run the steps one by one.                        */
CAKE_API int cake_kmeans_inertia_batched(const float* dist, long long B, long long N, double* out_inertia,
                               int inertia_stride, cake_stream_t stream);
CAKE_API int cake_kmeans_update_finish_batched(const float* sums, const int* counts, const cake_bf16* C_prev,
                               long long B, int K, int D, float* out_C, cake_bf16* out_C_bf16,
                               cake_stream_t stream);

/*
 * lloyd over rows that are spread over several devices, one process per device: this call runs one rank's share.
 * Every rank holds N_local rows and all K centroids.  Per iteration: assign and the per-cluster sums and counts of
 * the local rows (this library's kernels), then `allreduce` -- called on the host, once per iteration, after that
 * work has been enqueued -- must enqueue on `stream` an in-place sum over all ranks of sums[n_sums] (fp32) and
 * counts[n_counts] (int32), both device pointers (an NCCL all-reduce, or anything ordered after the work already on
 * the stream); then every rank divides, so all ranks hold the same centroids without a broadcast.  It returns 0, or
 * non-zero to abort (the call then returns CAKE_ERR_CUDA).  allreduce = NULL: a single rank.
 *   out_idx, out_dist: the local rows' last assignment; out_C, out_C_bf16, out_counts: global (same on all ranks);
 *   out_inertia [iters]: the LOCAL rows' sums of distances (the caller adds them up over the ranks at the end).
 * iters >= 1.  The exchange is K (D + 1) numbers per iteration whatever N is, which is why it is a collective
 * between two launches and not a fused kernel: there is no tile-by-tile transfer to overlap with the math.
 */
typedef int (*cake_allreduce_fn)(void* user, float* sums, long long n_sums, int* counts, long long n_counts,
                                 cake_stream_t stream);
CAKE_API int cake_kmeans_lloyd_sharded(const cake_bf16* X_local, const cake_bf16* C0, long long N_local, int D, int K,
                      int iters, float* out_C, cake_bf16* out_C_bf16, int* out_idx, float* out_dist,
                      int* out_counts, double* out_inertia, cake_allreduce_fn allreduce, void* user, void* ws,
                      size_t ws_bytes, cake_stream_t stream, unsigned flags);

/*
 * lloyd (same paragraph: a Lloyd iteration is assign followed by centroid_update).
 * For t = 0 .. iters-1: assign against C_t (C_0 = C0), out_inertia[t] = sum_i out_dist_t[i],
 * then update -> C_{t+1}; the next assign reads C_{t+1} rounded to bf16.  Exactly `iters`
 * iterations run; there is no convergence test.
 *   out_C       [B][K][D] fp32: C_iters (fp32 means of the last update)
 *   out_C_bf16  [B][K][D] bf16, may be NULL: its bf16 rounding
 *   out_idx     [B][N], out_dist [B][N] (may be NULL): those of the LAST assign (against C_{iters-1})
 *   out_counts  [B][K]: counts of the last update
 *   out_inertia [B][iters] fp64, may be NULL
 * iters = 0 copies C0 to the outputs and leaves idx / dist / counts untouched.
 */
CAKE_API int cake_kmeans_lloyd(const cake_bf16* X, const cake_bf16* C0, long long N, int D, int K, int iters,
                      float* out_C, cake_bf16* out_C_bf16, int* out_idx, float* out_dist,
                      int* out_counts, double* out_inertia, void* ws, size_t ws_bytes,
                      cake_stream_t stream, unsigned flags);
CAKE_API int cake_kmeans_lloyd_batched(const cake_bf16* X, const cake_bf16* C0, long long B, long long N,
                              int D, int K, int iters, float* out_C, cake_bf16* out_C_bf16,
                              int* out_idx, float* out_dist, int* out_counts, double* out_inertia,
                              void* ws, size_t ws_bytes, cake_stream_t stream, unsigned flags);

/*
 * lloyd with a convergence test (the paper fixes iteration counts and has no stopping rule; this is a reading of
 * this library).  Iterations run in blocks of `check_every`; after each block the host reads the block's inertia
 * values (one stream synchronisation per block) and stops once some iteration t >= 1 of the run had
 * inertia[t-1] - inertia[t] <= tol * inertia[t-1].  At most max_iters iterations; *out_iters (host) receives the
 * number run, a multiple of check_every unless max_iters cut the last block.  One problem (no batch).
 * out_C_bf16, out_inertia ([max_iters]) and out_iters are required; the other outputs as for cake_kmeans_lloyd
 * with iters = *out_iters.  Returns after the last block's synchronisation.
 */
CAKE_API int cake_kmeans_lloyd_tol(const cake_bf16* X, const cake_bf16* C0, long long N, int D, int K, int max_iters,
                      double tol, int check_every, float* out_C, cake_bf16* out_C_bf16, int* out_idx,
                      float* out_dist, int* out_counts, double* out_inertia, int* out_iters, void* ws,
                      size_t ws_bytes, cake_stream_t stream, unsigned flags);

/*
 * k-means++ seeding (the paper's workload starts from sampled rows and names no seeding; this is the textbook
 * D^2 sampling, offered as an initialiser).  The random numbers are the caller's:
 *   u        [K] fp32 uniforms in [0,1), device, in
 *   out_C0   [K][D] bf16, out: row 0 is X[floor(u[0] N)]; row k >= 1 is X[i] for the first i whose running sum
 *            mind[0] + ... + mind[i] exceeds u[k] * sum(mind), mind[i] being the squared distance from x_i to
 *            the nearest of the k rows chosen so far (a uniform row if that sum is zero)
 *   out_rows [K] int32, out, may be NULL: the chosen row numbers
 * Distances come from the assign kernel (fp32), the sums are fp64.  Asynchronous on `stream`, no host
 * synchronisation; 3 to 4 kernel launches per centroid.  `ws` as for the other calls (same size).
 */
CAKE_API int cake_kmeans_init_plusplus(const cake_bf16* X, long long N, int D, int K, const float* u,
                      cake_bf16* out_C0, int* out_rows, void* ws, size_t ws_bytes, cake_stream_t stream);

/*
 * lloyd with HOST buffers (same operation; measures the end-to-end cost a caller with data in
 * host memory sees).  X_host, C0_host and every out_*_host pointer are HOST pointers (pinned
 * memory makes the copies asynchronous); `dev` is device scratch of at least
 * cake_kmeans_lloyd_host_device_bytes(...) bytes, 256-byte aligned, into which the library copies
 * the inputs, runs cake_kmeans_lloyd_batched and from which it copies the results back, all on
 * `stream`.  The call returns after enqueueing; synchronise the stream before reading outputs.
 * Nullable outputs as in cake_kmeans_lloyd.
 */
CAKE_API int cake_kmeans_lloyd_host_device_bytes(long long B, long long N, int D, int K, int iters,
                                        size_t* out_bytes);
CAKE_API int cake_kmeans_lloyd_host(const cake_bf16* X_host, const cake_bf16* C0_host, long long B,
                           long long N, int D, int K, int iters, float* out_C_host,
                           cake_bf16* out_C_bf16_host, int* out_idx_host, float* out_dist_host,
                           int* out_counts_host, double* out_inertia_host, void* dev,
                           size_t dev_bytes, cake_stream_t stream, unsigned flags);

/*
 * Exact k-nearest-neighbour search (Section 6 names a KNN search family beside K-means, with recall 1.0:
 * the exact result; Appendix F lists its routes by name only).  Same distance and same tensor-core
 * pipeline as assign, with the database rows in the place of the centroids and a top-k epilogue.
 *   Q        [N][D] bf16, in: queries           X [M][D] bf16, in: database rows
 *   k        neighbours per query, 1..32 (more: CAKE_ERR_UNSUPPORTED)
 *   out_idx  [N][k] int32, out: the k nearest database rows, ascending by (distance, row number): among
 *            equal distances the lower row comes first; -1 where M < k
 *   out_dist [N][k] fp32, out, may be NULL: max(0, squared distance); +inf where M < k
 *   ws       scratch of at least cake_knn_workspace_bytes(...) bytes, 256-byte aligned, first 256 bytes
 *            zeroed once by the caller; word 0 is the sticky device status (cake_kmeans_device_status)
 * D <= 512 (D % 8 != 0 runs on zero-padded copies kept in ws); larger D: CAKE_ERR_UNSUPPORTED.
 * Distances are fp32 numbers compared with all their bits; their error follows |q|^2 + |x|^2 of the pair.
 * Asynchronous on `stream`; N = 0 does nothing.
 */
CAKE_API int cake_knn_workspace_bytes(long long N, long long M, int D, int k, size_t* out_bytes);
CAKE_API int cake_knn_search(const cake_bf16* Q, const cake_bf16* X, long long N, long long M, int D, int k,
                             int* out_idx, float* out_dist, void* ws, size_t ws_bytes, cake_stream_t stream);

/*
 * Reads the sticky device status word of a workspace: synchronises `stream`, copies the word to
 * *host_out (host pointer) and clears it.  *host_out is CAKE_OK, CAKE_ERR_BAD_INDEX or
 * CAKE_ERR_TIMEOUT.  No paper counterpart.
 */
CAKE_API int cake_kmeans_device_status(void* ws, cake_stream_t stream, int* host_out);

/*
 * Self-test of the bounded in-kernel wait: one thread waits on an mbarrier that nothing ever
 * completes, for at most `limit_ms` milliseconds, then records CAKE_ERR_TIMEOUT in the status
 * word of `ws` and returns normally (the context stays usable).  No paper counterpart.
 */
CAKE_API int cake_kmeans_selftest_bounded_wait(void* ws, size_t ws_bytes, int limit_ms, cake_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* CAKE_KMEANS_H_ */
