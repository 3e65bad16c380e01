// The C ABI: argument checks, workspace carving, path selection and the Lloyd loop.
// Every step of the path runs in this library's kernels; nothing here allocates.
#include <limits.h>

#include "internal.h"

namespace cake {
namespace {

constexpr size_t kAlign = 256;
inline size_t up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

struct Workspace {
    int* status;          // [64] header, zeroed by the caller once: word 0 = sticky device status
    void* caug;           // [B][Kpad/256][4 KiB] half-norm operand of the tensor-core assign
    float* sums;          // [B][K][D]
    int* nvalid;          // [B]
    int* cursor;          // [B][K]
    int2* pairs;          // [B][N] (row, cluster) in cluster order
    int* part;            // [B][slabs][K] per-slab histograms of the sort route
    int* done;            // [B][K] arrival counters of heavy clusters (sort route, K > 8192)
    int* rank;            // [B][N] rank of every row inside its cluster (sort route, K > 8192)
    cake_bf16* cbuf[2];   // [B][K][D] each
    float* dist;          // [B][N]
    cake_bf16* xpad;      // [B][N][padded_d(D)] zero-padded copy of X for the tensor-core assign when D % 8 != 0
    cake_bf16* cpad;      // [B][K][round_up(D, 64)] zero-padded copy of C it streams when D % 64 != 0
    cake_bf16* ccont;     // [B][K][D] centroids a Lloyd run continues from (convergence test between blocks of iterations)
    double* pp_part;      // [kPlusPlusMaxSlabs] slab sums of the k-means++ seeding
    float* fpart;         // fused update (one problem, K <= 128, D <= 128): partial sums [kFuseMaxCtas][128][round_up(D, 16)]
    int* fcnt;            // ... and partial counts [kFuseMaxCtas][128]
    void* xaug;           // rows of more than 512 columns: [B][round_up(N, 256)][16 B] X-side operand of the extra k-step
    float* xrowm;         // ... and the rows' margins [B][round_up(N, 256)]
    size_t bytes;
};

// what an earlier step of the same call has already derived from X in the workspace
struct XPrep {
    bool padded = false;   // xpad holds the zero-padded copy (D % 8 != 0)
    bool aug = false;      // xaug / xrowm are written (rows of more than 512 columns)
};

Workspace carve(void* base, i64 B, i64 N, int D, int K) {
    Workspace w;
    size_t o = 0;
    char* p = static_cast<char*>(base);
    auto take = [&](size_t n) { char* r = p ? p + o : nullptr; o += up(n); return r; };
    const size_t kd = static_cast<size_t>(B) * K * D;
    w.status = reinterpret_cast<int*>(take(256));
    w.caug = take(assign_tc_aug_bytes(B, K));
    // rows of padded_d(D) columns: for D % 8 != 0 the update may add up the padded copy of X
    w.sums = reinterpret_cast<float*>(take(static_cast<size_t>(B) * K * padded_d(D) * 4));
    w.nvalid = reinterpret_cast<int*>(take(static_cast<size_t>(B) * 4));
    w.cursor = reinterpret_cast<int*>(take(static_cast<size_t>(B) * K * 4));
    w.pairs = reinterpret_cast<int2*>(take(static_cast<size_t>(B) * N * 8));
    w.part = reinterpret_cast<int*>(take(update_sort_part_bytes(B, N, K)));
    w.done = reinterpret_cast<int*>(take(static_cast<size_t>(B) * K * 4));
    w.rank = reinterpret_cast<int*>(take(update_sort_rank_bytes(B, N, K)));
    w.cbuf[0] = reinterpret_cast<cake_bf16*>(take(kd * 2));
    w.cbuf[1] = reinterpret_cast<cake_bf16*>(take(kd * 2));
    w.dist = reinterpret_cast<float*>(take(static_cast<size_t>(B) * N * 4));
    const size_t dpad = assign_pad_supports(D) ? static_cast<size_t>(padded_d(D)) : 0;
    w.xpad = reinterpret_cast<cake_bf16*>(take(static_cast<size_t>(B) * N * dpad * 2));
    w.cpad = reinterpret_cast<cake_bf16*>(take(static_cast<size_t>(B) * K * assign_cpad_columns(D) * 2));
    w.ccont = reinterpret_cast<cake_bf16*>(take(kd * 2));
    w.pp_part = reinterpret_cast<double*>(take(static_cast<size_t>(kPlusPlusMaxSlabs) * 8));
    // (one partial per CTA of the assign kernel: at most one CTA per row tile and per SM)
    const bool fuse = fuse_shape_ok(B, D, K);
    const i64 row_tiles = (N + 127) / 128;
    const size_t fctas = fuse ? static_cast<size_t>(row_tiles < kFuseMaxCtas ? row_tiles : kFuseMaxCtas) : 0;
    w.fpart = reinterpret_cast<float*>(take(fctas * 128 * round_up(D, 16) * 4));
    w.fcnt = reinterpret_cast<int*>(take(fctas * 128 * 4));
    const bool wide = assign_wide_supports(padded_d(D));
    w.xaug = take(wide ? assign_wide_aug_bytes(B, N) : 0);
    w.xrowm = reinterpret_cast<float*>(take(wide ? assign_wide_margin_bytes(B, N) : 0));
    w.bytes = o;
    return w;
}

int check_shape(i64 B, i64 N, int D, int K) {
    if (B < 1 || N < 0 || D < 1 || K < 1) return CAKE_ERR_SHAPE;
    if (B > 65535 || N > INT_MAX - 1024 || static_cast<i64>(K) > INT_MAX - 1024) return CAKE_ERR_SHAPE;
    if (static_cast<double>(B) * K * D > 4.0e12 || static_cast<double>(B) * N * D > 4.0e13) return CAKE_ERR_SHAPE;
    return CAKE_OK;
}
inline bool misaligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) != 0; }

int check_ws(void* ws, size_t ws_bytes, i64 B, i64 N, int D, int K, Workspace* out) {
    if (!ws) return CAKE_ERR_NULL;
    if (misaligned(ws, kAlign)) return CAKE_ERR_ALIGN;
    *out = carve(ws, B, N, D, K);
    if (ws_bytes < out->bytes) return CAKE_ERR_WORKSPACE;
    return CAKE_OK;
}

// inertia (nullable): inertia[b * inertia_stride] += sum of problem b's distances.  The tensor-core
// kernel adds it up itself; the fallback needs `dist` (out_dist or scratch) and a reduction kernel.
// zero_inertia: the entries still have to be cleared (the tensor-core prologue does it on the way).
// aug_ready: the update ahead prepared this assign (see NextAssign): the tensor-core route skips its prologue
// xprep (in/out): what the workspace already holds of this X (an earlier step of the call made it)
// fuse_ctas (nullable): ask the tensor-core kernel to add the rows to per-cluster partial sums as well (fused update,
// see launch_assign_tc); *fuse_ctas > 0 on return if it did
int do_assign(const cake_bf16* X, const cake_bf16* C, int B, i64 N, int D, int K, int* out_idx,
              float* out_dist, double* inertia, int inertia_stride, bool zero_inertia, bool aug_ready,
              XPrep* xprep, const Workspace& w, cudaStream_t s, unsigned flags, int* fuse_ctas = nullptr) {
    if (fuse_ctas) *fuse_ctas = 0;
    unsigned path = flags & CAKE_ASSIGN_MASK;
    int Dx = 0;   // columns of the padded copy of X, if one is used
    if (path == CAKE_ASSIGN_AUTO && assign_pad_supports(D) && N > 0) {
        Dx = padded_d(D);
        if (!xprep->padded && launch_pad_rows(X, static_cast<i64>(B) * N, D, Dx, w.xpad, s) != cudaSuccess) return CAKE_ERR_CUDA;
        xprep->padded = true;
        X = w.xpad;
        path = CAKE_ASSIGN_TCGEN05;
    }
    // rows of more than 512 columns: the CTA-pair kernel's wide mode (X streamed beside the centroids), chosen
    // automatically and by either tensor-core flag
    const bool wide = assign_wide_supports(Dx ? Dx : D);
    if (path == CAKE_ASSIGN_AUTO) path = (assign_tc_supports(D) || wide) ? CAKE_ASSIGN_TCGEN05 : CAKE_ASSIGN_SIMT;
    if (zero_inertia && inertia && (path == CAKE_ASSIGN_SIMT || N == 0)) {
        if (cudaMemset2DAsync(inertia, static_cast<size_t>(inertia_stride) * sizeof(double), 0, sizeof(double),
                              static_cast<size_t>(B), s) != cudaSuccess)
            return CAKE_ERR_CUDA;
    }
    if (path == CAKE_ASSIGN_SIMT) {
        float* dist = out_dist ? out_dist : (inertia ? w.dist : nullptr);
        int rc = launch_assign_simt(X, C, B, N, D, K, out_idx, dist, s);
        if (rc == CAKE_OK && inertia && launch_inertia(dist, B, N, inertia, inertia_stride, s) != cudaSuccess)
            rc = CAKE_ERR_CUDA;
        return rc;
    }
    const bool pair = path == CAKE_ASSIGN_TCGEN05_PAIR || path == CAKE_ASSIGN_TCGEN05_PAIR_EXACT;
    if (path != CAKE_ASSIGN_TCGEN05 && path != CAKE_ASSIGN_TCGEN05_EXACT && !pair) return CAKE_ERR_UNSUPPORTED;
    if (!assign_tc_supports(Dx ? Dx : D) && !wide) return CAKE_ERR_UNSUPPORTED;
    if (N == 0) return CAKE_OK;
    // the packed epilogue (values compared with 17 significant bits) is the automatic choice; the exact
    // one compares full fp32 values and is slower
    const bool exact = path == CAKE_ASSIGN_TCGEN05_EXACT || path == CAKE_ASSIGN_TCGEN05_PAIR_EXACT;
    const bool fuse = fuse_ctas && !exact && fuse_shape_ok(B, D, K) && w.fpart && N > 0 && !pair;
    const int rc = launch_assign_tc(X, C, B, N, D, K, w.caug, exact, out_idx, out_dist, inertia, inertia_stride, zero_inertia,
                                    aug_ready, w.status, s, Dx,
                                    assign_cpad_columns(D) ? w.cpad : nullptr, 0, fuse ? w.fpart : nullptr, fuse ? w.fcnt : nullptr,
                                    fuse ? fuse_ctas : nullptr, pair, w.xaug, w.xrowm, xprep->aug);
    if (rc == CAKE_OK && wide) xprep->aug = true;
    return rc;
}

// next / prepared: see launch_finalize
int do_update(const cake_bf16* X, const int* idx, int B, i64 N, int D, int K, const cake_bf16* C_prev,
              float* out_C, cake_bf16* out_C_bf16, int* out_counts, const Workspace& w, cudaStream_t s,
              unsigned flags, XPrep* xprep, const NextAssign* next = nullptr, bool* prepared = nullptr) {
    if (prepared) *prepared = false;
    DeviceInfo di;
    int rc = current_device_info(&di);
    if (rc != CAKE_OK) return rc;
    unsigned path = flags & CAKE_UPDATE_MASK;
    bool divided = false;
    int Ds = D;   // columns of a row of sums
    if (path == CAKE_UPDATE_AUTO && assign_pad_supports(D) && update_slab_preferred(B, N, padded_d(D), K)) {
        // D % 8 != 0: the slab route on the zero-padded copy of X (its padding columns add up to zero and are
        // dropped by the division kernel); faster than the element-wise reduction even when the copy has to be made
        Ds = padded_d(D);
        if (!xprep->padded && launch_pad_rows(X, static_cast<i64>(B) * N, D, Ds, w.xpad, s) != cudaSuccess) return CAKE_ERR_CUDA;
        xprep->padded = true;
        X = w.xpad;
        path = CAKE_UPDATE_SLAB;
    }
    if (path == CAKE_UPDATE_AUTO) {
        // the slab route while a slab holds several rows per cluster, else the global sort; the
        // shared-memory table never measured faster than either and is only taken on request
        path = update_slab_preferred(B, N, D, K) ? CAKE_UPDATE_SLAB : CAKE_UPDATE_SORT;
    }
    if (path == CAKE_UPDATE_SMEM) {
        rc = launch_update_smem(X, idx, B, N, D, K, w.sums, out_counts, w.status, s);
    } else if (path == CAKE_UPDATE_SORT) {
        UpdateScratch scr{w.sums, w.nvalid, w.cursor, w.pairs, w.part, w.done, w.rank};
        rc = launch_update_sort(X, idx, B, N, D, K, scr, out_counts, C_prev, out_C, out_C_bf16, &divided, w.status, s);
    } else if (path == CAKE_UPDATE_SLAB || path == CAKE_UPDATE_SLAB_F1 || path == CAKE_UPDATE_SLAB_F2 ||
               path == CAKE_UPDATE_SLAB_F4) {
        const int force_f = path == CAKE_UPDATE_SLAB ? 0 : path == CAKE_UPDATE_SLAB_F1 ? 1 : path == CAKE_UPDATE_SLAB_F2 ? 2 : 4;
        rc = launch_update_slab(X, idx, B, N, Ds, K, w.sums, out_counts, w.status, force_f, s);
    } else {
        rc = CAKE_ERR_UNSUPPORTED;
    }
    if (rc != CAKE_OK) return rc;
    if (divided) return CAKE_OK;
    const bool slab = path != CAKE_UPDATE_SMEM && path != CAKE_UPDATE_SORT;
    if (launch_finalize(w.sums, out_counts, C_prev, B, K, D, out_C, out_C_bf16, slab, next, prepared, s, Ds) != cudaSuccess)
        return CAKE_ERR_CUDA;
    return CAKE_OK;
}

}  // namespace
}  // namespace cake

using namespace cake;

extern "C" {

int cake_version(void) { return 100; }

unsigned long long cake_kmeans_kernel_launches(void) { return launches_so_far(); }

const char* cake_strerror(int code) {
    switch (code) {
        case CAKE_OK: return "ok";
        case CAKE_ERR_NULL: return "a required pointer is NULL";
        case CAKE_ERR_SHAPE: return "invalid or too large shape";
        case CAKE_ERR_ALIGN: return "a base pointer is not sufficiently aligned";
        case CAKE_ERR_UNSUPPORTED: return "the requested path does not support this shape";
        case CAKE_ERR_WORKSPACE: return "workspace too small";
        case CAKE_ERR_CUDA: return "a CUDA call failed";
        case CAKE_ERR_BAD_INDEX: return "an index was outside [0,K) and was skipped";
        case CAKE_ERR_TIMEOUT: return "a bounded in-kernel wait expired";
        case CAKE_ERR_DEVICE: return "no usable CUDA device (compute capability 10.x needed)";
        default: return "unknown cake_kmeans code";
    }
}

int cake_kmeans_workspace_bytes(long long B, long long N, int D, int K, size_t* out_bytes) {
    if (!out_bytes) return CAKE_ERR_NULL;
    int rc = check_shape(B, N, D, K);
    if (rc != CAKE_OK) return rc;
    *out_bytes = carve(nullptr, B, N, D, K).bytes;
    return CAKE_OK;
}

int cake_kmeans_assign_batched(const cake_bf16* X, const cake_bf16* C, long long B, long long N, int D,
                               int K, int* out_idx, float* out_dist, void* ws, size_t ws_bytes,
                               cake_stream_t stream, unsigned flags) {
    int rc = check_shape(B, N, D, K);
    if (rc != CAKE_OK) return rc;
    if (!C || !ws || (N > 0 && (!X || !out_idx))) return CAKE_ERR_NULL;
    if (misaligned(X, 16) || misaligned(C, 16) || misaligned(out_idx, 4) || misaligned(out_dist, 4))
        return CAKE_ERR_ALIGN;
    Workspace w;
    rc = check_ws(ws, ws_bytes, B, N, D, K, &w);
    if (rc != CAKE_OK) return rc;
    XPrep x_padded;
    return do_assign(X, C, static_cast<int>(B), N, D, K, out_idx, out_dist, nullptr, 0, false, false, &x_padded, w,
                     reinterpret_cast<cudaStream_t>(stream), flags);
}

int cake_kmeans_assign(const cake_bf16* X, const cake_bf16* C, long long N, int D, int K, int* out_idx,
                       float* out_dist, void* ws, size_t ws_bytes, cake_stream_t stream, unsigned flags) {
    return cake_kmeans_assign_batched(X, C, 1, N, D, K, out_idx, out_dist, ws, ws_bytes, stream, flags);
}

int cake_kmeans_update_batched(const cake_bf16* X, const int* idx, long long B, long long N, int D, int K,
                               const cake_bf16* C_prev, float* out_C, cake_bf16* out_C_bf16,
                               int* out_counts, void* ws, size_t ws_bytes, cake_stream_t stream,
                               unsigned flags) {
    int rc = check_shape(B, N, D, K);
    if (rc != CAKE_OK) return rc;
    if (!out_C || !out_counts || !ws || (N > 0 && (!X || !idx))) return CAKE_ERR_NULL;
    if (misaligned(X, 16) || misaligned(C_prev, 16) || misaligned(out_C, 16) || misaligned(out_C_bf16, 16) ||
        misaligned(idx, 4) || misaligned(out_counts, 4))
        return CAKE_ERR_ALIGN;
    Workspace w;
    rc = check_ws(ws, ws_bytes, B, N, D, K, &w);
    if (rc != CAKE_OK) return rc;
    XPrep x_padded;
    return do_update(X, idx, static_cast<int>(B), N, D, K, C_prev, out_C, out_C_bf16, out_counts, w,
                     reinterpret_cast<cudaStream_t>(stream), flags, &x_padded);
}

int cake_kmeans_update(const cake_bf16* X, const int* idx, long long N, int D, int K,
                       const cake_bf16* C_prev, float* out_C, cake_bf16* out_C_bf16, int* out_counts,
                       void* ws, size_t ws_bytes, cake_stream_t stream, unsigned flags) {
    return cake_kmeans_update_batched(X, idx, 1, N, D, K, C_prev, out_C, out_C_bf16, out_counts, ws,
                                      ws_bytes, stream, flags);
}

namespace {
// sums and counts of the rows given (no division): the slab route while its runs are long enough (the measured
// threshold of the one-call update; with rows spread over ranks the runs get shorter), else the sort route
int do_update_partial(const cake_bf16* X, const int* idx, int B, i64 N, int D, int K, float* out_sums, int* out_counts,
                      const Workspace& w, cudaStream_t s, unsigned flags) {
    unsigned path = flags & CAKE_UPDATE_MASK;
    if (path == CAKE_UPDATE_AUTO)
        path = (update_slab_supports(D, K) && update_slab_preferred(B, N, D, K)) ? CAKE_UPDATE_SLAB : CAKE_UPDATE_SORT;
    if (path == CAKE_UPDATE_SLAB)
        return launch_update_slab(X, idx, B, N, D, K, out_sums, out_counts, w.status, 0, s);
    if (path == CAKE_UPDATE_SORT) {
        UpdateScratch scr{out_sums, w.nvalid, w.cursor, w.pairs, w.part, w.done, w.rank};
        bool divided = false;
        int rc = launch_update_sort(X, idx, B, N, D, K, scr, out_counts, nullptr, nullptr, nullptr, &divided, w.status, s);
        return (rc == CAKE_OK && divided) ? CAKE_ERR_UNSUPPORTED : rc;
    }
    return CAKE_ERR_UNSUPPORTED;
}
}  // namespace

int cake_kmeans_update_partial_batched(const cake_bf16* X, const int* idx, long long B, long long N, int D,
                                       int K, float* out_sums, int* out_counts, void* ws, size_t ws_bytes,
                                       cake_stream_t stream, unsigned flags) {
    int rc = check_shape(B, N, D, K);
    if (rc != CAKE_OK) return rc;
    if (!out_sums || !out_counts || !ws || (N > 0 && (!X || !idx))) return CAKE_ERR_NULL;
    if (misaligned(X, 16) || misaligned(idx, 4) || misaligned(out_sums, 16) || misaligned(out_counts, 4))
        return CAKE_ERR_ALIGN;
    Workspace w;
    rc = check_ws(ws, ws_bytes, B, N, D, K, &w);
    if (rc != CAKE_OK) return rc;
    return do_update_partial(X, idx, static_cast<int>(B), N, D, K, out_sums, out_counts, w,
                             reinterpret_cast<cudaStream_t>(stream), flags);
}

int cake_kmeans_lloyd_sharded(const cake_bf16* X_local, const cake_bf16* C0, long long N_local, int D, int K, int iters,
                              float* out_C, cake_bf16* out_C_bf16, int* out_idx, float* out_dist, int* out_counts,
                              double* out_inertia, cake_allreduce_fn allreduce, void* user, void* ws, size_t ws_bytes,
                              cake_stream_t stream, unsigned flags) {
    int rc = check_shape(1, N_local, D, K);
    if (rc != CAKE_OK) return rc;
    if (iters < 1) return CAKE_ERR_SHAPE;
    if (!C0 || !out_C || !out_counts || !ws || (N_local > 0 && (!X_local || !out_idx))) return CAKE_ERR_NULL;
    if (misaligned(X_local, 16) || misaligned(C0, 16) || misaligned(out_C, 16) || misaligned(out_C_bf16, 16) ||
        misaligned(out_idx, 4) || misaligned(out_dist, 4) || misaligned(out_counts, 4) || misaligned(out_inertia, 8))
        return CAKE_ERR_ALIGN;
    Workspace w;
    rc = check_ws(ws, ws_bytes, 1, N_local, D, K, &w);
    if (rc != CAKE_OK) return rc;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const i64 N = N_local;
    const unsigned apath = flags & CAKE_ASSIGN_MASK;
    const bool tc_assign = N > 0 && (((assign_tc_supports(D) || assign_wide_supports(D)) && (apath == CAKE_ASSIGN_AUTO || apath == CAKE_ASSIGN_TCGEN05 ||
                                                                apath == CAKE_ASSIGN_TCGEN05_EXACT || apath == CAKE_ASSIGN_TCGEN05_PAIR ||
                                                                apath == CAKE_ASSIGN_TCGEN05_PAIR_EXACT)) ||
                                     (assign_pad_supports(D) && apath == CAKE_ASSIGN_AUTO));
    const int cpad_columns = assign_cpad_columns(D);
    const cake_bf16* cur = C0;
    int nxt = 0;
    bool prepared = false;
    XPrep x_padded;
    for (int t = 0; t < iters; ++t) {
        rc = do_assign(X_local, cur, 1, N, D, K, out_idx, out_dist, out_inertia ? out_inertia + t : nullptr, iters, true,
                       prepared, &x_padded, w, s, flags);
        if (rc != CAKE_OK) return rc;
        // this rank's sums and counts (rows of D columns: the padded copy of X is not used here)
        rc = do_update_partial(X_local, out_idx, 1, N, D, K, w.sums, out_counts, w, s, flags);
        if (rc != CAKE_OK) return rc;
        // the one exchange of the iteration: the caller adds up sums and counts of all ranks, in place, in stream order
        if (allreduce && allreduce(user, w.sums, static_cast<long long>(K) * D, out_counts, K, stream) != 0) return CAKE_ERR_CUDA;
        cake_bf16* dst = (t == iters - 1 && out_C_bf16) ? out_C_bf16 : w.cbuf[nxt];
        NextAssign next{w.caug, out_inertia ? out_inertia + t + 1 : nullptr, iters, cpad_columns ? w.cpad : nullptr, cpad_columns};
        const bool want = tc_assign && t + 1 < iters;
        if (launch_finalize(w.sums, out_counts, cur, 1, K, D, out_C, dst, false, want ? &next : nullptr, &prepared, s) != cudaSuccess)
            return CAKE_ERR_CUDA;
        cur = dst;
        nxt ^= 1;
    }
    return CAKE_OK;
}

int cake_kmeans_update_finish_batched(const float* sums, const int* counts, const cake_bf16* C_prev, long long B,
                                      int K, int D, float* out_C, cake_bf16* out_C_bf16, cake_stream_t stream) {
    int rc = check_shape(B, 0, D, K);
    if (rc != CAKE_OK) return rc;
    if (!sums || !counts || !out_C) return CAKE_ERR_NULL;
    if (misaligned(sums, 16) || misaligned(counts, 4) || misaligned(C_prev, 16) || misaligned(out_C, 16) ||
        misaligned(out_C_bf16, 16))
        return CAKE_ERR_ALIGN;
    if (launch_finalize(sums, counts, C_prev, static_cast<int>(B), K, D, out_C, out_C_bf16, false, nullptr, nullptr,
                        reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess)
        return CAKE_ERR_CUDA;
    return CAKE_OK;
}

int cake_kmeans_inertia_batched(const float* dist, long long B, long long N, double* out_inertia, int inertia_stride,
                                cake_stream_t stream) {
    if (B < 1 || B > 65535 || N < 0 || inertia_stride < 1) return CAKE_ERR_SHAPE;
    if (!out_inertia || (N > 0 && !dist)) return CAKE_ERR_NULL;
    if (misaligned(dist, 4) || misaligned(out_inertia, 8)) return CAKE_ERR_ALIGN;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (cudaMemset2DAsync(out_inertia, static_cast<size_t>(inertia_stride) * sizeof(double), 0, sizeof(double),
                          static_cast<size_t>(B), s) != cudaSuccess)
        return CAKE_ERR_CUDA;
    return launch_inertia(dist, static_cast<int>(B), N, out_inertia, inertia_stride, s) == cudaSuccess ? CAKE_OK : CAKE_ERR_CUDA;
}

int cake_kmeans_lloyd_batched(const cake_bf16* X, const cake_bf16* C0, long long B, long long N, int D,
                              int K, int iters, float* out_C, cake_bf16* out_C_bf16, int* out_idx,
                              float* out_dist, int* out_counts, double* out_inertia, void* ws,
                              size_t ws_bytes, cake_stream_t stream, unsigned flags) {
    int rc = check_shape(B, N, D, K);
    if (rc != CAKE_OK) return rc;
    if (iters < 0) return CAKE_ERR_SHAPE;
    if (!C0 || !out_C || !ws) return CAKE_ERR_NULL;
    if (iters > 0 && (!out_counts || (N > 0 && (!X || !out_idx)))) return CAKE_ERR_NULL;
    if (misaligned(X, 16) || misaligned(C0, 16) || misaligned(out_C, 16) || misaligned(out_C_bf16, 16) ||
        misaligned(out_idx, 4) || misaligned(out_dist, 4) || misaligned(out_counts, 4) ||
        misaligned(out_inertia, 8))
        return CAKE_ERR_ALIGN;
    Workspace w;
    rc = check_ws(ws, ws_bytes, B, N, D, K, &w);
    if (rc != CAKE_OK) return rc;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const int Bi = static_cast<int>(B);
    const size_t kd = static_cast<size_t>(B) * K * D;

    if (iters == 0) {
        // out_C = C0 widened: the division kernel with all-zero counts takes the keep-previous branch
        if (cudaMemsetAsync(w.cursor, 0, static_cast<size_t>(B) * K * 4, s) != cudaSuccess) return CAKE_ERR_CUDA;
        if (launch_finalize(w.sums, w.cursor, C0, Bi, K, D, out_C, nullptr, false, nullptr, nullptr, s) != cudaSuccess)
            return CAKE_ERR_CUDA;
        if (out_C_bf16 && cudaMemcpyAsync(out_C_bf16, C0, kd * 2, cudaMemcpyDeviceToDevice, s) != cudaSuccess)
            return CAKE_ERR_CUDA;
        return CAKE_OK;
    }
    // No copies: the first iteration reads C0 itself, the bf16 centroids ping-pong between the two
    // workspace buffers and the last iteration writes the caller's buffer directly.  Each iteration's
    // inertia entries are cleared by its own assign step.
    // The division kernel of iteration t also writes what the tensor-core assign of iteration t + 1 would
    // otherwise compute in a prologue launch of its own.
    const unsigned apath = flags & CAKE_ASSIGN_MASK;
    const bool tc_assign = N > 0 && (((assign_tc_supports(D) || assign_wide_supports(D)) && (apath == CAKE_ASSIGN_AUTO || apath == CAKE_ASSIGN_TCGEN05 ||
                                                                apath == CAKE_ASSIGN_TCGEN05_EXACT || apath == CAKE_ASSIGN_TCGEN05_PAIR ||
                                                                apath == CAKE_ASSIGN_TCGEN05_PAIR_EXACT)) ||
                                     (assign_pad_supports(D) && apath == CAKE_ASSIGN_AUTO));
    const int cpad_columns = assign_cpad_columns(D);
    const cake_bf16* cur = C0;
    int nxt = 0;
    bool prepared = false;
    XPrep x_padded;   // what the workspace holds of X (padded copy, wide-row operand), made by the first step that needs it
    // One problem of at most 128 clusters and 128 features: a single pass over X per iteration.  The assign kernel adds
    // the rows of every tile to per-cluster partial sums while the tile is in shared memory, and one small kernel adds
    // the partials up and divides (two launches per iteration instead of four).
    const bool try_fuse = tc_assign && !(flags & CAKE_LLOYD_NO_FUSE) && (flags & CAKE_UPDATE_MASK) == CAKE_UPDATE_AUTO &&
                          apath != CAKE_ASSIGN_TCGEN05_EXACT && fuse_shape_ok(B, D, K);
    // ... and where the CTAs can keep all rows in shared memory, every iteration in one cooperative launch
    if (try_fuse && !(flags & CAKE_LLOYD_NO_RESIDENT) && (apath == CAKE_ASSIGN_AUTO || apath == CAKE_ASSIGN_TCGEN05) && w.fpart) {
        DeviceInfo di;
        rc = current_device_info(&di);
        if (rc != CAKE_OK) return rc;
        if (lloyd_small_supports(di, N, D, K)) {
            rc = launch_lloyd_small(X, C0, N, D, K, iters, w.fpart, w.fcnt, w.cbuf[0], reinterpret_cast<unsigned*>(w.status + 32),
                                    out_C, out_C_bf16, out_idx, out_dist, out_counts, out_inertia, w.status, di, s);
            if (rc == CAKE_OK) return rc;
            // (a cooperative launch the device refuses: the general path below; what was enqueued so far are two clears)
        }
    }
    for (int t = 0; t < iters; ++t) {
        int fuse_ctas = 0;
        rc = do_assign(X, cur, Bi, N, D, K, out_idx, out_dist, out_inertia ? out_inertia + t : nullptr, iters,
                       true, prepared, &x_padded, w, s, flags, try_fuse ? &fuse_ctas : nullptr);
        if (rc != CAKE_OK) return rc;
        cake_bf16* dst = (t == iters - 1 && out_C_bf16) ? out_C_bf16 : w.cbuf[nxt];
        NextAssign next{w.caug, out_inertia ? out_inertia + t + 1 : nullptr, iters,
                        cpad_columns ? w.cpad : nullptr, cpad_columns};
        const bool want = tc_assign && t + 1 < iters;
        if (fuse_ctas > 0) {
            if (launch_finalize_partials(w.fpart, w.fcnt, fuse_ctas, cur, K, D, out_C, dst, out_counts, want ? &next : nullptr,
                                         &prepared, s) != cudaSuccess)
                return CAKE_ERR_CUDA;
        } else {
            rc = do_update(X, out_idx, Bi, N, D, K, cur, out_C, dst, out_counts, w, s, flags, &x_padded, want ? &next : nullptr, &prepared);
            if (rc != CAKE_OK) return rc;
        }
        cur = dst;
        nxt ^= 1;
    }
    return CAKE_OK;
}

int cake_kmeans_lloyd(const cake_bf16* X, const cake_bf16* C0, long long N, int D, int K, int iters,
                      float* out_C, cake_bf16* out_C_bf16, int* out_idx, float* out_dist, int* out_counts,
                      double* out_inertia, void* ws, size_t ws_bytes, cake_stream_t stream, unsigned flags) {
    return cake_kmeans_lloyd_batched(X, C0, 1, N, D, K, iters, out_C, out_C_bf16, out_idx, out_dist,
                                     out_counts, out_inertia, ws, ws_bytes, stream, flags);
}

int cake_kmeans_lloyd_tol(const cake_bf16* X, const cake_bf16* C0, long long N, int D, int K, int max_iters, double tol,
                          int check_every, float* out_C, cake_bf16* out_C_bf16, int* out_idx, float* out_dist,
                          int* out_counts, double* out_inertia, int* out_iters, void* ws, size_t ws_bytes,
                          cake_stream_t stream, unsigned flags) {
    int rc = check_shape(1, N, D, K);
    if (rc != CAKE_OK) return rc;
    if (max_iters < 1 || check_every < 1 || !(tol >= 0.0)) return CAKE_ERR_SHAPE;
    if (!out_C_bf16 || !out_inertia || !out_iters) return CAKE_ERR_NULL;
    Workspace w;
    rc = check_ws(ws, ws_bytes, 1, N, D, K, &w);
    if (rc != CAKE_OK) return rc;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const size_t kd = static_cast<size_t>(K) * D;
    const cake_bf16* cur = C0;
    int done = 0;
    double prev = 0.0;
    bool have_prev = false;
    while (done < max_iters) {
        const int block = max_iters - done < check_every ? max_iters - done : check_every;
        rc = cake_kmeans_lloyd_batched(X, cur, 1, N, D, K, block, out_C, out_C_bf16, out_idx, out_dist, out_counts,
                                       out_inertia + done, ws, ws_bytes, stream, flags);
        if (rc != CAKE_OK) return rc;
        // the host looks at the block's inertia values: the one synchronisation per block
        double host[64];
        bool stop = false;
        for (int o = 0; o < block && !stop; o += 64) {
            const int n = block - o < 64 ? block - o : 64;
            if (cudaMemcpyAsync(host, out_inertia + done + o, static_cast<size_t>(n) * 8, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
                cudaStreamSynchronize(s) != cudaSuccess)
                return CAKE_ERR_CUDA;
            for (int j = 0; j < n; ++j) {
                if (have_prev && prev - host[j] <= tol * prev) stop = true;   // looked at only at the block's end
                prev = host[j];
                have_prev = true;
            }
        }
        done += block;
        if (stop) break;
        if (done < max_iters) {
            if (cudaMemcpyAsync(w.ccont, out_C_bf16, kd * 2, cudaMemcpyDeviceToDevice, s) != cudaSuccess) return CAKE_ERR_CUDA;
            cur = w.ccont;
        }
    }
    *out_iters = done;
    return CAKE_OK;
}

int cake_kmeans_init_plusplus(const cake_bf16* X, long long N, int D, int K, const float* u, cake_bf16* out_C0,
                              int* out_rows, void* ws, size_t ws_bytes, cake_stream_t stream) {
    int rc = check_shape(1, N, D, K);
    if (rc != CAKE_OK) return rc;
    if (N < 1) return CAKE_ERR_SHAPE;
    if (!X || !u || !out_C0 || !ws) return CAKE_ERR_NULL;
    if (misaligned(X, 16) || misaligned(out_C0, 16) || misaligned(u, 4) || misaligned(out_rows, 4)) return CAKE_ERR_ALIGN;
    Workspace w;
    rc = check_ws(ws, ws_bytes, 1, N, D, K, &w);
    if (rc != CAKE_OK) return rc;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    // scratch: the (row, cluster) pairs of the sort route hold an index per row (unused result of the one-centroid
    // assign) and the running minimum; `dist` the distances to the row chosen last
    int* idx_scr = reinterpret_cast<int*>(w.pairs);
    float* mind = reinterpret_cast<float*>(w.pairs) + N;
    if (launch_pp_pick(X, mind, w.pp_part, N, D, u, 0, out_C0, out_rows, s) != cudaSuccess) return CAKE_ERR_CUDA;
    XPrep x_padded;
    // the centroid of a one-centroid assign must start on a 16-byte boundary: rows of D % 8 != 0 columns go through
    // the continuation buffer
    const bool via_copy = (static_cast<size_t>(D) * 2) % 16 != 0;
    for (int k = 1; k < K; ++k) {
        const cake_bf16* c = out_C0 + static_cast<size_t>(k - 1) * D;
        if (via_copy) {
            if (cudaMemcpyAsync(w.ccont, c, static_cast<size_t>(D) * 2, cudaMemcpyDeviceToDevice, s) != cudaSuccess) return CAKE_ERR_CUDA;
            c = w.ccont;
        }
        rc = do_assign(X, c, 1, N, D, 1, idx_scr, w.dist, nullptr, 0, false, false, &x_padded, w, s,
                       assign_tc_supports(D) ? CAKE_ASSIGN_TCGEN05_EXACT : CAKE_ASSIGN_AUTO);
        if (rc != CAKE_OK) return rc;
        if (launch_pp_accumulate(w.dist, mind, N, k == 1, w.pp_part, s) != cudaSuccess) return CAKE_ERR_CUDA;
        if (launch_pp_pick(X, mind, w.pp_part, N, D, u, k, out_C0 + static_cast<size_t>(k) * D, out_rows, s) != cudaSuccess)
            return CAKE_ERR_CUDA;
    }
    return CAKE_OK;
}

namespace {
struct HostDev {
    cake_bf16 *X, *C0, *Cb;
    float *C, *dist;
    int *idx, *counts;
    double* inertia;
    void* ws;
    size_t ws_bytes, bytes;
};
HostDev carve_host(void* base, i64 B, i64 N, int D, int K, int iters) {
    HostDev h;
    size_t o = 0;
    char* p = static_cast<char*>(base);
    auto take = [&](size_t n) { char* r = p ? p + o : nullptr; o += up(n); return r; };
    const size_t kd = static_cast<size_t>(B) * K * D, nd = static_cast<size_t>(B) * N * D;
    h.X = reinterpret_cast<cake_bf16*>(take(nd * 2));
    h.C0 = reinterpret_cast<cake_bf16*>(take(kd * 2));
    h.Cb = reinterpret_cast<cake_bf16*>(take(kd * 2));
    h.C = reinterpret_cast<float*>(take(kd * 4));
    h.dist = reinterpret_cast<float*>(take(static_cast<size_t>(B) * N * 4));
    h.idx = reinterpret_cast<int*>(take(static_cast<size_t>(B) * N * 4));
    h.counts = reinterpret_cast<int*>(take(static_cast<size_t>(B) * K * 4));
    h.inertia = reinterpret_cast<double*>(take(static_cast<size_t>(B) * (iters > 0 ? iters : 1) * 8));
    h.ws_bytes = carve(nullptr, B, N, D, K).bytes;
    h.ws = take(h.ws_bytes);
    h.bytes = o;
    return h;
}
}  // namespace

int cake_kmeans_lloyd_host_device_bytes(long long B, long long N, int D, int K, int iters, size_t* out_bytes) {
    if (!out_bytes) return CAKE_ERR_NULL;
    int rc = check_shape(B, N, D, K);
    if (rc != CAKE_OK) return rc;
    if (iters < 0) return CAKE_ERR_SHAPE;
    *out_bytes = carve_host(nullptr, B, N, D, K, iters).bytes;
    return CAKE_OK;
}

int cake_kmeans_lloyd_host(const cake_bf16* X_host, const cake_bf16* C0_host, long long B, long long N,
                           int D, int K, int iters, float* out_C_host, cake_bf16* out_C_bf16_host,
                           int* out_idx_host, float* out_dist_host, int* out_counts_host,
                           double* out_inertia_host, void* dev, size_t dev_bytes, cake_stream_t stream,
                           unsigned flags) {
    int rc = check_shape(B, N, D, K);
    if (rc != CAKE_OK) return rc;
    if (iters < 0) return CAKE_ERR_SHAPE;
    if (!C0_host || !out_C_host || !dev || (N > 0 && !X_host)) return CAKE_ERR_NULL;
    if (misaligned(dev, kAlign)) return CAKE_ERR_ALIGN;
    HostDev h = carve_host(dev, B, N, D, K, iters);
    if (dev_bytes < h.bytes) return CAKE_ERR_WORKSPACE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const size_t kd = static_cast<size_t>(B) * K * D, nd = static_cast<size_t>(B) * N * D;
    const size_t bn = static_cast<size_t>(B) * N, bk = static_cast<size_t>(B) * K;
    if (nd && cudaMemcpyAsync(h.X, X_host, nd * 2, cudaMemcpyHostToDevice, s) != cudaSuccess) return CAKE_ERR_CUDA;
    if (cudaMemcpyAsync(h.C0, C0_host, kd * 2, cudaMemcpyHostToDevice, s) != cudaSuccess) return CAKE_ERR_CUDA;
    if (cudaMemsetAsync(h.ws, 0, 256, s) != cudaSuccess) return CAKE_ERR_CUDA;
    rc = cake_kmeans_lloyd_batched(h.X, h.C0, B, N, D, K, iters, h.C, out_C_bf16_host ? h.Cb : nullptr, h.idx,
                                   out_dist_host ? h.dist : nullptr, h.counts,
                                   out_inertia_host ? h.inertia : nullptr, h.ws, h.ws_bytes, stream, flags);
    if (rc != CAKE_OK) return rc;
    bool ok = cudaMemcpyAsync(out_C_host, h.C, kd * 4, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    if (out_C_bf16_host) ok = ok && cudaMemcpyAsync(out_C_bf16_host, h.Cb, kd * 2, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    if (iters > 0) {
        if (out_idx_host && bn) ok = ok && cudaMemcpyAsync(out_idx_host, h.idx, bn * 4, cudaMemcpyDeviceToHost, s) == cudaSuccess;
        if (out_dist_host && bn) ok = ok && cudaMemcpyAsync(out_dist_host, h.dist, bn * 4, cudaMemcpyDeviceToHost, s) == cudaSuccess;
        if (out_counts_host) ok = ok && cudaMemcpyAsync(out_counts_host, h.counts, bk * 4, cudaMemcpyDeviceToHost, s) == cudaSuccess;
        if (out_inertia_host) ok = ok && cudaMemcpyAsync(out_inertia_host, h.inertia, static_cast<size_t>(B) * iters * 8, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    }
    return ok ? CAKE_OK : CAKE_ERR_CUDA;
}

int cake_kmeans_device_status(void* ws, cake_stream_t stream, int* host_out) {
    if (!ws || !host_out) return CAKE_ERR_NULL;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    int v = 0;
    if (cudaMemcpyAsync(&v, ws, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return CAKE_ERR_CUDA;
    if (cudaMemsetAsync(ws, 0, sizeof(int), s) != cudaSuccess) return CAKE_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return CAKE_ERR_CUDA;
    *host_out = v;
    return CAKE_OK;
}

int cake_kmeans_selftest_bounded_wait(void* ws, size_t ws_bytes, int limit_ms, cake_stream_t stream) {
    if (!ws) return CAKE_ERR_NULL;
    if (ws_bytes < 256) return CAKE_ERR_WORKSPACE;
    if (limit_ms < 1 || limit_ms > 1000) return CAKE_ERR_SHAPE;
    if (launch_bounded_wait_selftest(static_cast<int*>(ws), limit_ms, reinterpret_cast<cudaStream_t>(stream)) !=
        cudaSuccess)
        return CAKE_ERR_CUDA;
    return CAKE_OK;
}

}  // extern "C"
