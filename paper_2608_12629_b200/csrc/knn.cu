// Exact k-nearest-neighbour search on the assign kernel's pipeline (the paper's Section 6 lists a "KNN search"
// family with recall 1.0 beside K-means: the same distance GEMM, a top-k epilogue instead of the arg-min).
//
// The database rows take the place of the centroids: they are streamed in 256-row tiles against 128-query row
// tiles, the whole m + d/2 is accumulated in tensor memory, and each epilogue thread keeps the 8 or 32 smallest
// values of its query and of its 128-column half of the tiles (assign_tc.cu, TOPK).  The two sorted half-lists of a
// query are merged here.  Everything is ordered by (distance, database row): equal distances go to the lower row.
#include <limits.h>

#include "internal.h"

namespace cake {
namespace {

constexpr size_t kAlign = 256;
inline size_t up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }
constexpr int kMaxK = 32;

// one thread per query: two sorted lists of kl (distance, row) pairs -> the k <= kl smallest, sorted
__global__ void __launch_bounds__(256)
knn_merge_kernel(const int* __restrict__ half_idx, const float* __restrict__ half_dist, i64 N, int kl, int k,
                 int* __restrict__ out_idx, float* __restrict__ out_dist) {
    const i64 row = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (row >= N) return;
    const int* ia = half_idx + row * 2 * kl;
    const float* da = half_dist + row * 2 * kl;
    const int* ib = ia + kl;
    const float* db = da + kl;
    int a = 0, b = 0;
    for (int s = 0; s < k; ++s) {
        // unused places carry row -1 and distance +inf and sort behind everything
        const bool has_a = a < kl && ia[a] >= 0, has_b = b < kl && ib[b] >= 0;
        int pick_i = -1;
        float pick_d = __int_as_float(0x7f800000);
        if (has_a && (!has_b || da[a] < db[b] || (da[a] == db[b] && ia[a] < ib[b]))) {
            pick_i = ia[a];
            pick_d = da[a];
            ++a;
        } else if (has_b) {
            pick_i = ib[b];
            pick_d = db[b];
            ++b;
        }
        out_idx[row * k + s] = pick_i;
        if (out_dist) out_dist[row * k + s] = pick_d;
    }
}

struct KnnWorkspace {
    int* status;          // [64] header: word 0 = sticky device status (zeroed by the caller once)
    void* aug;            // [ceil(M/256)][4 KiB] half-norm operand of the database rows
    int* half_idx;        // [N][2][kl], kl = list_len(k)
    float* half_dist;     // [N][2][kl]
    cake_bf16* qpad;      // [N][padded_d(D)] when D % 8 != 0
    cake_bf16* cpad;      // [M][round_up(D, 64)] when D % 64 != 0: the copy of the database the kernel streams
    size_t bytes;
};

// length of the per-half lists the kernel keeps: 8 or 32 (k = 1 is the arg-min and takes the assign kernel itself)
inline int list_len(int k) { return k <= 1 ? 0 : (k <= 8 ? 8 : 32); }

KnnWorkspace carve(void* base, i64 N, i64 M, int D, int k) {
    KnnWorkspace w;
    size_t o = 0;
    char* p = static_cast<char*>(base);
    auto take = [&](size_t n) { char* r = p ? p + o : nullptr; o += up(n); return r; };
    w.status = reinterpret_cast<int*>(take(256));
    w.aug = take(assign_tc_aug_bytes(1, static_cast<int>(M)));
    w.half_idx = reinterpret_cast<int*>(take(static_cast<size_t>(N) * 2 * list_len(k) * 4));
    w.half_dist = reinterpret_cast<float*>(take(static_cast<size_t>(N) * 2 * list_len(k) * 4));
    const size_t dpad = assign_pad_supports(D) ? static_cast<size_t>(padded_d(D)) : 0;
    w.qpad = reinterpret_cast<cake_bf16*>(take(static_cast<size_t>(N) * dpad * 2));
    w.cpad = reinterpret_cast<cake_bf16*>(take(static_cast<size_t>(M) * assign_cpad_columns(D) * 2));
    w.bytes = o;
    return w;
}

int check_shape(i64 N, i64 M, int D, int k) {
    if (N < 0 || M < 1 || D < 1 || k < 1) return CAKE_ERR_SHAPE;
    if (N > INT_MAX - 1024 || M > INT_MAX - 1024) return CAKE_ERR_SHAPE;
    if (static_cast<double>(N) * D > 4.0e13 || static_cast<double>(M) * D > 4.0e13) return CAKE_ERR_SHAPE;
    if (k > kMaxK) return CAKE_ERR_UNSUPPORTED;
    if (padded_d(D) > kAssignResidentMaxD) return CAKE_ERR_UNSUPPORTED;   // the top-k epilogue exists for a resident X tile only
    return CAKE_OK;
}

}  // namespace

cudaError_t launch_knn_merge(const int* half_idx, const float* half_dist, i64 N, int kl, int k, int* out_idx,
                             float* out_dist, cudaStream_t s) {
    if (N == 0) return cudaSuccess;
    knn_merge_kernel<<<static_cast<unsigned>((N + 255) / 256), 256, 0, s>>>(half_idx, half_dist, N, kl, k, out_idx, out_dist);
    note_launches(1);
    return cudaGetLastError();
}

}  // namespace cake

using namespace cake;

extern "C" {

int cake_knn_workspace_bytes(long long N, long long M, int D, int k, size_t* out_bytes) {
    if (!out_bytes) return CAKE_ERR_NULL;
    int rc = check_shape(N, M, D, k);
    if (rc != CAKE_OK) return rc;
    *out_bytes = carve(nullptr, N, M, D, k).bytes;
    return CAKE_OK;
}

int cake_knn_search(const cake_bf16* Q, const cake_bf16* X, long long N, long long M, int D, int k, int* out_idx,
                    float* out_dist, void* ws, size_t ws_bytes, cake_stream_t stream) {
    int rc = check_shape(N, M, D, k);
    if (rc != CAKE_OK) return rc;
    if (!X || !ws || (N > 0 && (!Q || !out_idx))) return CAKE_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(Q) | reinterpret_cast<uintptr_t>(X)) % 16 != 0) return CAKE_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(out_idx) | reinterpret_cast<uintptr_t>(out_dist)) % 4 != 0) return CAKE_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(ws) % kAlign != 0) return CAKE_ERR_ALIGN;
    KnnWorkspace w = carve(ws, N, M, D, k);
    if (ws_bytes < w.bytes) return CAKE_ERR_WORKSPACE;
    if (N == 0) return CAKE_OK;
    DeviceInfo di;
    rc = current_device_info(&di);
    if (rc != CAKE_OK) return rc;
    if (di.cc_major != 10) return CAKE_ERR_DEVICE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    int Dx = 0;
    if (assign_pad_supports(D)) {
        // rows that are no multiple of 16 bytes: a zero-padded copy of the queries here, of the database rows in the
        // kernel's prologue (zeros change no distance)
        Dx = padded_d(D);
        if (launch_pad_rows(Q, N, D, Dx, w.qpad, s) != cudaSuccess) return CAKE_ERR_CUDA;
        Q = w.qpad;
    }
    cake_bf16* cpad = assign_cpad_columns(D) ? w.cpad : nullptr;
    if (k == 1)   // the nearest row alone is the arg-min: the assign kernel with its full-precision epilogue, [N][1] = [N]
        return launch_assign_tc(Q, X, 1, N, D, static_cast<int>(M), w.aug, true, out_idx, out_dist, nullptr, 0, false, false,
                                w.status, s, Dx, cpad, 0);
    const int kl = list_len(k);
    rc = launch_assign_tc(Q, X, 1, N, D, static_cast<int>(M), w.aug, false, w.half_idx, w.half_dist, nullptr, 0, false,
                          false, w.status, s, Dx, cpad, kl);
    if (rc != CAKE_OK) return rc;
    if (launch_knn_merge(w.half_idx, w.half_dist, N, kl, k, out_idx, out_dist, s) != cudaSuccess) return CAKE_ERR_CUDA;
    return CAKE_OK;
}

}  // extern "C"
