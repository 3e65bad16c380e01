// k-means++ seeding (D^2 sampling) around the assign kernel.  The paper's K-means workload starts from sampled rows
// and names no seeding (Section 5, "Flash-KMeans clean-start workload"); this is the textbook initialiser, with the
// random numbers supplied by the caller.
//
// Per draw k >= 1 the library's assign kernel (one centroid: the row chosen last) gives every row's distance to it;
// pp_accumulate_kernel folds that into the running minimum mind[i] and sums it slab by slab (fp64);
// pp_pick_kernel finds the first row whose running sum of mind exceeds u[k] * sum(mind) and copies that row to the
// output.  Everything stays on the device: no host synchronisation between draws.
#include "internal.h"

namespace cake {
namespace {

constexpr int PP_THREADS = 1024;

// mind[i] = min(mind[i], dist[i]) (first draw: = dist[i]); part[b] = sum of the slab's mind, fp64
__global__ void __launch_bounds__(256)
pp_accumulate_kernel(const float* __restrict__ dist, float* __restrict__ mind, i64 N, i64 slab, int first,
                     double* __restrict__ part) {
    const i64 lo = static_cast<i64>(blockIdx.x) * slab;
    const i64 hi = lo + slab < N ? lo + slab : N;
    double acc = 0.0;
    for (i64 i = lo + threadIdx.x; i < hi; i += blockDim.x) {
        const float d = dist[i];
        const float m = first ? d : fminf(mind[i], d);
        mind[i] = m;
        acc += static_cast<double>(m);
    }
    __shared__ double red[256];
    red[threadIdx.x] = acc;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (static_cast<int>(threadIdx.x) < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) part[blockIdx.x] = red[0];
}

// One CTA.  k = 0: row = floor(u[0] * N).  k >= 1: target = u[k] * sum(part); the slab in which the running sum
// crosses the target is found from `part`, then the row inside it: every thread sums a run of consecutive rows, the
// runs are scanned, and the thread whose run crosses walks it.  The chosen row is recorded and copied to out_row.
__global__ void __launch_bounds__(PP_THREADS)
pp_pick_kernel(const cake_bf16* __restrict__ X, const float* __restrict__ mind, const double* __restrict__ part,
               int n_slabs, i64 slab, i64 N, int D, const float* __restrict__ u, int k, cake_bf16* __restrict__ out_row,
               int* __restrict__ rows_out) {
    __shared__ double run[PP_THREADS];
    __shared__ i64 chosen;
    __shared__ double base;
    __shared__ int slab_sel;
    const int t = threadIdx.x;
    const double uk = static_cast<double>(u[k]);
    if (t == 0) {
        i64 row = static_cast<i64>(uk * static_cast<double>(N));
        chosen = row < N ? row : N - 1;       // k = 0, or nothing to weigh by
        slab_sel = -1;
        if (k > 0) {
            double total = 0.0;
            for (int b = 0; b < n_slabs; ++b) total += part[b];
            if (total > 0.0) {
                const double target = uk * total;
                double acc = 0.0;
                int b = 0;
                for (; b < n_slabs - 1; ++b) {
                    if (acc + part[b] > target) break;
                    acc += part[b];
                }
                slab_sel = b;
                base = target - acc;          // what the rows of this slab have to exceed
            }
        }
    }
    __syncthreads();
    if (slab_sel >= 0) {
        const i64 lo = static_cast<i64>(slab_sel) * slab;
        const i64 hi = lo + slab < N ? lo + slab : N;
        const i64 per = (hi - lo + PP_THREADS - 1) / PP_THREADS;
        const i64 a = lo + static_cast<i64>(t) * per;
        const i64 e = a + per < hi ? a + per : hi;
        double acc = 0.0;
        for (i64 i = a; i < e; ++i) acc += static_cast<double>(mind[i]);
        run[t] = acc;
        __syncthreads();
        if (t == 0) {
            // the first run whose end exceeds the target; the last row with mass if rounding leaves none
            double before = 0.0;
            int sel = PP_THREADS - 1;
            for (int j = 0; j < PP_THREADS; ++j) {
                if (before + run[j] > base) { sel = j; break; }
                before += run[j];
            }
            const i64 ra = lo + static_cast<i64>(sel) * per;
            const i64 re = ra + per < hi ? ra + per : hi;
            i64 pick = hi - 1;
            double accr = before;
            for (i64 i = ra; i < re; ++i) {
                accr += static_cast<double>(mind[i]);
                if (accr > base) { pick = i; break; }
            }
            chosen = pick;
        }
        __syncthreads();
    }
    const i64 row = chosen;
    if (t == 0 && rows_out) rows_out[k] = static_cast<int>(row);
    for (int d = t; d < D; d += PP_THREADS) out_row[d] = X[static_cast<size_t>(row) * D + d];
}

}  // namespace

int pp_slabs(i64 N, i64* slab) {
    i64 n = (N + 2047) / 2048;
    if (n > kPlusPlusMaxSlabs) n = kPlusPlusMaxSlabs;
    if (n < 1) n = 1;
    *slab = (N + n - 1) / n;
    return static_cast<int>((N + *slab - 1) / *slab);
}

cudaError_t launch_pp_accumulate(const float* dist, float* mind, i64 N, bool first, double* part, cudaStream_t s) {
    i64 slab;
    const int n = pp_slabs(N, &slab);
    pp_accumulate_kernel<<<n, 256, 0, s>>>(dist, mind, N, slab, first ? 1 : 0, part);
    note_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_pp_pick(const cake_bf16* X, const float* mind, const double* part, i64 N, int D, const float* u, int k,
                           cake_bf16* out_row, int* rows_out, cudaStream_t s) {
    i64 slab;
    const int n = pp_slabs(N, &slab);
    pp_pick_kernel<<<1, PP_THREADS, 0, s>>>(X, mind, part, n, slab, N, D, u, k, out_row, rows_out);
    note_launches(1);
    return cudaGetLastError();
}

}  // namespace cake
