// Small kernels around the two hot ones: the CUDA-core assign fallback,
// the inertia reduction and the bounded-wait self test; plus the cached device query.
#include <atomic>
#include <mutex>

#include "internal.h"
#include "ptx.cuh"

namespace cake {

static std::atomic<unsigned long long> g_launches{0};
void note_launches(int n) { g_launches.fetch_add(static_cast<unsigned long long>(n), std::memory_order_relaxed); }
unsigned long long launches_so_far() { return g_launches.load(std::memory_order_relaxed); }

int current_device_info(DeviceInfo* out) {
    static std::mutex mu;
    static DeviceInfo cache[64];
    static bool have[64] = {false};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) {
        cudaGetLastError();
        return CAKE_ERR_DEVICE;
    }
    std::lock_guard<std::mutex> lock(mu);
    if (dev < 64 && have[dev]) {
        *out = cache[dev];
        return CAKE_OK;
    }
    DeviceInfo d;
    d.device = dev;
    if (cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&d.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return CAKE_ERR_CUDA;
    if (dev < 64) {
        cache[dev] = d;
        have[dev] = true;
    }
    *out = d;
    return CAKE_OK;
}

namespace {

__device__ __forceinline__ float bf16f(cake_bf16 b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }

// CUDA-core fallback: one warp per point, lanes stride the features, direct differences in fp32.
__global__ void __launch_bounds__(256)
assign_simt_kernel(const cake_bf16* __restrict__ X, const cake_bf16* __restrict__ C, int B, i64 N, int D,
                   int K, int* __restrict__ out_idx, float* __restrict__ out_dist) {
    const int lane = threadIdx.x & 31;
    const i64 warps_total = (static_cast<i64>(gridDim.x) * blockDim.x) >> 5;
    for (i64 w = (static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5; w < static_cast<i64>(B) * N;
         w += warps_total) {
        const i64 b = w / N;
        const cake_bf16* x = X + static_cast<size_t>(w) * D;
        const cake_bf16* Cb = C + static_cast<size_t>(b) * K * D;
        float best = __int_as_float(0x7f800000);
        int bidx = 0;
        for (int k = 0; k < K; ++k) {
            const cake_bf16* c = Cb + static_cast<size_t>(k) * D;
            float acc = 0.f;
            for (int d = lane; d < D; d += 32) {
                const float t = bf16f(x[d]) - bf16f(c[d]);
                acc = fmaf(t, t, acc);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            if (acc < best) {
                best = acc;
                bidx = k;
            }
        }
        if (lane == 0) {
            out_idx[w] = bidx;
            if (out_dist) out_dist[w] = best;
        }
    }
}

__global__ void __launch_bounds__(256)
inertia_kernel(const float* __restrict__ dist, i64 N, double* __restrict__ acc, int acc_stride) {
    __shared__ double part[8];
    const int b = blockIdx.y;
    const float* d = dist + static_cast<size_t>(b) * N;
    double s = 0.0;
    for (i64 i = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; i < N;
         i += static_cast<i64>(gridDim.x) * blockDim.x)
        s += static_cast<double>(d[i]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int i = 0; i < 8; ++i) t += part[i];
        atomicAdd(acc + static_cast<size_t>(b) * acc_stride, t);
    }
}

// Waits on an mbarrier that nothing completes, for at most limit_ns, then reports the expiry.
// one thread per 16-byte granule of the padded copy (the source rows are only 2-byte aligned)
__global__ void __launch_bounds__(256)
pad_rows_kernel(const cake_bf16* __restrict__ src, i64 rows, int D, int Gpad, uint4* __restrict__ dst) {
    const i64 total = rows * Gpad;
    for (i64 e = static_cast<i64>(blockIdx.x) * blockDim.x + threadIdx.x; e < total;
         e += static_cast<i64>(gridDim.x) * blockDim.x) {
        const i64 r = e / Gpad;
        const int c0 = static_cast<int>(e - r * Gpad) * 8;
        const cake_bf16* row = src + static_cast<size_t>(r) * D;
        uint32_t w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = c0 + 2 * j;
            const uint32_t lo = c < D ? __ldg(row + c) : 0u;
            const uint32_t hi = c + 1 < D ? __ldg(row + c + 1) : 0u;
            w[j] = lo | (hi << 16);
        }
        dst[e] = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

__global__ void bounded_wait_selftest_kernel(int* status, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        const uint32_t a = ptx::smem_u32(&bar);
        ptx::mbar_init(a, 1);
        ptx::fence_mbar_init();
        const uint64_t t0 = ptx::globaltimer_ns();
        bool done = false;
        while (!done) {
            if (ptx::mbar_try_wait(a, 0)) break;  // never true: no arrival is ever made
            if (ptx::globaltimer_ns() - t0 > limit_ns) {
                atomicCAS(status, CAKE_OK, CAKE_ERR_TIMEOUT);
                done = true;
            }
        }
    }
}

}  // namespace

int launch_assign_simt(const cake_bf16* X, const cake_bf16* C, int B, i64 N, int D, int K, int* out_idx,
                       float* out_dist, cudaStream_t s) {
    const i64 rows = static_cast<i64>(B) * N;
    if (rows == 0) return CAKE_OK;
    i64 ctas = (rows + 7) / 8;
    if (ctas > 148 * 64) ctas = 148 * 64;
    assign_simt_kernel<<<static_cast<unsigned>(ctas), 256, 0, s>>>(X, C, B, N, D, K, out_idx, out_dist);
    note_launches(1);
    return cudaGetLastError() == cudaSuccess ? CAKE_OK : CAKE_ERR_CUDA;
}

cudaError_t launch_inertia(const float* dist, int B, i64 N, double* acc, int acc_stride, cudaStream_t s) {
    if (N == 0) return cudaSuccess;
    i64 ctas = (N + 256 * 8 - 1) / (256 * 8);
    if (ctas > 296) ctas = 296;
    inertia_kernel<<<dim3(static_cast<unsigned>(ctas), B), 256, 0, s>>>(dist, N, acc, acc_stride);
    note_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_pad_rows(const cake_bf16* src, i64 rows, int D, int Dpad, cake_bf16* dst, cudaStream_t s) {
    const i64 total = rows * (Dpad / 8);
    if (total == 0) return cudaSuccess;
    i64 ctas = (total + 255) / 256;
    if (ctas > 148 * 32) ctas = 148 * 32;
    pad_rows_kernel<<<static_cast<unsigned>(ctas), 256, 0, s>>>(src, rows, D, Dpad / 8, reinterpret_cast<uint4*>(dst));
    note_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_bounded_wait_selftest(int* status, int limit_ms, cudaStream_t s) {
    bounded_wait_selftest_kernel<<<1, 32, 0, s>>>(status, static_cast<unsigned long long>(limit_ms) * 1000000ull);
    note_launches(1);
    return cudaGetLastError();
}

}  // namespace cake
