// cake_kmeans_assign_static: nearest-centroid assignment for callers that cannot allocate.
//
// Some callers have no way to hand this library a workspace: code that runs where cudaMalloc is
// forbidden (inside another framework's memory-pool callback, in a process whose device memory is
// fully pre-partitioned, in an embedding whose allocator hooks must not be re-entered).  For them
// the scratch the assign kernel needs -- the centroid half-norm operand and the status word -- lives in a fixed
// array that is part of the loaded library image, so nothing is allocated at any point.
//
// The array is `static __device__`: every GPU that loads the library holds these 262,400 bytes until
// the process exits.  In host code the array's name is only a host-side handle, not a device
// address, so the address is obtained once per device with cudaGetSymbolAddress (with that device
// current) and that pointer is what the kernels receive.
#include <mutex>

#include "internal.h"

namespace cake {
namespace {

constexpr int kStaticMaxK = 16384;                         // largest K this entry point accepts
constexpr size_t kStaticHeader = 256;                      // status word, padded
constexpr size_t kStaticBytes =
    kStaticHeader + static_cast<size_t>(kStaticMaxK / kAssignBlockN) * kAssignAugTileBytes;   // 256 B + 256 KiB

static __device__ __align__(256) unsigned char g_assign_scratch[kStaticBytes];

// Device address of g_assign_scratch on the current device; resolved on the first call per device.
int scratch_for_current_device(unsigned char** out) {
    static std::mutex mu;
    static unsigned char* ptrs[64] = {nullptr};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return CAKE_ERR_DEVICE;
    }
    std::lock_guard<std::mutex> lock(mu);
    if (!ptrs[dev]) {
        void* p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&p, g_assign_scratch);
        if (e != cudaSuccess || !p) {
            cudaGetLastError();
            return CAKE_ERR_CUDA;
        }
        ptrs[dev] = static_cast<unsigned char*>(p);
    }
    *out = ptrs[dev];
    return CAKE_OK;
}

}  // namespace
}  // namespace cake

using namespace cake;

extern "C" int cake_kmeans_assign_static(const cake_bf16* X, const cake_bf16* C, long long N, int D, int K,
                                         int* out_idx, float* out_dist, cake_stream_t stream) {
    if (N < 0 || D < 1 || K < 1 || N > 2147482623LL) return CAKE_ERR_SHAPE;
    if (K > kStaticMaxK) return CAKE_ERR_UNSUPPORTED;      // beyond the fixed scratch: use cake_kmeans_assign
    if (!C || (N > 0 && (!X || !out_idx))) return CAKE_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(C)) % 16 != 0) return CAKE_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(out_idx) | reinterpret_cast<uintptr_t>(out_dist)) % 4 != 0) return CAKE_ERR_ALIGN;
    if (N == 0) return CAKE_OK;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (!assign_tc_supports(D)) return launch_assign_simt(X, C, 1, N, D, K, out_idx, out_dist, s);

    unsigned char* scratch = nullptr;
    int rc = scratch_for_current_device(&scratch);
    if (rc != CAKE_OK) return rc;
    // Word 0 of the array is the sticky device status: zero when the library is loaded, raised by a kernel
    // whose bounded wait expired, read and cleared by cake_kmeans_assign_static_status.  The half-norm operand
    // behind the header is rewritten in full (all ceil(K/256) tiles, padding rows included) by the prologue
    // that launch_assign_tc runs first, so nothing of an earlier call survives where this one reads.
    // (launch_assign_tc makes its host-side checks before it enqueues anything.)
    return launch_assign_tc(X, C, 1, N, D, K, scratch + kStaticHeader, false, out_idx, out_dist, nullptr, 0,
                            false, false, reinterpret_cast<int*>(scratch), s);
}

extern "C" int cake_kmeans_assign_static_status(cake_stream_t stream, int* host_out) {
    if (!host_out) return CAKE_ERR_NULL;
    unsigned char* scratch = nullptr;
    int rc = scratch_for_current_device(&scratch);
    if (rc != CAKE_OK) return rc;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    int v = 0;
    if (cudaMemcpyAsync(&v, scratch, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return CAKE_ERR_CUDA;
    if (cudaMemsetAsync(scratch, 0, sizeof(int), s) != cudaSuccess) return CAKE_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return CAKE_ERR_CUDA;
    *host_out = v;
    return CAKE_OK;
}
