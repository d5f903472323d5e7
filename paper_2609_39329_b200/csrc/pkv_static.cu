// pkv_gram_noalloc: the sufficient statistics of Eq. 9 for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need the statistics:
// a plug-in inside a serving engine that owns every byte of device memory through its own pool, or a
// latency-critical loop where an allocation (an implicit device synchronisation) is not acceptable.  pkv_gram needs a context, and a
// context allocates its workspace.  This variant keeps the scratch the kernels need — the
// token-contiguous bf16 hi/lo copies of X and R and the device status word — in a fixed array that is
// part of the library image, so it needs neither a context nor any allocation.
//
// Consequences of the fixed array, all documented in pkv.h as well:
//   * sizes are bounded (PKV_NOALLOC_MAX_N / _F / _D); larger problems are rejected;
//   * every GPU that loads the library carries the array (about 4.2 MB) until the process exits;
//   * all calls share it: two calls whose kernels can overlap on the GPU (different streams) race.
#include <cuda_runtime.h>

#include "pkv_tc.h"

namespace {

constexpr size_t kStatusBytes = 256;
constexpr size_t kPairElems = (size_t)PKV_NOALLOC_MAX_F * PKV_NOALLOC_MAX_N;      // XT parts
constexpr size_t kPairElemsR = (size_t)PKV_NOALLOC_MAX_D * PKV_NOALLOC_MAX_N;     // RT parts
constexpr size_t kScratchBytes = kStatusBytes + 2 * kPairElems * 2 + 2 * kPairElemsR * 2;

// In host code this name is only a handle for the runtime's symbol calls; the device address is
// obtained with cudaGetSymbolAddress below and handed to the kernels as an ordinary pointer.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
unsigned char* g_scratch_addr[kMaxDevices];   // per device, filled at first use on that device

// Once per device, with that device current: resolve the array's device address.
int setup_device(int dev, unsigned char** out) {
    if (dev < 0 || dev >= kMaxDevices) return PKV_ERR_UNSUPPORTED;
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess || !p) {
            cudaGetLastError();
            return PKV_ERR_CUDA;
        }
        g_scratch_addr[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_scratch_addr[dev];
    return PKV_OK;
}

}  // namespace

extern "C" int pkv_gram_noalloc(const float* X, const float* R, int32_t n, int32_t F, int32_t d, float* S_H,
                                float* S_T, int accumulate, void* cuda_stream) {
    using namespace pkv;
    if (!X || !R || !S_H || !S_T) return PKV_ERR_INVALID_ARG;
    if (n <= 0 || F <= 0 || d <= 0) return PKV_ERR_INVALID_ARG;
    if (n > PKV_NOALLOC_MAX_N || F > PKV_NOALLOC_MAX_F || d > PKV_NOALLOC_MAX_D) return PKV_ERR_UNSUPPORTED;
    if (F % 8 || d % 8) return PKV_ERR_UNSUPPORTED;
    const void* ptrs[] = {X, R, S_H, S_T};
    for (const void* q : ptrs)
        if ((uintptr_t)q & 15) return PKV_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PKV_ERR_CUDA;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return PKV_ERR_CUDA;
    const cudaError_t before = cudaPeekAtLastError();      // an error the caller already carries is not this call's
    if (major != 10 || !tc_encode_available()) return PKV_ERR_UNSUPPORTED;
    unsigned char* base = nullptr;
    int rc = setup_device(dev, &base);
    if (rc != PKV_OK) return rc;

    cudaStream_t st = (cudaStream_t)cuda_stream;
    DevStatus* status = reinterpret_cast<DevStatus*>(base);
    __nv_bfloat16* b16 = reinterpret_cast<__nv_bfloat16*>(base + kStatusBytes);
    Pair XT{b16, b16 + kPairElems};
    Pair RT{b16 + 2 * kPairElems, b16 + 2 * kPairElems + kPairElemsR};
    const int ldT = (n + 7) / 8 * 8;
    // the array keeps the previous call's contents: the status word must start at zero (the operand
    // copies are fully rewritten for the rows and columns this call reads)
    if (cudaMemsetAsync(status, 0, sizeof(DevStatus), st) != cudaSuccess) return PKV_ERR_CUDA;
    Lc lc{st, nullptr, nullptr};
    rc = tc_gram_with_buffers(lc, XT, RT, ldT, X, R, n, F, d, S_H, S_T, accumulate != 0, status);
    if (rc != PKV_OK) return rc;
    DevStatus host;      // plain host memory: the copy below is synchronous with respect to the host
    if (cudaMemcpyAsync(&host, status, sizeof(DevStatus), cudaMemcpyDeviceToHost, st) != cudaSuccess) return PKV_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return PKV_ERR_CUDA;
    const cudaError_t after = cudaPeekAtLastError();
    if (after != cudaSuccess && after != before) return PKV_ERR_CUDA;
    return host.code;
}
