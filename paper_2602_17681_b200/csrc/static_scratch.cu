// latmix_linear_static: the whole layer for callers that may not allocate device memory.
//
// Some callers of this library cannot hand it a workspace: code that runs under an allocator it does not
// own (an inference server's plugin, a real-time loop with a frozen memory map), or that simply must not
// reach cudaMalloc because an allocation synchronises the device.  For them the scratch that latmix_linear
// keeps in the caller's workspace -- the status word and the activation codes and scales between the two
// kernels -- lives in one file-scope device array of fixed size.  Every GPU that loads the library holds that
// array until the process exits; every call on a device shares it.
#include <atomic>
#include <mutex>

#include "internal.h"

namespace latmix {

// 16 MiB of activation codes + scales (enough for 4096 x 4096 MXFP4 or 4096 x 3968 8-bit elements)
// behind the 256-byte header that holds the status word.
constexpr size_t kStaticScratchBytes = LATMIX_STATIC_SCRATCH_BYTES;
static_assert(kStaticScratchBytes > kWorkspaceHeaderBytes, "header must fit");

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code `g_static_scratch` is only a handle for the runtime, not a device address; the address the
// kernels need comes from cudaGetSymbolAddress, asked once per device with that device current.
static cudaError_t static_scratch_address(void** out) {
    constexpr int kMaxDevices = 64;
    static void* addr[kMaxDevices];
    static std::atomic<int> known[kMaxDevices];
    static std::mutex mu;
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (known[dev].load(std::memory_order_acquire) == 0) {
        std::lock_guard<std::mutex> lock(mu);
        if (known[dev].load(std::memory_order_relaxed) == 0) {
            void* p = nullptr;
            e = cudaGetSymbolAddress(&p, g_static_scratch);
            if (e != cudaSuccess) return e;
            addr[dev] = p;
            known[dev].store(1, std::memory_order_release);
        }
    }
    *out = addr[dev];
    return cudaSuccess;
}

}  // namespace latmix

using namespace latmix;

extern "C" latmix_status_t latmix_linear_static(const void* X, latmix_dtype_t x_dtype, const void* A, const float* b,
                                                const void* Wq_codes, const void* Wq_scales, const float* c, int64_t M,
                                                int64_t K, int64_t N, latmix_format_t fmt, float* out, int64_t ldo,
                                                uint32_t flags, latmix_status_t* device_status, void* cuda_stream) {
    if (fmt == LATMIX_NVFP4) return LATMIX_ERR_UNSUPPORTED;     // its tensor scale would need the header this call clears
    // what latmix_linear cannot do without: the header, the activation codes and their scales
    size_t code_bytes = 0, scale_bytes = 0;
    latmix_status_t s = latmix_mx_sizes(M, K, fmt, LATMIX_SF_TCGEN05, &code_bytes, &scale_bytes);
    if (s != LATMIX_OK) return s;
    const size_t need = kWorkspaceHeaderBytes + (code_bytes + 255) / 256 * 256 + (scale_bytes + 255) / 256 * 256;
    if (need > kStaticScratchBytes) return LATMIX_ERR_WORKSPACE;      // beyond the built-in scratch: use latmix_linear
    void* scratch = nullptr;
    if (static_scratch_address(&scratch) != cudaSuccess) return LATMIX_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // the array keeps whatever the previous call left: the status word must start at zero
    if (cudaMemsetAsync(scratch, 0, kWorkspaceHeaderBytes, st) != cudaSuccess) return LATMIX_ERR_CUDA;
    s = latmix_linear(X, x_dtype, A, b, Wq_codes, Wq_scales, c, M, K, N, fmt, out, ldo, scratch, kStaticScratchBytes, flags,
                      cuda_stream);
    if (s != LATMIX_OK) return s;
    if (device_status != nullptr) *device_status = latmix_device_status(scratch, cuda_stream);
    return LATMIX_OK;
}
