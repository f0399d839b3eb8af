// amx_quant_gemm_static: the quantize + GEMM layer call for callers that cannot give the
// library a workspace because they cannot allocate device memory at all.
//
// Who that is: code that runs after the application has handed the whole device to its own
// arena (an inference server that sizes its pools once at start-up), plug-ins and callbacks
// that are forbidden to touch the allocator, and latency-critical loops where an allocation -
// which may synchronise the device and takes an unbounded time - is not acceptable.  For them
// the scratch that amx_quant_gemm takes from its `workspace` argument (the GEMM's status word, the
// quantized copy of the activation and, when the FP4 kernel is picked, both operands in that kernel's
// form) lives in a fixed array inside the library image.
//
// The price: every GPU that loads the library carries the array (kStaticScratchBytes) until the
// process exits, problem sizes are capped by it, and all calls share it - two calls whose
// kernels overlap on the GPU (different streams, different host threads) race on it.
#include <mutex>

#include "gemm.cuh"

namespace amx {
namespace {

constexpr size_t kStaticScratchBytes = size_t(16) << 20;   // 16 MiB per GPU
constexpr int kMaxDevices = 64;

// In host code this name is only a handle for the runtime's symbol lookup, never an address a
// kernel may be given: the device address is fetched once per device below.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_mutex;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of the array on the current device; looked up on the first call per device.  With lazy
// module loading that lookup is also what brings this translation unit's module - and with it the array -
// onto the device, so it can fail for lack of memory when the application has already taken all of it.
int static_scratch(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return AMX_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();                 // do not leave the failure for the next launch check to trip over
            return AMX_ERR_CUDA;
        }
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return AMX_OK;
}

}  // namespace
}  // namespace amx

extern "C" size_t amx_quant_gemm_static_capacity(void) { return amx::kStaticScratchBytes; }

extern "C" int amx_quant_gemm_static(const void* A, int64_t ld_a, const uint8_t* w_codes,
                                     const uint8_t* w_scales, int64_t M, int64_t N, int64_t K,
                                     int group_size, uint32_t flags, float* C, int64_t ld_c, void* stream) {
    using namespace amx;
    if (flags & ~(AMX_GEMM_SIMT | AMX_GEMM_TC)) return AMX_ERR_FLAGS;
    if (!valid_group_size(group_size, K) || M < 0 || N < 0 || K <= 0 || K % group_size || K % 8) return AMX_ERR_SHAPE;
    if (M == 0 || N == 0) return AMX_OK;
    // Nothing below needs to start at zero except the GEMM's status word, which the GEMM launcher
    // clears itself on `stream`; the quantized activation is fully overwritten before it is read.
    if (amx_quant_gemm_workspace_bytes(M, N, K, group_size, flags) > kStaticScratchBytes) return AMX_ERR_TOO_LARGE;
    void* scratch = nullptr;
    const int rc = static_scratch(&scratch);
    if (rc != AMX_OK) return rc;
    return amx_quant_gemm(A, ld_a, w_codes, w_scales, nullptr, 0, M, N, K, group_size, flags, C, ld_c, scratch,
                          kStaticScratchBytes, stream);
}

// The status word of the most recent call on the current device (first word of the array).
extern "C" int amx_quant_gemm_static_status(void* stream) {
    void* scratch = nullptr;
    const int rc = amx::static_scratch(&scratch);
    if (rc != AMX_OK) return rc;
    return amx_gemm_status(scratch, stream);
}
