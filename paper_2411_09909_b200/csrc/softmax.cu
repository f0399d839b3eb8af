// Row softmax in fp32 with bf16 output: the step between the two attention products.  The
// normalised self-attention map is what gets quantized (arXiv 2411.09909, Appendix C), and the
// quantizer reads bf16, so P is rounded to bf16 (nearest even) here.
#include <cuda_bf16.h>

#include "amx_common.cuh"

namespace amx {
namespace {

constexpr int kT = 256;

__device__ __forceinline__ float block_reduce(float v, bool is_max, float* sh) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        const float o = __shfl_xor_sync(0xFFFFFFFFu, v, d);
        v = is_max ? fmaxf(v, o) : v + o;
    }
    __syncthreads();  // sh may still be read from a previous reduction
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    v = sh[0];
#pragma unroll
    for (int i = 1; i < kT / 32; ++i) v = is_max ? fmaxf(v, sh[i]) : v + sh[i];
    return v;
}

__global__ void __launch_bounds__(kT)
softmax_bf16_kernel(const float* __restrict__ S, int64_t cols, int64_t ld_s, float alpha,
                    __nv_bfloat16* __restrict__ P, int64_t ld_p) {
    __shared__ float sh[kT / 32];
    const float* s = S + (int64_t)blockIdx.x * ld_s;
    __nv_bfloat16* p = P + (int64_t)blockIdx.x * ld_p;
    float mx = -INFINITY;
    for (int64_t c = threadIdx.x; c < cols; c += kT) mx = fmaxf(mx, alpha * s[c]);
    mx = block_reduce(mx, true, sh);
    float sum = 0.f;
    for (int64_t c = threadIdx.x; c < cols; c += kT) sum += expf(alpha * s[c] - mx);
    sum = block_reduce(sum, false, sh);
    for (int64_t c = threadIdx.x; c < cols; c += kT)
        p[c] = __float2bfloat16_rn(expf(alpha * s[c] - mx) / sum);
}

}  // namespace
}  // namespace amx

extern "C" int amx_softmax_bf16(const float* S, int64_t rows, int64_t cols, int64_t ld_s, float alpha,
                                void* P, int64_t ld_p, void* stream) {
    using namespace amx;
    if (rows < 0 || cols <= 0 || ld_s < cols || ld_p < cols || rows > 0x7FFFFFFF) return AMX_ERR_SHAPE;
    if (rows == 0) return AMX_OK;
    if (!S || !P) return AMX_ERR_NULL;
    if (!aligned(S, 4) || !aligned(P, 2)) return AMX_ERR_ALIGN;
    softmax_bf16_kernel<<<(unsigned)rows, kT, 0, static_cast<cudaStream_t>(stream)>>>(
        S, cols, ld_s, alpha, reinterpret_cast<__nv_bfloat16*>(P), ld_p);
    return launch_status();
}
