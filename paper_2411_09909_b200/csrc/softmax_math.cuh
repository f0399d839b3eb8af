// Row softmax in fp32, the step between the two attention products (arXiv 2411.09909, Appendix C: the
// normalised self-attention map is what gets quantized).  Shared by the stand-alone kernel (bf16 output) and by
// the kernel that casts the map to AMXFP4 in the same pass, so that both produce the same bits: one block of kT
// threads per row; thread t owns the 32-column groups t, t + kT, ...; maxima and sums are taken first over the
// thread's own columns in order, then over the warp (xor tree), then over the warps in order.
#pragma once
#include <cuda_bf16.h>

#include "amx_common.cuh"

namespace amx {
namespace softmax {

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

// alpha * s for the 32 columns of group g of a row; -inf past the last column (contributes exp() = 0).
// vec: the row is 16-byte aligned and holds whole groups, so the group is read with eight 16-byte loads.
__device__ __forceinline__ void load_group(const float* __restrict__ s, int64_t g, int64_t cols, bool vec, float alpha,
                                           float (&t)[32]) {
    if (vec) {
        const float4* p = reinterpret_cast<const float4*>(s + g * 32);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float4 q = __ldg(p + j);
            t[4 * j] = alpha * q.x; t[4 * j + 1] = alpha * q.y; t[4 * j + 2] = alpha * q.z; t[4 * j + 3] = alpha * q.w;
        }
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const int64_t c = g * 32 + i;
            t[i] = c < cols ? alpha * s[c] : -INFINITY;
        }
    }
}

// Row maximum and the sum of exp(alpha * s - max) for the row this block owns.
__device__ __forceinline__ void row_stats(const float* __restrict__ s, int64_t cols, bool vec, float alpha, float* sh,
                                          float& mx, float& sum) {
    const int64_t G = (cols + 31) / 32;
    float t[32];
    mx = -INFINITY;
    for (int64_t g = threadIdx.x; g < G; g += kT) {
        load_group(s, g, cols, vec, alpha, t);
#pragma unroll
        for (int i = 0; i < 32; ++i) mx = fmaxf(mx, t[i]);
    }
    mx = block_reduce(mx, true, sh);
    sum = 0.f;
    for (int64_t g = threadIdx.x; g < G; g += kT) {
        load_group(s, g, cols, vec, alpha, t);
#pragma unroll
        for (int i = 0; i < 32; ++i) sum += expf(t[i] - mx);
    }
    sum = block_reduce(sum, false, sh);
}

// e / sum for the 32 values e = exp(alpha * s - max) of one group, rounded to bf16 (nearest even), as 16 bf16x2
// words.
__device__ __forceinline__ void normalised_group_e(const float (&e)[32], float sum, uint32_t (&w)[16]) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const __nv_bfloat16 lo = __float2bfloat16_rn(e[2 * i] / sum);
        const __nv_bfloat16 hi = __float2bfloat16_rn(e[2 * i + 1] / sum);
        w[i] = (uint32_t)__bfloat16_as_ushort(lo) | ((uint32_t)__bfloat16_as_ushort(hi) << 16);
    }
}
// The same from t = alpha * s.
__device__ __forceinline__ void normalised_group(float (&t)[32], float mx, float sum, uint32_t (&w)[16]) {
#pragma unroll
    for (int i = 0; i < 32; ++i) t[i] = expf(t[i] - mx);
    normalised_group_e(t, sum, w);
}

}  // namespace softmax
}  // namespace amx
