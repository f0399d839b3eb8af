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

// exp(t - mx) as 2^(t * log2(e) - mx * log2(e)): one fused multiply-add (the product is not rounded) and the
// hardware's base-2 exponential (relative error 2^-22; results below the smallest normal float flush to zero).
// neg_mx_l2e = -(mx * log2(e)), rounded once per row: the rounding error is a common factor of the whole row and
// cancels in the normalisation.  What remains is the rounding of the exponent itself, |t - mx| * 2^-24 relative,
// which any fp32 evaluation of exp(t - mx) has as well.
__device__ __forceinline__ float neg_max_log2e(float mx) { return -(mx * 1.4426950408889634f); }
__device__ __forceinline__ float exp_rel(float t, float neg_mx_l2e) {
    const float y = fmaf(t, 1.4426950408889634f, neg_mx_l2e);
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(y));
    return r;
}

// alpha * s for the 32 columns of group g of a row; -inf past the last column (contributes exp() = 0).
// vec: the row is 16-byte aligned and holds whole groups, so the group is read with eight 16-byte loads.
// seen: columns from `seen` on are masked (a causal row sees its own and earlier keys only): -inf as well.
__device__ __forceinline__ void load_group(const float* __restrict__ s, int64_t g, int64_t cols, bool vec, float alpha,
                                           float (&t)[32], int64_t seen) {
    if (seen < cols) cols = seen;
    if (vec && (g + 1) * 32 <= cols) {
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

// Softmax of a row of at most kT groups with the thread's group kept in registers: on return e holds
// exp(alpha * s - max) of the thread's own group (zeros for a thread without one); returns the row sum.
__device__ __forceinline__ float cached_row_exp(const float* __restrict__ s, int G, bool vec, float alpha, float* sh,
                                                float (&e)[32], int64_t seen) {
    if ((int)threadIdx.x < G) {
        load_group(s, threadIdx.x, (int64_t)G * 32, vec, alpha, e, seen);
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) e[i] = -INFINITY;
    }
    float mx = -INFINITY, sum = 0.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) mx = fmaxf(mx, e[i]);
    mx = block_reduce(mx, true, sh);
    const float nm = neg_max_log2e(mx);
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        e[i] = exp_rel(e[i], nm);
        sum += e[i];
    }
    return block_reduce(sum, false, sh);
}

// Row maximum and the sum of exp(alpha * s - max) for the row this block owns.
__device__ __forceinline__ void row_stats(const float* __restrict__ s, int64_t cols, bool vec, float alpha, float* sh,
                                          float& mx, float& sum, int64_t seen) {
    const int64_t G = (cols + 31) / 32;
    float t[32];
    mx = -INFINITY;
    for (int64_t g = threadIdx.x; g < G; g += kT) {
        load_group(s, g, cols, vec, alpha, t, seen);
#pragma unroll
        for (int i = 0; i < 32; ++i) mx = fmaxf(mx, t[i]);
    }
    mx = block_reduce(mx, true, sh);
    sum = 0.f;
    const float nm = neg_max_log2e(mx);
    for (int64_t g = threadIdx.x; g < G; g += kT) {
        load_group(s, g, cols, vec, alpha, t, seen);
#pragma unroll
        for (int i = 0; i < 32; ++i) sum += exp_rel(t[i], nm);
    }
    sum = block_reduce(sum, false, sh);
}

// e / sum for the 32 values e = exp(alpha * s - max) of one group, rounded to bf16 (nearest even), as 16 bf16x2
// words.
// The division is one reciprocal per row and a multiply per element (within 1.5 fp32 ulp of the quotient, far
// inside the bf16 rounding that follows).
__device__ __forceinline__ void normalised_group_e(const float (&e)[32], float sum, uint32_t (&w)[16]) {
    const float inv = 1.0f / sum;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const __nv_bfloat162 pr = __floats2bfloat162_rn(e[2 * i] * inv, e[2 * i + 1] * inv);   // .x = low half
        w[i] = *reinterpret_cast<const uint32_t*>(&pr);
    }
}
// The same from t = alpha * s.
__device__ __forceinline__ void normalised_group(float (&t)[32], float mx, float sum, uint32_t (&w)[16]) {
    const float nm = neg_max_log2e(mx);
#pragma unroll
    for (int i = 0; i < 32; ++i) t[i] = exp_rel(t[i], nm);
    normalised_group_e(t, sum, w);
}

}  // namespace softmax
}  // namespace amx
