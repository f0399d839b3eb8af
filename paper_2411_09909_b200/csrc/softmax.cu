// Row softmax in fp32 with bf16 output: the step between the two attention products.  The
// normalised self-attention map is what gets quantized (arXiv 2411.09909, Appendix C), and the
// quantizer reads bf16, so P is rounded to bf16 (nearest even) here.  The arithmetic is in
// softmax_math.cuh; the kernel that also casts the map is in quantize.cu.
#include "softmax_math.cuh"

namespace amx {
namespace {

using namespace softmax;

__device__ __forceinline__ void store_group(uint16_t* __restrict__ p, int64_t g, int64_t cols, bool vec_out,
                                            const uint32_t (&w)[16]) {
    if (vec_out) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            reinterpret_cast<uint4*>(p + g * 32)[j] = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const int64_t c = g * 32 + i;
            if (c < cols) p[c] = (uint16_t)(w[i >> 1] >> ((i & 1) * 16));
        }
    }
}

// Rows of whole groups, at most kT of them: each thread keeps its group in registers between the passes.
__global__ void __launch_bounds__(kT)
softmax_bf16_cached_kernel(const float* __restrict__ S, int G, int64_t ld_s, float alpha, uint16_t* __restrict__ P,
                           int64_t ld_p, int vec_in, int vec_out) {
    __shared__ float sh[kT / 32];
    float e[32];
    const float sum = cached_row_exp(S + (int64_t)blockIdx.x * ld_s, G, vec_in != 0, alpha, sh, e, (int64_t)G * 32);
    if ((int)threadIdx.x < G) {
        uint32_t w[16];
        normalised_group_e(e, sum, w);
        store_group(P + (int64_t)blockIdx.x * ld_p, threadIdx.x, (int64_t)G * 32, vec_out != 0, w);
    }
}

__global__ void __launch_bounds__(kT)
softmax_bf16_kernel(const float* __restrict__ S, int64_t cols, int64_t ld_s, float alpha,
                    uint16_t* __restrict__ P, int64_t ld_p, int vec_in, int vec_out) {
    __shared__ float sh[kT / 32];
    const float* s = S + (int64_t)blockIdx.x * ld_s;
    uint16_t* p = P + (int64_t)blockIdx.x * ld_p;
    float mx, sum;
    row_stats(s, cols, vec_in != 0, alpha, sh, mx, sum, cols);
    const int64_t G = (cols + 31) / 32;
    for (int64_t g = threadIdx.x; g < G; g += kT) {
        float t[32];
        uint32_t w[16];
        load_group(s, g, cols, vec_in != 0, alpha, t, cols);
        normalised_group(t, mx, sum, w);
        store_group(p, g, cols, vec_out != 0, w);
    }
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
    const int whole = cols % 32 == 0;
    const int vec_in = whole && aligned(S, 16) && ld_s % 4 == 0;
    const int vec_out = whole && aligned(P, 16) && ld_p % 8 == 0;
    if (whole && cols / 32 <= softmax::kT)
        softmax_bf16_cached_kernel<<<(unsigned)rows, softmax::kT, 0, static_cast<cudaStream_t>(stream)>>>(
            S, (int)(cols / 32), ld_s, alpha, reinterpret_cast<uint16_t*>(P), ld_p, vec_in, vec_out);
    else
        softmax_bf16_kernel<<<(unsigned)rows, softmax::kT, 0, static_cast<cudaStream_t>(stream)>>>(
            S, cols, ld_s, alpha, reinterpret_cast<uint16_t*>(P), ld_p, vec_in, vec_out);
    return launch_status();
}
