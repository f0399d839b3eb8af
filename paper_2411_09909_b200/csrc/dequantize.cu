// AMXFP4 -> bf16 / fp32 (Eq. 1 of arXiv 2411.09909): value = (-1)^s * E2M1 * scale_s.
// The product has at most 5 significant bits, so the fp32 multiply and the bf16 store are exact.
#include <cuda_bf16.h>

#include "amx_common.cuh"

namespace amx {
namespace {

template <bool F32>
__global__ void __launch_bounds__(256)
dequantize_kernel(const uint32_t* __restrict__ codes, const uint16_t* __restrict__ scales,
                  int64_t n_vec, int64_t vec_per_row, int vec_per_group, int64_t ld_out,
                  void* __restrict__ out) {
    const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;  // 8 elements per thread
    if (v >= n_vec) return;
    const uint32_t nib = codes[v];
    const uint32_t sc = scales[v / vec_per_group];
    const float sp = e5m2_to_float(sc & 0xFFu), sn = e5m2_to_float(sc >> 8);
    float f[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t c = (nib >> (4 * i)) & 15u;
        const float mag = e2m1_mag_to_float(c & 7u);
        f[i] = (c & 8u) ? -(mag * sn) : mag * sp;
    }
    const int64_t row = v / vec_per_row, col = (v % vec_per_row) * 8;
    if (F32) {
        float4* o = reinterpret_cast<float4*>(reinterpret_cast<float*>(out) + row * ld_out + col);
        o[0] = make_float4(f[0], f[1], f[2], f[3]);
        o[1] = make_float4(f[4], f[5], f[6], f[7]);
    } else {
        uint4 p;
        __nv_bfloat162 t;
        t = __floats2bfloat162_rn(f[0], f[1]); p.x = *reinterpret_cast<uint32_t*>(&t);
        t = __floats2bfloat162_rn(f[2], f[3]); p.y = *reinterpret_cast<uint32_t*>(&t);
        t = __floats2bfloat162_rn(f[4], f[5]); p.z = *reinterpret_cast<uint32_t*>(&t);
        t = __floats2bfloat162_rn(f[6], f[7]); p.w = *reinterpret_cast<uint32_t*>(&t);
        *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(out) + row * ld_out + col) = p;
    }
}

}  // namespace
}  // namespace amx

extern "C" int amx_dequantize(const uint8_t* codes, const uint8_t* scales, int64_t rows, int64_t K,
                              int group_size, uint32_t flags, void* out, int64_t ld_out, void* stream) {
    using namespace amx;
    if (!valid_group_size(group_size, K) || rows < 0 || K <= 0 || K % group_size || K % 8 || ld_out < K)
        return AMX_ERR_SHAPE;
    if (flags & ~AMX_OUT_F32) return AMX_ERR_FLAGS;
    if (rows == 0) return AMX_OK;
    if (!codes || !scales || !out) return AMX_ERR_NULL;
    if (!aligned(codes, 4) || !aligned(scales, 2) || !aligned(out, 16) || ld_out % 8) return AMX_ERR_ALIGN;
    const int64_t n_vec = rows * (K / 8);
    const int64_t blocks = (n_vec + 255) / 256;
    if (blocks > 0x7FFFFFFF) return AMX_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    auto* cv = reinterpret_cast<const uint32_t*>(codes);
    auto* sv = reinterpret_cast<const uint16_t*>(scales);
    if (flags & AMX_OUT_F32)
        dequantize_kernel<true><<<(unsigned)blocks, 256, 0, st>>>(cv, sv, n_vec, K / 8, group_size / 8, ld_out, out);
    else
        dequantize_kernel<false><<<(unsigned)blocks, 256, 0, st>>>(cv, sv, n_vec, K / 8, group_size / 8, ld_out, out);
    return launch_status();
}
