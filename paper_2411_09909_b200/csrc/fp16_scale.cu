// FP4 elements with binary16 shared scales, one per group or one per sign: the "FP16" row of the paper's ablation
// of the shared-scale encoding (arXiv 2411.09909, appendix "Ablation Study on Shared-Scale Bit-Encoding"), there to
// show how close the 8-bit E5M2 scale comes to a 16-bit one.  The quantizer is that of Sections 4.2-4.3 with every
// "nearest E5M2" replaced by "nearest binary16" (ties to even, subnormals kept, saturating at 65504).  The same
// table has a row for the other FP8 scale type, E4M3 ("1-4-3"): an option of the cast here, stored as the binary16
// pattern of the E4M3 value (every E4M3 value is a binary16 value), so that nothing else changes.
//
// Layout: codes as everywhere ([rows, K/2], element 2j in the low nibble), scales uint16 [rows, K/gs, 2] = binary16
// bit patterns {positive side, negative side} (equal in the symmetric format).
//
// Exactness.  Scale: max / 6 is divided in fp32 (correctly rounded) and converted to binary16 (round to nearest
// even); the double rounding is harmless because max has 8 significant bits: a quotient that is not itself a
// 12-bit number is at least 2^-14 (relative) away from every binary16 rounding boundary.  Element: |x| / scale in
// fp32, then the hardware's nearest-even conversion to E2M1; a boundary of that conversion times the scale has at
// most 14 significant bits, so a quotient that is not exactly on a boundary is at least 2^-14 away from it, and one
// that is comes out of the division exactly.  Decoded values (E2M1 x binary16: 13 significant bits) are exact in
// fp32, not in bf16: dequantization writes fp32 and the product runs on the CUDA cores with fp32 accumulation.
#include <cuda_fp16.h>

#include "cast_math.cuh"
#include "gemm.cuh"

namespace amx {
namespace {

// binary16 pattern of the scale of a side maximum.  E4M3: the nearest FP8 E4M3 value instead (the hardware's
// convert: nearest even, subnormals, saturating at 448), widened exactly to binary16.  The double rounding through
// fp32 is harmless for the same reason as above (an E4M3 boundary has even fewer bits).
template <bool E4M3>
__device__ __forceinline__ uint32_t scale_bits(float side_max) {
    const float q = __fdiv_rn(side_max, 6.0f);
    if (E4M3) {
        unsigned short b;
        uint32_t h2;
        asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(b) : "f"(0.0f), "f"(q));
        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(b));
        return h2 & 0xFFFFu;
    }
    return (uint32_t)__half_as_ushort(__float2half_rn(fminf(q, 65504.0f)));
}
__device__ __forceinline__ float half_bits_to_float(uint32_t h) { return __half2float(__ushort_as_half((unsigned short)h)); }

// One thread per group: a sweep for the side maxima, a second one (the group is in the L1 by then) for the codes.
template <bool ASYM, bool E4M3>
__global__ void __launch_bounds__(256) quantize_f16s_kernel(const uint16_t* __restrict__ x, int64_t n_groups, int64_t G,
                                                            int64_t ld_x, int gs, uint32_t* __restrict__ codes,
                                                            uint32_t* __restrict__ scales) {
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= n_groups) return;
    const int64_t row = idx / G, g = idx % G;
    const uint4* xp = reinterpret_cast<const uint4*>(x + row * ld_x + g * gs);
    float pmax = 0.f, nmax = 0.f;
    for (int c = 0; c < gs / 8; ++c) {
        const uint4 q = __ldg(xp + c);
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t b = (i & 1) ? w[i >> 1] >> 16 : w[i >> 1] & 0xFFFFu;
            const float a = __uint_as_float((b & 0x7FFFu) << 16);
            if (b >> 15) nmax = fmaxf(nmax, a);
            else pmax = fmaxf(pmax, a);
        }
    }
    if (!ASYM) pmax = nmax = fmaxf(pmax, nmax);
    const uint32_t hp = scale_bits<E4M3>(pmax), hn = scale_bits<E4M3>(nmax);
    const float sp = half_bits_to_float(hp), sn = half_bits_to_float(hn);
    uint32_t* out = codes + (row * G * gs + g * gs) / 8;
    for (int c = 0; c < gs / 8; ++c) {
        const uint4 q = __ldg(xp + c);
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
        uint32_t qb[8], signs = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t b = (i & 1) ? w[i >> 1] >> 16 : w[i >> 1] & 0xFFFFu;
            const float a = __uint_as_float((b & 0x7FFFu) << 16), s = (b >> 15) ? sn : sp;
            qb[i] = s > 0.f ? __float_as_uint(__fdiv_rn(a, s)) : 0u;     // zero scale: zero magnitude
            signs |= (b >> 15) << (4 * i + 3);
        }
        out[c] = cast::cvt_e2m1x8(cast::pack_f32x2(qb[0], qb[1]), cast::pack_f32x2(qb[2], qb[3]),
                                  cast::pack_f32x2(qb[4], qb[5]), cast::pack_f32x2(qb[6], qb[7])) | signs;
    }
    scales[idx] = hp | (hn << 16);
}

// Eq. 1 with binary16 scales; 8 elements per thread, fp32 out.
__global__ void __launch_bounds__(256) dequantize_f16s_kernel(const uint32_t* __restrict__ codes,
                                                              const uint32_t* __restrict__ scales, int64_t n_vec,
                                                              int64_t vec_per_row, int vec_per_group, int64_t ld_out,
                                                              float* __restrict__ out) {
    const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= n_vec) return;
    const uint32_t nib = codes[v], sc = scales[v / vec_per_group];
    const float sp = half_bits_to_float(sc & 0xFFFFu), sn = half_bits_to_float(sc >> 16);
    float f[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t c = (nib >> (4 * i)) & 15u;
        const float mag = e2m1_mag_to_float(c & 7u);
        f[i] = (c & 8u) ? -(mag * sn) : mag * sp;
    }
    float4* o = reinterpret_cast<float4*>(out + (v / vec_per_row) * ld_out + (v % vec_per_row) * 8);
    o[0] = make_float4(f[0], f[1], f[2], f[3]);
    o[1] = make_float4(f[4], f[5], f[6], f[7]);
}

}  // namespace
}  // namespace amx

using namespace amx;

extern "C" int amx_quantize_f16s(const void* x, int64_t rows, int64_t K, int64_t ld_x, int group_size, uint32_t flags,
                                 uint8_t* codes, uint16_t* scales, void* stream) {
    if (!fixed_group_size(group_size) || rows < 0 || K <= 0 || K % group_size || ld_x < K) return AMX_ERR_SHAPE;
    if (flags & ~(AMX_F16S_ASYMMETRIC | AMX_F16S_SCALE_E4M3)) return AMX_ERR_FLAGS;
    if (rows == 0) return AMX_OK;
    if (!x || !codes || !scales) return AMX_ERR_NULL;
    if (!aligned(x, 16) || ld_x % 8 || !aligned(codes, 4) || !aligned(scales, 4)) return AMX_ERR_ALIGN;
    const int64_t G = K / group_size, n_groups = rows * G, blocks = (n_groups + 255) / 256;
    if (blocks > 0x7FFFFFFF) return AMX_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    auto* xv = static_cast<const uint16_t*>(x);
    auto* cv = reinterpret_cast<uint32_t*>(codes);
    auto* sv = reinterpret_cast<uint32_t*>(scales);
    const bool asym = flags & AMX_F16S_ASYMMETRIC, e4m3 = flags & AMX_F16S_SCALE_E4M3;
    auto* kernel = asym ? (e4m3 ? quantize_f16s_kernel<true, true> : quantize_f16s_kernel<true, false>)
                        : (e4m3 ? quantize_f16s_kernel<false, true> : quantize_f16s_kernel<false, false>);
    kernel<<<(unsigned)blocks, 256, 0, st>>>(xv, n_groups, G, ld_x, group_size, cv, sv);
    return launch_status();
}

extern "C" int amx_dequantize_f16s(const uint8_t* codes, const uint16_t* scales, int64_t rows, int64_t K, int group_size,
                                   float* out, int64_t ld_out, void* stream) {
    if (!fixed_group_size(group_size) || rows < 0 || K <= 0 || K % group_size || ld_out < K) return AMX_ERR_SHAPE;
    if (rows == 0) return AMX_OK;
    if (!codes || !scales || !out) return AMX_ERR_NULL;
    if (!aligned(codes, 4) || !aligned(scales, 4) || !aligned(out, 16) || ld_out % 4) return AMX_ERR_ALIGN;
    const int64_t n_vec = rows * (K / 8), blocks = (n_vec + 255) / 256;
    if (blocks > 0x7FFFFFFF) return AMX_ERR_SHAPE;
    dequantize_f16s_kernel<<<(unsigned)blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        reinterpret_cast<const uint32_t*>(codes), reinterpret_cast<const uint32_t*>(scales), n_vec, K / 8, group_size / 8,
        ld_out, out);
    return launch_status();
}

extern "C" int amx_gemm_f16s(const uint8_t* a_codes, const uint16_t* a_scales, const uint8_t* w_codes,
                             const uint16_t* w_scales, int64_t M, int64_t N, int64_t K, int group_size, float* C,
                             int64_t ld_c, void* stream) {
    if (!fixed_group_size(group_size) || M < 0 || N < 0 || K <= 0 || K % group_size || ld_c < N) return AMX_ERR_SHAPE;
    if (M == 0 || N == 0) return AMX_OK;
    if (!a_codes || !a_scales || !w_codes || !w_scales || !C) return AMX_ERR_NULL;
    if (!aligned(a_codes, 4) || !aligned(w_codes, 4) || !aligned(a_scales, 2) || !aligned(w_scales, 2) || !aligned(C, 4))
        return AMX_ERR_ALIGN;
    return gemm_simt_f16s(a_codes, a_scales, w_codes, w_scales, M, N, K, group_size, C, ld_c,
                          static_cast<cudaStream_t>(stream));
}
