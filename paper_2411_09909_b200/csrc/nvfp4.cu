// NVFP4 and its asymmetric variant ANVFP4: the format arXiv 2411.09909 compares AMXFP4 with in Section 5 (its table
// of NVFP4 / ANVFP4 results) - FP4 E2M1 elements in groups of 16, one FP8 E4M3 scale per group (ANVFP4: one per sign,
// as in AMXFP4) and one fp32 scale for the whole tensor.  Group size 16 and the E4M3 scale type are what the
// block-scaled FP4 MMA takes natively (scale_vec::4X, UE4M3), so the prepared operand carries the scale bytes as
// they are: no per-row offset, nothing is flushed, and symmetric NVFP4 needs ONE product per tile pair where
// AMXFP4's E5M2 scales and sign split need four.
//
// The paper names the parts of the format but no arithmetic.  The reading implemented here (the same as the CPU
// reference's, operation by operation, every operation an IEEE fp32 one rounded to nearest even, so that both take
// every rounding decision identically):
//     t  = max|x| / 2688 (= 448 * 6; 1 for an all-zero tensor),  rt = 1 / t
//     g  = (max_side * fl(1/6)) * rt            -> E4M3 byte (nearest even, saturating at 448, subnormals)
//     d  = E4M3(byte) * t,  rd = 1 / d (0 for a zero byte)
//     q  = x * rd                               -> E2M1 code (nearest even, clamped at 6), sign bit = sign of x
// decoded value = (-1)^s * E2M1 * E4M3(scale_s) * t.
// Two launches: the tensor maximum (a read of the whole tensor), then the cast.
#include <cuda_bf16.h>

#include "cast_math.cuh"
#include "fp4_operand.cuh"
#include "gemm.cuh"

namespace amx {
namespace {

using namespace cast;
using namespace fp4;

// max |x| over the tensor as a bf16 bit pattern (non-negative floats order like their patterns): atomicMax into
// bits[1], which the caller zeroed.
__global__ void __launch_bounds__(256)
absmax_kernel(const uint4* __restrict__ x, int64_t n_vec, int64_t vec_per_row, int64_t ld_vec, unsigned* __restrict__ bits) {
    uint32_t m = 0;
    for (int64_t v = (int64_t)blockIdx.x * 256 + threadIdx.x; v < n_vec; v += (int64_t)gridDim.x * 256) {
        const uint4 q = __ldg(x + (v / vec_per_row) * ld_vec + v % vec_per_row);
        m = __vmaxu2(m, __vmaxu2(__vmaxu2(q.x & 0x7FFF7FFFu, q.y & 0x7FFF7FFFu), __vmaxu2(q.z & 0x7FFF7FFFu, q.w & 0x7FFF7FFFu)));
    }
    m = max(m & 0xFFFFu, m >> 16);
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    __shared__ uint32_t red[8];
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < 8; ++i) m = max(m, red[i]);
        if (m) atomicMax(bits + 1, m << 16);          // as an fp32 pattern
    }
}

// two fp32 values -> two E4M3 bytes (hi in bits 15..8)
__device__ __forceinline__ uint32_t cvt_e4m3x2(float hi, float lo) {
    unsigned short d;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(d) : "f"(hi), "f"(lo));
    return d;
}
__device__ __forceinline__ float e4m3_to_float(uint32_t byte) {
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((unsigned short)byte));
    float f;
    asm("cvt.f32.f16 %0, %1;" : "=f"(f) : "h"((unsigned short)(h2 & 0xFFFFu)));
    return f;
}

// One thread per 64 consecutive elements of a row (four groups of 16): canonical codes (32 bytes) and scale bytes
// (8 bytes) and, when the prepared form is asked for, the two sign planes (NVFP4: its signed codes as one plane),
// the four scale bytes per plane as one word of the tensor cores' scale-factor layout, and the row word.
template <bool ASYM>
__global__ void __launch_bounds__(256)
cast_nv_kernel(const uint4* __restrict__ x, int64_t rows, int chunks_per_row, int64_t ld_vec, float* __restrict__ tensor_scale,
               uint4* __restrict__ codes, uint2* __restrict__ scales, uint4* __restrict__ pos, uint4* __restrict__ neg,
               uint8_t* __restrict__ sf_pos, uint8_t* __restrict__ sf_neg, int* __restrict__ row_exp, int nk64,
               float* __restrict__ prepared_scale) {
    const int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
    const float amax = tensor_scale[1];
    const float t = amax > 0.0f ? __fdiv_rn(amax, 2688.0f) : 1.0f;
    if (idx == 0) {
        tensor_scale[0] = t;
        if (prepared_scale) *prepared_scale = t;
    }
    if (idx >= rows * chunks_per_row) return;
    const float rt = __fdiv_rn(1.0f, t), sixth = __fdiv_rn(1.0f, 6.0f);
    const int64_t row = idx / chunks_per_row;
    const int c = (int)(idx - row * chunks_per_row);
    const uint4* src = x + row * ld_vec + (int64_t)c * 8;
    uint32_t w[32];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint4 q = __ldg(src + j);
        w[4 * j] = q.x; w[4 * j + 1] = q.y; w[4 * j + 2] = q.z; w[4 * j + 3] = q.w;
    }
    uint32_t nib[8], pp[8], nn[8], sc8[2] = {0, 0}, sfp = 0, sfn = 0;
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        uint32_t wg[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) wg[i] = w[8 * g + i];
        const uint32_t mx = side_maxima<8>(wg);                       // {nmax : pmax} bf16 patterns
        float pmax = __uint_as_float(mx << 16), nmax = __uint_as_float(mx & 0xFFFF0000u);
        if (!ASYM) pmax = nmax = fmaxf(pmax, nmax);
        const uint32_t by = cvt_e4m3x2(__fmul_rn(__fmul_rn(nmax, sixth), rt), __fmul_rn(__fmul_rn(pmax, sixth), rt));
        const uint32_t bp = by & 0xFFu, bn = by >> 8;
        const float rdp = bp ? __fdiv_rn(1.0f, __fmul_rn(e4m3_to_float(bp), t)) : 0.0f;
        const float rdn = bn ? __fdiv_rn(1.0f, __fmul_rn(e4m3_to_float(bn), t)) : 0.0f;
        const uint64_t ip2 = pack_f32x2(__float_as_uint(rdp), __float_as_uint(rdp)), in2 = pack_f32x2(__float_as_uint(rdn), __float_as_uint(rdn));
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t cp, cn;
            encode8_both(wg + 4 * h, ip2, in2, cp, cn);
            const uint32_t m = negative_nibbles(cp);
            const uint32_t code = (cp & ~m) | (cn & m);
            nib[2 * g + h] = code;
            pp[2 * g + h] = ASYM ? (cp & ~m) : code;                  // NVFP4: no split, the signed codes are the one plane
            nn[2 * g + h] = ASYM ? (cn & m) : 0u;
        }
        sc8[g >> 1] |= (bp | (bn << 8)) << (16 * (g & 1));
        sfp |= bp << (8 * g);
        sfn |= (ASYM ? bn : 0u) << (8 * g);
    }
    const int64_t v = idx * 2;                                        // 16-byte pieces of codes
    if (codes) {
        codes[v] = make_uint4(nib[0], nib[1], nib[2], nib[3]);
        codes[v + 1] = make_uint4(nib[4], nib[5], nib[6], nib[7]);
    }
    if (scales) scales[idx] = make_uint2(sc8[0], sc8[1]);
    if (pos) {
        pos[v] = make_uint4(pp[0], pp[1], pp[2], pp[3]);
        pos[v + 1] = make_uint4(pp[4], pp[5], pp[6], pp[7]);
        neg[v] = make_uint4(nn[0], nn[1], nn[2], nn[3]);
        neg[v + 1] = make_uint4(nn[4], nn[5], nn[6], nn[7]);
        const int64_t off = sf_row_offset(row, nk64) + (int64_t)c * kSfChunkBytes;
        *reinterpret_cast<uint32_t*>(sf_pos + off) = sfp;
        *reinterpret_cast<uint32_t*>(sf_neg + off) = sfn;
        // row word: no offset (exponent key 25 stands for 2^0); without a split only the first plane is in use
        if (c == 0) row_exp[row] = row_word(25, ASYM ? (kRowHasPos | kRowHasNeg) : kRowHasPos);
    }
}

template <bool F32>
__global__ void __launch_bounds__(256)
dequantize_nv_kernel(const uint32_t* __restrict__ codes, const uint16_t* __restrict__ scales, const float* __restrict__ tensor_scale,
                     int64_t n_vec, int64_t vec_per_row, int64_t ld_out, void* __restrict__ out) {
    const int64_t v = (int64_t)blockIdx.x * 256 + threadIdx.x;       // 8 elements per thread, half a group
    if (v >= n_vec) return;
    const uint32_t nib = codes[v], sc = scales[v >> 1];
    const float t = tensor_scale[0], sp = e4m3_to_float(sc & 0xFFu), sn = e4m3_to_float(sc >> 8);
    float f[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t c = (nib >> (4 * i)) & 15u;
        const float mag = e2m1_mag_to_float(c & 7u);
        f[i] = __fmul_rn((c & 8u) ? -(mag * sn) : mag * sp, t);      // the first product is exact, one rounding
    }
    const int64_t row = v / vec_per_row, col = (v % vec_per_row) * 8;
    if (F32) {
        float4* o = reinterpret_cast<float4*>(reinterpret_cast<float*>(out) + row * ld_out + col);
        o[0] = make_float4(f[0], f[1], f[2], f[3]);
        o[1] = make_float4(f[4], f[5], f[6], f[7]);
    } else {
        uint4 pk;
        __nv_bfloat162 b;
        b = __floats2bfloat162_rn(f[0], f[1]); pk.x = *reinterpret_cast<uint32_t*>(&b);
        b = __floats2bfloat162_rn(f[2], f[3]); pk.y = *reinterpret_cast<uint32_t*>(&b);
        b = __floats2bfloat162_rn(f[4], f[5]); pk.z = *reinterpret_cast<uint32_t*>(&b);
        b = __floats2bfloat162_rn(f[6], f[7]); pk.w = *reinterpret_cast<uint32_t*>(&b);
        *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(out) + row * ld_out + col) = pk;
    }
}

constexpr size_t kTrailer = 256;      // behind the prepared operand: its tensor scale (one float)

}  // namespace
}  // namespace amx

using namespace amx;

extern "C" size_t amx_nvfp4_prepared_bytes(int64_t rows, int64_t K, int is_weight) {
    if (rows <= 0 || K <= 0 || K % 64) return 0;
    return fp4::operand_layout(rows, K, is_weight ? 256 : 128).total + kTrailer;
}

extern "C" int amx_quantize_nvfp4(const void* x, int64_t rows, int64_t K, int64_t ld_x, uint32_t flags, uint8_t* codes,
                                  uint8_t* scales, float* tensor_scale, int is_weight, void* prepared, size_t prepared_bytes,
                                  void* stream) {
    if (flags & ~AMX_NV_ASYMMETRIC) return AMX_ERR_FLAGS;
    if (rows <= 0 || K <= 0 || K % 64 || ld_x < K || rows * (K / 64) > 0x7FFFFFFFll * 256) return AMX_ERR_SHAPE;
    if (!x || !tensor_scale) return AMX_ERR_NULL;
    if (prepared && prepared_bytes < amx_nvfp4_prepared_bytes(rows, K, is_weight)) return AMX_ERR_WORKSPACE;
    if (!aligned(x, 16) || ld_x % 8 || !aligned(codes, 16) || !aligned(scales, 8) || !aligned(tensor_scale, 8) ||
        !aligned(prepared, 256))
        return AMX_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const fp4::OperandLayout o = fp4::operand_layout(rows, K, is_weight ? 256 : 128);
    uint8_t* base = static_cast<uint8_t*>(prepared);
    if (cudaMemsetAsync(tensor_scale, 0, 8, st) != cudaSuccess) return AMX_ERR_CUDA;
    // padding rows and padding chunks of the scale factors are zero (both planes)
    if (prepared && cudaMemsetAsync(base + 2 * o.plane, 0, 2 * o.sf, st) != cudaSuccess) return AMX_ERR_CUDA;
    const int64_t n_vec = rows * (K / 8);
    int64_t blocks = (n_vec + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    absmax_kernel<<<(unsigned)blocks, 256, 0, st>>>(static_cast<const uint4*>(x), n_vec, K / 8, ld_x / 8,
                                                    reinterpret_cast<unsigned*>(tensor_scale));
    int rc = launch_status();
    if (rc != AMX_OK) return rc;
    const int64_t items = rows * (K / 64);
    auto* kernel = (flags & AMX_NV_ASYMMETRIC) ? cast_nv_kernel<true> : cast_nv_kernel<false>;
    kernel<<<(unsigned)((items + 255) / 256), 256, 0, st>>>(
        static_cast<const uint4*>(x), rows, (int)(K / 64), ld_x / 8, tensor_scale, reinterpret_cast<uint4*>(codes),
        reinterpret_cast<uint2*>(scales), reinterpret_cast<uint4*>(base), prepared ? reinterpret_cast<uint4*>(base + o.plane) : nullptr,
        prepared ? base + 2 * o.plane : nullptr, prepared ? base + 2 * o.plane + o.sf : nullptr,
        prepared ? reinterpret_cast<int*>(base + 2 * o.plane + 2 * o.sf) : nullptr, o.nk64,
        prepared ? reinterpret_cast<float*>(base + o.total) : nullptr);
    return launch_status();
}

extern "C" int amx_dequantize_nvfp4(const uint8_t* codes, const uint8_t* scales, const float* tensor_scale, int64_t rows,
                                    int64_t K, uint32_t flags, void* out, int64_t ld_out, void* stream) {
    if (rows < 0 || K <= 0 || K % 16 || ld_out < K) return AMX_ERR_SHAPE;
    if (flags & ~AMX_OUT_F32) return AMX_ERR_FLAGS;
    if (rows == 0) return AMX_OK;
    if (!codes || !scales || !tensor_scale || !out) return AMX_ERR_NULL;
    if (!aligned(codes, 4) || !aligned(scales, 2) || !aligned(tensor_scale, 4) || !aligned(out, 16) || ld_out % 8) return AMX_ERR_ALIGN;
    const int64_t n_vec = rows * (K / 8), blocks = (n_vec + 255) / 256;
    if (blocks > 0x7FFFFFFF) return AMX_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    auto* cv = reinterpret_cast<const uint32_t*>(codes);
    auto* sv = reinterpret_cast<const uint16_t*>(scales);
    if (flags & AMX_OUT_F32) dequantize_nv_kernel<true><<<(unsigned)blocks, 256, 0, st>>>(cv, sv, tensor_scale, n_vec, K / 8, ld_out, out);
    else dequantize_nv_kernel<false><<<(unsigned)blocks, 256, 0, st>>>(cv, sv, tensor_scale, n_vec, K / 8, ld_out, out);
    return launch_status();
}

namespace {
int gemm_nvfp4(const void* a_prepared, const void* w_prepared, int64_t M, int64_t N, int64_t K, float* C, int64_t ld_c,
               void* workspace, size_t workspace_bytes, void* stream, bool one_plane) {
    if (M <= 0 || N <= 0 || K <= 0 || K % 64 || ld_c < N || !gemm_fp4_supported(M, N, K, 32)) return AMX_ERR_SHAPE;
    if (!a_prepared || !w_prepared || !C) return AMX_ERR_NULL;
    if (!workspace || workspace_bytes < 256) return AMX_ERR_WORKSPACE;
    if (!aligned(a_prepared, 256) || !aligned(w_prepared, 256) || !aligned(workspace, 256) || !aligned(C, 4)) return AMX_ERR_ALIGN;
    const float* sa = reinterpret_cast<const float*>(static_cast<const uint8_t*>(a_prepared) + fp4::operand_layout(M, K, 128).total);
    const float* sw = reinterpret_cast<const float*>(static_cast<const uint8_t*>(w_prepared) + fp4::operand_layout(N, K, 256).total);
    return gemm_fp4_prepared_at({a_prepared, M, M, 0}, {w_prepared, N, N, 0}, M, N, K, C, ld_c, workspace,
                                static_cast<cudaStream_t>(stream), 256, nullptr, sa, sw, one_plane);
}
}  // namespace

extern "C" int amx_gemm_nvfp4(const void* a_prepared, const void* w_prepared, int64_t M, int64_t N, int64_t K, float* C,
                              int64_t ld_c, void* workspace, size_t workspace_bytes, void* stream) {
    return gemm_nvfp4(a_prepared, w_prepared, M, N, K, C, ld_c, workspace, workspace_bytes, stream, false);
}
extern "C" int amx_gemm_nvfp4_sym(const void* a_prepared, const void* w_prepared, int64_t M, int64_t N, int64_t K, float* C,
                                  int64_t ld_c, void* workspace, size_t workspace_bytes, void* stream) {
    return gemm_nvfp4(a_prepared, w_prepared, M, N, K, C, ld_c, workspace, workspace_bytes, stream, true);
}
