// bf16 -> AMXFP4 direct cast (arXiv 2411.09909, Sections 4.2-4.3; Algorithm 1 applied per sign
// with the FP8 E5M2 shared scale).  HBM-bound: 2 B read + 0.5625 B written per element.
//
// Exactness of the arithmetic (all decisions are bit-identical to exact rational arithmetic):
//   * Side maxima are taken on the bf16 bit patterns as signed 16-bit integers.  Non-negative
//     floats order like their bit patterns, negative ones become non-negative after flipping
//     the sign bit, and the other side is removed by the max with 0.
//   * scale = RNE_E5M2(max / 6) and magnitude = RNE_E2M1(|x| / scale) are evaluated as
//     "multiply by a reciprocal that is slightly too large, then truncate to 12 significant
//     bits".  max and x have 8 significant bits and every rounding midpoint times its divisor
//     has at most 6, so a quotient is either exactly a midpoint (the tie: the product then
//     overshoots by < 2^-18 relative and truncation returns the midpoint itself, which the
//     converter resolves to even) or at least 2^-8 relative away from every midpoint
//     (overshoot + truncation move it by < 2^-11: it stays on its side).
//   * The final roundings are the hardware converts cvt.rn.satfinite.{e5m2x2,e2m1x2}.f32.
#include <cuda_bf16.h>

#include "amx_common.cuh"

namespace amx {
namespace {

constexpr int kThreads = 256;

// 1/6 rounded up a few ulps (0x3E2AAAAB is the nearest float, already above 1/6).
__device__ __forceinline__ float sixth_up() { return __uint_as_float(0x3E2AAAAFu); }

__device__ __forceinline__ float trunc12(float v) {
    return __uint_as_float(__float_as_uint(v) & 0xFFFFF000u);
}

// {hi, lo} -> two E5M2 bytes, hi in bits 15..8.
__device__ __forceinline__ uint32_t cvt_e5m2x2(float hi, float lo) {
    unsigned short d;
    asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(d) : "f"(hi), "f"(lo));
    return d;
}

// Four pairs of quotients -> eight E2M1 nibbles; element i lands in nibble i.
__device__ __forceinline__ uint32_t cvt_e2m1x8(const float (&r)[8]) {
    uint32_t d;
    asm("{\n"
        ".reg .b8 b0, b1, b2, b3;\n"
        "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n"
        "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n"
        "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n"
        "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n"
        "mov.b32 %0, {b0, b1, b2, b3};\n"
        "}"
        : "=r"(d)
        : "f"(r[0]), "f"(r[1]), "f"(r[2]), "f"(r[3]), "f"(r[4]), "f"(r[5]), "f"(r[6]), "f"(r[7]));
    return d;
}

// Reciprocal of an E5M2 value, biased upward by < 2^-18 relative; 0 for a zero scale.
__device__ __forceinline__ float inv_scale_up(float s) {
    float r;
    asm("rcp.approx.f32 %0, %1;" : "=f"(r) : "f"(s));
    r = __uint_as_float(__float_as_uint(r) + 16u);
    return s > 0.0f ? r : 0.0f;
}

// Side maxima of NW bf16x2 words as one word {nmax bits : pmax bits}.  Signed 16-bit max over the
// raw patterns, clamped at 0, is the largest non-negative value; unsigned 16-bit max is the negative
// value of largest magnitude whenever a negative one exists (its sign bit is then flipped away).
template <int NW>
__device__ __forceinline__ uint32_t side_maxima(const uint32_t (&w)[NW]) {
    uint32_t pm = w[0], nm = w[0];
#pragma unroll
    for (int i = 1; i + 1 < NW; i += 2) {
        pm = __vimax3_s16x2(pm, w[i], w[i + 1]);
        nm = __vimax3_u16x2(nm, w[i], w[i + 1]);
    }
    if (NW % 2 == 0) {
        pm = __vmaxs2(pm, w[NW - 1]);
        nm = __vmaxu2(nm, w[NW - 1]);
    }
    nm ^= 0x80008000u;
    pm = __vimax_s16x2_relu(pm, pm);
    nm = __vimax_s16x2_relu(nm, nm);
    return __vmaxs2(__byte_perm(pm, nm, 0x5410), __byte_perm(pm, nm, 0x7632));
}

// The two E5M2 scale bytes of a group from its side maxima {nmax : pmax} (positive side in bits
// 7..0, negative side in bits 15..8), and the two biased reciprocals the elements are multiplied by.
__device__ __forceinline__ uint32_t group_scales(uint32_t c, float& inv_p, float& inv_n) {
    const float pmax = __uint_as_float(c << 16);
    const float nmax = __uint_as_float(c & 0xFFFF0000u);
    const uint32_t sc = cvt_e5m2x2(trunc12(nmax * sixth_up()), trunc12(pmax * sixth_up()));
    inv_p = inv_scale_up(e5m2_to_float(sc & 0xFFu));
    inv_n = inv_scale_up(e5m2_to_float(sc >> 8));
    return sc;
}

// x * (sign(x) ? inv_n : inv_p).  The choice is an integer multiply-add on the reciprocals' bit
// patterns (inv_p + sign * (inv_n - inv_p)): it runs on the FMA pipe, which this kernel leaves
// mostly idle, instead of adding a compare and a select to the saturated integer/logic pipe.
__device__ __forceinline__ float scale_by_side(uint32_t x_bits, uint32_t inv_p, uint32_t inv_diff) {
    uint32_t sel;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(sel) : "r"(x_bits >> 31), "r"(inv_diff), "r"(inv_p));
    return __uint_as_float(x_bits) * __uint_as_float(sel);
}

// 8 consecutive elements (4 bf16x2 words) -> 8 nibbles.
__device__ __forceinline__ uint32_t encode8(const uint32_t* w, float inv_p, float inv_n) {
    const uint32_t ip = __float_as_uint(inv_p), idiff = __float_as_uint(inv_n) - ip;
    float r[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        r[2 * i] = trunc12(scale_by_side(w[i] << 16, ip, idiff));
        r[2 * i + 1] = trunc12(scale_by_side(w[i] & 0xFFFF0000u, ip, idiff));
    }
    return cvt_e2m1x8(r);
}

// Quantizes 8 consecutive elements held as 4 bf16x2 words.  TPG threads (8*TPG = group size) hold
// one group and sit in consecutive lanes.  Returns the 8 nibbles; `sc` receives the scale bytes.
template <int TPG>
__device__ __forceinline__ uint32_t quantize8(const uint4 q, uint32_t& sc) {
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
    uint32_t c = side_maxima<4>(w);
#pragma unroll
    for (int d = 1; d < TPG; d <<= 1) c = __vmaxs2(c, __shfl_xor_sync(0xFFFFFFFFu, c, d));
    float inv_p, inv_n;
    sc = group_scales(c, inv_p, inv_n);
    return encode8(w, inv_p, inv_n);
}

// Groups along the contiguous axis.  Each thread owns EPT = min(gs, 32) consecutive elements
// (EPT/8 16-byte loads, one EPT/2-byte store); a group is TPG = gs / EPT consecutive lanes, so a
// 16- or 32-group needs no shuffle and its scales are computed once.  n_items = rows * K / EPT.
// With PREP (32-groups, contiguous rows) the kernel also writes what the FP4 GEMM's operand preparation
// would otherwise derive in a second pass over the codes: the two sign planes (every nibble in the plane of
// its sign bit, zero in the other) and, per row, the largest exponent key of the row's scales (atomic max).
template <int EPT, int TPG, bool CONTIG, bool PREP = false>
__global__ void __launch_bounds__(kThreads)
quantize_rows_kernel(const uint4* __restrict__ x, int64_t n_items, int64_t items_per_row,
                     int64_t ld_vec, uint4* __restrict__ codes, uint16_t* __restrict__ scales,
                     uint4* __restrict__ pos = nullptr, uint4* __restrict__ neg = nullptr,
                     int* __restrict__ row_kmax = nullptr) {
    constexpr int NV = EPT / 8;
    const int64_t v = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    uint32_t w[NV * 4];
    const bool live = v < n_items;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        uint4 q = make_uint4(0, 0, 0, 0);
        if (live) {
            int64_t off = v * NV + j;
            if (!CONTIG) off = (v / items_per_row) * ld_vec + (v % items_per_row) * NV + j;
            q = __ldg(x + off);
        }
        w[4 * j] = q.x; w[4 * j + 1] = q.y; w[4 * j + 2] = q.z; w[4 * j + 3] = q.w;
    }
    uint32_t c = side_maxima<NV * 4>(w);
#pragma unroll
    for (int d = 1; d < TPG; d <<= 1) c = __vmaxs2(c, __shfl_xor_sync(0xFFFFFFFFu, c, d));
    float inv_p, inv_n;
    const uint32_t sc = group_scales(c, inv_p, inv_n);
    uint32_t nib[NV];
#pragma unroll
    for (int j = 0; j < NV; ++j) nib[j] = encode8(w + 4 * j, inv_p, inv_n);
    if (live) {
        if (NV == 4) codes[v] = make_uint4(nib[0], nib[1], nib[2], nib[NV - 1]);
        else *reinterpret_cast<uint2*>(reinterpret_cast<uint8_t*>(codes) + v * 8) = make_uint2(nib[0], nib[NV - 1]);
        if ((threadIdx.x & (TPG - 1)) == 0) scales[v / TPG] = (uint16_t)sc;
    }
    if (PREP) {
        static_assert(!PREP || (NV == 4 && TPG == 1 && CONTIG), "prepared output: 32-groups of contiguous rows");
        if (live) {
            uint32_t pp[4], nn[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t m = ((nib[j] >> 3) & 0x11111111u) * 15u;   // 0xF on negative nibbles
                nn[j] = nib[j] & m;
                pp[j] = nib[j] & ~m;
            }
            pos[v] = make_uint4(pp[0], pp[1], pp[2], pp[3]);
            neg[v] = make_uint4(nn[0], nn[1], nn[2], nn[3]);
        }
        // row maximum of the scale exponent keys: one atomic per warp when the warp sits inside one row
        const int key = live ? max(scale_key(sc & 0xFFu), scale_key(sc >> 8)) : 0;
        const int64_t row = v / items_per_row;
        const int64_t v_first = v - (threadIdx.x & 31), v_last = min(v_first + 31, n_items - 1);
        if (v_first < n_items) {
            if (v_first / items_per_row == v_last / items_per_row) {
                const int wmax = __reduce_max_sync(0xFFFFFFFFu, key);
                if ((threadIdx.x & 31) == 0 && wmax > 0) atomicMax(row_kmax + row, wmax);
            } else if (live && key > 0) {
                atomicMax(row_kmax + row, key);
            }
        }
    }
}

// Groups DOWN the rows (strided axis): x is [R, C]; output is the canonical layout of x^T.
// A block stages a [64 rows x 64 columns] tile in shared memory and re-reads it column-wise.
constexpr int kTR = 64, kTC = 64;

template <int TPG>
__global__ void __launch_bounds__(kThreads)
quantize_cols_kernel(const __nv_bfloat16* __restrict__ x, int64_t R, int64_t C, int64_t ld,
                     uint32_t* __restrict__ codes, uint16_t* __restrict__ scales, int gs) {
    __shared__ uint16_t tile[kTC][kTR + 2];  // [column][row], padded
    const int64_t r0 = (int64_t)blockIdx.y * kTR, c0 = (int64_t)blockIdx.x * kTC;
    const uint16_t* xs = reinterpret_cast<const uint16_t*>(x);
    for (int i = threadIdx.x; i < kTR * kTC; i += kThreads) {
        const int rr = i / kTC, cc = i % kTC;
        uint16_t v = 0;
        if (r0 + rr < R && c0 + cc < C) v = xs[(r0 + rr) * ld + c0 + cc];
        tile[cc][rr] = v;
    }
    __syncthreads();
    // kTR/8 = 8 threads cover one column's 64 rows; 256 threads -> 32 columns per pass
    for (int pass = 0; pass < kTC / (kThreads / (kTR / 8)); ++pass) {
        const int cc = pass * (kThreads / (kTR / 8)) + threadIdx.x / (kTR / 8);
        const int seg = threadIdx.x % (kTR / 8);
        const uint16_t* t = &tile[cc][seg * 8];
        uint4 q;
        q.x = t[0] | ((uint32_t)t[1] << 16);
        q.y = t[2] | ((uint32_t)t[3] << 16);
        q.z = t[4] | ((uint32_t)t[5] << 16);
        q.w = t[6] | ((uint32_t)t[7] << 16);
        uint32_t sc;
        const uint32_t nib = quantize8<TPG>(q, sc);
        const int64_t col = c0 + cc, row = r0 + seg * 8;
        if (col < C && row < R) {  // R % 8 == 0, so the 8 rows are all valid or all invalid
            codes[(col * R + row) / 8] = nib;
            if ((seg & (TPG - 1)) == 0) scales[(col * R + row) / gs] = (uint16_t)sc;
        }
    }
}

template <int EPT, int TPG>
int launch_rows(const void* x, int64_t rows, int64_t K, int64_t ld, uint8_t* codes,
                uint8_t* scales, cudaStream_t st) {
    const int64_t n_items = rows * (K / EPT);
    const int64_t blocks = (n_items + kThreads - 1) / kThreads;
    if (blocks > 0x7FFFFFFF) return AMX_ERR_SHAPE;
    auto* xv = reinterpret_cast<const uint4*>(x);
    auto* cv = reinterpret_cast<uint4*>(codes);
    auto* sv = reinterpret_cast<uint16_t*>(scales);
    if (ld == K)
        quantize_rows_kernel<EPT, TPG, true><<<(unsigned)blocks, kThreads, 0, st>>>(xv, n_items, K / EPT, ld / 8, cv, sv);
    else
        quantize_rows_kernel<EPT, TPG, false><<<(unsigned)blocks, kThreads, 0, st>>>(xv, n_items, K / EPT, ld / 8, cv, sv);
    return launch_status();
}

}  // namespace

// Cast with fused FP4-operand preparation (gs = 32, contiguous rows): canonical codes and scales plus the
// sign planes and the per-row maximum exponent keys (row_kmax must be zero on entry).
int quantize_rows_prepared(const void* x, int64_t rows, int64_t K, uint8_t* codes, uint8_t* scales, void* pos,
                           void* neg, int* row_kmax, cudaStream_t st) {
    const int64_t n_items = rows * (K / 32);
    const int64_t blocks = (n_items + kThreads - 1) / kThreads;
    if (blocks > 0x7FFFFFFF) return AMX_ERR_SHAPE;
    quantize_rows_kernel<32, 1, true, true><<<(unsigned)blocks, kThreads, 0, st>>>(
        reinterpret_cast<const uint4*>(x), n_items, K / 32, K / 8, reinterpret_cast<uint4*>(codes),
        reinterpret_cast<uint16_t*>(scales), reinterpret_cast<uint4*>(pos), reinterpret_cast<uint4*>(neg), row_kmax);
    return launch_status();
}

namespace {

template <int TPG>
int launch_cols(const void* x, int64_t R, int64_t C, int64_t ld, int gs, uint8_t* codes,
                uint8_t* scales, cudaStream_t st) {
    dim3 grid((unsigned)((C + kTC - 1) / kTC), (unsigned)((R + kTR - 1) / kTR));
    if (grid.y > 65535) return AMX_ERR_SHAPE;
    quantize_cols_kernel<TPG><<<grid, kThreads, 0, st>>>(
        reinterpret_cast<const __nv_bfloat16*>(x), R, C, ld, reinterpret_cast<uint32_t*>(codes),
        reinterpret_cast<uint16_t*>(scales), gs);
    return launch_status();
}

}  // namespace
}  // namespace amx

extern "C" int amx_quantize(const void* x, int64_t rows, int64_t K, int64_t ld_x, int group_size,
                            uint8_t* codes, uint8_t* scales, void* stream) {
    using namespace amx;
    if (!valid_group_size(group_size) || rows < 0 || K <= 0 || K % group_size || K % 8 || ld_x < K)
        return AMX_ERR_SHAPE;
    if (rows == 0) return AMX_OK;
    if (!x || !codes || !scales) return AMX_ERR_NULL;
    if (!aligned(x, 16) || ld_x % 8 || !aligned(codes, group_size == 16 ? 8 : 16) || !aligned(scales, 2)) return AMX_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    switch (group_size) {
        case 16: return launch_rows<16, 1>(x, rows, K, ld_x, codes, scales, st);
        case 32: return launch_rows<32, 1>(x, rows, K, ld_x, codes, scales, st);
        case 64: return launch_rows<32, 2>(x, rows, K, ld_x, codes, scales, st);
        default: return launch_rows<32, 4>(x, rows, K, ld_x, codes, scales, st);
    }
}

extern "C" int amx_quantize_t(const void* x, int64_t R, int64_t C, int64_t ld_x, int group_size,
                              uint8_t* codes, uint8_t* scales, void* stream) {
    using namespace amx;
    if (!valid_group_size(group_size) || R < 0 || C < 0 || R % group_size || ld_x < C) return AMX_ERR_SHAPE;
    if (R == 0 || C == 0) return AMX_OK;
    if (!x || !codes || !scales) return AMX_ERR_NULL;
    if (!aligned(x, 2) || !aligned(codes, 4) || !aligned(scales, 2)) return AMX_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    switch (group_size) {  // a 64-row tile holds whole groups only for gs <= 64
        case 16: return launch_cols<2>(x, R, C, ld_x, group_size, codes, scales, st);
        case 32: return launch_cols<4>(x, R, C, ld_x, group_size, codes, scales, st);
        case 64: return launch_cols<8>(x, R, C, ld_x, group_size, codes, scales, st);
        default: return AMX_ERR_SHAPE;
    }
}
