// Arithmetic of the bf16 -> AMXFP4 direct cast for one group (arXiv 2411.09909, Section 4.2; Algorithm 1
// applied per sign with the FP8 E5M2 shared scale), shared by the cast kernels and by the GEMM whose
// producers cast the activation tile themselves.
//
// Exactness (all decisions are bit-identical to exact rational arithmetic):
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
#pragma once
#include "amx_common.cuh"

namespace amx {
namespace cast {

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

// E5M2 byte of the power-of-two scale of Algorithm 1 for a side (or group) maximum given as a non-negative bf16
// pattern: X = 2^(floor(log2 max) - 2), from the exponent field E of the pattern: X's E5M2 exponent field is
// E - 127 - 2 + 15 = E - 114; fields 0 and -1 are the subnormals 2^-15 (byte 2) and 2^-16 (byte 1), smaller ones
// store a zero scale, larger than 30 store 2^15.  ROUND: the exponent is rounded instead of floored (appendix on
// floor vs. round), i.e. one more when max >= sqrt(2) x its power of two: (128 + m)^2 >= 2 x 128^2 for the 7
// mantissa bits m, which is m >= 54.
template <bool ROUND>
__device__ __forceinline__ uint32_t pot_scale_byte(uint32_t bits) {
    const int e5 = (int)(bits >> 7) - 114 + ((ROUND && (bits & 0x7Fu) >= 54u) ? 1 : 0);
    return e5 > 30 ? 0x78u : e5 >= 1 ? (uint32_t)e5 << 2 : e5 == 0 ? 2u : e5 == -1 ? 1u : 0u;
}

// Whether a format stores one shared scale per group (in both bytes) or one per sign.
__host__ __device__ constexpr bool format_is_symmetric(int fmt) { return fmt == 1 || fmt == 2 || fmt == 4; }

// Scale bytes and reciprocals for the comparison formats (FMT: AMX_FMT_*):
//   SYM_FP8 (1)          the FP8 scale of the larger side maximum, used by both sides;
//   MXFP4 (2)            Algorithm 1's power-of-two floor scale of the group maximum;
//   AMXFP4_POT (3)       the same per sign;
//   MXFP4_POT_ROUND (4), AMXFP4_POT_ROUND (5)   exponent rounded instead of floored, per group / per sign.
template <int FMT>
__device__ __forceinline__ uint32_t group_scales_fmt(uint32_t c, float& inv_p, float& inv_n) {
    if (FMT == 0) return group_scales(c, inv_p, inv_n);
    if (FMT == 3 || FMT == 5) {
        const uint32_t bp = pot_scale_byte<FMT == 5>(c & 0xFFFFu), bn = pot_scale_byte<FMT == 5>(c >> 16);
        inv_p = inv_scale_up(e5m2_to_float(bp));
        inv_n = inv_scale_up(e5m2_to_float(bn));
        return bp | (bn << 8);
    }
    const uint32_t amax = max(c & 0xFFFFu, c >> 16);              // both halves are non-negative bf16 patterns
    uint32_t b;
    if (FMT == 1) b = cvt_e5m2x2(0.0f, trunc12(__uint_as_float(amax << 16) * sixth_up())) & 0xFFu;
    else b = pot_scale_byte<FMT == 4>(amax);
    inv_p = inv_n = inv_scale_up(e5m2_to_float(b));
    return b | (b << 8);
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

// One group of an FP4-GEMM operand from its 16 bf16x2 words: canonical codes and scale bytes at group index v,
// and the sign planes that are asked for (pos / neg may be nullptr).  Returns the scale bytes {neg : pos}.
// With a symmetric format (FMT != 0) the operand needs no split: the signed codes go to the "positive" plane
// as they are, the other plane is zero, and the returned bytes name the one scale as the positive side's only.
template <int FMT = 0>
__device__ __forceinline__ uint32_t emit_group(const uint32_t (&w)[16], int64_t v, uint4* __restrict__ codes,
                                               uint16_t* __restrict__ scales, uint4* __restrict__ pos,
                                               uint4* __restrict__ neg) {
    float inv_p, inv_n;
    const uint32_t sc = group_scales_fmt<FMT>(side_maxima<16>(w), inv_p, inv_n);
    uint32_t nib[4], pp[4], nn[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        nib[j] = encode8(w + 4 * j, inv_p, inv_n);
        const uint32_t m = FMT ? 0u : ((nib[j] >> 3) & 0x11111111u) * 15u;   // 0xF on negative nibbles
        nn[j] = nib[j] & m;
        pp[j] = nib[j] & ~m;
    }
    codes[v] = make_uint4(nib[0], nib[1], nib[2], nib[3]);
    if (pos) pos[v] = make_uint4(pp[0], pp[1], pp[2], pp[3]);
    if (neg) neg[v] = make_uint4(nn[0], nn[1], nn[2], nn[3]);
    scales[v] = (uint16_t)sc;
    return FMT ? (sc & 0xFFu) : sc;
}

// The same for a group without negative elements (a softmax output) when only the FP4 GEMM's operand is wanted:
// its positive sign plane is its code word, the negative plane and scale are zero.  Same arithmetic as above,
// minus everything the negative side needs.  Stores the plane at group index v (and, when asked, the same word as
// the group's canonical codes: without a set sign bit the two are equal), returns the positive scale byte.
__device__ __forceinline__ uint32_t emit_nonneg_plane(const uint32_t (&w)[16], int64_t v, uint4* __restrict__ plane,
                                                      uint4* __restrict__ codes = nullptr) {
    uint32_t pm = w[0];
#pragma unroll
    for (int i = 1; i + 1 < 16; i += 2) pm = __vimax3_s16x2(pm, w[i], w[i + 1]);
    pm = __vmaxs2(pm, w[15]);
    pm = __vmaxs2(pm, pm >> 16) & 0xFFFFu;                       // the group maximum's bf16 bits
    const uint32_t sc = cvt_e5m2x2(0.0f, trunc12(__uint_as_float(pm << 16) * sixth_up())) & 0xFFu;
    const float inv = inv_scale_up(e5m2_to_float(sc));
    uint32_t nib[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        float r[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            r[2 * i] = trunc12(__uint_as_float(w[4 * j + i] << 16) * inv);
            r[2 * i + 1] = trunc12(__uint_as_float(w[4 * j + i] & 0xFFFF0000u) * inv);
        }
        nib[j] = cvt_e2m1x8(r);
    }
    plane[v] = make_uint4(nib[0], nib[1], nib[2], nib[3]);
    if (codes) codes[v] = make_uint4(nib[0], nib[1], nib[2], nib[3]);
    return sc;
}

}  // namespace cast
}  // namespace amx
