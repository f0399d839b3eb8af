// Arithmetic of the bf16 -> AMXFP4 direct cast for one group (arXiv 2411.09909, Section 4.2; Algorithm 1
// applied per sign with the FP8 E5M2 shared scale), shared by the cast kernels and by the GEMM whose
// producers cast the activation tile themselves.
//
// Exactness (all decisions are bit-identical to exact rational arithmetic):
//   * Side maxima are taken on the bf16 bit patterns as signed 16-bit integers.  Non-negative
//     floats order like their bit patterns, negative ones become non-negative after flipping
//     the sign bit, and the other side is removed by the max with 0.
//   * max and x have 8 significant bits and every rounding midpoint times its divisor has at most
//     6, so a quotient is either exactly a midpoint (a tie, which the converter must see as the
//     midpoint itself to resolve it to even) or at least 2^-8 relative away from every midpoint
//     (any evaluation with a relative error far below that stays on the right side).
//   * scale = RNE_E5M2(max / 6): multiply by a reciprocal of 6 that is slightly too large, then
//     truncate to 12 significant bits - at a tie the product overshoots by < 2^-18 relative and
//     truncation returns the midpoint itself.
//   * magnitude = RNE_E2M1(|x| / scale): one fp32 multiply by the correctly rounded reciprocal of
//     the scale's significand (1, 1.25, 1.5 or 1.75) times the exact power of two.  For these four
//     reciprocals the rounded product IS the midpoint at every tie (checked for every bf16 value
//     on the host in IEEE arithmetic, and on the device by the exhaustive parity sweep), so no
//     truncation is needed; away from ties the error is < 2^-23.
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

// Reciprocal of the value of an E5M2 scale byte: the fp32 nearest to 1 / significand (significand 1, 1.25, 1.5,
// 1.75: the byte's two low bits) times the exact power of two; 0 for a zero scale.  scale_norm() gives the
// normalised form (exponent key << 2 | significand bits) of normal and subnormal bytes alike; the value is
// significand x 2^(key - 17).
__device__ __forceinline__ float inv_scale(uint32_t byte) {
    const uint32_t n = scale_norm(byte), m = n & 3u;
    const uint32_t r = m == 0 ? 0x3F800000u : m == 1 ? 0x3F4CCCCDu : m == 2 ? 0x3F2AAAABu : 0x3F124925u;   // 1, 0.8, 2/3, 4/7
    return byte ? __uint_as_float(r + ((17u - (n >> 2)) << 23)) : 0.0f;
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
    inv_p = inv_scale(sc & 0xFFu);
    inv_n = inv_scale(sc >> 8);
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
        inv_p = inv_scale(bp);
        inv_n = inv_scale(bn);
        return bp | (bn << 8);
    }
    const uint32_t amax = max(c & 0xFFFFu, c >> 16);              // both halves are non-negative bf16 patterns
    uint32_t b;
    if (FMT == 1) b = cvt_e5m2x2(0.0f, trunc12(__uint_as_float(amax << 16) * sixth_up())) & 0xFFu;
    else b = pot_scale_byte<FMT == 4>(amax);
    inv_p = inv_n = inv_scale(b);
    return b | (b << 8);
}

// Packed fp32 pairs (sm_100: two independent IEEE multiplies per instruction, same rounding as the scalar one).
__device__ __forceinline__ uint64_t pack_f32x2(uint32_t lo, uint32_t hi) {
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
    return d;
}
__device__ __forceinline__ uint64_t mul_f32x2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi) {
    uint32_t l, h;
    asm("mov.b64 {%0, %1}, %2;" : "=r"(l), "=r"(h) : "l"(v));
    lo = __uint_as_float(l);
    hi = __uint_as_float(h);
}
// Four packed pairs of quotients -> eight E2M1 nibbles; element i lands in nibble i.
__device__ __forceinline__ uint32_t cvt_e2m1x8(uint64_t q0, uint64_t q1, uint64_t q2, uint64_t q3) {
    uint32_t d;
    asm("{\n"
        ".reg .b8 b0, b1, b2, b3;\n"
        ".reg .f32 l0, h0, l1, h1, l2, h2, l3, h3;\n"
        "mov.b64 {l0, h0}, %1;\n"
        "mov.b64 {l1, h1}, %2;\n"
        "mov.b64 {l2, h2}, %3;\n"
        "mov.b64 {l3, h3}, %4;\n"
        "cvt.rn.satfinite.e2m1x2.f32 b0, h0, l0;\n"
        "cvt.rn.satfinite.e2m1x2.f32 b1, h1, l1;\n"
        "cvt.rn.satfinite.e2m1x2.f32 b2, h2, l2;\n"
        "cvt.rn.satfinite.e2m1x2.f32 b3, h3, l3;\n"
        "mov.b32 %0, {b0, b1, b2, b3};\n"
        "}"
        : "=r"(d) : "l"(q0), "l"(q1), "l"(q2), "l"(q3));
    return d;
}
// 0xF on the nibbles of `codes` whose sign bit is set.  The shift is a multiply (FMA pipe; the logic pipe is the busy one).
__device__ __forceinline__ uint32_t negative_nibbles(uint32_t codes) { return (__umulhi(codes, 1u << 29) & 0x11111111u) * 15u; }

// The two bf16 values of a word as a packed pair of fp32 bit patterns {low element, high element}.  Shifts written
// as multiplies by a constant the assembler cannot see (it lives in constant memory): they run on the FMA pipe,
// which this arithmetic leaves mostly idle, instead of the saturated integer/logic pipe.
static __constant__ uint32_t kTwo16 = 65536u;
__device__ __forceinline__ uint64_t bf16x2_to_f32x2(uint32_t w) {
    const uint32_t k = kTwo16;
    return pack_f32x2(w * k, __umulhi(w, k) * k);
}

// 8 consecutive elements (4 bf16x2 words) -> their 8 nibbles twice: as if every element used the positive-side
// reciprocal (cp) and as if every element used the negative-side one (cn).  An element's own code is its nibble
// of cp when its sign bit is clear and of cn when it is set; the sign bit of a nibble is the element's in both.
// (Two packed multiplies and two converts per element pair cost less than picking the reciprocal per element.)
__device__ __forceinline__ void encode8_both(const uint32_t* w, uint64_t inv_p2, uint64_t inv_n2, uint32_t& cp, uint32_t& cn) {
    uint64_t x[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) x[i] = bf16x2_to_f32x2(w[i]);
    cp = cvt_e2m1x8(mul_f32x2(x[0], inv_p2), mul_f32x2(x[1], inv_p2), mul_f32x2(x[2], inv_p2), mul_f32x2(x[3], inv_p2));
    cn = cvt_e2m1x8(mul_f32x2(x[0], inv_n2), mul_f32x2(x[1], inv_n2), mul_f32x2(x[2], inv_n2), mul_f32x2(x[3], inv_n2));
}
// The same with one reciprocal for both signs (the symmetric formats).
__device__ __forceinline__ uint32_t encode8_one(const uint32_t* w, uint64_t inv2) {
    return cvt_e2m1x8(mul_f32x2(bf16x2_to_f32x2(w[0]), inv2), mul_f32x2(bf16x2_to_f32x2(w[1]), inv2),
                      mul_f32x2(bf16x2_to_f32x2(w[2]), inv2), mul_f32x2(bf16x2_to_f32x2(w[3]), inv2));
}

// 8 consecutive elements (4 bf16x2 words) -> 8 nibbles, every element divided by the scale of its own sign.
__device__ __forceinline__ uint32_t encode8(const uint32_t* w, float inv_p, float inv_n) {
    const uint32_t ip = __float_as_uint(inv_p), in = __float_as_uint(inv_n);
    uint32_t cp, cn;
    encode8_both(w, pack_f32x2(ip, ip), pack_f32x2(in, in), cp, cn);
    const uint32_t m = negative_nibbles(cp);
    return (cp & ~m) | (cn & m);
}

// One group of an FP4-GEMM operand from its 16 bf16x2 words: canonical codes (when asked for) and scale bytes at
// group index v, and the sign planes that are asked for (codes / pos / neg may be nullptr).  Returns the scale
// bytes {neg : pos}.
// With a symmetric format (FMT != 0) the operand needs no split: the signed codes go to the "positive" plane
// as they are, the other plane is zero, and the returned bytes name the one scale as the positive side's only.
template <int FMT = 0>
__device__ __forceinline__ uint32_t emit_group(const uint32_t (&w)[16], int64_t v, uint4* __restrict__ codes,
                                               uint16_t* __restrict__ scales, uint4* __restrict__ pos,
                                               uint4* __restrict__ neg) {
    float inv_p, inv_n;
    const uint32_t sc = group_scales_fmt<FMT>(side_maxima<16>(w), inv_p, inv_n);
    const uint32_t ip = __float_as_uint(inv_p), in = __float_as_uint(inv_n);
    const uint64_t inv_p2 = pack_f32x2(ip, ip), inv_n2 = pack_f32x2(in, in);
    uint32_t nib[4], pp[4], nn[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        if (FMT) {                               // one scale, no split: the signed codes are the "positive" plane
            nib[j] = pp[j] = encode8_one(w + 4 * j, inv_p2);
            nn[j] = 0;
        } else {
            uint32_t cp, cn;
            encode8_both(w + 4 * j, inv_p2, inv_n2, cp, cn);
            const uint32_t m = negative_nibbles(cp);
            pp[j] = cp & ~m;
            nn[j] = cn & m;
            nib[j] = pp[j] | nn[j];
        }
    }
    if (codes) codes[v] = make_uint4(nib[0], nib[1], nib[2], nib[3]);
    if (pos) pos[v] = make_uint4(pp[0], pp[1], pp[2], pp[3]);
    if (neg) neg[v] = make_uint4(nn[0], nn[1], nn[2], nn[3]);
    scales[v] = (uint16_t)sc;
    return FMT ? (sc & 0xFFu) : sc;
}

// The cast of a group without negative elements (a softmax output) when only the FP4 kernels' operand is wanted:
// its positive sign plane is its code word, the negative plane and scale are zero.  Same arithmetic as above,
// minus everything the negative side needs.  nib: the group's 32 codes; returns the positive scale byte.
// (The bf16 pairs are split with a shift and a mask here: this runs in the attention epilogue, where the logic pipe
// has room and instruction issue is what counts.)
__device__ __forceinline__ uint32_t cast_nonneg_group(const uint32_t (&w)[16], uint32_t (&nib)[4]) {
    uint32_t pm = w[0];
#pragma unroll
    for (int i = 1; i + 1 < 16; i += 2) pm = __vimax3_s16x2(pm, w[i], w[i + 1]);
    pm = __vmaxs2(pm, w[15]);
    pm = __vmaxs2(pm, pm >> 16) & 0xFFFFu;                       // the group maximum's bf16 bits
    const uint32_t sc = cvt_e5m2x2(0.0f, trunc12(__uint_as_float(pm << 16) * sixth_up())) & 0xFFu;
    const uint32_t inv = __float_as_uint(inv_scale(sc));
    const uint64_t inv2 = pack_f32x2(inv, inv);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        uint64_t q[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) q[i] = mul_f32x2(pack_f32x2(w[4 * j + i] << 16, w[4 * j + i] & 0xFFFF0000u), inv2);
        nib[j] = cvt_e2m1x8(q[0], q[1], q[2], q[3]);
    }
    return sc;
}
// Stores the plane at group index v (and, when asked, the same word as the group's canonical codes: without a set
// sign bit the two are equal), returns the positive scale byte.
__device__ __forceinline__ uint32_t emit_nonneg_plane(const uint32_t (&w)[16], int64_t v, uint4* __restrict__ plane,
                                                      uint4* __restrict__ codes = nullptr) {
    uint32_t nib[4];
    const uint32_t sc = cast_nonneg_group(w, nib);
    plane[v] = make_uint4(nib[0], nib[1], nib[2], nib[3]);
    if (codes) codes[v] = make_uint4(nib[0], nib[1], nib[2], nib[3]);
    return sc;
}

}  // namespace cast
}  // namespace amx
