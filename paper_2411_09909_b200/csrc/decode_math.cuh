// Exact decode of AMXFP4 codes to bf16 (Eq. 1): shared by the kernels that multiply on bf16 operands.
//
// Per 32-element group the 2 x 8 possible values (magnitude x side scale) are computed once with packed bf16
// multiplies and held as byte-plane lookup tables in registers; elements are then looked up four at a time with
// byte permutes and the side is chosen with a mask built from the sign bits.  A decoded value has at most 5
// significant bits, so bf16 holds it exactly.
#pragma once

#include <cuda_bf16.h>

#include "amx_common.cuh"

namespace amx {
namespace decode {

// prmt.b32: result byte i = byte (selector nibble i & 7) of {b, a}; when bit 3 of the nibble is set the
// byte's sign bit is replicated over the whole result byte instead.
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
struct GroupTables {   // byte planes of the 8 values per side: [side][plane lo/hi][2 regs]
    uint32_t lo_p0, lo_p1, hi_p0, hi_p1, lo_n0, lo_n1, hi_n0, hi_n1;
};

// bf16x2 {s, s} of an E5M2 byte (exact: E5M2 is the top byte of a half; a half widens exactly).
__device__ __forceinline__ uint32_t scale_pair(uint32_t byte) {
    const uint32_t f = __float_as_uint(e5m2_to_float(byte));
    return prmt(f, f, 0x3232);
}
__device__ __forceinline__ uint32_t mul_bf16x2(uint32_t a, uint32_t b) {
    __nv_bfloat162 r = __hmul2(*reinterpret_cast<__nv_bfloat162*>(&a), *reinterpret_cast<__nv_bfloat162*>(&b));
    return *reinterpret_cast<uint32_t*>(&r);
}
__device__ __forceinline__ GroupTables make_tables(uint32_t sc) {
    // E2M1 magnitudes as bf16 pairs: {0, .5} {1, 1.5} {2, 3} {4, 6}
    const uint32_t c01 = 0x3F000000u, c23 = 0x3FC03F80u, c45 = 0x40404000u, c67 = 0x40C04080u;
    const uint32_t sp = scale_pair(sc & 0xFFu), sn = scale_pair(sc >> 8) ^ 0x80008000u;
    GroupTables t;
    uint32_t a = mul_bf16x2(c01, sp), b = mul_bf16x2(c23, sp), c = mul_bf16x2(c45, sp), d = mul_bf16x2(c67, sp);
    t.lo_p0 = prmt(a, b, 0x6420); t.hi_p0 = prmt(a, b, 0x7531);
    t.lo_p1 = prmt(c, d, 0x6420); t.hi_p1 = prmt(c, d, 0x7531);
    a = mul_bf16x2(c01, sn); b = mul_bf16x2(c23, sn); c = mul_bf16x2(c45, sn); d = mul_bf16x2(c67, sn);
    t.lo_n0 = prmt(a, b, 0x6420); t.hi_n0 = prmt(a, b, 0x7531);
    t.lo_n1 = prmt(c, d, 0x6420); t.hi_n1 = prmt(c, d, 0x7531);
    return t;
}
// 8 codes (one 32-bit word) -> 8 bf16 values (16 bytes).
__device__ __forceinline__ uint4 decode_word(uint32_t w, const GroupTables& t) {
    const uint32_t sel = w & 0x77777777u, selh = sel >> 16, ws = w << 4;
    const uint32_t m0 = prmt(ws, w, 0xD9C8), m1 = prmt(ws, w, 0xFBEA);  // 0xFF where negative
    uint32_t lo, hi;
    uint4 o;
    lo = (prmt(t.lo_p0, t.lo_p1, sel) & ~m0) | (prmt(t.lo_n0, t.lo_n1, sel) & m0);
    hi = (prmt(t.hi_p0, t.hi_p1, sel) & ~m0) | (prmt(t.hi_n0, t.hi_n1, sel) & m0);
    o.x = prmt(lo, hi, 0x5140); o.y = prmt(lo, hi, 0x7362);
    lo = (prmt(t.lo_p0, t.lo_p1, selh) & ~m1) | (prmt(t.lo_n0, t.lo_n1, selh) & m1);
    hi = (prmt(t.hi_p0, t.hi_p1, selh) & ~m1) | (prmt(t.hi_n0, t.hi_n1, selh) & m1);
    o.z = prmt(lo, hi, 0x5140); o.w = prmt(lo, hi, 0x7362);
    return o;
}

// Decode by packed multiplies, for kernels that the integer/logic pipe bounds: the multiplication by the scale
// is a packed bf16 multiply (FMA pipe) instead of table look-ups, at the price of a fixed permutation of the eight
// elements of a word (harmless for a contraction whose two operands are decoded the same way) and of a factor
// 2^-63 on every value (exact; the other operand carries 2^+63):
//   - a 3-bit E2M1 code placed at bits 8..6 of a bf16 reads as (its value) x 2^-126: codes 0 and 1 are the bf16
//     subnormals 0 and 2^-127, the others have exponent field 1..3 and the code's mantissa bit;
//   - one shift and one mask put the codes of elements q and q + 4 of a word there (pair q);
//   - the element's scale (positive or negative side, the sign folded into the latter) is chosen with a mask that
//     a byte permute in sign-replicating mode builds from the two sign bits;
//   - scales are held as bf16 pairs times 2^63 (2^126 would overflow); decode_pairs_up multiplies once more,
//     by 2^126, for the operand that carries the other 2^63.
struct GroupScales {
    uint32_t pos, neg;     // {s_p, s_p} x 2^63 and {-s_n, -s_n} x 2^63 as bf16 pairs
};
__device__ __forceinline__ GroupScales make_scales(uint32_t sc) {
    const float two63 = 9223372036854775808.f;
    const uint32_t p = __float_as_uint(e5m2_to_float(sc & 0xFFu) * two63);
    const uint32_t n = __float_as_uint(e5m2_to_float((sc >> 8) & 0xFFu) * -two63);
    return {prmt(p, p, 0x3232), prmt(n, n, 0x3232)};
}
__device__ __forceinline__ uint4 decode_pairs(uint32_t w, const GroupScales& gs) {
    const uint32_t kMag = 0x01C001C0u, ws = w << 4;
    const uint32_t m0 = prmt(ws, ws, 0xAA88), m1 = prmt(w, w, 0xAA88);     // 0xFFFF where the element is negative
    const uint32_t m2 = prmt(ws, ws, 0xBB99), m3 = prmt(w, w, 0xBB99);
    uint4 o;
    o.x = mul_bf16x2((w << 6) & kMag, (gs.pos & ~m0) | (gs.neg & m0));
    o.y = mul_bf16x2((w << 2) & kMag, (gs.pos & ~m1) | (gs.neg & m1));
    o.z = mul_bf16x2((w >> 2) & kMag, (gs.pos & ~m2) | (gs.neg & m2));
    o.w = mul_bf16x2((w >> 6) & kMag, (gs.pos & ~m3) | (gs.neg & m3));
    return o;
}
// The same pairs times 2^+63 (true value x 2^63): the other operand of a product with decode_pairs.
__device__ __forceinline__ uint4 decode_pairs_up(uint32_t w, const GroupScales& gs) {
    const uint32_t two126 = 0x7E807E80u;
    uint4 o = decode_pairs(w, gs);
    o.x = mul_bf16x2(o.x, two126); o.y = mul_bf16x2(o.y, two126);
    o.z = mul_bf16x2(o.z, two126); o.w = mul_bf16x2(o.w, two126);
    return o;
}

}  // namespace decode
}  // namespace amx
