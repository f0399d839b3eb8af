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

}  // namespace decode
}  // namespace amx
