// Shared host/device helpers of the AMXFP4 CUDA library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "amx.h"

namespace amx {

// Group sizes: 16, 32, 64 or 128 elements, or the whole row as one group (group_size == K, K a multiple of 8:
// the grouping of the paper's worked example), which only the generic kernels take.
inline bool fixed_group_size(int gs) { return gs == 16 || gs == 32 || gs == 64 || gs == 128; }
inline bool valid_group_size(int gs, int64_t K) { return fixed_group_size(gs) || (gs > 0 && gs == K && K % 8 == 0); }

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Returns AMX_OK when the last launch was accepted, AMX_ERR_CUDA otherwise.
inline int launch_status() { return cudaGetLastError() == cudaSuccess ? AMX_OK : AMX_ERR_CUDA; }

// ---- device-side number formats -------------------------------------------------------------

// fp32 value of an E5M2 byte: E5M2 is the upper byte of an IEEE half.
__device__ __forceinline__ float e5m2_to_float(uint32_t byte) {
    float f;
    unsigned short h = (unsigned short)(byte << 8);
    asm("cvt.f32.f16 %0, %1;" : "=f"(f) : "h"(h));
    return f;
}

// fp32 magnitude of a 3-bit E2M1 code EEM: 0, .5, 1, 1.5, 2, 3, 4, 6.
// For EE > 0 the bits placed at fp32 exponent/mantissa positions give 2^(EE-1) * (1 + M/2);
// EE == 0 is the subnormal M * 0.5.
__device__ __forceinline__ float e2m1_mag_to_float(uint32_t c3) {
    uint32_t bits = (c3 << 22) + (126u << 23);   // exponent field EE + 126, mantissa msb = M
    float v = __uint_as_float(bits);
    return (c3 & 6u) ? v : 0.5f * (float)(c3 & 1u);
}

// An E5M2 scale byte as (key << 2) | mantissa of its normalised form: key = unbiased exponent + 17 (so that
// 2^-16 has key 1) and two mantissa bits.  Normal bytes (b >= 4) are b + 8; the subnormals 1, 2, 3 x 2^-16 are
// 1.0 x 2^-16, 1.0 x 2^-15 and 1.5 x 2^-15: 4, 8 and 10 (read from a packed table); 0 for a zero scale.
__device__ __forceinline__ uint32_t scale_norm(uint32_t b) {
    return b >= 4 ? b + 8 : (0x0A080400u >> (b * 8)) & 0xFFu;
}
// Exponent key of an E5M2 scale byte, 0 for a zero scale.
__device__ __forceinline__ int scale_key(uint32_t b) { return (int)(scale_norm(b) >> 2); }
// Per-row word of a prepared FP4-GEMM operand: bits 15..0 the row's power-of-two offset (largest exponent key
// - 25; 0 for an all-zero row) as a signed 16-bit number, bit 16 set when some group of the row has a nonzero
// positive-side scale, bit 17 the same for the negative side.  A tile whose rows all lack a side has an
// all-zero plane for it, and the GEMM does not issue that plane's products.  Bits 31..18: how many nonzero
// scales of the row did not fit the UE4M3 range under the row's offset and were flushed to zero (see
// to_ue4m3), saturating at kRowFlushedMax.
constexpr int kRowHasPos = 1 << 16, kRowHasNeg = 1 << 17;
constexpr int kRowFlushedShift = 18, kRowFlushedMax = 0x3FFF;
__host__ __device__ __forceinline__ int row_word(int kmax, int side_bits, int flushed = 0) {
    const int f = flushed > kRowFlushedMax ? kRowFlushedMax : flushed;
    return ((kmax ? kmax - 25 : 0) & 0xFFFF) | side_bits | (int)((unsigned)f << kRowFlushedShift);
}
__host__ __device__ __forceinline__ int row_word_exp(int w) { return (int)(short)(w & 0xFFFF); }
__host__ __device__ __forceinline__ int row_word_flushed(int w) { return (int)((unsigned)w >> kRowFlushedShift); }
// side bits of a group's scale bytes {neg : pos}
__device__ __forceinline__ int side_bits_of(uint32_t sc) {
    return ((sc & 0xFFu) ? kRowHasPos : 0) | ((sc >> 8) ? kRowHasNeg : 0);
}

// Scale factors of a prepared operand: chunks of 512 bytes per [128 rows x 64 elements], the chunks of one block
// of 128 rows consecutive along K; inside a chunk byte (r % 32) * 16 + (r / 32) * 4 + (k16 % 4), one scale per 16
// elements.  Offset of row `row`'s bytes of its first chunk, and of 32-group g's two bytes relative to that.
constexpr int kSfChunkBytes = 512;
__host__ __device__ __forceinline__ int64_t sf_row_offset(int64_t row, int nk64) {
    const int rr = (int)(row & 127);
    return (row >> 7) * nk64 * (int64_t)kSfChunkBytes + (rr & 31) * 16 + (rr >> 5) * 4;
}
__host__ __device__ __forceinline__ int64_t sf_group_offset(int g) { return (int64_t)(g >> 1) * kSfChunkBytes + (g & 1) * 2; }

// UE4M3 byte of the E5M2 byte b for a row whose largest key is kmax (0 when it does not fit): exponent field
// key - kmax + 15 (at least 1), the two mantissa bits in bits 2..1.
__device__ __forceinline__ uint32_t to_ue4m3(uint32_t b, int kmax) {
    const int t = (int)scale_norm(b) + ((15 - kmax) << 2);       // (exponent field << 2) | mantissa
    return (b != 0 && t >= 4) ? (uint32_t)t << 1 : 0u;
}
// Whether to_ue4m3 flushes the nonzero scale byte b: its key lies 15 or more below the row's largest.
__device__ __forceinline__ bool ue4m3_flushes(uint32_t b, int kmax) {
    return b != 0 && (int)scale_norm(b) + ((15 - kmax) << 2) < 4;
}

}  // namespace amx
