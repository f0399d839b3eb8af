// bf16 -> AMXFP4 direct cast (arXiv 2411.09909, Sections 4.2-4.3; Algorithm 1 applied per sign
// with the FP8 E5M2 shared scale).  HBM-bound: 2 B read + 0.5625 B written per element.  The per-group
// arithmetic, with the argument for its exactness, is in cast_math.cuh.
#include <cuda_bf16.h>

#include "cast_math.cuh"
#include "cp_async.cuh"
#include "softmax_math.cuh"

namespace amx {
namespace {

using namespace cast;

constexpr int kThreads = 256;

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
template <int EPT, int TPG, bool CONTIG, int FMT = 0>
__global__ void __launch_bounds__(kThreads)
quantize_rows_kernel(const uint4* __restrict__ x, int64_t n_items, int64_t items_per_row,
                     int64_t ld_vec, uint4* __restrict__ codes, uint16_t* __restrict__ scales) {
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
    const uint32_t sc = group_scales_fmt<FMT>(c, inv_p, inv_n);
    uint32_t nib[NV];
#pragma unroll
    for (int j = 0; j < NV; ++j) nib[j] = encode8(w + 4 * j, inv_p, inv_n);
    if (live) {
        if (NV == 4) codes[v] = make_uint4(nib[0], nib[1], nib[2], nib[NV - 1]);
        else *reinterpret_cast<uint2*>(reinterpret_cast<uint8_t*>(codes) + v * 8) = make_uint2(nib[0], nib[NV - 1]);
        if ((threadIdx.x & (TPG - 1)) == 0) scales[v / TPG] = (uint16_t)sc;
    }
}

// The whole row as one group (group_size == K; the grouping of the worked example in Appendix B.3): one block per
// row, two sweeps - the row's side maxima (block reduction), then the codes.  The second sweep re-reads the row
// from the caches.  Generic path, any K that is a multiple of 8.
template <int FMT>
__global__ void __launch_bounds__(kThreads)
quantize_whole_rows_kernel(const uint4* __restrict__ x, int64_t vec_per_row, int64_t ld_vec, uint32_t* __restrict__ codes,
                           uint16_t* __restrict__ scales) {
    __shared__ uint32_t red[kThreads / 32];
    const int64_t row = blockIdx.x;
    const uint4* xr = x + row * ld_vec;
    uint32_t c = 0;
    for (int64_t i = threadIdx.x; i < vec_per_row; i += kThreads) {
        const uint4 q = __ldg(xr + i);
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
        c = __vmaxs2(c, side_maxima<4>(w));
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) c = __vmaxs2(c, __shfl_xor_sync(0xFFFFFFFFu, c, d));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = c;
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kThreads / 32; ++i) c = __vmaxs2(c, red[i]);
    float inv_p, inv_n;
    const uint32_t sc = group_scales_fmt<FMT>(c, inv_p, inv_n);
    for (int64_t i = threadIdx.x; i < vec_per_row; i += kThreads) {
        const uint4 q = __ldg(xr + i);
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
        codes[row * vec_per_row + i] = encode8(w, inv_p, inv_n);
    }
    if (threadIdx.x == 0) scales[row] = (uint16_t)sc;
}

// Groups DOWN the rows (strided axis): x is [R, C]; output is the canonical layout of x^T.
// A block stages a [64 rows x 64 columns] tile in shared memory and re-reads it column-wise.
constexpr int kTR = 64, kTC = 64;

template <int TPG>
__global__ void __launch_bounds__(kThreads)
quantize_cols_kernel(const __nv_bfloat16* __restrict__ x, int64_t R, int64_t C, int64_t ld,
                     uint32_t* __restrict__ codes, uint16_t* __restrict__ scales, int gs) {
    // blockIdx.z: one of several [R, C] matrices stored one after another (R * ld elements apart); their
    // transposed outputs follow one another as well
    __shared__ uint16_t tile[kTC][kTR + 2];  // [column][row], padded
    const int64_t r0 = (int64_t)blockIdx.y * kTR, c0 = (int64_t)blockIdx.x * kTC;
    const uint16_t* xs = reinterpret_cast<const uint16_t*>(x) + (int64_t)blockIdx.z * R * ld;
    codes += (int64_t)blockIdx.z * (C * R / 8);
    scales += (int64_t)blockIdx.z * (C * R / gs);
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

// The cast for an operand of the FP4 GEMM (32-groups, contiguous rows).  Besides the canonical codes and scales
// it writes, in the same pass, everything the GEMM reads: the two sign planes (every nibble in the plane of its
// sign bit, zero in the other), the UE4M3 scale factors of both planes - byte (r%32)*16 + (r/32)*4 + k16%4 of
// the 512-byte chunk of [128 rows x 64 elements]; one scale per 16 elements, so a 32-group's scale is stored
// twice - and per row the power of two by which those scale factors understate the true scales
// (row_exp = largest exponent key of the row - 25).  The scale factors depend on the row's largest scale, so
// whole rows belong to one warp (cast_prepared_kernel) or, in the softmax variant, to one block
// (finish_prepared_row).  Rows past the last row, and groups past the last group, get zero scale factors, so that
// padded tile rows and columns multiply zero codes by a finite scale.

// Second half of a prepared cast, for the GX threads (a multiple of 32) that own row `row` (`top`: the largest
// positive-side scale byte the thread has seen in bits 7..0, the largest negative-side one in bits 15..8;
// slot: the row's four shared-memory words, zero on entry): row maximum of the exponent keys and which sides
// occur, the row's scale factors in the tensor cores' layout, padding included, and the row word (with the
// number of scales that did not fit the UE4M3 range and were flushed: the last warp of the row to finish
// writes it, so no third block barrier is needed).
__device__ __forceinline__ void finish_prepared_row(int64_t row, bool row_live, int G, int gx, int GX, uint32_t top,
                                                    uint32_t sc_first, const uint16_t* __restrict__ scales,
                                                    int* slot, uint8_t* __restrict__ sf_pos,
                                                    uint8_t* __restrict__ sf_neg, int* __restrict__ row_exp, int nk64,
                                                    int* __restrict__ flushed_total = nullptr) {
    // Two shared-memory atomics per warp.  The key of an E5M2 byte grows with the byte (scales carry no sign
    // bit), so the largest byte has the largest key.
    const uint32_t top_p = __reduce_max_sync(0xFFFFFFFFu, top & 0xFFu), top_n = __reduce_max_sync(0xFFFFFFFFu, top >> 8);
    __syncthreads();                               // the slot was zeroed at the top of the kernel
    if ((gx & 31) == 0 && (top_p | top_n)) {
        atomicMax(&slot[0], scale_key(max(top_p, top_n)));
        atomicOr(&slot[1], side_bits_of(top_p | (top_n << 8)));
    }
    __syncthreads();
    const int kmax = slot[0];
    // offset of this row's bytes inside a chunk; the chunks of one block of 128 rows are consecutive along K
    const int64_t sf_row = sf_row_offset(row, nk64);
    const int64_t v_row = row * G;
    int flushed = 0;
    for (int g = gx; g < nk64 * 2; g += GX) {      // groups past G: padding to whole 256-element blocks
        uint32_t up = 0, un = 0;
        if (row_live && g < G) {
            // a later group of a striding thread: re-read the scale bytes this thread stored before
            const uint32_t sc = (g == gx) ? sc_first : scales[v_row + g];
            up = to_ue4m3(sc & 0xFFu, kmax);
            un = to_ue4m3(sc >> 8, kmax);
            flushed += (int)((sc & 0xFFu) != 0 && up == 0) + (int)((sc >> 8) != 0 && un == 0);
        }
        const int64_t off = sf_row + sf_group_offset(g);
        *reinterpret_cast<uint16_t*>(sf_pos + off) = (uint16_t)(up | (up << 8));
        *reinterpret_cast<uint16_t*>(sf_neg + off) = (uint16_t)(un | (un << 8));
    }
    if (!row_live) return;                         // uniform over the row's warps
    flushed = __reduce_add_sync(0xFFFFFFFFu, flushed);
    if ((gx & 31) == 0) {
        if (flushed) atomicAdd(&slot[2], flushed);
        __threadfence_block();
        if (atomicAdd(&slot[3], 1) == GX / 32 - 1) {
            const int total = atomicAdd(&slot[2], 0);
            row_exp[row] = row_word(kmax, slot[1], total);
            if (total && flushed_total) atomicAdd(flushed_total, total);
        }
    }
}

// The cast for an operand of the FP4 GEMM.  A row (or, when rows are short, several rows) belongs to one warp:
// LPR = 2^lpr_log2 lanes per row, lane lr of them owns the groups lr, lr + LPR, ...  A lane streams its groups
// through a private ring in shared memory with asynchronous copies (kCastDepth groups ahead; the loads hold no
// registers).  First sweep: per group the cast, the stores of the planes, the scale bytes and (when asked for)
// the canonical codes; the scale bytes stay in registers (GPL of them per lane; GPL = 0: any number, re-read from
// the scales just stored).  Then the row's largest exponent key by a warp reduction, and the second sweep turns
// the scale bytes into the row's scale factors, padding included, and writes the row word.
// Scale factors leave the block in whole 32-byte sectors: the tensor cores' layout interleaves eight rows (r, r+1,
// r+32, r+33, r+64, r+65, r+96, r+97, r even) in every sector, so a block of eight warps owns exactly such sets of
// rows - warp (q, h) has the rows 32 q + 2 k + h of a 128-row block, for the block's RPW = 32 / LPR values of k -
// collects the converted bytes in shared memory and stores them 16 bytes per thread.  (Written 2 bytes at a
// time straight from the owning lanes, the scale factors were 4 % of the bytes and doubled the kernel's L2
// write requests.)  Rows past the last row get zero scale factors.
constexpr int kCastDepth = 2;                              // groups in flight per lane
constexpr int kCastWarps = 8;
constexpr int kCastRingBytes = kCastWarps * kCastDepth * 32 * 64;
constexpr int kCastMaxExchangeBytes = 96 * 1024;           // above this (K > 49152 at LPR = 32) the lanes store their bytes themselves

template <int FMT, int GPL>
__global__ void __launch_bounds__(kCastWarps * 32)
cast_prepared_kernel(const uint4* __restrict__ x, int64_t R, int G, int lpr_log2, int exchange,
                     uint4* __restrict__ codes, uint16_t* __restrict__ scales, uint4* __restrict__ pos,
                     uint4* __restrict__ neg, uint8_t* __restrict__ sf_pos, uint8_t* __restrict__ sf_neg,
                     int* __restrict__ row_exp, int nk64, int* __restrict__ flushed_total) {
    extern __shared__ __align__(16) uint8_t smem_raw[];
    const int lane = threadIdx.x & 31, wi = threadIdx.x >> 5, LPR = 1 << lpr_log2, lr = lane & (LPR - 1);
    const int RPW = 32 >> lpr_log2, sg = lane >> lpr_log2;      // rows per warp; which of them this lane works on
    // the block's rows: 128-row block rb, sector sets k0 .. k0 + RPW - 1 (16 / RPW blocks share a 128-row block)
    const int64_t rb = (int64_t)blockIdx.x >> (lpr_log2 - 1);
    const int k0 = ((int)blockIdx.x & ((16 >> (5 - lpr_log2)) - 1)) << (5 - lpr_log2);
    const int r_in = 32 * (wi >> 1) + 2 * (k0 + sg) + (wi & 1);  // row inside the 128-row block
    const int64_t row = rb * 128 + r_in;
    const bool live = row < R;
    const unsigned seg_mask = LPR == 32 ? 0xFFFFFFFFu : ((1u << LPR) - 1u) << (lane & ~(LPR - 1));
    const int64_t v_row = row * G;
    // this lane's ring: kCastDepth slots of 64 bytes (one group).  Piece j of a group sits at 16-byte position
    // j ^ ((lane >> 1) & 3) of the slot, so that the lanes of a quarter warp read eight different bank groups.
    uint8_t* ring = smem_raw + ((wi * kCastDepth * 32) + lane) * 64;
    uint8_t* xchg = smem_raw + kCastRingBytes;        // [plane][chunk][sector set][h][q] words of 4 scale-factor bytes
    const int swz = (lane >> 1) & 3;
    const int n_own = (live && lr < G) ? ((G - lr + LPR - 1) >> lpr_log2) : 0;   // groups this lane owns
    auto issue = [&](int i) {                        // copies of the lane's i-th group, one commit group per call
        if (i < n_own) {
            const uint4* src = x + (v_row + lr + ((int64_t)i << lpr_log2)) * 4;
            uint8_t* slot = ring + (i % kCastDepth) * (32 * 64);
#pragma unroll
            for (int j = 0; j < 4; ++j) cp_async16(slot + ((j ^ swz) << 4), src + j);
        }
        cp_async_commit();
    };
    auto cast_group = [&](int i) -> uint32_t {       // the i-th group has landed: read it back, cast, store
        const uint8_t* slot = ring + (i % kCastDepth) * (32 * 64);
        uint32_t w[16];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint4 q = *reinterpret_cast<const uint4*>(slot + ((j ^ swz) << 4));
            w[4 * j] = q.x; w[4 * j + 1] = q.y; w[4 * j + 2] = q.z; w[4 * j + 3] = q.w;
        }
        return emit_group<FMT>(w, v_row + lr + ((int64_t)i << lpr_log2), codes, scales, pos, neg);
    };
    uint32_t sc_reg[GPL > 0 ? GPL : 1];
    uint32_t top = 0;                               // largest scale bytes seen by this lane, {neg : pos}
#pragma unroll
    for (int i = 0; i < kCastDepth - 1; ++i) issue(i);
    if (GPL > 0) {
#pragma unroll
        for (int i = 0; i < GPL; ++i) {
            issue(i + kCastDepth - 1);
            cp_async_wait<kCastDepth - 1>();
            sc_reg[i] = i < n_own ? cast_group(i) : 0u;
            top = __vmaxu4(top, sc_reg[i]);         // byte-wise maximum
        }
    } else {
        for (int i = 0; i < n_own; ++i) {
            issue(i + kCastDepth - 1);
            cp_async_wait<kCastDepth - 1>();
            top = __vmaxu4(top, cast_group(i));
        }
    }
    cp_async_wait<0>();
    // The key of an E5M2 byte grows with the byte (scales carry no sign bit): the largest byte has the largest key.
    const uint32_t top_p = __reduce_max_sync(seg_mask, top & 0xFFu), top_n = __reduce_max_sync(seg_mask, (top >> 8) & 0xFFu);
    const int kmax = scale_key(max(top_p, top_n));
    const int64_t sf_row = sf_row_offset(row, nk64);
    // word of the exchange buffer that holds this row's bytes of chunk c: ((c * RPW + sg) * 2 + h) * 4 + q
    const int x_row = (sg * 2 + (wi & 1)) * 4 + (wi >> 1), x_plane = nk64 * RPW * 8;   // in words
    int flushed = 0;
    auto put = [&](int g, uint32_t sc) {            // scale factors of group g (zero past the row's last group)
        const uint32_t up = to_ue4m3(sc & 0xFFu, kmax), un = to_ue4m3(sc >> 8, kmax);
        flushed += (int)((sc & 0xFFu) != 0 && up == 0) + (int)((sc >> 8) != 0 && un == 0);
        if (exchange) {
            uint16_t* w16 = reinterpret_cast<uint16_t*>(xchg) + (((g >> 1) * RPW * 8 + x_row) << 1) + (g & 1);
            w16[0] = (uint16_t)(up | (up << 8));
            w16[x_plane << 1] = (uint16_t)(un | (un << 8));
        } else {
            const int64_t off = sf_row + sf_group_offset(g);
            *reinterpret_cast<uint16_t*>(sf_pos + off) = (uint16_t)(up | (up << 8));
            *reinterpret_cast<uint16_t*>(sf_neg + off) = (uint16_t)(un | (un << 8));
        }
    };
    const int g_end = nk64 * 2;                     // groups past G: padding to whole 256-element blocks
    if (GPL > 0) {
#pragma unroll
        for (int i = 0; i < GPL; ++i) {
            const int g = lr + (i << lpr_log2);
            if (g < g_end) put(g, sc_reg[i]);       // zero for a group past G and for a padding row
        }
        for (int g = lr + (GPL << lpr_log2); g < g_end; g += LPR) put(g, 0u);
    } else {
        for (int g = lr; g < g_end; g += LPR) put(g, (live && g < G) ? (uint32_t)scales[v_row + g] : 0u);
    }
    flushed = __reduce_add_sync(seg_mask, flushed);
    if (lr == 0 && live) {
        row_exp[row] = row_word(kmax, side_bits_of(top_p | (top_n << 8)), flushed);
        if (flushed && flushed_total) atomicAdd(flushed_total, flushed);
    }
    if (!exchange) return;                          // uniform over the block
    __syncthreads();
    // 16 bytes per thread: the words of rows q = 0..3 (32 rows apart) for one (plane, chunk, sector set, h);
    // two neighbouring threads (h = 0, 1) fill one sector
    const int per_plane = nk64 * RPW * 2;
    for (int item = threadIdx.x; item < 2 * per_plane; item += kCastWarps * 32) {
        const int plane = item >= per_plane, rest = item - plane * per_plane;
        const int c = rest / (RPW * 2), sh = rest - c * (RPW * 2);      // sh = sector set * 2 + h
        const uint4 v = reinterpret_cast<const uint4*>(xchg)[item];
        uint8_t* dst = (plane ? sf_neg : sf_pos) + (rb * nk64 + c) * (int64_t)kSfChunkBytes + (2 * k0 + sh) * 16;
        *reinterpret_cast<uint4*>(dst) = v;
    }
}

// Attention glue in one pass (Appendix C): row softmax of the fp32 logits (times alpha), rounding of the
// normalised map to bf16 - the cast's input type - and the cast of that row to AMXFP4, without the map ever
// reaching global memory as fp32 or bf16.  One block of softmax::kT threads per row (grid = padded rows when the
// prepared form is written, blocks past the last row only zero scale-factor padding).  Same bits as the
// stand-alone softmax kernel followed by the cast: both use softmax_math.cuh and cast_math.cuh.
// CACHED: the row has at most kT groups, so each thread keeps its one group in registers between the passes.
template <bool CACHED>
__global__ void __launch_bounds__(softmax::kT)
softmax_cast_kernel(const float* __restrict__ S, int64_t R, int G, int64_t ld_s, float alpha, int vec, int causal,
                    uint4* __restrict__ codes, uint16_t* __restrict__ scales, uint4* __restrict__ pos,
                    uint4* __restrict__ neg, uint8_t* __restrict__ sf_pos, uint8_t* __restrict__ sf_neg,
                    int* __restrict__ row_exp, int nk64) {
    __shared__ float sh[softmax::kT / 32];
    __shared__ int slot_s[4];
    const int gx = threadIdx.x;
    const int64_t row = blockIdx.x;
    const bool row_live = row < R;                  // uniform over the block
    if (gx < 4) slot_s[gx] = 0;
    uint32_t sc_first = 0, top = 0;
    if (row_live) {
        const float* s = S + row * ld_s;
        const int64_t cols = (int64_t)G * 32, v_row = row * G;
        const int64_t seen = causal ? min(cols, row + 1) : cols;     // causal: query `row` sees keys 0 .. row
        if (CACHED) {
            float e[32];
            const float sum = softmax::cached_row_exp(s, G, vec != 0, alpha, sh, e, seen);
            if (gx < G) {
                uint32_t w[16];
                softmax::normalised_group_e(e, sum, w);
                sc_first = emit_group(w, v_row + gx, codes, scales, pos, neg);
                top = sc_first;
            }
        } else {
            float mx, sum;
            softmax::row_stats(s, cols, vec != 0, alpha, sh, mx, sum, seen);
            for (int g = gx; g < G; g += softmax::kT) {
                float t[32];
                uint32_t w[16];
                softmax::load_group(s, g, cols, vec != 0, alpha, t, seen);
                softmax::normalised_group(t, mx, sum, w);
                const uint32_t sc = emit_group(w, v_row + g, codes, scales, pos, neg);
                if (g == gx) sc_first = sc;
                top = __vmaxu4(top, sc);
            }
        }
    }
    if (!pos) return;                               // canonical output only
    finish_prepared_row(row, row_live, G, gx, softmax::kT, top, sc_first, scales, slot_s, sf_pos, sf_neg, row_exp, nk64);
}

template <int EPT, int TPG, int FMT = 0>
int launch_rows(const void* x, int64_t rows, int64_t K, int64_t ld, uint8_t* codes,
                uint8_t* scales, cudaStream_t st) {
    const int64_t n_items = rows * (K / EPT);
    const int64_t blocks = (n_items + kThreads - 1) / kThreads;
    if (blocks > 0x7FFFFFFF) return AMX_ERR_SHAPE;
    auto* xv = reinterpret_cast<const uint4*>(x);
    auto* cv = reinterpret_cast<uint4*>(codes);
    auto* sv = reinterpret_cast<uint16_t*>(scales);
    if (ld == K)
        quantize_rows_kernel<EPT, TPG, true, FMT><<<(unsigned)blocks, kThreads, 0, st>>>(xv, n_items, K / EPT, ld / 8, cv, sv);
    else
        quantize_rows_kernel<EPT, TPG, false, FMT><<<(unsigned)blocks, kThreads, 0, st>>>(xv, n_items, K / EPT, ld / 8, cv, sv);
    return launch_status();
}

}  // namespace

// Cast with the FP4 GEMM's operand preparation in the same launch (gs = 32, contiguous rows): canonical codes
// and scales, the two sign planes, the UE4M3 scale factors of both planes in the tensor cores' layout (nk64
// chunks of 512 B per block of 128 rows, rows padded to padded_rows) and the rows' power-of-two offsets.
namespace {
template <int FMT>
int launch_cast_prepared(const void* x, int64_t rows, int64_t G, uint8_t* codes, uint8_t* scales, void* pos, void* neg,
                         uint8_t* sf_pos, uint8_t* sf_neg, int* row_exp, int nk64, int64_t padded_rows, cudaStream_t st,
                         int* flushed_total) {
    int lpr_log2 = 1;
    while (lpr_log2 < 5 && (1 << lpr_log2) < G) ++lpr_log2;          // lanes per row: a power of two, 2 .. 32
    const int gpl = (int)((G + (1 << lpr_log2) - 1) >> lpr_log2);   // groups per lane
    const int rpw = 32 >> lpr_log2;                                  // rows per warp
    const int64_t blocks = (padded_rows / 128) * (16 / rpw);         // a block has 8 * rpw rows of one 128-row block
    if (blocks > 0x7FFFFFFF) return AMX_ERR_SHAPE;
    const size_t exchange_bytes = (size_t)64 * rpw * nk64;           // both planes, 4 bytes per row and 64 elements
    const int exchange = exchange_bytes <= (size_t)kCastMaxExchangeBytes;
    const int smem = kCastRingBytes + (exchange ? (int)exchange_bytes : 0);
    auto* kernel = gpl <= 1 ? cast_prepared_kernel<FMT, 1> : gpl <= 2 ? cast_prepared_kernel<FMT, 2>
                 : gpl <= 4 ? cast_prepared_kernel<FMT, 4> : gpl <= 8 ? cast_prepared_kernel<FMT, 8>
                 : cast_prepared_kernel<FMT, 0>;      // longer rows: the scale bytes are re-read, not kept in registers
    static bool configured[64][5] = {};                 // the opt-in to > 48 KB of dynamic shared memory: per device, kernel
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return AMX_ERR_CUDA;
    const int slot = gpl <= 1 ? 0 : gpl <= 2 ? 1 : gpl <= 4 ? 2 : gpl <= 8 ? 3 : 4;
    if (!configured[dev][slot]) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kCastRingBytes + kCastMaxExchangeBytes) !=
            cudaSuccess) {
            cudaGetLastError();
            return AMX_ERR_CUDA;
        }
        configured[dev][slot] = true;
    }
    kernel<<<(unsigned)blocks, kCastWarps * 32, smem, st>>>(
        reinterpret_cast<const uint4*>(x), rows, (int)G, lpr_log2, exchange, reinterpret_cast<uint4*>(codes),
        reinterpret_cast<uint16_t*>(scales), reinterpret_cast<uint4*>(pos), reinterpret_cast<uint4*>(neg), sf_pos, sf_neg,
        row_exp, nk64, flushed_total);
    return launch_status();
}
}  // namespace

// codes may be nullptr: the canonical codes are then not written (the planes hold the same nibbles).
int quantize_rows_prepared(const void* x, int64_t rows, int64_t K, uint8_t* codes, uint8_t* scales, void* pos,
                           void* neg, uint8_t* sf_pos, uint8_t* sf_neg, int* row_exp, int nk64, int64_t padded_rows,
                           cudaStream_t st, int format, int* flushed_total) {
    const int64_t G = K / 32;
    if (format == AMX_FMT_SYM_FP8)
        return launch_cast_prepared<1>(x, rows, G, codes, scales, pos, neg, sf_pos, sf_neg, row_exp, nk64, padded_rows, st, flushed_total);
    if (format == AMX_FMT_MXFP4)
        return launch_cast_prepared<2>(x, rows, G, codes, scales, pos, neg, sf_pos, sf_neg, row_exp, nk64, padded_rows, st, flushed_total);
    return launch_cast_prepared<0>(x, rows, G, codes, scales, pos, neg, sf_pos, sf_neg, row_exp, nk64, padded_rows, st, flushed_total);
}

// Softmax of the rows of S (fp32 [rows, ld_s], cols % 32 == 0), rounded to bf16 and cast, in one launch.  With
// pos == nullptr only the canonical codes and scales are written.
int softmax_cast_rows(const float* S, int64_t rows, int64_t cols, int64_t ld_s, float alpha, uint8_t* codes,
                      uint8_t* scales, void* pos, void* neg, uint8_t* sf_pos, uint8_t* sf_neg, int* row_exp, int nk64,
                      int64_t padded_rows, cudaStream_t st, int causal) {
    const int64_t G = cols / 32, blocks = pos ? padded_rows : rows;
    if (blocks > 0x7FFFFFFF || G > 0x7FFFFFFF / 32) return AMX_ERR_SHAPE;
    const int vec = aligned(S, 16) && ld_s % 4 == 0;
    auto* kernel = G <= softmax::kT ? softmax_cast_kernel<true> : softmax_cast_kernel<false>;
    kernel<<<(unsigned)blocks, softmax::kT, 0, st>>>(S, rows, (int)G, ld_s, alpha, vec, causal, reinterpret_cast<uint4*>(codes),
                                                     reinterpret_cast<uint16_t*>(scales), reinterpret_cast<uint4*>(pos),
                                                     reinterpret_cast<uint4*>(neg), sf_pos, sf_neg, row_exp, nk64);
    return launch_status();
}

namespace {

template <int TPG>
int launch_cols(const void* x, int64_t R, int64_t C, int64_t ld, int gs, uint8_t* codes,
                uint8_t* scales, cudaStream_t st, int64_t batch = 1) {
    dim3 grid((unsigned)((C + kTC - 1) / kTC), (unsigned)((R + kTR - 1) / kTR), (unsigned)batch);
    if (grid.y > 65535 || batch > 65535) return AMX_ERR_SHAPE;
    quantize_cols_kernel<TPG><<<grid, kThreads, 0, st>>>(
        reinterpret_cast<const __nv_bfloat16*>(x), R, C, ld, reinterpret_cast<uint32_t*>(codes),
        reinterpret_cast<uint16_t*>(scales), gs);
    return launch_status();
}

}  // namespace

// amx_quantize_t with group size 32 on `batch` matrices [R, C] stored one after another (contiguous rows); the
// canonical outputs of their transposes follow one another too.
int quantize_cols_batched(const void* x, int64_t batch, int64_t R, int64_t C, uint8_t* codes, uint8_t* scales,
                          cudaStream_t st) {
    return launch_cols<4>(x, R, C, C, 32, codes, scales, st, batch);
}

}  // namespace amx

namespace amx {
namespace {
template <int FMT>
int launch_rows_gs(const void* x, int64_t rows, int64_t K, int64_t ld_x, int group_size, uint8_t* codes, uint8_t* scales,
                   cudaStream_t st) {
    if (group_size == K && !fixed_group_size(group_size)) {          // whole-row grouping
        if (rows > 0x7FFFFFFF) return AMX_ERR_SHAPE;
        quantize_whole_rows_kernel<FMT><<<(unsigned)rows, kThreads, 0, st>>>(
            reinterpret_cast<const uint4*>(x), K / 8, ld_x / 8, reinterpret_cast<uint32_t*>(codes),
            reinterpret_cast<uint16_t*>(scales));
        return launch_status();
    }
    switch (group_size) {
        case 16: return launch_rows<16, 1, FMT>(x, rows, K, ld_x, codes, scales, st);
        case 32: return launch_rows<32, 1, FMT>(x, rows, K, ld_x, codes, scales, st);
        case 64: return launch_rows<32, 2, FMT>(x, rows, K, ld_x, codes, scales, st);
        default: return launch_rows<32, 4, FMT>(x, rows, K, ld_x, codes, scales, st);
    }
}
}  // namespace
}  // namespace amx

extern "C" int amx_quantize(const void* x, int64_t rows, int64_t K, int64_t ld_x, int group_size,
                            uint8_t* codes, uint8_t* scales, void* stream) {
    return amx_quantize_fmt(x, rows, K, ld_x, group_size, AMX_FMT_AMXFP4, codes, scales, stream);
}

extern "C" int amx_quantize_fmt(const void* x, int64_t rows, int64_t K, int64_t ld_x, int group_size, int format,
                                uint8_t* codes, uint8_t* scales, void* stream) {
    using namespace amx;
    if (format < AMX_FMT_AMXFP4 || format > AMX_FMT_AMXFP4_POT_ROUND) return AMX_ERR_FLAGS;
    if (!valid_group_size(group_size, K) || rows < 0 || K <= 0 || K % group_size || K % 8 || ld_x < K)
        return AMX_ERR_SHAPE;
    if (rows == 0) return AMX_OK;
    if (!x || !codes || !scales) return AMX_ERR_NULL;
    const int code_align = fixed_group_size(group_size) ? (group_size == 16 ? 8 : 16) : 4;
    if (!aligned(x, 16) || ld_x % 8 || !aligned(codes, code_align) || !aligned(scales, 2)) return AMX_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (format == AMX_FMT_SYM_FP8) return launch_rows_gs<1>(x, rows, K, ld_x, group_size, codes, scales, st);
    if (format == AMX_FMT_MXFP4) return launch_rows_gs<2>(x, rows, K, ld_x, group_size, codes, scales, st);
    if (format == AMX_FMT_AMXFP4_POT) return launch_rows_gs<3>(x, rows, K, ld_x, group_size, codes, scales, st);
    if (format == AMX_FMT_MXFP4_POT_ROUND) return launch_rows_gs<4>(x, rows, K, ld_x, group_size, codes, scales, st);
    if (format == AMX_FMT_AMXFP4_POT_ROUND) return launch_rows_gs<5>(x, rows, K, ld_x, group_size, codes, scales, st);
    return launch_rows_gs<0>(x, rows, K, ld_x, group_size, codes, scales, st);
}

extern "C" int amx_quantize_t(const void* x, int64_t R, int64_t C, int64_t ld_x, int group_size,
                              uint8_t* codes, uint8_t* scales, void* stream) {
    using namespace amx;
    if (!fixed_group_size(group_size) || R < 0 || C < 0 || R % group_size || ld_x < C) return AMX_ERR_SHAPE;
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
