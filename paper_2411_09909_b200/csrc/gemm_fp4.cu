// AMXFP4 x AMXFP4 -> fp32 on the FP4 tensor-core pipe (tcgen05 block-scaled MMA, sm_100a).
//
// The format picks one of two group scales per ELEMENT (by the element's sign; arXiv 2411.09909,
// Section 4.3), while a block-scaled MMA operand has one scale per (row, K block).  So each decoded
// operand is written as the sum of two single-scale operands,
//     Ahat = S_p o A+  +  S_n o A-      (A+ / A- = the codes with the other sign's nibbles zeroed),
// and the product becomes four block-scaled FP4 MMAs accumulating into one TMEM tile:
//     Ahat What^T = A+ W+^T + A+ W-^T + A- W+^T + A- W-^T.
//
// Scales: the MMA takes UE4M3 scales, one per 16 elements.  An E5M2 scale has the same four
// significands but a wider exponent range, so every operand row gets a power-of-two offset that
// maps its largest scale to the top UE4M3 binade; scale * 2^-offset is written as UE4M3 (each
// 32-group's scale twice) and the fp32 accumulator is multiplied by 2^(offset_A[m] + offset_W[n])
// in the epilogue (exact).  Scales more than 14 binades below their row's largest scale do not fit
// and are flushed to zero: their groups contribute less than 2^-14 of the row's largest group.
//
// Persistent CTAs (one per SM) walk over 128 x 256 tiles of C; K blocks of 128 elements cycle through
// four 48 KB shared-memory stages:
//   warp 0   TMA producer: per stage one 3-D tile {A+, A-} and one {W+, W-} (64-byte swizzle),
//            completion on the stage's `full` mbarrier
//   warp 1   allocates TMEM; one lane issues the stage's MMAs (4 sign pairs x K steps of 64), then
//            commits to the stage's `empty` mbarrier
//   warps 2-9  (two groups of four, alternating K blocks) move each stage's scale factors shared -> registers -> tensor memory (tcgen05.st; this
//            keeps the copies off the in-order MMA queue) and arrive on the stage's `full` barrier; they follow only the
//            `full` barriers and so run ahead into the next tile
//   warps 10-17 epilogue: TMEM -> registers (double-buffered loads), power-of-two rescale, 32-byte fp32
//            stores.  While a tile's accumulator is read out the producer already prefetches the next
//            tile's stages, and the MMA issuer starts the next tile as soon as the columns the two tiles
//            share have been read (see "Tensor memory" below).
// A preparation kernel per operand derives the planes, the UE4M3 scale-factor
// blocks in the 128 x 4 interleaved layout the MMA reads, and the row offsets from the canonical
// codes and scales.  Every device-side wait is bounded.
#include <cuda_bf16.h>

#include <cstdlib>

#include "fp4_operand.cuh"
#include "gemm.cuh"
#include "tcgen05.cuh"

namespace amx {
namespace {

using namespace tc;
using namespace fp4;

constexpr int BM = 128, BN = 256;
constexpr int kSfGroups = 2, kSfWarps = 4 * kSfGroups, kEpilogueWarps = 8;
constexpr int kThreads = (2 + kSfWarps + kEpilogueWarps) * 32;
constexpr int kTmemCols = 512;
// Tensor memory.  Two fp32 accumulators of 256 columns are all 512 columns, and the block-scaled MMA reads its
// scale factors from tensor memory too.  So consecutive tiles of a CTA alternate between two accumulator windows
// that overlap: columns [0, 256) for its even tiles, [160, 416) for the odd ones; the scale factors of the K blocks
// in flight take the 96 columns from 416.  The epilogue reads the 96 shared columns of a finished tile first and
// releases them (`ovl_free`); the next tile's MMAs start then, while the other 160 columns are still being read
// and stored (`rest_free` guards their reuse by the tile after next).  Only the read of 96 of 256 columns stays
// between two tiles, instead of the whole drain.  (Tiles of 128 columns use [0, 128) and [160, 288): no overlap.)
constexpr int kAccWindow = 160;        // first column of the odd tiles' accumulator
constexpr uint32_t kTmemSf = 416;      // scale-factor columns
constexpr int kTmemSfCols = 96;

// Shared-memory stage geometry for a K block of BK = 128 elements (BK/2 = 64 bytes of codes per row and plane,
// 64-byte swizzle): 4 stages of 48 KB.  (K blocks of 256 elements in two 96 KB stages measured slower.)
// ONE_PLANE (BK = 128): a stage holds one plane of each operand, 8 stages of 24 KB.  For two operands in a symmetric
// format, whose one product per K step leaves the tensor pipe waiting for loads: twice as many K blocks in flight.
template <int BK_, bool ONE_PLANE = false>
struct Cfg {
    static constexpr int BK = BK_;
    static constexpr int kPlanes = ONE_PLANE ? 1 : 2;
    static constexpr int kRowBytes = BK / 2;
    static constexpr int kSteps = BK / 64;                            // MMAs (K = 64) per K block and sign pair
    static constexpr int kStages = ONE_PLANE ? 8 : 4;
    static constexpr int kTileA = BM * kRowBytes, kTileB = BN * kRowBytes;   // one plane
    static constexpr int kOffAp = 0, kOffAn = ONE_PLANE ? 0 : kTileA, kOffWp = kPlanes * kTileA,
                         kOffWn = kOffWp + (ONE_PLANE ? 0 : kTileB);
    static constexpr int kStageBytes = kPlanes * (kTileA + kTileB);   // {A+, A-} and {W+, W-}: one TMA each
    static constexpr int kSmemBytes = kStages * kStageBytes + 1024 + 2048 + 256;   // + alignment slack + Control
    // TMEM columns of one stage's scale factors: A planes (4 columns per K step), then W planes (8)
    static constexpr int kSfColsA = kPlanes * kSteps * 4, kSfCols = kSfColsA + kPlanes * kSteps * 8;
    // the scale factors of kSfSlots K blocks are in tensor memory at a time (fewer than shared-memory stages: the
    // scale-factor warps store block i once the MMAs of block i - kSfSlots are done, while block i - 1 is multiplied)
    static constexpr int kSfSlots = kTmemSfCols / kSfCols;
    static_assert(kSfSlots >= 2 && kSfSlots % kSfGroups == 0 && kSfSlots <= kStages, "scale-factor ring");
    static_assert(kAccWindow + BN <= (int)kTmemSf && kTmemSf + kSfSlots * kSfCols <= kTmemCols, "tensor memory map");
    static_assert(BK == 128, "stages are laid out for 128-element K blocks (64-byte rows, 64-byte swizzle)");
};
constexpr int kMaxStages = 8;

struct __align__(16) Control {
    uint64_t full[kMaxStages], empty[kMaxStages], accum_full;
    uint64_t ovl_free;              // the columns a finished tile shares with the next tile's accumulator have been read
    uint64_t rest_free[2];          // its other columns have been read ([i]: tiles with number % 2 == i)
    uint64_t sides_ready[2];        // the epilogue warps have written sides[i] for the CTA's tile number 2 k + i
    uint32_t tmem_base;
    volatile int abort;
    volatile int sides[2][8];       // per epilogue warp: which sign planes its share of the tile's rows uses
    alignas(16) int w_exp[2][BN];   // read as int4 in the epilogue
};
static_assert(sizeof(Control) <= 2048 + 256, "Control must fit its reserved space");

// K-major operand rows of 64 bytes with the 64-byte swizzle: groups of 8 rows are 512 B apart.
__device__ __forceinline__ uint64_t smem_desc_sw64(uint32_t addr) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | (1ull << 16) | ((uint64_t)(512 >> 4) << 32) | (1ull << 46) | (4ull << 61);
}

// Instruction descriptor, kind::mxf4nvf4 block-scaled: A and B E2M1 (format code 1), K-major,
// UE4M3 scale factors (bit 23 = 0), N >> 3 at bit 17, M >> 4 at bit 24, K = 64 (bit 31 = 0).
__host__ __device__ constexpr uint32_t instr_desc(int n) { return (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24); }

// ------------------------------------------------------------------------- preparation --
// One launch per operand; one block per 32 operand rows (rows beyond R, up to the padded row count,
// get zero scale factors so that padded tile rows multiply zero codes by a finite scale).
//   1. row words: a warp per row finds the largest exponent key kmax among the row's scales (kmax - 25 is the
//      power of two by which the row's UE4M3 scales understate the true ones) and which sides occur at all
//   2. sign planes: every nibble goes to the plane of its sign bit, zero in the other plane
//   3. scale factors of both planes in the layout the MMA reads:
//      [plane][row block of 128][K/64 block][512 B], byte (r%32)*16 + (r/32)*4 + (k16 % 4);
//      one scale per 16 elements, so each 32-group's scale is written twice
constexpr int kPrepRows = 8;
__global__ void __launch_bounds__(256)
prepare_operand_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ scales, int64_t R, int64_t K,
                       int nk64, uint4* __restrict__ pos, uint4* __restrict__ neg, uint8_t* __restrict__ sf_pos,
                       uint8_t* __restrict__ sf_neg, int* __restrict__ row_exp, int* __restrict__ flushed_total) {
    __shared__ int kmax_s[kPrepRows];
    __shared__ int unsplit_s[kPrepRows];
    const int64_t row0 = (int64_t)blockIdx.x * kPrepRows, G = K / 32;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int r = warp; r < kPrepRows; r += 8) {
        const int64_t row = row0 + r;
        int kmax = 0, sides = 0;
        uint32_t differ = 0;
        if (row < R) {
            const unsigned short* s2 = reinterpret_cast<const unsigned short*>(scales + row * G * 2);
            for (int64_t g = lane; g < G; g += 32) {
                const uint32_t v = __ldg(s2 + g);
                kmax = max(kmax, max(scale_key(v & 0xFF), scale_key(v >> 8)));
                sides |= side_bits_of(v);
                differ |= (v & 0xFF) ^ (v >> 8);
            }
        }
        kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
        sides = __reduce_or_sync(0xFFFFFFFFu, sides);
        differ = __reduce_or_sync(0xFFFFFFFFu, differ);
        // A row whose two scales agree in every group (a symmetric format) needs no split: sum over both signs of
        // code x scale_side = code x scale.  Its signed codes go to the positive plane as they are.
        const bool unsplit = !differ;
        if (unsplit) sides &= kRowHasPos;
        // nonzero scales that the row's offset pushes below the UE4M3 range (they are flushed in step 3)
        int flushed = 0;
        if (row < R) {
            const unsigned short* s2 = reinterpret_cast<const unsigned short*>(scales + row * G * 2);
            for (int64_t g = lane; g < G; g += 32) {
                const uint32_t v = __ldg(s2 + g);
                flushed += (int)ue4m3_flushes(v & 0xFF, kmax) + (int)(!unsplit && ue4m3_flushes(v >> 8, kmax));
            }
        }
        flushed = __reduce_add_sync(0xFFFFFFFFu, flushed);
        if (lane == 0) {
            kmax_s[r] = kmax;
            unsplit_s[r] = unsplit;
            if (row < R) row_exp[row] = row_word(kmax, sides, flushed);
            if (flushed && flushed_total) atomicAdd(flushed_total, flushed);
        }
    }
    // sign planes of this block's rows (contiguous in memory: rows are K/2 bytes apart)
    __syncthreads();                                             // unsplit_s is complete
    const int64_t rows_here = min((int64_t)kPrepRows, R - row0);
    if (rows_here > 0) {
        const int64_t v0 = row0 * (K / 32), n_vec = rows_here * (K / 32);
        const uint4* src = reinterpret_cast<const uint4*>(codes) + v0;
        for (int64_t i = threadIdx.x; i < n_vec; i += 256) {
            const uint4 w = __ldg(src + i);
            const uint32_t v[4] = {w.x, w.y, w.z, w.w};
            const uint32_t keep = unsplit_s[(int)i / (int)G] ? 0u : 0xFFFFFFFFu;   // i < 8 rows x G: 32-bit division
            uint32_t p[4], n[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t m = ((v[j] >> 3) & 0x11111111u) * 15u & keep;   // 0xF on negative nibbles
                n[j] = v[j] & m;
                p[j] = v[j] & ~m;
            }
            pos[v0 + i] = make_uint4(p[0], p[1], p[2], p[3]);
            neg[v0 + i] = make_uint4(n[0], n[1], n[2], n[3]);
        }
    }
    __syncthreads();
    // scale factors: item = (K/64 block c, row r); consecutive threads take consecutive rows
    const int64_t rb = row0 / 128;
    const int r_in_blk0 = (int)(row0 % 128);
    for (int item = threadIdx.x; item < nk64 * kPrepRows; item += 256) {
        const int c = item / kPrepRows, r = item % kPrepRows;
        const int64_t row = row0 + r;
        uint32_t wp = 0, wn = 0;
        if (row < R) {
            const int kmax = kmax_s[r];
#pragma unroll
            for (int h = 0; h < 2; ++h) {                        // the two 32-groups of this 64-element block
                const int64_t g = (int64_t)c * 2 + h;
                if (g < G) {
                    const uint32_t v = __ldg(reinterpret_cast<const unsigned short*>(scales + (row * G + g) * 2));
                    const uint32_t up = to_ue4m3(v & 0xFF, kmax), un = unsplit_s[r] ? 0u : to_ue4m3(v >> 8, kmax);
                    wp |= (up | (up << 8)) << (16 * h);
                    wn |= (un | (un << 8)) << (16 * h);
                }
            }
        }
        const int rr = r_in_blk0 + r;                            // row inside its block of 128
        const int64_t off = (rb * nk64 + c) * (int64_t)kSfChunk + (rr % 32) * 16 + (rr / 32) * 4;
        *reinterpret_cast<uint32_t*>(sf_pos + off) = wp;
        *reinterpret_cast<uint32_t*>(sf_neg + off) = wn;
    }
}

// -------------------------------------------------------------------------------- GEMM --
struct Params {
    const uint8_t *sfa_pos, *sfa_neg, *sfb_pos, *sfb_neg;
    const int *a_exp, *w_exp;
    int64_t M, N, K, ld_c;
    int64_t a_row0, w_row0;      // first rows of this product's operands inside the (stacked) prepared operands

    float* C;
    int nk64, vec_store;
    int out_bf16;                // C holds bf16 (each fp32 result rounded to nearest even) instead of fp32
    int band;                    // tile order: row blocks of A per band, see blk_m / blk_n
    int slices;                  // SLICED instantiation: K is cut into this many ranges, each (tile, range) a work item
    int64_t slice_stride;        //   whose partial product goes to C + range * slice_stride
    int* status;
    const float *scale_a, *scale_w;   // not NULL: one fp32 factor per operand (the tensor scales of NVFP4 operands);
                                 // the store epilogue multiplies every result by their product
    const int* gate;             // not NULL: the kernel returns at once when this word is nonzero (the caller then
                                 // runs the exact bf16-decode kernel on the same operands, gated the other way)
};
// 16 consecutive fp32 results of one row -> global memory, as two 32-byte stores when allowed.
__device__ __forceinline__ void store_row16(float* out, const float (&f)[16], bool vec, int64_t n_left) {
    if (vec && n_left >= 16) {
#pragma unroll
        for (int j = 0; j < 16; j += 8)
            asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(out + j), "f"(f[j]), "f"(f[j + 1]),
                         "f"(f[j + 2]), "f"(f[j + 3]), "f"(f[j + 4]), "f"(f[j + 5]), "f"(f[j + 6]), "f"(f[j + 7]) : "memory");
    } else {
#pragma unroll
        for (int j = 0; j < 16; ++j)
            if (j < n_left) out[j] = f[j];
    }
}

// The same 16 results rounded to bf16 (nearest even): one 32-byte store.
__device__ __forceinline__ void store_row16_bf16(__nv_bfloat16* out, const float (&f)[16], bool vec, int64_t n_left) {
    if (vec && n_left >= 16) {
        uint32_t w[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * j], f[2 * j + 1]);
            w[j] = *reinterpret_cast<const uint32_t*>(&h);
        }
        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(out), "r"(w[0]), "r"(w[1]), "r"(w[2]),
                     "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]) : "memory");
    } else {
#pragma unroll
        for (int j = 0; j < 16; ++j)
            if (j < n_left) out[j] = __float2bfloat16_rn(f[j]);
    }
}

// NHALF: tiles of 128 x 128 for products with at most 128 columns: the W box, the MMA and the epilogue are half as
// wide, the stage layout keeps its size.
// ONE_PLANE: the caller states that neither operand has a second sign plane (Cfg above): only the first planes and
// their scale factors are read, one product per K step.  A tile whose row words show a second plane after all puts
// AMX_ERR_FLAGS into the status word (the kernel runs to its end; C is then not the product).
template <int BK_, bool SLICED = false, bool NHALF = false, bool ONE_PLANE = false>
__global__ void __launch_bounds__(kThreads, 1)
gemm_fp4_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_w,
                const __grid_constant__ CUtensorMap tm_a1, const __grid_constant__ CUtensorMap tm_w1, const Params p) {
    using C_ = Cfg<BK_, ONE_PLANE>;
    constexpr int kPlanes = C_::kPlanes;
    if (p.gate && *p.gate != 0) return;                          // uniform over the grid: nothing was set up yet
    constexpr int BNT = NHALF ? BN / 2 : BN;                     // tile width
    constexpr int kOffWnT = NHALF ? C_::kOffWp + C_::kTileB / 2 : C_::kOffWn;   // the box packs its two planes
    constexpr uint32_t kIdescT = instr_desc(BNT);
    constexpr int BK = C_::BK, kRowBytes = C_::kRowBytes, kSteps = C_::kSteps, kStages = C_::kStages;
    constexpr int kStageBytes = C_::kStageBytes;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Control* ctl = reinterpret_cast<Control*>(tiles + kStages * kStageBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Work items: tile x K range (one range unless SLICED); an item index is tile * S + range, num_kb the K blocks
    // of one item when there is one range.
    const int S = SLICED ? p.slices : 1;
    const int kb_total = (int)((p.K + BK - 1) / BK);
    const int num_kb = kb_total / S;                             // per item; SLICED: ranges differ by at most one block
    auto kb_begin = [&](int64_t tile) -> int { return SLICED ? (int)((int)(tile % S) * kb_total / S) : 0; };
    // Persistent CTA: tiles blockIdx.x, blockIdx.x + gridDim.x, ...; neighbouring tiles share their A rows.
    const int64_t n_tiles = (p.N + BNT - 1) / BNT, m_tiles = (p.M + BM - 1) / BM;
    const int64_t total_tiles = m_tiles * n_tiles * S;
    // Tile order.  The CTAs work on ~148 consecutive tiles at a time and advance through K roughly together, so what
    // they read from DRAM per wave is the operand rows the wave touches, once.  Tiles are ordered in bands of
    // p.band row blocks of A: inside a band the tile index walks down the band's row blocks first, then along N.
    // A wave then touches band x 128 rows of A and (148 / band) x 256 rows of W (with 16: 2048 + 2368 rows, near
    // the minimum), and consecutive waves of a band share its rows of A in L2.  Walking along N first, a wave of a
    // tall product touched a few row blocks of A and ALL of W: 3.6 GB of DRAM reads for 0.23 GB of operands at
    // 16384 x 10240 x 8192.  A band as tall as the matrix is the plain "down M first" order (small M).
    // (two 32-bit divisions per call: the host rejects products with 2^31 tiles or more)
    const uint32_t band = (uint32_t)p.band, per_band = band * (uint32_t)n_tiles;
    auto banded = [&](int64_t tile, uint32_t& m, uint32_t& n) {
        const uint32_t t = (uint32_t)tile / (uint32_t)S, b = t / per_band, r = t - b * per_band;
        const uint32_t rows_here = min(band, (uint32_t)m_tiles - b * band);      // the last band may be shorter
        n = r / rows_here;
        m = b * band + (r - n * rows_here);
    };
    auto blk_m = [&](int64_t tile) -> int64_t {
        uint32_t m, n;
        banded(tile, m, n);
        return m;
    };
    auto blk_n = [&](int64_t tile) -> int64_t {
        uint32_t m, n;
        banded(tile, m, n);
        return n;
    };
    // K blocks of a tile (of an item)
    auto nkb_of = [&](int64_t tile) -> int {
        if (SLICED) return (int)(((int)(tile % S) + 1) * kb_total / S) - kb_begin(tile);
        return num_kb;
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&ctl->full[s], 1 + 4);               // producer (with the TMA byte count) + four scale-factor warps
            mbar_init(&ctl->empty[s], 1);
        }
        mbar_init(&ctl->accum_full, 1);
        mbar_init(&ctl->ovl_free, kEpilogueWarps);
        mbar_init(&ctl->rest_free[0], kEpilogueWarps);
        mbar_init(&ctl->rest_free[1], kEpilogueWarps);
        mbar_init(&ctl->sides_ready[0], kEpilogueWarps);
        mbar_init(&ctl->sides_ready[1], kEpilogueWarps);
        ctl->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&ctl->tmem_base, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ctl->tmem_base;

    // Which sign planes a tile's rows use at all (bits of the row words, OR-ed over the tile's 128 + 256 rows; each
    // lane its share, to be OR-ed over the warp): bit 0/1: A has +/-, bit 2/3: W has +/-.  The products with a plane
    // that is zero for the whole tile are not issued, and that plane is not even loaded: an operand in a symmetric
    // format, or the all-positive attention map, moves half the bytes.
    auto tile_sides = [&](int64_t tile) {
        int bits = 0;
        if (tile < total_tiles) {
            const int64_t m0 = blk_m(tile) * BM, n0 = blk_n(tile) * BNT;
#pragma unroll
            for (int i = 0; i < BM / 32; ++i)
                if (m0 + i * 32 + lane < p.M) bits |= (__ldg(p.a_exp + m0 + i * 32 + lane) >> 16) & 3;
#pragma unroll
            for (int i = 0; i < BNT / 32; ++i)
                if (n0 + i * 32 + lane < p.N) bits |= ((__ldg(p.w_exp + n0 + i * 32 + lane) >> 16) & 3) << 2;
        }
        return bits;
    };
    auto whole_sides = [&](int lane_bits) {                         // over the warp; an all-zero operand keeps one plane
        int sides = __reduce_or_sync(0xFFFFFFFFu, lane_bits);
        if (!(sides & 3)) sides |= 1;
        if (!(sides & 12)) sides |= 4;
        return sides;
    };

    if (warp == 0) {
        // -------------------------------------------------------------- TMA producer
        // Which planes of a tile are not zero comes from the epilogue warps, which read the tile's row words a tile
        // ahead anyway (sides[] in the control block): nothing on this lane's path but a barrier that has long
        // completed and eight shared-memory words.
        if (lane == 0) {
            constexpr int kTileWT = NHALF ? C_::kTileB / 2 : C_::kTileB;   // one plane of the W tile as loaded
            int it = 0, j = 0;                                   // K blocks issued so far over all tiles; tiles so far
            bool ok = true;
            for (int64_t tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++j) {
                int sides = 5;                                   // ONE_PLANE: the first plane of each operand, always
                if (!ONE_PLANE) {
                    if (!mbar_wait(&ctl->sides_ready[j & 1], (j >> 1) & 1, &ctl->abort, p.status)) break;
                    sides = 0;
#pragma unroll
                    for (int i = 0; i < 8; ++i) sides |= ctl->sides[j & 1][i];
                    if (!(sides & 3)) sides |= 1;                // as the MMA warp: an all-zero operand keeps one plane
                    if (!(sides & 12)) sides |= 4;
                }
                const int a_planes = sides & 3, w_planes = (sides >> 2) & 3;
                const uint32_t bytes = (a_planes == 3 ? 2 : 1) * C_::kTileA + (w_planes == 3 ? 2 : 1) * kTileWT;
                const int64_t m_blk = blk_m(tile), n_blk = blk_n(tile);
                const int kb0 = kb_begin(tile), nkb = nkb_of(tile);
                const int ya = (int)(p.a_row0 + m_blk * BM), yw = (int)(p.w_row0 + n_blk * BNT);
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % kStages;
                    if (it >= kStages && !mbar_wait(&ctl->empty[s], ((it / kStages) - 1) & 1, &ctl->abort, p.status)) {
                        ok = false;
                        break;
                    }
                    uint8_t* st = tiles + s * kStageBytes;
                    mbar_expect_tx(&ctl->full[s], bytes);
                    const int x = (kb0 + kb) * kRowBytes;
                    // one 3-D tile per operand: {row bytes, rows, both sign planes} - or the one plane that is not zero
                    if (a_planes == 3) tma_load_3d(st + C_::kOffAp, &tm_a, x, ya, 0, &ctl->full[s]);
                    else tma_load_3d(st + (a_planes == 2 ? C_::kOffAn : C_::kOffAp), &tm_a1, x, ya, a_planes == 2 ? 1 : 0, &ctl->full[s]);
                    if (w_planes == 3) tma_load_3d(st + C_::kOffWp, &tm_w, x, yw, 0, &ctl->full[s]);
                    else tma_load_3d(st + (w_planes == 2 ? kOffWnT : C_::kOffWp), &tm_w1, x, yw, w_planes == 2 ? 1 : 0, &ctl->full[s]);
                }
            }
            // after an abort: let the copies already in flight land before shared memory is released
            if (ctl->abort)
                for (int i = max(0, it - kStages); i < it; ++i)
                    for (uint32_t n = 0; n < kSpinLimit && !mbar_try_wait(&ctl->full[i % kStages], (i / kStages) & 1); ++n) {}
        }
    } else if (warp == 1) {
        // -------------------------------------------------------------- MMA issuer
        // The whole warp runs the loop (so that addresses and descriptors stay warp-uniform); one elected
        // lane issues.  All operand descriptors differ from the first stage's only in their 14-bit address
        // field (bytes >> 4); the per-plane and per-K-step offsets are compile-time constants.
        const uint64_t desc0 = smem_desc_sw64(smem_u32(tiles));
        int it = 0, t = 0;
        bool ok = true, ready = false;                           // ready: the next K block's barrier was seen complete
        // (the planes of a tile: tile_sides above; the words of the next tile are fetched while the current one runs)
        int sides_next = ONE_PLANE ? 0 : tile_sides(blockIdx.x);
        for (int64_t tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
            const int sides = ONE_PLANE ? 5 : whole_sides(sides_next);   // an all-zero operand: one product, which zeroes the tile
            if (!ONE_PLANE) sides_next = tile_sides(tile + gridDim.x);
            const int nkb = nkb_of(tile);
            const int n_mma = ((sides & 1) + ((sides >> 1) & 1)) * (((sides >> 2) & 1) + ((sides >> 3) & 1)) * kSteps;
            // this tile's accumulator window: the columns it shares with the previous tile's must have been read, and
            // so must the rest of the window's last use (tile t - 2).  Neither barrier can run a phase ahead of this
            // wait: its next completion needs this tile's own MMAs.
            const uint32_t acc = tmem + ((t & 1) ? kAccWindow : 0);
            if (t > 0) ok = mbar_wait(&ctl->ovl_free, (t - 1) & 1, &ctl->abort, p.status);
            if (t > 1 && ok) ok = mbar_wait(&ctl->rest_free[t & 1], ((t >> 1) - 1) & 1, &ctl->abort, p.status);
            tc_fence_after();
            uint32_t accumulate = 0;
            for (int kb = 0; kb < nkb && ok; ++kb, ++it) {
                const int s = it % kStages;
                // tiles landed (TMA byte count) and scale factors stored (four warp arrivals); usually already
                // seen by the poll that was slipped between the previous block's MMAs
                if (!ready) ok = mbar_wait(&ctl->full[s], (it / kStages) & 1, &ctl->abort, p.status);
                if (!ok) break;
                tc_fence_after();
                const uint64_t dstage = desc0 + (uint64_t)((s * kStageBytes) >> 4);
                const uint32_t sfa = tmem + kTmemSf + (it % C_::kSfSlots) * C_::kSfCols, sfb = sfa + C_::kSfColsA;
                const int s_next = (it + 1) % kStages;
                const uint32_t parity_next = ((it + 1) / kStages) & 1;
                uint32_t seen = 0;
                if (elect_one()) {
                    int idx = 0;                                 // MMAs issued so far in this K block
#pragma unroll
                    for (int pa = 0; pa < kPlanes; ++pa)
#pragma unroll
                        for (int pw = 0; pw < kPlanes; ++pw)
#pragma unroll
                            for (int kk = 0; kk < kSteps; ++kk) {   // 64 elements = 32 bytes along the swizzled row
                                if (((sides >> pa) & 1) && ((sides >> (2 + pw)) & 1)) {
                                    mma_fp4_block16(acc, dstage + (((pa ? C_::kOffAn : C_::kOffAp) + kk * 32) >> 4),
                                                    dstage + (((pw ? kOffWnT : C_::kOffWp) + kk * 32) >> 4), kIdescT,
                                                    sfa + (pa * kSteps + kk) * 4, sfb + (pw * kSteps + kk) * 8,
                                                    idx ? 1u : accumulate);
                                    // with two MMAs still to go (they keep the pipe busy meanwhile), look whether the
                                    // next K block is complete, so that its MMAs can follow without a wait
                                    if (idx == max(n_mma - 3, 0)) seen = mbar_try_wait(&ctl->full[s_next], parity_next);
                                    ++idx;
                                }
                            }
                    mma_commit(&ctl->empty[s]);
                }
                ready = __any_sync(0xFFFFFFFFu, seen) != 0;
                accumulate = 1;
            }
            if (ok && elect_one()) mma_commit(&ctl->accum_full);
            __syncwarp();
            ++t;
        }
    } else if (warp < 2 + kSfWarps) {
        // -------------------------------------------------------------- scale factors
        // Warp w serves the 32-lane quarter w % 4 of tensor memory: every quarter has to hold a copy of
        // the scale-factor columns.  Per K block a lane reads 16 bytes of each 512-byte scale-factor block
        // straight from global memory (the 4-byte scale words of rows lane, lane+32, lane+64, lane+96) and
        // stores them to its quarter with tcgen05.st.  The values for the group's next K block are fetched
        // before the wait for the TMEM buffer, so the global latency stays off the critical path, and the
        // scale factors are normally in place before the TMA tiles of the same stage land.
        // Two groups of four warps take alternate K blocks.
        const int q = warp & 3, group = (warp - 2) >> 2;
        constexpr int kBlocks = kPlanes * kSteps * 3;                  // per K block: A (1) + W (2 row blocks), x planes x steps
        uint4 sfv[kBlocks];
        auto fetch = [&](int64_t tile, int kb) {
            const int64_t m_blk = blk_m(tile), n_blk = blk_n(tile);
#pragma unroll
            for (int pl = 0; pl < kPlanes; ++pl)
#pragma unroll
                for (int kk = 0; kk < kSteps; ++kk) {
                    const int64_t c = ((int64_t)kb_begin(tile) + kb) * kSteps + kk;
                    const uint8_t* a = (pl ? p.sfa_neg : p.sfa_pos) + (m_blk * p.nk64 + c) * kSfChunk + lane * 16;
                    const uint8_t* w = (pl ? p.sfb_neg : p.sfb_pos) + (n_blk * (BNT / 128) * p.nk64 + c) * kSfChunk + lane * 16;
                    sfv[(pl * kSteps + kk) * 3 + 0] = __ldg(reinterpret_cast<const uint4*>(a));
                    sfv[(pl * kSteps + kk) * 3 + 1] = __ldg(reinterpret_cast<const uint4*>(w));
                    sfv[(pl * kSteps + kk) * 3 + 2] =           // second block of 128 rows (none in a half-width tile)
                        __ldg(reinterpret_cast<const uint4*>(w + (NHALF ? 0 : (int64_t)p.nk64 * kSfChunk)));
                }
        };
        // this group's K blocks, in order, over all tiles: (tile, kb) with global index it = group, group + 2, ...
        int64_t tile = blockIdx.x;
        int kb = group;
        while (tile < total_tiles && kb >= nkb_of(tile)) { kb -= nkb_of(tile); tile += gridDim.x; }
        int it = group;
        bool ok = true;
        if (tile < total_tiles) fetch(tile, kb);
        while (tile < total_tiles && ok) {
            const int s = it % kStages;
            // the slot of the scale-factor ring is free once the MMAs of K block it - kSfSlots are done (the `empty`
            // barrier of that block's stage; it cannot complete again before this block's factors are stored)
            if (it >= C_::kSfSlots) {
                const int j = it - C_::kSfSlots;
                ok = mbar_wait(&ctl->empty[j % kStages], (j / kStages) & 1, &ctl->abort, p.status);
            }
            if (!ok) break;
            tc_fence_after();
            const uint32_t sfa = tmem + ((uint32_t)(q * 32) << 16) + kTmemSf + (it % C_::kSfSlots) * C_::kSfCols, sfb = sfa + C_::kSfColsA;
#pragma unroll
            for (int i = 0; i < kPlanes * kSteps; ++i) {
                tmem_st4(sfa + i * 4, sfv[i * 3].x, sfv[i * 3].y, sfv[i * 3].z, sfv[i * 3].w);
                tmem_st4(sfb + i * 8, sfv[i * 3 + 1].x, sfv[i * 3 + 1].y, sfv[i * 3 + 1].z, sfv[i * 3 + 1].w);
                tmem_st4(sfb + i * 8 + 4, sfv[i * 3 + 2].x, sfv[i * 3 + 2].y, sfv[i * 3 + 2].z, sfv[i * 3 + 2].w);
            }
            // next K block of this group
            it += kSfGroups;
            kb += kSfGroups;
            while (tile < total_tiles && kb >= nkb_of(tile)) { kb -= nkb_of(tile); tile += gridDim.x; }
            if (tile < total_tiles) fetch(tile, kb);             // in flight during the wait below
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl->full[s]);
        }
    } else {
        // -------------------------------------------------------------- epilogue
        // Eight warps: quarter q = warp % 4 of the lanes (= rows), one half of the columns each.
        const int e = warp - (2 + kSfWarps);                     // 0..7
        const int q = warp & 3;
        constexpr int kOvl = BNT > kAccWindow ? BNT - kAccWindow : 0;        // columns two consecutive tiles share
        constexpr int kC1 = kOvl / 2 / 16, kC2 = (BNT - kOvl) / 2 / 16;       // this warp's chunks of either part
        static_assert(kOvl % 32 == 0 && (BNT - kOvl) % 32 == 0, "both parts split into two halves of 16-column chunks");
        const int tid_e = threadIdx.x - (2 + kSfWarps) * 32;
        int t = 0;
        bool ok = true;
        static_assert(kEpilogueWarps * 32 == BN, "one column offset per epilogue thread");   // BNT <= BN
        // The per-tile constants (this thread's column offset and row offset) are fetched one tile ahead, so that
        // their latency is off the path between two tiles.
        struct TileConsts {
            int w_ex, a_ex, planes;     // planes: bit 0/1 this thread's row of A has +/-, bit 2/3 its row of W has
        };
        auto load_consts = [&](int64_t tl) {
            TileConsts c = {0, 0, 0};
            if (tl < total_tiles) {
                const int64_t n = blk_n(tl) * BNT + tid_e, mm = blk_m(tl) * BM + q * 32 + lane;
                if (tid_e < BNT && n < p.N) {
                    const int w = __ldg(p.w_exp + n);
                    c.w_ex = row_word_exp(w);
                    c.planes |= ((w >> 16) & 3) << 2;
                }
                if (mm < p.M) {
                    const int w = __ldg(p.a_exp + mm);
                    c.a_ex = row_word_exp(w);
                    c.planes |= (w >> 16) & 3;
                }
            }
            return c;
        };
        // The eight warps' row words cover the tile's 128 + 256 rows: each tells the producer which planes its rows
        // use (tile number j of this CTA); the producer reads them before the tile's first load.
        auto publish = [&](const TileConsts& c, int64_t tl, int j) {
            if (tl >= total_tiles) return;
            const int bits = __reduce_or_sync(0xFFFFFFFFu, c.planes);
            if (ONE_PLANE) {                                     // nobody waits for the planes; a second one is an error
                if (lane == 0 && (bits & 10)) atomicExch(p.status, (int)AMX_ERR_FLAGS);
                return;
            }
            if (lane == 0) {
                ctl->sides[j & 1][e] = bits;
                mbar_arrive(&ctl->sides_ready[j & 1]);
            }
        };
        const float out_scale = p.scale_a ? __ldg(p.scale_a) * __ldg(p.scale_w) : 1.0f;
        int64_t tile = blockIdx.x;
        TileConsts nxt = load_consts(tile);
        publish(nxt, tile, 0);
        while (tile < total_tiles && ok) {
            const TileConsts cur = nxt;
            const int64_t tile_after = tile + gridDim.x;
            nxt = load_consts(tile_after);                       // in flight while this tile is worked on
            publish(nxt, tile_after, t + 1);
            const int64_t m0 = blk_m(tile) * BM, n0 = blk_n(tile) * BNT;
            float* const C_item = p.C + (SLICED ? (tile % S) * p.slice_stride : 0);
            int* w_exp = ctl->w_exp[t & 1];
            w_exp[tid_e] = cur.w_ex;
            const int64_t m = m0 + q * 32 + lane;
            const int a_exp = cur.a_ex;
            ok = mbar_wait(&ctl->accum_full, t & 1, &ctl->abort, p.status);
            tc_fence_after();
            // every epilogue warp has written its part of w_exp (named barrier: the other roles do not join)
            asm volatile("bar.sync 1, %0;" ::"n"(kEpilogueWarps * 32) : "memory");
            if (ok) {
                // The tile's window starts at column 0 (even t) or kAccWindow (odd t).  The kOvl columns it shares with
                // the next tile's window - its last ones when even, its first ones when odd - are read first; this warp
                // takes its half h of both parts, kC1 + kC2 chunks of 16 columns.
                const int h = e >> 2, odd = t & 1;
                const int o1 = odd ? 0 : BNT - kOvl, o2 = odd ? kOvl : 0;
                auto chunk_col = [&](int i) {                    // first column (inside the tile) of this warp's chunk i
                    return i < kC1 ? o1 + h * (kOvl / 2) + 16 * i : o2 + h * ((BNT - kOvl) / 2) + 16 * (i - kC1);
                };
                const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(odd ? kAccWindow : 0);
                uint32_t v[2][16];
                if (kC1 == 0) {                                  // nothing shared: the next tile may start at once
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ctl->ovl_free);
                }
                tmem_ld16(taddr + chunk_col(0), v[0]);
#pragma unroll
                for (int i = 0; i < kC1 + kC2; ++i) {
                    const int buf = i & 1;
                    tmem_ld_wait();
                    if (i + 1 == kC1) {                          // the shared columns are in registers
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&ctl->ovl_free);
                    }
                    if (i + 1 == kC1 + kC2) {                    // so is the rest: tile t + 2 may overwrite the window
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&ctl->rest_free[odd]);
                    }
                    if (i + 1 < kC1 + kC2) tmem_ld16(taddr + chunk_col(i + 1), v[buf ^ 1]);   // loads while this chunk is stored
                    const int col = chunk_col(i);
                    float f[16];
#pragma unroll
                    for (int j = 0; j < 16; j += 4) {
                        const int4 we = *reinterpret_cast<const int4*>(&w_exp[col + j]);
                        const int ex[4] = {we.x, we.y, we.z, we.w};
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const int sh = min(127, max(-126, a_exp + ex[k]));
                            f[j + k] = __uint_as_float(v[buf][j + k]) * __uint_as_float((uint32_t)(sh + 127) << 23) * out_scale;
                        }
                    }
                    if (m < p.M) {
                        if (p.out_bf16)
                            store_row16_bf16(reinterpret_cast<__nv_bfloat16*>(C_item) + m * p.ld_c + n0 + col, f, p.vec_store != 0,
                                             p.N - (n0 + col));
                        else
                            store_row16(C_item + m * p.ld_c + n0 + col, f, p.vec_store != 0, p.N - (n0 + col));
                    }
                }
            }
            ++t;
            tile = tile_after;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

// ---------------------------------------------------------------------------------- host --
int prepare(const uint8_t* codes, const uint8_t* scales, int64_t rows, int64_t K, const OperandLayout& o,
            uint8_t* base, cudaStream_t st, int* flushed_total = nullptr) {
    const int64_t padded_rows = o.row_blocks * 128;
    prepare_operand_kernel<<<(unsigned)(padded_rows / kPrepRows), 256, 0, st>>>(
        codes, scales, rows, K, o.nk64, reinterpret_cast<uint4*>(base), reinterpret_cast<uint4*>(base + o.plane),
        base + 2 * o.plane, base + 2 * o.plane + o.sf, reinterpret_cast<int*>(base + 2 * o.plane + 2 * o.sf),
        flushed_total);
    return launch_status();
}

}  // namespace

bool gemm_fp4_supported(int64_t M, int64_t N, int64_t K, int gs) {
    return gs == 32 && M > 0 && N > 0 && K > 0 && K % 32 == 0 && (M + BM - 1) / BM <= 65535 &&
           M < (1ll << 31) && N < (1ll << 31) && K < (1ll << 31);
}

size_t gemm_fp4_workspace_bytes(int64_t M, int64_t N, int64_t K) {
    return 256 + operand_layout(M, K, BM).total + operand_layout(N, K, BN).total;
}

namespace {

template <int BK_, bool SLICED = false, bool NHALF = false, bool ONE_PLANE = false>
int launch_fp4(const uint8_t* pa, const uint8_t* pw, const OperandLayout& oa, const OperandLayout& ow, int64_t a_rows,
               int64_t w_rows, Params p, int dev, cudaStream_t st) {
    using C_ = Cfg<BK_, ONE_PLANE>;
    constexpr int BNT = NHALF ? BN / 2 : BN;
    static bool configured[64] = {};
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(gemm_fp4_kernel<BK_, SLICED, NHALF, ONE_PLANE>, cudaFuncAttributeMaxDynamicSharedMemorySize, C_::kSmemBytes) != cudaSuccess)
            return AMX_ERR_CUDA;
        configured[dev] = true;
    }
    CUtensorMap tm_a, tm_w, tm_a1, tm_w1;                       // both planes of a tile in one box, and one plane alone
    if (!make_map(&tm_a, pa, a_rows, p.K, oa.plane, BM, C_::kRowBytes) || !make_map(&tm_w, pw, w_rows, p.K, ow.plane, BNT, C_::kRowBytes) ||
        !make_map(&tm_a1, pa, a_rows, p.K, oa.plane, BM, C_::kRowBytes, 1) ||
        !make_map(&tm_w1, pw, w_rows, p.K, ow.plane, BNT, C_::kRowBytes, 1))
        return AMX_ERR_CUDA;
    static int sm_count[64] = {};
    if (!sm_count[dev] && cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return AMX_ERR_CUDA;
    const int64_t tiles = ((p.N + BNT - 1) / BNT) * ((p.M + BM - 1) / BM) * (SLICED ? p.slices : 1);
    const unsigned grid = (unsigned)(tiles < sm_count[dev] ? tiles : sm_count[dev]);   // one persistent CTA per SM
    gemm_fp4_kernel<BK_, SLICED, NHALF, ONE_PLANE><<<grid, kThreads, C_::kSmemBytes, st>>>(tm_a, tm_w, tm_a1, tm_w1, p);
    return launch_status();
}

}  // namespace

namespace {
// Kernel parameters for the product of row ranges of two prepared operands.
int fill_params(const Fp4Operand& a, const Fp4Operand& w, int64_t M, int64_t N, int64_t K, float* C, int64_t ld_c,
                void* workspace, cudaStream_t st, Params& p, OperandLayout& oa, OperandLayout& ow, int& dev) {
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return AMX_ERR_CUDA;
    if (a.row0 % 128 || w.row0 % 128) return AMX_ERR_SHAPE;
    if (((M + BM - 1) / BM) * ((N + BN - 1) / BN) >= (1ll << 27)) return AMX_ERR_SHAPE;   // tile indices are 32-bit
    oa = operand_layout(a.layout_rows, K, BM);
    ow = operand_layout(w.layout_rows, K, BN);
    const uint8_t* pa = static_cast<const uint8_t*>(a.prepared);
    const uint8_t* pw = static_cast<const uint8_t*>(w.prepared);
    int* status = static_cast<int*>(workspace);
    if (cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return AMX_ERR_CUDA;
    p = Params{};
    // scale factors come in chunks per 128 rows, row words per row: the range starts at a pointer offset
    const size_t a_sf0 = (size_t)(a.row0 / 128) * oa.nk64 * kSfChunk, w_sf0 = (size_t)(w.row0 / 128) * ow.nk64 * kSfChunk;
    p.sfa_pos = pa + 2 * oa.plane + a_sf0;
    p.sfa_neg = p.sfa_pos + oa.sf;
    p.a_exp = reinterpret_cast<const int*>(pa + 2 * oa.plane + 2 * oa.sf) + a.row0;
    p.sfb_pos = pw + 2 * ow.plane + w_sf0;
    p.sfb_neg = p.sfb_pos + ow.sf;
    p.w_exp = reinterpret_cast<const int*>(pw + 2 * ow.plane + 2 * ow.sf) + w.row0;
    p.M = M; p.N = N; p.K = K; p.ld_c = ld_c; p.C = C;
    p.a_row0 = a.row0; p.w_row0 = w.row0;
    p.nk64 = oa.nk64;
    p.vec_store = C && aligned(C, 32) && ld_c % 8 == 0;     // 32-byte stores in the epilogue
    p.status = status;
    {
        const char* e = getenv("AMX_FP4_BAND");              // row blocks of A per band of the tile order (default 16)
        const int64_t want = e && atoi(e) > 0 ? atoi(e) : 16, m_tiles = (M + BM - 1) / BM;
        p.band = (int)(want < m_tiles ? want : m_tiles);
    }
    return AMX_OK;
}

}  // namespace

// Few output tiles and a long K (a few token rows against a big weight): K ranges as separate work items, so
// that more SMs stream the operands; their partial products go to the workspace and are added in range order.
// Returns the number of ranges (1: none); ranges hold the same number of 128-element K blocks up to one.
int gemm_fp4_slices(int64_t M, int64_t N, int64_t K) {
    const int64_t tiles = ((N + BN - 1) / BN) * ((M + BM - 1) / BM);
    const int num_kb = (int)((K + 127) / 128);
    int s = (int)(148 / tiles);
    if (s > num_kb / 6) s = num_kb / 6;                  // at least six K blocks per range
    if (s > 8) s = 8;
    return s < 2 ? 1 : s;
}
size_t gemm_fp4_prepared_workspace_bytes(int64_t M, int64_t N, int64_t K) {
    const int s = gemm_fp4_slices(M, N, K);
    return 256 + (s > 1 ? (size_t)s * M * N * 4 : 0);
}

// The GEMM proper on two prepared operands (each laid out by operand_layout()), or on row ranges of them.
// workspace_bytes >= gemm_fp4_prepared_workspace_bytes() enables the K ranges; 256 bytes always suffice.
int gemm_fp4_prepared_at(const Fp4Operand& a, const Fp4Operand& w, int64_t M, int64_t N, int64_t K, float* C,
                         int64_t ld_c, void* workspace, cudaStream_t st, size_t workspace_bytes, const int* gate,
                         const float* scale_a, const float* scale_w, bool one_plane, bool out_bf16) {
    Params p;
    OperandLayout oa, ow;
    int dev;
    const int rc = fill_params(a, w, M, N, K, C, ld_c, workspace, st, p, oa, ow, dev);
    if (rc != AMX_OK) return rc;
    p.gate = gate;
    p.scale_a = scale_a;
    p.scale_w = scale_w;
    if (out_bf16) {                                         // 32-byte stores hold 16 results
        p.out_bf16 = 1;
        p.vec_store = aligned(C, 32) && ld_c % 16 == 0;
    }
    const uint8_t* pa = static_cast<const uint8_t*>(a.prepared);
    const uint8_t* pw = static_cast<const uint8_t*>(w.prepared);
    const int slices = gemm_fp4_slices(M, N, K);
    // at most 128 columns: tiles of 128 x 128, so that no half of a W tile is padding
    const bool half = N <= BN / 2 && !getenv("AMX_FP4_NO_HALF_TILE");
    if (!gate && !scale_a && !out_bf16 && slices > 1 && workspace_bytes >= gemm_fp4_prepared_workspace_bytes(M, N, K)) {
        float* part = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + 256);
        p.C = part;
        p.ld_c = N;
        p.vec_store = N % 8 == 0;
        p.slices = slices;
        p.slice_stride = M * N;
        const int r2 = launch_fp4<128, true>(pa, pw, oa, ow, a.rows_total, w.rows_total, p, dev, st);
        return r2 != AMX_OK ? r2 : reduce_slices(part, slices, M, N, C, ld_c, st);
    }
    // both operands stated to be single planes: the deeper pipeline (full-width tiles; the other shapes are short
    // products, where the depth does not matter, and run the general kernel, which skips absent planes by itself)
    if (one_plane && !half) return launch_fp4<128, false, false, true>(pa, pw, oa, ow, a.rows_total, w.rows_total, p, dev, st);
    return half ? launch_fp4<128, false, true>(pa, pw, oa, ow, a.rows_total, w.rows_total, p, dev, st)
                : launch_fp4<128>(pa, pw, oa, ow, a.rows_total, w.rows_total, p, dev, st);
}

int gemm_fp4_prepared(const void* a_prepared, const void* w_prepared, int64_t M, int64_t N, int64_t K, float* C,
                      int64_t ld_c, void* workspace, cudaStream_t st, size_t workspace_bytes, const int* gate) {
    return gemm_fp4_prepared_at({a_prepared, M, M, 0}, {w_prepared, N, N, 0}, M, N, K, C, ld_c, workspace, st,
                                workspace_bytes, gate);
}

// Size of a prepared operand: as the A operand (rows padded to 128) or the W operand (rows padded to 256).
size_t gemm_fp4_prepared_bytes(int64_t rows, int64_t K, bool is_weight) {
    return operand_layout(rows, K, is_weight ? BN : BM).total;
}

// Fused form: one launch of the cast kernel writes the canonical operand and the prepared one.
int gemm_fp4_quantize_prepared(const void* x, int64_t rows, int64_t K, bool is_weight, uint8_t* codes, uint8_t* scales,
                               void* prepared, cudaStream_t st, int64_t layout_rows, int format, int* flushed_total) {
    const OperandLayout o = operand_layout(layout_rows ? layout_rows : rows, K, is_weight ? BN : BM);
    uint8_t* base = static_cast<uint8_t*>(prepared);
    return quantize_rows_prepared(x, rows, K, codes, scales, base, base + o.plane, base + 2 * o.plane,
                                  base + 2 * o.plane + o.sf, reinterpret_cast<int*>(base + 2 * o.plane + 2 * o.sf), o.nk64,
                                  o.row_blocks * 128, st, format, flushed_total);
}

// Row words of a prepared operand (rows of them, device memory).
const int* gemm_fp4_row_words(const void* prepared, int64_t rows, int64_t K, bool is_weight) {
    const OperandLayout o = operand_layout(rows, K, is_weight ? BN : BM);
    return reinterpret_cast<const int*>(static_cast<const uint8_t*>(prepared) + 2 * o.plane + 2 * o.sf);
}

int gemm_fp4_softmax_prepared(const float* S, int64_t rows, int64_t cols, int64_t ld_s, float alpha, bool is_weight,
                              uint8_t* codes, uint8_t* scales, void* prepared, cudaStream_t st, int causal) {
    const OperandLayout o = operand_layout(rows, cols, is_weight ? BN : BM);
    uint8_t* base = static_cast<uint8_t*>(prepared);
    return softmax_cast_rows(S, rows, cols, ld_s, alpha, codes, scales, base, base + o.plane, base + 2 * o.plane,
                             base + 2 * o.plane + o.sf, reinterpret_cast<int*>(base + 2 * o.plane + 2 * o.sf), o.nk64,
                             o.row_blocks * 128, st, causal);
}

int gemm_fp4_prepare(const uint8_t* codes, const uint8_t* scales, int64_t rows, int64_t K, bool is_weight,
                     void* prepared, cudaStream_t st, int64_t layout_rows, int* flushed_total) {
    return prepare(codes, scales, rows, K, operand_layout(layout_rows ? layout_rows : rows, K, is_weight ? BN : BM),
                   static_cast<uint8_t*>(prepared), st, flushed_total);
}

// Workspace: word 0 the status, word 1 the number of scales flushed while preparing the two operands (see
// to_ue4m3), then the prepared operands.  gate_on_flushed: the GEMM kernel returns at once when that count is
// not zero (the caller follows with the exact kernel, gated the other way).
int gemm_fp4(const uint8_t* a_codes, const uint8_t* a_scales, const uint8_t* w_codes, const uint8_t* w_scales,
             int64_t M, int64_t N, int64_t K, float* C, int64_t ld_c, void* workspace, cudaStream_t st,
             bool gate_on_flushed) {
    const OperandLayout oa = operand_layout(M, K, BM), ow = operand_layout(N, K, BN);
    uint8_t* base = static_cast<uint8_t*>(workspace);
    uint8_t* pa = base + 256;
    uint8_t* pw = pa + oa.total;
    int* flushed = reinterpret_cast<int*>(base) + 1;
    if (cudaMemsetAsync(base, 0, 8, st) != cudaSuccess) return AMX_ERR_CUDA;
    int rc = prepare(a_codes, a_scales, M, K, oa, pa, st, flushed);
    if (rc == AMX_OK) rc = prepare(w_codes, w_scales, N, K, ow, pw, st, flushed);
    if (rc != AMX_OK) return rc;
    return gemm_fp4_prepared(pa, pw, M, N, K, C, ld_c, base, st, 256, gate_on_flushed ? flushed : nullptr);
}

}  // namespace amx
