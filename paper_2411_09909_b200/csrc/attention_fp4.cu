// Fully quantized attention on the FP4 tensor-core pipe for head dimension 128 (arXiv 2411.09909, Appendix C:
// Query, Key, the self-attention map and Value are all cast to AMXFP4; Section 1: at long context these products
// are a large share of the prefill work).  Neither the logits nor the attention map ever reach global memory.
//
// What is quantized is the NORMALISED map P = softmax(Q K^T / sqrt(d)), rounded to bf16, with groups of 32 along
// the keys.  Its scales depend on the final row maximum and sum, so the product Q K^T runs twice:
//   pass 1  S tiles -> per-row maximum and sum of exponentials (kept per thread over all key tiles of a row);
//   pass 2  S tiles again -> P tile = 2^(s - max) / sum, rounded to bf16 and cast to AMXFP4 in registers (P has no
//           negative element: one sign plane), written to shared memory in the layout the MMA reads, its scale
//           factors copied to tensor memory, and O += P V on the tensor cores in the same kernel.
// Both products use the sign split of the GEMM (gemm_fp4.cu): S = Q+K+ + Q+K- + Q-K+ + Q-K- (8 block-scaled MMAs
// per 128 x 128 tile at K = 128), O += P V+ + P V- (4 MMAs per tile of 128 keys).
//
// One persistent CTA per SM walks over (head, block of 128 queries) items; per item it loops over the key tiles:
//   warp 0      TMA: the item's Q tile; per key tile the K tile and (pass 2) the V^T tile, {+, -} planes each, into a
//               ring of kStages stages
//   warp 1      issues the MMAs two key tiles ahead: S(j+2) is issued before the wait for P(j), so the tensor cores
//               work on the next logits while the epilogue warps turn the current ones into P
//   warps 2-5   scale factors of Q, K, V^T: global -> registers -> tensor memory (tcgen05.st), and the per-key column
//               factors alpha * log2(e) * 2^(K row offset) of the tile
//   warps 6-21  epilogue, two groups of eight warps: group g takes the key tiles with (tile count) % 2 == g from the S
//               accumulator g, so the two groups are in different phases of their tiles (tensor-memory loads and
//               maxima in one, exponentials in the other) and keep both the issue slots and the special-function
//               unit busy; a thread owns one query row and 64 keys of its tiles: tensor memory -> registers (the
//               accumulator is released right after the loads), softmax arithmetic, the cast, stores to shared memory
//   after the last key tile of an item the epilogue warps read out O, rescale by the rows' powers of two and store.
// Tensor memory: S0, S1, O (128 columns each), scale factors of Q (16), of kStages K/V^T stages (32 each), of the
// two P tiles (8 each): 512 columns.  Every wait is bounded; on a timeout all roles run their loops out without
// work, tensor memory is released and the status word reports AMX_ERR_TIMEOUT.
#include <cuda_bf16.h>

#include "cast_math.cuh"
#include "fp4_operand.cuh"
#include "gemm.cuh"
#include "tcgen05.cuh"

namespace amx {
namespace {

using namespace tc;
using namespace fp4;

constexpr int BM = 128, BNK = 128, HD = 128;         // queries per item, keys per tile, head dimension
constexpr int kStages = 3;
// Ring of the per-tile column factors: its writers (scale-factor warps) run at most kStages tiles ahead of the MMAs
// and those at most 2 tiles ahead of the readers (epilogue), so 8 slots never collide and need no barrier of their own.
constexpr int kKcRing = 8;
constexpr int kSfWarps = 4, kEpiWarps = 16;
constexpr int kThreads = (2 + kSfWarps + kEpiWarps) * 32;
constexpr int kPlane = 128 * 64;                      // one sign plane of a 128 x 128 tile: 64-byte rows
constexpr int kTileBytes = 2 * kPlane;                // {+, -}
// tensor-memory columns
constexpr uint32_t kColS = 0, kColO = 256, kColSfQ = 384, kColSfKV = 400, kColSfP = 496, kTmemCols = 512;
static_assert(kColSfKV + kStages * 32 == kColSfP && kColSfP + 2 * 8 == kTmemCols, "tensor-memory budget");

struct __align__(16) Control {
    uint64_t q_full, q_empty, kv_full[kStages], kv_empty[kStages], s_full[2], s_empty[2], p_full[2], p_empty[2], o_full, o_empty;
    uint32_t tmem_base;
    volatile int abort;
};

// shared-memory layout (offsets from the 1024-aligned base)
template <int PASS>
struct Smem {
    static constexpr int kStageBytes = PASS == 2 ? 2 * kTileBytes : kTileBytes;   // K tile, then the V^T tile
    static constexpr int kOffQ = 0;
    static constexpr int kOffKV = kTileBytes;
    static constexpr int kOffP = kOffKV + kStages * kStageBytes;                  // two P planes (pass 2)
    static constexpr int kOffSfP = kOffP + (PASS == 2 ? 2 * kPlane : 0);          // two buffers x two 512-byte chunks
    static constexpr int kOffKc = kOffSfP + (PASS == 2 ? 2 * 2 * 512 : 0);        // per stage: 128 column factors
    static constexpr int kOffCtl = kOffKc + kKcRing * 512;
    static constexpr int kBytes = kOffCtl + 512 + 1024;                           // + Control + alignment slack
};
static_assert(sizeof(Control) <= 512, "Control must fit its reserved space");

// K-major operand rows of 64 bytes with the 64-byte swizzle: groups of 8 rows are 512 B apart.
__device__ __forceinline__ uint64_t desc_sw64(uint32_t addr) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | (1ull << 16) | ((uint64_t)(512 >> 4) << 32) | (1ull << 46) | (4ull << 61);
}
// kind::mxf4nvf4 block-scaled, A and B E2M1, K-major, UE4M3 scale factors, M = N = 128, K = 64 per instruction
constexpr uint32_t kIdesc = (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

struct Params {
    // prepared operands (fp4_operand.cuh); row ranges of stacked heads: head h of the launch has its queries at
    // rows q_row0 + h * L of Q, its keys at k_row0 + (h / kv_group) * L of K, its 128 V^T rows at
    // v_row0 + (h / kv_group) * 128 (kv_group query heads share one head of keys and values: grouped-query attention)
    const uint8_t *sfq[2], *sfk[2], *sfv[2];         // scale-factor chunks of the planes, from the operand's first chunk
    const int *q_words, *k_words, *v_words;          // row words, from the operand's first row
    int64_t q_row0, k_row0, v_row0;
    int nk64_q, nk64_k, nk64_v;
    int heads, m_tiles, causal, kv_group;
    int64_t L;
    float alpha;
    float2* part;            // [heads * L][4]: per row and key-group column {max, sum of 2^(t - max)}, base-2 units
    float* O;                // pass 2 out: [heads][L][128]
    int* status;
    // optional outputs of pass 2 for head 0 of the launch (verification): the bf16 map the cast started from
    // [L][L/2 words], canonical codes [L][L/32] x 16 bytes, scale bytes, and the prepared form of P (plane, scale
    // factors, row words)
    uint4 *p_bits, *p_codes, *p_plane;
    uint16_t* p_scales;
    uint8_t* p_sf;
    int* p_words;
    int p_nk64;
};

template <int PASS, bool CAUSAL>
__global__ void __launch_bounds__(kThreads, 1)
attention_fp4_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                     const __grid_constant__ CUtensorMap tm_v, const Params p) {
    using S_ = Smem<PASS>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Control* ctl = reinterpret_cast<Control*>(sm + S_::kOffCtl);
    float* kc_all = reinterpret_cast<float*>(sm + S_::kOffKc);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_items = p.heads * p.m_tiles;
    // item -> (head, query block); under a causal mask the long items (late query blocks) come first
    auto item_head = [&](int id) { return id % p.heads; };
    auto item_m = [&](int id) { const int mi = id / p.heads; return (CAUSAL && p.causal) ? p.m_tiles - 1 - mi : mi; };
    auto tiles_of = [&](int m_blk) { return (CAUSAL && p.causal) ? m_blk + 1 : (int)(p.L / BNK); };

    if (threadIdx.x == 0) {
        mbar_init(&ctl->q_full, 1 + kSfWarps);
        mbar_init(&ctl->q_empty, 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&ctl->kv_full[s], 1 + kSfWarps);
            mbar_init(&ctl->kv_empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&ctl->s_full[b], 1);
            mbar_init(&ctl->s_empty[b], kEpiWarps / 2);          // the accumulator's own epilogue group
            mbar_init(&ctl->p_full[b], kEpiWarps / 2);
            mbar_init(&ctl->p_empty[b], 1);
        }
        mbar_init(&ctl->o_full, 1);
        mbar_init(&ctl->o_empty, kEpiWarps);
        ctl->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&ctl->tmem_base, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ctl->tmem_base;

    if (warp == 0) {
        // ---------------------------------------------------------------------------------- TMA producer
        if (lane == 0) {
            int it = 0, ii = 0;
            bool ok = true;
            for (int id = blockIdx.x; id < n_items && ok; id += gridDim.x, ++ii) {
                const int h = item_head(id), m_blk = item_m(id);
                // the previous item's logits MMAs have read the Q tile
                if (ii > 0 && !mbar_wait(&ctl->q_empty, (ii - 1) & 1, &ctl->abort, p.status)) break;
                mbar_expect_tx(&ctl->q_full, kTileBytes);
                tma_load_3d(sm + S_::kOffQ, &tm_q, 0, (int)(p.q_row0 + (int64_t)h * p.L + m_blk * BM), 0, &ctl->q_full);
                const int T = tiles_of(m_blk);
                for (int j = 0; j < T; ++j, ++it) {
                    const int s = it % kStages;
                    if (it >= kStages && !mbar_wait(&ctl->kv_empty[s], ((it / kStages) - 1) & 1, &ctl->abort, p.status)) {
                        ok = false;
                        break;
                    }
                    uint8_t* st = sm + S_::kOffKV + s * S_::kStageBytes;
                    mbar_expect_tx(&ctl->kv_full[s], S_::kStageBytes);
                    tma_load_3d(st, &tm_k, 0, (int)(p.k_row0 + (int64_t)(h / p.kv_group) * p.L + j * BNK), 0, &ctl->kv_full[s]);
                    if (PASS == 2) tma_load_3d(st + kTileBytes, &tm_v, j * 64, (int)(p.v_row0 + (int64_t)(h / p.kv_group) * HD), 0, &ctl->kv_full[s]);
                }
            }
            // after a timeout: let the copies already in flight land before shared memory is released
            if (ctl->abort) {
                for (int i = max(0, it - kStages); i < it; ++i)
                    for (uint32_t n = 0; n < kSpinLimit && !mbar_try_wait(&ctl->kv_full[i % kStages], (i / kStages) & 1); ++n) {}
                if (ii > 0)
                    for (uint32_t n = 0; n < kSpinLimit && !mbar_try_wait(&ctl->q_full, (ii - 1) & 1); ++n) {}
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------------------------- MMA issuer
        // The whole warp runs the loops (addresses stay warp-uniform); one elected lane issues.
        const uint32_t base = smem_u32(sm);
        int it_s = 0, it_p = 0, ii = 0;
        bool ok = true;
        // logits of key tile number `it` (global count): S[it % 2] = Q K^T, four sign pairs x two K steps of 64
        auto issue_s = [&](int it) {
            const int s = it % kStages, b = it & 1;
            if (ok) ok = mbar_wait(&ctl->kv_full[s], (it / kStages) & 1, &ctl->abort, p.status);
            if (ok && it >= 2) ok = mbar_wait(&ctl->s_empty[b], ((it >> 1) - 1) & 1, &ctl->abort, p.status);
            if (!ok) return;
            tc_fence_after();
            if (elect_one()) {
                const uint32_t q_addr = base + S_::kOffQ, k_addr = base + S_::kOffKV + s * S_::kStageBytes;
                const uint32_t sfq = tmem + kColSfQ, sfk = tmem + kColSfKV + s * 32;
                uint32_t acc = 0;
#pragma unroll
                for (int pa = 0; pa < 2; ++pa)
#pragma unroll
                    for (int pw = 0; pw < 2; ++pw)
#pragma unroll
                        for (int kk = 0; kk < 2; ++kk) {
                            mma_fp4_block16(tmem + kColS + b * 128, desc_sw64(q_addr + pa * kPlane + kk * 32),
                                            desc_sw64(k_addr + pw * kPlane + kk * 32), kIdesc, sfq + (pa * 2 + kk) * 4,
                                            sfk + (pw * 2 + kk) * 4, acc);
                            acc = 1;
                        }
                mma_commit(&ctl->s_full[b]);
                if (PASS == 1) mma_commit(&ctl->kv_empty[s]);    // nothing else reads the stage
            }
            __syncwarp();
        };
        // O (+)= P V for key tile number `it`: P from the epilogue warps (shared memory + scale-factor chunks)
        auto issue_pv = [&](int it, bool first) {
            const int s = it % kStages, b = it & 1;
            if (ok) ok = mbar_wait(&ctl->p_full[b], (it >> 1) & 1, &ctl->abort, p.status);
            // the previous item's O has been read out before it is overwritten
            if (ok && first && ii > 0) ok = mbar_wait(&ctl->o_empty, (ii - 1) & 1, &ctl->abort, p.status);
            if (!ok) return;
            tc_fence_after();
            if (elect_one()) {
                const uint32_t p_addr = base + S_::kOffP + b * kPlane, v_addr = base + S_::kOffKV + s * S_::kStageBytes + kTileBytes;
                const uint32_t sfp = tmem + kColSfP + b * 8, sfv = tmem + kColSfKV + s * 32 + 16;
#pragma unroll
                for (int kk = 0; kk < 2; ++kk)
                    tmem_cp_32x128b_warpx4(sfp + kk * 4, smem_desc_rows16(base + S_::kOffSfP + (b * 2 + kk) * 512));
                uint32_t acc = first ? 0u : 1u;
#pragma unroll
                for (int pv = 0; pv < 2; ++pv)
#pragma unroll
                    for (int kk = 0; kk < 2; ++kk) {
                        mma_fp4_block16(tmem + kColO, desc_sw64(p_addr + kk * 32), desc_sw64(v_addr + pv * kPlane + kk * 32),
                                        kIdesc, sfp + kk * 4, sfv + (pv * 2 + kk) * 4, acc);
                        acc = 1;
                    }
                mma_commit(&ctl->kv_empty[s]);
                mma_commit(&ctl->p_empty[b]);
            }
            __syncwarp();
        };
        for (int id = blockIdx.x; id < n_items; id += gridDim.x, ++ii) {
            const int T = tiles_of(item_m(id));
            if (ok) ok = mbar_wait(&ctl->q_full, ii & 1, &ctl->abort, p.status);
            // the logits run two key tiles ahead of P V (both accumulators in use); after the item's last S the Q
            // tile is free for the next item
            auto next_s = [&](int j) {
                if (j < T) issue_s(it_s++);
                if (j == T - 1 && ok && elect_one()) mma_commit(&ctl->q_empty);
                __syncwarp();
            };
            next_s(0);
            next_s(1);
            for (int j = 0; j < T; ++j) {
                if (PASS == 2) issue_pv(it_p++, j == 0);
                next_s(j + 2);
            }
            if (PASS == 2 && ok && elect_one()) mma_commit(&ctl->o_full);
            __syncwarp();
        }
    } else if (warp < 2 + kSfWarps) {
        // ---------------------------------------------------------------------------------- scale factors
        // Warp w serves the 32-lane quarter w % 4 of tensor memory (every quarter holds a copy of the scale-factor
        // columns): a lane reads 16 bytes of each 512-byte chunk (the words of rows lane, lane + 32, + 64, + 96)
        // and stores them to its quarter.  Thread t of the four warps also stages the column factor of key t.
        const int q = warp & 3, t = (warp - 2) * 32 + lane;
        const uint32_t tq = tmem + ((uint32_t)(q * 32) << 16);
        int it = 0, ii = 0;
        bool ok = true;
        auto chunk = [&](const uint8_t* sf, int64_t row0, int nk64, int k64) {
            return __ldg(reinterpret_cast<const uint4*>(sf + ((row0 >> 7) * nk64 + k64) * (int64_t)kSfChunk + lane * 16));
        };
        for (int id = blockIdx.x; id < n_items; id += gridDim.x, ++ii) {
            const int h = item_head(id), m_blk = item_m(id);
            const int64_t q_row = p.q_row0 + (int64_t)h * p.L + m_blk * BM;
            uint4 v[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) v[i] = chunk(p.sfq[i >> 1], q_row, p.nk64_q, i & 1);
            if (ok && ii > 0) ok = mbar_wait(&ctl->q_empty, (ii - 1) & 1, &ctl->abort, p.status);
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int i = 0; i < 4; ++i) tmem_st4(tq + kColSfQ + i * 4, v[i].x, v[i].y, v[i].z, v[i].w);
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->q_full);
            }
            const int T = tiles_of(m_blk);
            for (int j = 0; j < T; ++j, ++it) {
                const int s = it % kStages;
                const int64_t k_row = p.k_row0 + (int64_t)(h / p.kv_group) * p.L + j * BNK;
                uint4 vk[4], vv[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) vk[i] = chunk(p.sfk[i >> 1], k_row, p.nk64_k, i & 1);
                if (PASS == 2) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) vv[i] = chunk(p.sfv[i >> 1], p.v_row0 + (int64_t)(h / p.kv_group) * HD, p.nk64_v, j * 2 + (i & 1));
                }
                const int kw = row_word_exp(__ldg(p.k_words + k_row + t));
                if (ok && it >= kStages) ok = mbar_wait(&ctl->kv_empty[s], ((it / kStages) - 1) & 1, &ctl->abort, p.status);
                if (!ok) continue;
                tc_fence_after();
                kc_all[(it % kKcRing) * 128 + t] = p.alpha * 1.4426950408889634f * __uint_as_float((uint32_t)(kw + 127) << 23);
#pragma unroll
                for (int i = 0; i < 4; ++i) tmem_st4(tq + kColSfKV + s * 32 + i * 4, vk[i].x, vk[i].y, vk[i].z, vk[i].w);
                if (PASS == 2) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) tmem_st4(tq + kColSfKV + s * 32 + 16 + i * 4, vv[i].x, vv[i].y, vv[i].z, vv[i].w);
                }
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->kv_full[s]);
            }
        }
    } else {
        // ---------------------------------------------------------------------------------- epilogue
        // Warp e: group g = e / 8 (the key tiles whose global count is g modulo 2, accumulator g), lane quarter
        // q = warp % 4 (its rows), half = (e / 4) % 2 of the tile's 128 keys: a thread owns one query row and two
        // 32-key groups (64 columns) of each of its group's tiles.  For reading out O every warp takes 32 columns.
        const int e = warp - (2 + kSfWarps), q = warp & 3, grp = e >> 3, half = (e >> 2) & 1, cg_o = e >> 2;
        const int r = q * 32 + lane;                                 // row inside the item = tensor-memory lane
        const uint32_t tq = tmem + ((uint32_t)(q * 32) << 16);
        int it = 0, ii = 0;
        bool ok = true;
        auto exp2_approx = [](float y) {
            float v;
            asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(v) : "f"(y));
            return v;
        };
        for (int id = blockIdx.x; id < n_items; id += gridDim.x, ++ii) {
            const int h = item_head(id), m_blk = item_m(id);
            const int64_t m = (int64_t)m_blk * BM + r;                // query index inside the head
            const int64_t grow = (int64_t)h * p.L + m;               // row of the launch's stacked heads
            const int a_exp = row_word_exp(__ldg(p.q_words + p.q_row0 + grow));
            const float ra = __uint_as_float((uint32_t)(a_exp + 127) << 23);
            // pass 2: the row's statistics, merged from the four partial results of pass 1 in a fixed order
            float neg_mx = 0.f, inv = 0.f;
            int kmax = 0;
            if (PASS == 2) {
                const float4* pp = reinterpret_cast<const float4*>(p.part + grow * 4);
                const float4 a = __ldg(pp), b = __ldg(pp + 1);       // {max0, sum0, max1, sum1}, {max2, sum2, max3, sum3}
                const float mx = fmaxf(fmaxf(a.x, a.z), fmaxf(b.x, b.z));
                float sum = a.y * exp2f(a.x - mx);
                sum += a.w * exp2f(a.z - mx);
                sum += b.y * exp2f(b.x - mx);
                sum += b.w * exp2f(b.z - mx);
                inv = 1.0f / sum;
                neg_mx = -mx;
                // the row's largest element is 2^0 / sum: its group has the row's largest scale
                float ip, in;
                const uint32_t sc = cast::group_scales((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(inv)), ip, in);
                kmax = scale_key(sc & 0xFFu);
                if (p.p_words && h == 0 && (e >> 2) == 0) p.p_words[m] = row_word(kmax, kRowHasPos);
            }
            float run_mx = -INFINITY, run_sum = 0.f;                  // pass 1: over this thread's columns of its tiles
            const int T = tiles_of(m_blk);
            for (int j = 0; j < T; ++j, ++it) {
                if ((it & 1) != grp) continue;                        // the other group's tile
                const int b = grp;
                if (ok) ok = mbar_wait(&ctl->s_full[b], (it >> 1) & 1, &ctl->abort, p.status);
                if (!ok) continue;
                tc_fence_after();
                // (the tile's column factors were stored before the scale-factor warps arrived on the stage's barrier,
                // which the MMA warp waited for before it issued what s_full reports as complete)
                if (PASS == 2 && it >= 2) {                           // the previous P in this buffer has been multiplied
                    ok = mbar_wait(&ctl->p_empty[b], ((it >> 1) - 1) & 1, &ctl->abort, p.status);
                    if (!ok) continue;
                }
                // u = accumulator x (alpha log2(e) 2^(K row offset)): the logit in base-2 units up to the query row's
                // power of two ra, by which multiplying is exact: t = u ra.  (Packed fp32 pairs: same roundings as the
                // scalar operations, half the instructions.)
                uint32_t acc[32];
                uint64_t u2[16];
                auto scale_columns = [&](int cg) {
                    const ulonglong2* kc2 = reinterpret_cast<const ulonglong2*>(kc_all + (it % kKcRing) * 128 + cg * 32);
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const ulonglong2 k2 = kc2[c];                 // four column factors
                        u2[2 * c] = cast::mul_f32x2(cast::pack_f32x2(acc[4 * c], acc[4 * c + 1]), k2.x);
                        u2[2 * c + 1] = cast::mul_f32x2(cast::pack_f32x2(acc[4 * c + 2], acc[4 * c + 3]), k2.y);
                    }
                    if (CAUSAL && p.causal && j == m_blk) {            // the diagonal tile: keys after the query are masked
                        const int n_local = (int)(m - (int64_t)j * BNK) - cg * 32;   // last visible column of this group
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            float lo, hi;
                            cast::unpack_f32x2(u2[c], lo, hi);
                            if (2 * c > n_local) lo = -INFINITY;
                            if (2 * c + 1 > n_local) hi = -INFINITY;
                            u2[c] = cast::pack_f32x2(__float_as_uint(lo), __float_as_uint(hi));
                        }
                    }
                };
                const uint64_t ra2 = cast::pack_f32x2(__float_as_uint(ra), __float_as_uint(ra));
                auto work = [&](int cg) {                             // one 32-key group, from u2
                    if (PASS == 1) {
                        float u[32];
#pragma unroll
                        for (int c = 0; c < 16; ++c) cast::unpack_f32x2(u2[c], u[2 * c], u[2 * c + 1]);
                        float c4[4] = {u[0], u[1], u[2], u[3]};
#pragma unroll
                        for (int c = 4; c < 32; ++c) c4[c & 3] = fmaxf(c4[c & 3], u[c]);
                        const float cm = fmaxf(fmaxf(c4[0], c4[1]), fmaxf(c4[2], c4[3]));
                        const float nmx = fmaxf(run_mx, cm * ra);
                        // 2^(-inf) = 0 on the first tile; a maximum still at -inf (everything masked so far) must
                        // not meet itself in a difference
                        const float ref = nmx == -INFINITY ? 0.f : nmx;
                        run_sum *= exp2_approx(run_mx - ref);
                        run_mx = nmx;
                        const uint64_t nref2 = cast::pack_f32x2(__float_as_uint(-ref), __float_as_uint(-ref));
                        float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            float t0, t1;
                            cast::unpack_f32x2(cast::fma_f32x2(u2[c], ra2, nref2), t0, t1);
                            s4[(2 * c) & 3] += exp2_approx(t0);
                            s4[(2 * c + 1) & 3] += exp2_approx(t1);
                        }
                        run_sum += (s4[0] + s4[1]) + (s4[2] + s4[3]);
                    } else {
                        // normalise, round to bf16, cast (P has no negative element: one plane)
                        const uint64_t nm2 = cast::pack_f32x2(__float_as_uint(neg_mx), __float_as_uint(neg_mx));
                        const uint64_t inv2 = cast::pack_f32x2(__float_as_uint(inv), __float_as_uint(inv));
                        uint32_t w[16];
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            float t0, t1, p0, p1;
                            cast::unpack_f32x2(cast::fma_f32x2(u2[c], ra2, nm2), t0, t1);
                            cast::unpack_f32x2(cast::mul_f32x2(cast::pack_f32x2(__float_as_uint(exp2_approx(t0)),
                                                                                __float_as_uint(exp2_approx(t1))), inv2), p0, p1);
                            const __nv_bfloat162 pr = __floats2bfloat162_rn(p0, p1);
                            w[c] = *reinterpret_cast<const uint32_t*>(&pr);
                        }
                        uint32_t nib[4];
                        const uint32_t sc = cast::cast_nonneg_group(w, nib);
                        const uint32_t up = to_ue4m3(sc, kmax);
                        // plane: row r, 16-byte piece cg of its 64 bytes, 64-byte swizzle; scale factors: chunk of the
                        // K step cg / 2, byte (r % 32) * 16 + (r / 32) * 4 + (cg % 2) * 2, each scale twice (blocks of 16)
                        *reinterpret_cast<uint4*>(sm + S_::kOffP + b * kPlane + r * 64 + ((cg ^ ((r >> 1) & 3)) << 4)) =
                            make_uint4(nib[0], nib[1], nib[2], nib[3]);
                        *reinterpret_cast<uint16_t*>(sm + S_::kOffSfP + (b * 2 + (cg >> 1)) * 512 + (r & 31) * 16 + (r >> 5) * 4 +
                                                     (cg & 1) * 2) = (uint16_t)(up | (up << 8));
                        if (p.p_plane && h == 0) {                    // verification outputs (head 0 of the launch)
                            const int64_t g = (int64_t)j * 4 + cg, v = m * (p.L / 32) + g;
                            p.p_plane[v] = make_uint4(nib[0], nib[1], nib[2], nib[3]);
                            *reinterpret_cast<uint16_t*>(p.p_sf + sf_row_offset(m, p.p_nk64) + sf_group_offset((int)g)) = (uint16_t)(up | (up << 8));
                            if (p.p_codes) p.p_codes[v] = make_uint4(nib[0], nib[1], nib[2], nib[3]);
                            if (p.p_scales) p.p_scales[v] = (uint16_t)sc;
                            if (p.p_bits) {
#pragma unroll
                                for (int c = 0; c < 4; ++c) p.p_bits[v * 4 + c] = make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
                            }
                        }
                    }
                };
                // the second group's tensor-memory load is in flight while the first group is worked on
                const int cg0 = half * 2;
                tmem_ld32(tq + kColS + b * 128 + cg0 * 32, acc);
                tmem_ld_wait();
                scale_columns(cg0);
                tmem_ld32(tq + kColS + b * 128 + (cg0 + 1) * 32, acc);
                work(cg0);
                tmem_ld_wait();
                tc_fence_before();                                    // both halves are in registers: release the accumulator
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->s_empty[b]);
                scale_columns(cg0 + 1);
                work(cg0 + 1);
                if (PASS == 2) {
                    fence_proxy_async();                              // visible to the tensor core's reads
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ctl->p_full[b]);
                }
            }
            if (PASS == 1) {
                if (ok) p.part[grow * 4 + grp * 2 + half] = make_float2(run_mx, run_sum);
            } else {
                // O of the item: rows x (32 columns of the head dimension per thread), rescaled by 2^(row offset of P
                // + row offset of V^T) - exact - and stored
                if (ok) ok = mbar_wait(&ctl->o_full, ii & 1, &ctl->abort, p.status);
                if (!ok) continue;
                tc_fence_after();
                uint32_t acc[32];
                tmem_ld32(tq + kColO + cg_o * 32, acc);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->o_empty);
                const int4* vw = reinterpret_cast<const int4*>(p.v_words + p.v_row0 + (int64_t)(h / p.kv_group) * HD + cg_o * 32);
                float* out = p.O + ((int64_t)h * p.L + m) * HD + cg_o * 32;
                const int p_exp = kmax ? kmax - 25 : 0;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const int4 w4 = __ldg(vw + c);
                    const int ex[4] = {row_word_exp(w4.x), row_word_exp(w4.y), row_word_exp(w4.z), row_word_exp(w4.w)};
                    float f[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int sh = min(127, max(-126, p_exp + ex[i]));
                        f[i] = __uint_as_float(acc[4 * c + i]) * __uint_as_float((uint32_t)(sh + 127) << 23);
                    }
                    *reinterpret_cast<float4*>(out + 4 * c) = make_float4(f[0], f[1], f[2], f[3]);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

template <int PASS, bool CAUSAL>
int launch_pass(const CUtensorMap& tm_q, const CUtensorMap& tm_k, const CUtensorMap& tm_v, const Params& p, int dev, int sms,
                cudaStream_t st) {
    static bool configured[64] = {};
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(attention_fp4_kernel<PASS, CAUSAL>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<PASS>::kBytes) !=
            cudaSuccess) {
            cudaGetLastError();
            return AMX_ERR_CUDA;
        }
        configured[dev] = true;
    }
    const int items = p.heads * p.m_tiles;
    attention_fp4_kernel<PASS, CAUSAL><<<(unsigned)(items < sms ? items : sms), kThreads, Smem<PASS>::kBytes, st>>>(tm_q, tm_k, tm_v, p);
    return launch_status();
}

}  // namespace

bool attn_fused_supported(int64_t L, int64_t d) { return d == HD && L > 0 && L % BNK == 0 && L / BNK <= 32767; }

// per-row partial softmax statistics of the heads of one launch
size_t attn_fused_scratch_bytes(int64_t heads, int64_t L) { return up256((size_t)heads * L * 4 * sizeof(float2)); }

// Attention for `heads` stacked heads whose operands were prepared ahead: q (left-hand layout, heads * L rows, K = 128),
// k (right-hand layout, same rows), vt (right-hand layout, heads * 128 rows of V^T, K = L).  O: fp32 [heads][L][128].
// workspace: 256 bytes (status word).  dbg_*: optional verification outputs for head 0 (see Params).
int attn_fused(const Fp4Operand& q, const Fp4Operand& k, const Fp4Operand& vt, int heads, int64_t L, float alpha, int causal,
               void* scratch, float* O, void* workspace, cudaStream_t st, void* dbg_bits, uint8_t* dbg_codes, uint8_t* dbg_scales,
               void* dbg_prepared, int kv_group) {
    if (!attn_fused_supported(L, HD) || heads <= 0 || q.row0 % 128 || k.row0 % 128 || vt.row0 % 128) return AMX_ERR_SHAPE;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return AMX_ERR_CUDA;
    static int sm_count[64] = {};
    if (!sm_count[dev] && cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return AMX_ERR_CUDA;
    const OperandLayout oq = operand_layout(q.layout_rows, HD, 128), ok_ = operand_layout(k.layout_rows, HD, 256),
                        ov = operand_layout(vt.layout_rows, L, 256);
    const uint8_t* pq = static_cast<const uint8_t*>(q.prepared);
    const uint8_t* pk = static_cast<const uint8_t*>(k.prepared);
    const uint8_t* pv = static_cast<const uint8_t*>(vt.prepared);
    CUtensorMap tm_q, tm_k, tm_v;
    if (!make_map(&tm_q, pq, q.rows_total, HD, oq.plane, 128, 64) || !make_map(&tm_k, pk, k.rows_total, HD, ok_.plane, 128, 64) ||
        !make_map(&tm_v, pv, vt.rows_total, L, ov.plane, 128, 64))
        return AMX_ERR_CUDA;
    int* status = static_cast<int*>(workspace);
    if (cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return AMX_ERR_CUDA;
    Params p{};
    p.sfq[0] = pq + 2 * oq.plane;   p.sfq[1] = p.sfq[0] + oq.sf;
    p.sfk[0] = pk + 2 * ok_.plane;  p.sfk[1] = p.sfk[0] + ok_.sf;
    p.sfv[0] = pv + 2 * ov.plane;   p.sfv[1] = p.sfv[0] + ov.sf;
    p.q_words = reinterpret_cast<const int*>(pq + 2 * oq.plane + 2 * oq.sf);
    p.k_words = reinterpret_cast<const int*>(pk + 2 * ok_.plane + 2 * ok_.sf);
    p.v_words = reinterpret_cast<const int*>(pv + 2 * ov.plane + 2 * ov.sf);
    p.q_row0 = q.row0; p.k_row0 = k.row0; p.v_row0 = vt.row0;
    p.nk64_q = oq.nk64; p.nk64_k = ok_.nk64; p.nk64_v = ov.nk64;
    p.heads = heads; p.m_tiles = (int)(L / BM); p.causal = causal ? 1 : 0;
    p.kv_group = kv_group > 0 ? kv_group : 1;
    p.L = L; p.alpha = alpha;
    p.part = static_cast<float2*>(scratch);
    p.O = O;
    p.status = status;
    if (dbg_prepared) {
        const OperandLayout op = operand_layout(L, L, 128);
        uint8_t* pp = static_cast<uint8_t*>(dbg_prepared);
        p.p_plane = reinterpret_cast<uint4*>(pp);
        p.p_sf = pp + 2 * op.plane;
        p.p_words = reinterpret_cast<int*>(pp + 2 * op.plane + 2 * op.sf);
        p.p_nk64 = op.nk64;
        p.p_bits = static_cast<uint4*>(dbg_bits);
        p.p_codes = reinterpret_cast<uint4*>(dbg_codes);
        p.p_scales = reinterpret_cast<uint16_t*>(dbg_scales);
    }
    int rc = causal ? launch_pass<1, true>(tm_q, tm_k, tm_v, p, dev, sm_count[dev], st)
                    : launch_pass<1, false>(tm_q, tm_k, tm_v, p, dev, sm_count[dev], st);
    if (rc != AMX_OK) return rc;
    return causal ? launch_pass<2, true>(tm_q, tm_k, tm_v, p, dev, sm_count[dev], st)
                  : launch_pass<2, false>(tm_q, tm_k, tm_v, p, dev, sm_count[dev], st);
}

}  // namespace amx
