// AMXFP4 x AMXFP4 -> fp32 on the 5th-generation tensor cores (tcgen05, sm_100a), exact-decode
// variant: C[m,n] = sum_k Ahat[m,k] * What[n,k] (arXiv 2411.09909, Section 4.3).
//
// The format gives every element one of TWO group scales, picked by the element's own sign, so
// an operand tile is not a single block-scaled FP4 matrix.  Here each tile is decoded exactly to
// bf16 in shared memory (a decoded value has at most 5 significant bits) and multiplied with
// tcgen05.mma kind::f16, fp32 accumulators in tensor memory.
//
// One CTA computes one 128 x 256 tile of C.  Roles:
//   warps 0..7  producers: read 4-bit codes + E5M2 scales from global memory, decode one 64-wide
//               K block to bf16 in the 128-byte-swizzled K-major layout the MMA reads; afterwards
//               they are the epilogue (TMEM -> registers -> global)
//   warp 8      allocates tensor memory; one elected lane issues the MMAs and commits them to
//               mbarriers
// Two shared-memory stages (48 KB each) cycle through full/empty mbarriers.  The stage count leaves room for a
// second CTA on the SM, but a kernel that allocates tensor memory gets its SM to itself (measured: padding the
// shared memory to exclude a second CTA changes nothing; the occupancy calculator reports one).  Measured and
// dropped: four stages (no gain), twelve producer warps with two tasks per thread (377 against 507 TFLOP/s).
//
// Decode (decode_math.cuh): a 3-bit E2M1 code placed at bits 8..6 of a bf16 is the value x 2^-126, so a shift
// and a mask per element pair, the side's scale chosen by a mask built from the sign bits, and one packed bf16
// multiply give the decoded pair; the two tiles carry 2^+63 and 2^-63 (exact), and both get the same
// permutation of a word's eight elements, which a contraction does not see.  (Lookup tables by byte permutes,
// the earlier form, kept all of this on the integer/logic pipe, which bounds the kernel.)
//
// Every wait is bounded: when a limit expires the CTA records AMX_ERR_TIMEOUT in the status word,
// all roles leave their loops, tensor memory is released and the kernel returns.
#include <cuda_bf16.h>

#include "cast_math.cuh"
#include "decode_math.cuh"
#include "gemm.cuh"
#include "tcgen05.cuh"

namespace amx {
namespace {

using namespace tc;

constexpr int BM = 128, BN = 256, BK = 64;       // tile; BK bf16 = one 128-byte swizzle row
constexpr int kStages = 2;
constexpr int kProducerWarps = 8;
constexpr int kThreads = (kProducerWarps + 1) * 32;
constexpr int kTileA = BM * BK * 2, kTileB = BN * BK * 2, kStageBytes = kTileA + kTileB;
constexpr int kTmemCols = 256;

struct __align__(8) Control {
    uint64_t full[kStages], empty[kStages], accum;
    uint32_t tmem_base;
    volatile int abort;
};
constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + sizeof(Control);

// Instruction descriptor, kind::f16: D fp32, A and B bf16, both K-major, M x N.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

using namespace decode;   // group tables and decode_word (decode_math.cuh)

struct Task {      // one 32-element group of one tile row
    uint4 codes;
    uint32_t scales;
};
constexpr int kTasksPerThread = (BM + BN) * 2 / (kProducerWarps * 32);   // 3

__device__ __forceinline__ Task load_task(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ scales,
                                          int64_t row, int64_t rows, int64_t K, int64_t k) {
    Task t;
    t.codes = make_uint4(0, 0, 0, 0);
    t.scales = 0;
    if (row < rows && k < K) {
        t.codes = __ldg(reinterpret_cast<const uint4*>(codes + row * (K / 2) + k / 2));
        t.scales = __ldg(reinterpret_cast<const unsigned short*>(scales + (row * (K / 32) + k / 32) * 2));
    }
    return t;
}

// One 32-element group of a bf16 activation row, as loaded (CAST_A).
struct RawGroup {
    uint4 q[4];
};
__device__ __forceinline__ RawGroup load_raw(const uint16_t* __restrict__ x, int64_t ld, int64_t row, int64_t rows,
                                             int64_t K, int64_t k) {
    RawGroup g;
#pragma unroll
    for (int j = 0; j < 4; ++j) g.q[j] = make_uint4(0, 0, 0, 0);
    if (row < rows && k < K) {
        const uint4* p = reinterpret_cast<const uint4*>(x + row * ld + k);
#pragma unroll
        for (int j = 0; j < 4; ++j) g.q[j] = __ldg(p + j);
    }
    return g;
}
// The direct cast of one group (Section 4.2), same arithmetic as the cast kernel: codes and scale bytes.
__device__ __forceinline__ Task cast_task(const RawGroup& g) {
    uint32_t w[16];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        w[4 * j] = g.q[j].x; w[4 * j + 1] = g.q[j].y; w[4 * j + 2] = g.q[j].z; w[4 * j + 3] = g.q[j].w;
    }
    float inv_p, inv_n;
    Task t;
    t.scales = cast::group_scales(cast::side_maxima<16>(w), inv_p, inv_n);
    t.codes.x = cast::encode8(w, inv_p, inv_n);
    t.codes.y = cast::encode8(w + 4, inv_p, inv_n);
    t.codes.z = cast::encode8(w + 8, inv_p, inv_n);
    t.codes.w = cast::encode8(w + 12, inv_p, inv_n);
    return t;
}

// CAST_A: the A operand is the bf16 activation itself (a_x, leading dimension ld_a); the producer
// that owns a group casts it to AMXFP4 in registers and decodes the result, so the activation is read once
// from global memory and its codes never exist there (a_codes / a_scales are unused).
template <bool CAST_A>
__global__ void __launch_bounds__(kThreads, 2)
gemm_tc_kernel(const uint8_t* __restrict__ a_codes, const uint8_t* __restrict__ a_scales,
               const uint16_t* __restrict__ a_x, int64_t ld_a,
               const uint8_t* __restrict__ w_codes, const uint8_t* __restrict__ w_scales,
               int64_t M, int64_t N, int64_t K, float* __restrict__ C, int64_t ld_c, int vec_store,
               int* __restrict__ status, int kb_per_slice, int64_t slice_stride, const int* __restrict__ run_if_nonzero) {
    if (run_if_nonzero && *run_if_nonzero == 0) return;          // uniform over the grid: nothing was set up yet
    // blockIdx.z: slice of the K range (kb_per_slice K blocks each); slice z writes its partial product to
    // C + z * slice_stride (one slice: the result itself)
    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Control* ctl = reinterpret_cast<Control*>(tiles + kStages * kStageBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t m0 = (int64_t)blockIdx.y * BM, n0 = (int64_t)blockIdx.x * BN;
    const int kb_begin = (int)blockIdx.z * kb_per_slice;
    const int num_kb = min((int)((K + BK - 1) / BK) - kb_begin, kb_per_slice);   // K blocks of this slice
    C += (int64_t)blockIdx.z * slice_stride;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&ctl->full[s], kProducerWarps);
            mbar_init(&ctl->empty[s], 1);
        }
        mbar_init(&ctl->accum, 1);
        ctl->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kProducerWarps) tmem_alloc(&ctl->tmem_base, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ctl->tmem_base;

    if (warp < kProducerWarps) {
        // ------------------------------------------------------------------ producers
        // task i of this thread: tile row (tid >> 1) + 128 * i, group (tid & 1) of the K block
        const int tid = threadIdx.x, half = tid & 1, r = tid >> 1;
        Task cur[kTasksPerThread], nxt[kTasksPerThread];
        RawGroup raw;
        auto load_all = [&](Task (&t)[kTasksPerThread], int kb) {
            const int64_t k = (int64_t)(kb_begin + kb) * BK + half * 32;
            if (CAST_A) raw = load_raw(a_x, ld_a, m0 + r, M, K, k);
            else t[0] = load_task(a_codes, a_scales, m0 + r, M, K, k);
#pragma unroll
            for (int i = 1; i < kTasksPerThread; ++i)
                t[i] = load_task(w_codes, w_scales, n0 + r + 128 * (i - 1), N, K, k);
        };
        load_all(cur, 0);
        if (CAST_A) cur[0] = cast_task(raw);
        bool ok = true;
        for (int kb = 0; kb < num_kb && ok; ++kb) {
            const int s = kb % kStages;
            if (kb + 1 < num_kb) load_all(nxt, kb + 1);
            if (kb >= kStages) ok = mbar_wait(&ctl->empty[s], ((kb / kStages) - 1) & 1, &ctl->abort, status);
            if (!ok) break;
            uint8_t* stage = tiles + s * kStageBytes;
#pragma unroll
            for (int i = 0; i < kTasksPerThread; ++i) {
                const int row = r + 128 * i;                       // row inside [A tile | B tile]
                uint8_t* dst = stage + row * 128;                  // A tile is 128 rows: B rows follow it
                const bool live = i ? (n0 + r + 128 * (i - 1) < N) : (m0 + r < M);
                if (!live) {                                       // a row past the operand: zeros, no decode
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        *reinterpret_cast<uint4*>(dst + (((half * 4 + j) ^ (row & 7)) << 4)) = make_uint4(0, 0, 0, 0);
                    continue;
                }
                // packed-multiply decode: both tiles get the same permutation of a word's eight elements, the A
                // tile holds values x 2^63 and the B tile values x 2^-63 (exact), so every product is the true one
                const GroupScales gs = make_scales(cur[i].scales);
                const uint32_t w[4] = {cur[i].codes.x, cur[i].codes.y, cur[i].codes.z, cur[i].codes.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int chunk = half * 4 + j;                // 16-byte chunk inside the 128-byte row
                    *reinterpret_cast<uint4*>(dst + ((chunk ^ (row & 7)) << 4)) =
                        i ? decode_pairs(w[j], gs) : decode_pairs_up(w[j], gs);
                }
            }
            fence_proxy_async();          // make the generic-proxy stores visible to the tensor core
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl->full[s]);
#pragma unroll
            for (int i = 0; i < kTasksPerThread; ++i) cur[i] = nxt[i];
            if (CAST_A && kb + 1 < num_kb) cur[0] = cast_task(raw);
        }
        // ------------------------------------------------------------------ epilogue
        if (ok) ok = mbar_wait(&ctl->accum, 0, &ctl->abort, status);
        tc_fence_after();
        if (ok) {
            const int q = warp & 3, h = warp >> 2;                 // lane quarter, column half
            const int64_t m = m0 + q * 32 + lane;
#pragma unroll 1
            for (int c0 = 0; c0 < BN / 2; c0 += 32) {
                uint32_t v[32];
                const int col = h * (BN / 2) + c0;
                tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)col, v);
                tmem_ld_wait();
                if (m < M) {
                    float* out = C + m * ld_c + n0 + col;
                    if (vec_store && n0 + col + 32 <= N) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            *reinterpret_cast<float4*>(out + j) = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]),
                                                                              __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (n0 + col + j < N) out[j] = __uint_as_float(v[j]);
                    }
                }
            }
        }
    } else if (lane == 0) {
        // ------------------------------------------------------------------ MMA issuer
        bool ok = true;
        for (int kb = 0; kb < num_kb && ok; ++kb) {
            const int s = kb % kStages;
            ok = mbar_wait(&ctl->full[s], (kb / kStages) & 1, &ctl->abort, status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t a_addr = smem_u32(tiles + s * kStageBytes), b_addr = a_addr + kTileA;
#pragma unroll
            for (int k = 0; k < BK / 16; ++k)     // 16 bf16 = 32 bytes further along the swizzled row
                mma_bf16(tmem, smem_desc_sw128(a_addr + k * 32), smem_desc_sw128(b_addr + k * 32), kIdesc,
                         (kb | k) ? 1u : 0u);
            mma_commit(&ctl->empty[s]);           // frees the stage once these MMAs have read it
        }
        if (ok) mma_commit(&ctl->accum);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kProducerWarps) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

}  // namespace

bool gemm_tc_supported(int64_t M, int64_t N, int64_t K, int gs) {
    return gs == 32 && M > 0 && N > 0 && K > 0 && K % 32 == 0 && (M + BM - 1) / BM <= 65535;
}

namespace {

// Few output tiles and a long K (a handful of token rows against a big weight: the decode phase): the K range is
// cut into slices that run as separate CTAs, so that the whole machine streams and decodes the weight; the
// partial products go to the workspace and are added up in slice order (deterministic).  Returns the number of
// slices (1: none) and the K blocks per slice.
constexpr int kSmCount = 148;
int k_slices(int64_t M, int64_t N, int64_t K, int& kb_per_slice) {
    const int64_t tiles = ((N + BN - 1) / BN) * ((M + BM - 1) / BM);
    const int num_kb = (int)((K + BK - 1) / BK);
    kb_per_slice = num_kb;
    if (tiles >= kSmCount || num_kb < 16) return 1;
    int want = (int)(2 * kSmCount / tiles);                          // two CTAs per SM, one wave
    if (want > num_kb / 8) want = num_kb / 8;                        // at least 8 K blocks per slice
    if (want > 16) want = 16;
    if (want < 2) return 1;
    kb_per_slice = (num_kb + want - 1) / want;
    return (num_kb + kb_per_slice - 1) / kb_per_slice;
}

// C[m][n] = sum over slices, in slice order.
__global__ void __launch_bounds__(256)
reduce_slices_kernel(const float* __restrict__ part, int slices, int64_t M, int64_t N, float* __restrict__ C, int64_t ld_c,
                     const int* __restrict__ run_if_nonzero) {
    if (run_if_nonzero && *run_if_nonzero == 0) return;
    const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (i >= M * N) return;
    float acc = part[i];
    for (int z = 1; z < slices; ++z) acc += part[(int64_t)z * M * N + i];
    C[(i / N) * ld_c + i % N] = acc;
}

}  // namespace

size_t gemm_tc_workspace_bytes(int64_t M, int64_t N, int64_t K) {   // the status word, then the slices' partial products
    int kb_per;
    const int slices = k_slices(M, N, K, kb_per);
    return 256 + (slices > 1 ? (size_t)slices * M * N * 4 : 0);
}

namespace {

int launch_tc(const uint8_t* a_codes, const uint8_t* a_scales, const uint16_t* a_x, int64_t ld_a,
              const uint8_t* w_codes, const uint8_t* w_scales, int64_t M, int64_t N, int64_t K, float* C,
              int64_t ld_c, void* workspace, cudaStream_t st, const int* gate = nullptr, int* status_word = nullptr) {
    static bool configured[64] = {};   // the opt-in to > 48 KB of dynamic shared memory is per device
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return AMX_ERR_CUDA;
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(gemm_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess ||
            cudaFuncSetAttribute(gemm_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
            return AMX_ERR_CUDA;
        configured[dev] = true;
    }
    // status word: the first word of the workspace, cleared here, unless the caller shares one it cleared itself
    int* status = status_word ? status_word : static_cast<int*>(workspace);
    if (!status_word && cudaMemsetAsync(status, 0, 2 * sizeof(int), st) != cudaSuccess) return AMX_ERR_CUDA;   // + flushed count: none
    int kb_per;
    const int slices = k_slices(M, N, K, kb_per);
    dim3 grid((unsigned)((N + BN - 1) / BN), (unsigned)((M + BM - 1) / BM), (unsigned)slices);
    float* part = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + 256);
    float* out = slices > 1 ? part : C;
    const int64_t ld_out = slices > 1 ? N : ld_c, slice_stride = slices > 1 ? M * N : 0;
    const int vec_store = aligned(out, 16) && ld_out % 4 == 0;   // else the epilogue stores scalars
    if (a_x)
        gemm_tc_kernel<true><<<grid, kThreads, kSmemBytes, st>>>(nullptr, nullptr, a_x, ld_a, w_codes, w_scales, M, N, K, out,
                                                                 ld_out, vec_store, status, kb_per, slice_stride, gate);
    else
        gemm_tc_kernel<false><<<grid, kThreads, kSmemBytes, st>>>(a_codes, a_scales, nullptr, 0, w_codes, w_scales, M, N, K,
                                                                  out, ld_out, vec_store, status, kb_per, slice_stride, gate);
    int rc = launch_status();
    if (rc != AMX_OK || slices == 1) return rc;
    return reduce_slices(part, slices, M, N, C, ld_c, st, gate);
}

}  // namespace

int reduce_slices(const float* part, int slices, int64_t M, int64_t N, float* C, int64_t ld_c, cudaStream_t st,
                  const int* run_if_nonzero) {
    reduce_slices_kernel<<<(unsigned)((M * N + 255) / 256), 256, 0, st>>>(part, slices, M, N, C, ld_c, run_if_nonzero);
    return launch_status();
}

// run_if_nonzero: the launches do nothing when that device word is zero.  status_word: where a timeout is
// recorded instead of the workspace's first word (the caller has cleared it).
int gemm_tc(const uint8_t* a_codes, const uint8_t* a_scales, const uint8_t* w_codes, const uint8_t* w_scales,
            int64_t M, int64_t N, int64_t K, float* C, int64_t ld_c, void* workspace, cudaStream_t st,
            const int* run_if_nonzero, int* status_word) {
    return launch_tc(a_codes, a_scales, nullptr, 0, w_codes, w_scales, M, N, K, C, ld_c, workspace, st, run_if_nonzero,
                     status_word);
}

// C = cast(X) What^T with the cast of X done by the kernel's producers.  X: bf16 [M, ld_a], 16-byte aligned,
// ld_a % 8 == 0.
int gemm_tc_cast(const void* x, int64_t ld_a, const uint8_t* w_codes, const uint8_t* w_scales, int64_t M, int64_t N,
                 int64_t K, float* C, int64_t ld_c, void* workspace, cudaStream_t st) {
    return launch_tc(nullptr, nullptr, static_cast<const uint16_t*>(x), ld_a, w_codes, w_scales, M, N, K, C, ld_c,
                     workspace, st);
}

int gemm_tc_status(const void* workspace, cudaStream_t st) {
    if (!workspace) return AMX_OK;
    int v = 0;
    if (cudaMemcpyAsync(&v, workspace, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return AMX_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return AMX_ERR_CUDA;
    return v;
}

}  // namespace amx
