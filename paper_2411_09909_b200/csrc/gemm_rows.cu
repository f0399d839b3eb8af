// AMXFP4 x AMXFP4 -> fp32 for at most 64 rows of A against a large weight (the decode phase of inference):
// C[m,n] = sum_k Ahat[m,k] * What[n,k] (arXiv 2411.09909, Section 4.3), bound by streaming the 4.5-bit weight
// from HBM once, not by arithmetic.
//
// The weight is read in its canonical layout (codes [N, K/2], scales [N, K/32, 2]); nothing is prepared ahead.
// The few activation rows are cast and decoded to bf16 once by a small kernel (decoded values are exact in bf16,
// Eq. 1), already in the order the multiply instruction's fragments want.
//
// Streaming kernel: warp-level mma.sync m16n8k16 (bf16 in, fp32 accumulate) with 16 token rows as the M side and
// 8 weight rows as the N side; up to four tiles of 16 token rows reuse the decoded weight registers of a step.
// The contraction index may be permuted freely as long as both operands use the same permutation; here lane
// (g, t) (g = lane / 4, t = lane % 4) owns, for one step of 128 elements of K, the whole 32-element group
// 4 * step + t of weight row g of each of its two 8-row tiles: 16 bytes of codes and the group's two scales per
// tile, brought in by asynchronous copies into a per-warp ring in shared memory four steps ahead (no registers
// are held by loads in flight) and decoded in registers with packed bf16 multiplies (decode_pairs below).
// The matching activation values (rows g and g + 8, same group) are read from global memory in 16-byte pieces,
// 512 contiguous bytes per warp and load; every warp of every CTA on an SM reads the same few hundred KB, so they
// come from the L1 (staging them in shared memory needed a block barrier every few steps and measured slower).
// Eight MMAs per tile and step consume four elements per lane each.  What bounds the kernel is instruction
// issue (decode on the integer/logic pipe), not the tensor cores: the MMAs are a few percent of the instructions.
//
// A CTA of eight warps covers 128 weight rows and one range of K; the ranges of K of the same 128 rows are the
// CTAs of one thread-block cluster (up to 8), which add their partial products over distributed shared memory
// in rank order - deterministic, no scratch in global memory and no second launch.
//
// The two launches of a call are chained by programmatic dependent launch: the streaming kernel is allowed onto the
// SMs while the fragments kernel still runs, sets up and fills its weight rings (the weight does not depend on the
// fragments), and only then waits for the fragments kernel to complete; the fragments kernel in turn waits for
// whatever ran before it in the stream before it writes anything.  Measured on a 16-row step over four weights:
// 87 -> 71 us with plain launches; replayed from a CUDA graph the same step takes 71 us without these edges and
// 81 us with them, so a stream that is being captured gets ordinary launches.
#include <cooperative_groups.h>
#include <cuda_bf16.h>

#include "cast_math.cuh"
#include "cp_async.cuh"
#include "decode_math.cuh"
#include "gemm.cuh"

namespace cg = cooperative_groups;

namespace amx {
namespace {

using namespace decode;

constexpr int kMaxRows = 16;                 // token rows of one tile (the M side of one MMA)
constexpr int kMaxRowTiles = 4;              // up to 64 token rows
constexpr int kWarps = 8, kThreads = kWarps * 32;
constexpr int kTiles = 2;                    // 8-row weight tiles per warp
constexpr int kCtaRows = kWarps * kTiles * 8;   // 128 weight rows per CTA
constexpr int kStepK = 128;                  // elements of K per step: one group per lane of a quad
constexpr int kStepBytes = kMaxRows * kStepK * 2;   // activation fragments of one step: 4 KB
constexpr int kMaxSlices = 8;                // portable cluster size
constexpr int kPartPitch = 136;              // floats per token row of the partial-product tile (bank spread)

// Fragment order of the decoded activation, per step of 128 elements: [row tile mt][unit j = 0..3][half 0..1]
// [lane 0..31] pieces of 16 bytes; the piece of lane (g, t) holds elements 8j .. 8j+7 of group 4 * step + t of row
// 16 * mt + 8 * half + g (in the pair order and scaling of pair_order_scaled).  mts = row tiles (1, 2 or 4).
__device__ __forceinline__ int64_t fragment_piece(int64_t step, int mts, int mt, int j, int half, int g, int t) {
    return ((((step * mts + mt) * 4 + j) * 2 + half) * 32) + g * 4 + t;
}

// The streaming kernel decodes a word of eight weight codes into the bf16 pairs (e0, e4), (e1, e5), (e2, e6),
// (e3, e7), each value 2^-63 times the true one (decode_pairs in decode_math.cuh); the activation pieces are stored in the same
// pair order and multiplied by 2^63, so that every product is the true one.  Both scalings are exact: a decoded
// value times 2^+-63 stays far inside the bf16 range.
__device__ __forceinline__ uint4 pair_order_scaled(uint4 o) {      // o: pairs (e0,e1), (e2,e3), (e4,e5), (e6,e7)
    const uint32_t two63 = 0x5F005F00u;
    uint4 r;
    r.x = mul_bf16x2(prmt(o.x, o.z, 0x5410), two63);
    r.y = mul_bf16x2(prmt(o.x, o.z, 0x7632), two63);
    r.z = mul_bf16x2(prmt(o.y, o.w, 0x5410), two63);
    r.w = mul_bf16x2(prmt(o.y, o.w, 0x7632), two63);
    return r;
}

// One thread per 8 elements of the slab of 16 * mts rows (four adjacent lanes share a 32-element group and
// exchange their side maxima with two shuffles): decode, or cast then decode (CAST), and write one 16-byte piece.
// Rows past M are written as zeros.  The kernel is a few thousand threads of pure latency, so the work of a group
// is spread over lanes instead of being one long dependent chain.
// griddepcontrol.wait: returns once every grid this one programmatically depends on has completed and its writes
// are visible (at once when the launch carried no such dependency).  griddepcontrol.launch_dependents: the grid
// launched behind this one with programmatic serialization may start once every CTA here has said so or exited.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <bool CAST>
__global__ void __launch_bounds__(128) rows_fragments_kernel(const uint8_t* __restrict__ codes,
                                                             const uint8_t* __restrict__ scales,
                                                             const uint16_t* __restrict__ x, int64_t ld_x, int M,
                                                             int mts, int64_t K, uint4* __restrict__ frag,
                                                             int* __restrict__ status) {
    const int64_t groups = K / 32;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    grid_dependency_wait();                    // the previous call on this stream may still read the workspace
    grid_launch_dependents();                  // the streaming kernel may start filling its rings
    if (idx == 0) status[0] = status[1] = 0;   // no device-side wait that can expire, no scale is flushed: both words read 0
    const bool live = idx < groups * 4 * kMaxRows * mts;           // whole groups: the four lanes agree
    const int j = (int)(idx & 3);
    const int64_t gidx = idx >> 2;
    const int row = live ? (int)(gidx / groups) : M;
    const int64_t grp = gidx % groups;
    uint32_t word = 0, sc = 0;
    if (CAST) {
        uint32_t w[4] = {0, 0, 0, 0};
        if (row < M) {
            const uint4 q = __ldg(reinterpret_cast<const uint4*>(x + row * ld_x + grp * 32) + j);
            w[0] = q.x; w[1] = q.y; w[2] = q.z; w[3] = q.w;
        }
        uint32_t c = cast::side_maxima<4>(w);
        c = __vmaxs2(c, __shfl_xor_sync(0xFFFFFFFFu, c, 1));
        c = __vmaxs2(c, __shfl_xor_sync(0xFFFFFFFFu, c, 2));
        float inv_p, inv_n;
        sc = cast::group_scales(c, inv_p, inv_n);
        word = cast::encode8(w, inv_p, inv_n);
    } else if (row < M) {
        word = __ldg(reinterpret_cast<const uint32_t*>(codes + (row * groups + grp) * 16) + j);
        sc = __ldg(reinterpret_cast<const unsigned short*>(scales + (row * groups + grp) * 2));
    }
    if (!live) return;
    const GroupTables tb = make_tables(sc);
    const int64_t step = grp >> 2;
    const int t = (int)(grp & 3), g = row & 7, half = (row >> 3) & 1, mt = row >> 4;
    frag[fragment_piece(step, mts, mt, j, half, g, t)] = pair_order_scaled(decode_word(word, tb));
}

__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Shared memory of a CTA: one ring of kDepth steps per warp for the weight stream.  A ring slot holds, per 8-row
// tile, the 32 lanes' 16 bytes of codes and 4 bytes of scales (the two groups 4 * step + 2 * (t / 2) + {0, 1}; the
// lane uses the half t % 2).  Every lane reads back only what its own copies wrote, so the ring needs no barrier,
// only the lane's own wait.
constexpr int kDepth = 4;
constexpr int kSlotCodes = kTiles * 32 * 16, kSlotBytes = kSlotCodes + kTiles * 32 * 4;
constexpr int kRingBytes = kDepth * kSlotBytes;   // per warp
constexpr int kSmemBytes = kWarps * kRingBytes;
static_assert(4 * kMaxRows * kPartPitch * 4 <= kWarps * kRingBytes, "the partial-product tile reuses the rings");

// MT: tiles of 16 token rows (1, 2 or 4).  The decoded weight registers of a step are used by every row tile.
template <int MT>
__global__ void __launch_bounds__(kThreads, MT == 1 ? 4 : 2) gemm_rows_kernel(const uint4* __restrict__ frag,
                                                                const uint8_t* __restrict__ w_codes,
                                                                const uint8_t* __restrict__ w_scales, int M, int64_t N,
                                                                int64_t K, float* __restrict__ C, int64_t ld_c) {
    extern __shared__ __align__(16) uint8_t smem[];
    cg::cluster_group cluster = cg::this_cluster();
    const int slices = (int)gridDim.y, slice = (int)blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, t = lane & 3;
    const int64_t groups = K / 32, steps = K / kStepK;
    const int64_t s_begin = steps * slice / slices;
    const int n_total = (int)(steps * (slice + 1) / slices - s_begin);
    const int64_t row0 = (int64_t)blockIdx.x * kCtaRows + warp * (kTiles * 8);

    // this lane's stream positions at step s_begin: codes of group 4 * step + t, scales of the group pair
    const uint8_t* pc[kTiles];
    const uint8_t* ps[kTiles];
#pragma unroll
    for (int i = 0; i < kTiles; ++i) {
        int64_t r = row0 + i * 8 + g;
        r = r < N ? r : N - 1;               // rows past the weight read its last row; their sums are not stored
        pc[i] = w_codes + (r * groups + s_begin * 4 + t) * 16;
        ps[i] = w_scales + (r * groups + s_begin * 4 + (t & 2)) * 2;
    }
    uint8_t* ring = smem + warp * kRingBytes;
    auto issue = [&](int step) {             // step relative to s_begin; one commit group per call
        if (step < n_total) {
            uint8_t* slot = ring + (step % kDepth) * kSlotBytes;
#pragma unroll
            for (int i = 0; i < kTiles; ++i) {
                cp_async16(slot + i * 512 + lane * 16, pc[i] + (int64_t)step * 64);
                cp_async4(slot + kSlotCodes + i * 128 + lane * 4, ps[i] + (int64_t)step * 8);
            }
        }
        cp_async_commit();
    };
#pragma unroll
    for (int d = 0; d < kDepth; ++d) issue(d);
    grid_launch_dependents();                // whatever follows waits for this grid's completion by itself
    grid_dependency_wait();                  // the fragments (and the previous user of C) are complete from here on

    float acc[MT][kTiles][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int i = 0; i < kTiles; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[mt][i][j] = 0.f;

    for (int step = 0; step < n_total; ++step) {
        const uint4* a = frag + (s_begin + step) * (MT * kStepBytes / 16) + lane;
        uint4 a_lo[4], a_hi[4];                                  // rows g and g + 8 of a tile, elements 8j .. 8j + 7
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            a_lo[j] = __ldg(a + (j * 2) * 32);
            a_hi[j] = __ldg(a + (j * 2 + 1) * 32);
        }
        cp_async_wait<kDepth - 1>();                             // this step's group has landed
        const uint8_t* slot = ring + (step % kDepth) * kSlotBytes;
        uint4 b[kTiles][4];
#pragma unroll
        for (int i = 0; i < kTiles; ++i) {
            const uint4 cw = *reinterpret_cast<const uint4*>(slot + i * 512 + lane * 16);
            const uint32_t sw = *reinterpret_cast<const uint32_t*>(slot + kSlotCodes + i * 128 + lane * 4);
            const GroupScales gs = make_scales((t & 1) ? sw >> 16 : sw & 0xFFFFu);
            const uint32_t w[4] = {cw.x, cw.y, cw.z, cw.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) b[i][j] = decode_pairs(w[j], gs);
        }
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            if (mt > 0) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    a_lo[j] = __ldg(a + ((mt * 4 + j) * 2) * 32);
                    a_hi[j] = __ldg(a + ((mt * 4 + j) * 2 + 1) * 32);
                }
            }
#pragma unroll
            for (int i = 0; i < kTiles; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    mma_bf16(acc[mt][i], a_lo[j].x, a_hi[j].x, a_lo[j].y, a_hi[j].y, b[i][j].x, b[i][j].y);
                    mma_bf16(acc[mt][i], a_lo[j].z, a_hi[j].z, a_lo[j].w, a_hi[j].w, b[i][j].z, b[i][j].w);
                }
        }
        issue(step + kDepth);                                    // refill the slot just consumed
    }
    cp_async_wait<0>();

    // Partial products of this range of K: [16 token rows][128 weight rows] in shared memory (over the rings, which
    // are drained), then every CTA of
    // the cluster adds its share of the outputs over all ranks, in rank order.
    __syncthreads();
    float* part = reinterpret_cast<float*>(smem);
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int i = 0; i < kTiles; ++i) {
            const int col = warp * (kTiles * 8) + i * 8 + 2 * t;
            *reinterpret_cast<float2*>(part + (mt * 16 + g) * kPartPitch + col) = make_float2(acc[mt][i][0], acc[mt][i][1]);
            *reinterpret_cast<float2*>(part + (mt * 16 + g + 8) * kPartPitch + col) = make_float2(acc[mt][i][2], acc[mt][i][3]);
        }
    cluster.sync();
    const int per = MT * kMaxRows * kCtaRows / slices;           // outputs this CTA adds up (a multiple of 256)
    for (int o = slice * per + threadIdx.x; o < (slice + 1) * per; o += kThreads) {
        const int m = o / kCtaRows, col = o % kCtaRows;
        float v[kMaxSlices];
#pragma unroll
        for (int r = 0; r < kMaxSlices; ++r)                     // all remote reads in flight together
            v[r] = r < slices ? cluster.map_shared_rank(part, r)[m * kPartPitch + col] : 0.f;
        float sum = 0.f;
#pragma unroll
        for (int r = 0; r < kMaxSlices; ++r) sum += v[r];
        const int64_t n = (int64_t)blockIdx.x * kCtaRows + col;
        if (m < M && n < N) C[m * ld_c + n] = sum;
    }
    cluster.sync();                                              // no CTA leaves while its tile is still read
}

using RowsKernel = void (*)(const uint4*, const uint8_t*, const uint8_t*, int, int64_t, int64_t, float*, int64_t);

// Row tiles for M token rows (1, 2 or 4) and the kernel instantiation for them.
int row_tiles(int64_t M) { return M <= kMaxRows ? 1 : M <= 2 * kMaxRows ? 2 : 4; }
RowsKernel kernel_for_tiles(int mts) {
    return mts == 1 ? gemm_rows_kernel<1> : mts == 2 ? gemm_rows_kernel<2> : gemm_rows_kernel<4>;
}

// Programmatic dependent launch is used outside stream capture only (see the file header).
bool programmatic_launch_ok(cudaStream_t st) {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cs) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return cs == cudaStreamCaptureStatusNone;
}

void cluster_config(cudaLaunchConfig_t& cfg, cudaLaunchAttribute* attr, unsigned row_blocks, int slices, cudaStream_t st,
                    bool programmatic = false) {
    cfg = {};
    cfg.gridDim = dim3(row_blocks, (unsigned)slices, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = st;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = (unsigned)slices;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = programmatic ? 2 : 1;
}

// How many clusters of `slices` CTAs the device holds at once (asked once per kernel and cluster size; 0 if the
// query fails).
int resident_clusters(int mts, int slices) {
    static int cached[kMaxRowTiles + 1][kMaxSlices + 1] = {};
    int& c = cached[mts][slices];
    if (c) return c > 0 ? c : 0;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    cluster_config(cfg, attr, 1, slices, nullptr);
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kernel_for_tiles(mts), &cfg) != cudaSuccess || n <= 0) {
        cudaGetLastError();
        n = -1;
    }
    c = n;
    return n > 0 ? n : 0;
}

// Ranges of K per 128 weight rows: as many as give every range at least two steps and still let all clusters
// be resident at once (a second wave of CTAs would start its stream from an empty pipeline).
int slices_for(int mts, int64_t N, int64_t K) {
    const int64_t steps = K / kStepK, row_blocks = (N + kCtaRows - 1) / kCtaRows;
    int s = kMaxSlices;
    while (s > 1 && (steps < 2 * s || row_blocks > resident_clusters(mts, s))) s >>= 1;
    return s;
}

int launch_rows(const uint4* frag, const uint8_t* w_codes, const uint8_t* w_scales, int64_t M, int64_t N, int64_t K,
                float* C, int64_t ld_c, cudaStream_t st) {
    static bool configured[64] = {};         // the opt-in to > 48 KB of dynamic shared memory is per device
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return AMX_ERR_CUDA;
    if (!configured[dev]) {
        for (int mts = 1; mts <= kMaxRowTiles; mts *= 2)
            if (cudaFuncSetAttribute(kernel_for_tiles(mts), cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) !=
                cudaSuccess) {
                cudaGetLastError();
                return AMX_ERR_CUDA;
            }
        configured[dev] = true;
    }
    const int mts = row_tiles(M);
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    cluster_config(cfg, attr, (unsigned)((N + kCtaRows - 1) / kCtaRows), slices_for(mts, N, K), st, programmatic_launch_ok(st));
    if (cudaLaunchKernelEx(&cfg, kernel_for_tiles(mts), frag, w_codes, w_scales, (int)M, N, K, C, ld_c) != cudaSuccess) {
        cudaGetLastError();
        return AMX_ERR_CUDA;
    }
    return AMX_OK;
}

// Workspace: 256 bytes whose first word is the status word amx_gemm_status reads, then the decoded rows.
constexpr size_t kHeaderBytes = 256;
uint4* fragments_of(void* workspace) { return reinterpret_cast<uint4*>(static_cast<uint8_t*>(workspace) + kHeaderBytes); }

template <bool CAST>
int launch_fragments(const uint8_t* codes, const uint8_t* scales, const uint16_t* x, int64_t ld_x, int64_t M, int64_t K,
                     void* workspace, cudaStream_t st) {
    const int mts = row_tiles(M);
    const int64_t threads = (int64_t)kMaxRows * mts * (K / 32) * 4;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((threads + 127) / 128), 1, 1);
    cfg.blockDim = dim3(128, 1, 1);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = programmatic_launch_ok(st) ? 1 : 0;
    if (cudaLaunchKernelEx(&cfg, rows_fragments_kernel<CAST>, codes, scales, x, ld_x, (int)M, mts, K,
                           fragments_of(workspace), static_cast<int*>(workspace)) != cudaSuccess) {
        cudaGetLastError();
        return AMX_ERR_CUDA;
    }
    return AMX_OK;
}

}  // namespace

bool gemm_rows_supported(int64_t M, int64_t N, int64_t K, int gs) {
    return gs == 32 && M >= 1 && M <= kMaxRows * kMaxRowTiles && N >= 1 && K >= kStepK && K % kStepK == 0 &&
           (N + kCtaRows - 1) / kCtaRows <= 0x7FFFFFFF;
}

size_t gemm_rows_workspace_bytes(int64_t M, int64_t K) {
    return kHeaderBytes + (size_t)kMaxRows * row_tiles(M) * (size_t)K * 2;
}

int gemm_rows(const uint8_t* a_codes, const uint8_t* a_scales, const uint8_t* w_codes, const uint8_t* w_scales,
              int64_t M, int64_t N, int64_t K, float* C, int64_t ld_c, void* workspace, cudaStream_t st) {
    if (launch_fragments<false>(a_codes, a_scales, nullptr, 0, M, K, workspace, st) != AMX_OK) return AMX_ERR_CUDA;
    return launch_rows(fragments_of(workspace), w_codes, w_scales, M, N, K, C, ld_c, st);
}

int gemm_rows_cast(const void* x, int64_t ld_x, const uint8_t* w_codes, const uint8_t* w_scales, int64_t M, int64_t N,
                   int64_t K, float* C, int64_t ld_c, void* workspace, cudaStream_t st) {
    if (launch_fragments<true>(nullptr, nullptr, static_cast<const uint16_t*>(x), ld_x, M, K, workspace, st) != AMX_OK)
        return AMX_ERR_CUDA;
    return launch_rows(fragments_of(workspace), w_codes, w_scales, M, N, K, C, ld_c, st);
}

}  // namespace amx
