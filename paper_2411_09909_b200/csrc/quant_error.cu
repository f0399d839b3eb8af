// Squared error of a quantized tensor against its bf16 source, split into the max-clamping and the rounding
// part (arXiv 2411.09909, appendix "Determining PoT Shared Scale: Floor vs. Round": the output error of a shared
// scale decomposes into the error of elements beyond the largest representable magnitude and the rounding error
// of all others).  An element is clamped when |x| > 6 * (the scale of its side).
//
// Memory-bound reduction: 2 bytes of source, half a byte of codes and the scale bytes per element are read once.
// A thread takes 16 consecutive elements at a time (two 16-byte loads of the source, one 8-byte load of codes);
// x - xhat is exact in fp32 for the output of the casts (both have few significant bits and nearby exponents),
// squares and sums are fp64.  The summation order is fixed (grid-stride per thread, shuffles in a warp, warps in
// order, then one block over the per-block partial sums), so the result is the same bits on every run.
#include "amx_common.cuh"

namespace amx {
namespace {

constexpr int kThreads = 256, kMaxBlocks = 2048;

struct Sums {
    double x2, e2, clamp2, clamped;
};

__device__ __forceinline__ void add16(Sums& s, const uint4 (&xw)[2], uint2 cw, float sp, float sn) {
    const uint32_t xs[8] = {xw[0].x, xw[0].y, xw[0].z, xw[0].w, xw[1].x, xw[1].y, xw[1].z, xw[1].w};
    const uint32_t cs[2] = {cw.x, cw.y};
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float x = __uint_as_float((i & 1) ? (xs[i >> 1] & 0xFFFF0000u) : (xs[i >> 1] << 16));
        const uint32_t c = (cs[i >> 3] >> ((i & 7) * 4)) & 15u;
        const float scale = (c & 8u) ? sn : sp;
        const float mag = e2m1_mag_to_float(c & 7u) * scale;
        const double e = (double)(x - ((c & 8u) ? -mag : mag)), xd = (double)x;
        const double e2 = e * e;
        s.x2 += xd * xd;
        s.e2 += e2;
        if (fabsf(x) > 6.0f * scale) {
            s.clamp2 += e2;
            s.clamped += 1.0;
        }
    }
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Sum over the block; valid in thread 0.
__device__ __forceinline__ Sums block_sum(Sums s, double (*sh)[4]) {
    s.x2 = warp_sum(s.x2); s.e2 = warp_sum(s.e2); s.clamp2 = warp_sum(s.clamp2); s.clamped = warp_sum(s.clamped);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { sh[warp][0] = s.x2; sh[warp][1] = s.e2; sh[warp][2] = s.clamp2; sh[warp][3] = s.clamped; }
    __syncthreads();
    Sums t = {0, 0, 0, 0};
    if (threadIdx.x == 0)
        for (int w = 0; w < kThreads / 32; ++w) { t.x2 += sh[w][0]; t.e2 += sh[w][1]; t.clamp2 += sh[w][2]; t.clamped += sh[w][3]; }
    return t;
}

__global__ void __launch_bounds__(kThreads) quant_error_kernel(const uint16_t* __restrict__ x, int64_t rows, int64_t K,
                                                               int64_t ld_x, const uint8_t* __restrict__ codes,
                                                               const uint8_t* __restrict__ scales, int gs,
                                                               double* __restrict__ partial) {
    __shared__ double sh[kThreads / 32][4];
    const int64_t per_row = K / 16, chunks = rows * per_row, groups = K / gs;
    Sums s = {0, 0, 0, 0};
    for (int64_t c = (int64_t)blockIdx.x * kThreads + threadIdx.x; c < chunks; c += (int64_t)gridDim.x * kThreads) {
        const int64_t row = c / per_row, k = (c - row * per_row) * 16;
        const uint4* xp = reinterpret_cast<const uint4*>(x + row * ld_x + k);
        const uint4 xw[2] = {__ldg(xp), __ldg(xp + 1)};
        const uint2 cw = __ldg(reinterpret_cast<const uint2*>(codes + row * (K / 2) + k / 2));
        const uint32_t sc = __ldg(reinterpret_cast<const unsigned short*>(scales + (row * groups + k / gs) * 2));
        add16(s, xw, cw, e5m2_to_float(sc & 0xFFu), e5m2_to_float(sc >> 8));
    }
    const Sums t = block_sum(s, sh);
    if (threadIdx.x == 0) {
        double* p = partial + (int64_t)blockIdx.x * 4;
        p[0] = t.x2; p[1] = t.e2; p[2] = t.clamp2; p[3] = t.clamped;
    }
}

__global__ void __launch_bounds__(kThreads) quant_error_final_kernel(const double* __restrict__ partial, int blocks,
                                                                     double* __restrict__ out) {
    __shared__ double sh[kThreads / 32][4];
    Sums s = {0, 0, 0, 0};
    for (int b = threadIdx.x; b < blocks; b += kThreads) {
        s.x2 += partial[b * 4]; s.e2 += partial[b * 4 + 1]; s.clamp2 += partial[b * 4 + 2]; s.clamped += partial[b * 4 + 3];
    }
    const Sums t = block_sum(s, sh);
    if (threadIdx.x == 0) { out[0] = t.x2; out[1] = t.e2; out[2] = t.clamp2; out[3] = t.clamped; }
}

}  // namespace
}  // namespace amx

using namespace amx;

extern "C" size_t amx_quant_error_workspace_bytes(void) { return (size_t)kMaxBlocks * 4 * sizeof(double); }

extern "C" int amx_quant_error(const void* x, int64_t rows, int64_t K, int64_t ld_x, const uint8_t* codes,
                               const uint8_t* scales, int group_size, double* out, void* workspace,
                               size_t workspace_bytes, void* stream) {
    if (!valid_group_size(group_size) || rows < 0 || K <= 0 || K % group_size || ld_x < K) return AMX_ERR_SHAPE;
    if (!out) return AMX_ERR_NULL;
    if (rows > 0 && (!x || !codes || !scales)) return AMX_ERR_NULL;
    if (!workspace || workspace_bytes < amx_quant_error_workspace_bytes()) return AMX_ERR_WORKSPACE;
    if (!aligned(x, 16) || ld_x % 8 || !aligned(codes, 8) || !aligned(scales, 2) || !aligned(out, 8) ||
        !aligned(workspace, 8))
        return AMX_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t chunks = rows * (K / 16);
    int64_t blocks = (chunks + kThreads - 1) / kThreads;
    blocks = blocks < 1 ? 1 : blocks > kMaxBlocks ? kMaxBlocks : blocks;
    double* partial = static_cast<double*>(workspace);
    quant_error_kernel<<<(unsigned)blocks, kThreads, 0, st>>>(static_cast<const uint16_t*>(x), rows, K, ld_x, codes, scales,
                                                             group_size, partial);
    if (launch_status() != AMX_OK) return AMX_ERR_CUDA;
    quant_error_final_kernel<<<1, kThreads, 0, st>>>(partial, (int)blocks, out);
    return launch_status();
}
