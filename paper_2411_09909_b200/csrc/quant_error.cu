// Squared error of a quantized tensor against its bf16 source, split into the max-clamping and the rounding
// part (arXiv 2411.09909, appendix "Determining PoT Shared Scale: Floor vs. Round": the output error of a shared
// scale decomposes into the error of elements beyond the largest representable magnitude and the rounding error
// of all others).  An element is clamped when |x| > 6 * (the scale of its side).
//
// Memory-bound reduction: 2 bytes of source, half a byte of codes and the scale bytes per element are read once.
// A thread takes 16 consecutive elements at a time (two 16-byte loads of the source, one 8-byte load of codes);
// x - xhat is exact in fp32 for the output of the casts (both have few significant bits and nearby exponents).
// The 16 squares of a chunk are added in fp32 (relative error below 2^-20 of the chunk's sum: all terms are
// non-negative), everything above a chunk in fp64 - fp64 arithmetic per element would bound the kernel (the
// conversions alone cost more than the memory traffic).  The clamped count is an integer.  The summation order is fixed (grid-stride per thread, shuffles in a warp, warps in
// order, then one block over the per-block partial sums), so the result is the same bits on every run.
// F16S instantiation: binary16 shared scales ([rows, K/gs, 2] uint16); xhat then has up to 13 significant bits and
// x - xhat is still exact in fp32.
#include <cuda_fp16.h>

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
    float x2 = 0.f, e2 = 0.f, c2 = 0.f;
    int clamped = 0;
    // A 3-bit E2M1 code at bits 24..22 of an fp32 pattern reads as (its value) x 2^-126 (code 1 is the subnormal
    // 2^-127); the side scales carry the 2^126 in two exact halves.
    const float up = 9223372036854775808.f;                      // 2^63
    const float sp_up = sp * up, sn_up = -sn * up, sp6 = 6.0f * sp, sn6 = 6.0f * sn;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float x = __uint_as_float((i & 1) ? (xs[i >> 1] & 0xFFFF0000u) : (xs[i >> 1] << 16));
        const uint32_t w = cs[i >> 3] >> ((i & 7) * 4);
        const bool neg = w & 8u;
        const float mag_dn = __uint_as_float((w & 7u) << 22) * up;   // value x 2^-63, exact
        const float e = fmaf(-mag_dn, neg ? sn_up : sp_up, x), ee = e * e;
        x2 = fmaf(x, x, x2);
        e2 += ee;
        if (fabsf(x) > (neg ? sn6 : sp6)) {
            c2 += ee;
            ++clamped;
        }
    }
    s.x2 += (double)x2; s.e2 += (double)e2; s.clamp2 += (double)c2; s.clamped += (double)clamped;
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

template <bool F16S>
__global__ void __launch_bounds__(kThreads) quant_error_kernel(const uint16_t* __restrict__ x, int64_t rows, int64_t K,
                                                               int64_t ld_x, const uint8_t* __restrict__ codes,
                                                               const uint8_t* __restrict__ scales, int gs_log2,
                                                               double* __restrict__ partial) {
    __shared__ double sh[kThreads / 32][4];
    // grid x walks the 16-element chunks of a row, grid y the rows: no division per chunk
    const int64_t per_row = K / 16, groups = K >> gs_log2;
    Sums s = {0, 0, 0, 0};
    for (int64_t row = blockIdx.y; row < rows; row += gridDim.y) {
        const uint16_t* xr = x + row * ld_x;
        const uint8_t* cr = codes + row * (K / 2);
        const uint8_t* sr = scales + row * groups * (F16S ? 4 : 2);
        for (int64_t c = (int64_t)blockIdx.x * kThreads + threadIdx.x; c < per_row; c += (int64_t)gridDim.x * kThreads) {
            const int64_t k = c * 16;
            const uint4* xp = reinterpret_cast<const uint4*>(xr + k);
            const uint4 xw[2] = {__ldg(xp), __ldg(xp + 1)};
            const uint2 cw = __ldg(reinterpret_cast<const uint2*>(cr + k / 2));
            if (F16S) {
                const uint32_t sc = __ldg(reinterpret_cast<const uint32_t*>(sr + (k >> gs_log2) * 4));
                add16(s, xw, cw, __half2float(__ushort_as_half((unsigned short)(sc & 0xFFFFu))),
                      __half2float(__ushort_as_half((unsigned short)(sc >> 16))));
            } else {
                const uint32_t sc = __ldg(reinterpret_cast<const unsigned short*>(sr + (k >> gs_log2) * 2));
                add16(s, xw, cw, e5m2_to_float(sc & 0xFFu), e5m2_to_float(sc >> 8));
            }
        }
    }
    const Sums t = block_sum(s, sh);
    if (threadIdx.x == 0) {
        double* p = partial + ((int64_t)blockIdx.y * gridDim.x + blockIdx.x) * 4;
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

namespace {
int quant_error(const void* x, int64_t rows, int64_t K, int64_t ld_x, const uint8_t* codes, const void* scales,
                bool f16s, int group_size, double* out, void* workspace, size_t workspace_bytes, void* stream) {
    if (!fixed_group_size(group_size) || rows < 0 || K <= 0 || K % group_size || ld_x < K) return AMX_ERR_SHAPE;
    if (!out) return AMX_ERR_NULL;
    if (rows > 0 && (!x || !codes || !scales)) return AMX_ERR_NULL;
    if (!workspace || workspace_bytes < amx_quant_error_workspace_bytes()) return AMX_ERR_WORKSPACE;
    if (!aligned(x, 16) || ld_x % 8 || !aligned(codes, 8) || !aligned(scales, f16s ? 4 : 2) || !aligned(out, 8) ||
        !aligned(workspace, 8))
        return AMX_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t per_row = K / 16;
    int64_t bx = (per_row + kThreads - 1) / kThreads;
    bx = bx > 64 ? 64 : bx;
    int64_t by = rows < 1 ? 1 : rows > kMaxBlocks / bx ? kMaxBlocks / bx : rows;
    const int64_t blocks = bx * by;
    double* partial = static_cast<double*>(workspace);
    const int gs_log2 = group_size == 16 ? 4 : group_size == 32 ? 5 : group_size == 64 ? 6 : 7;
    const dim3 grid((unsigned)bx, (unsigned)by);
    if (f16s)
        quant_error_kernel<true><<<grid, kThreads, 0, st>>>(static_cast<const uint16_t*>(x), rows, K, ld_x, codes,
                                                            static_cast<const uint8_t*>(scales), gs_log2, partial);
    else
        quant_error_kernel<false><<<grid, kThreads, 0, st>>>(static_cast<const uint16_t*>(x), rows, K, ld_x, codes,
                                                             static_cast<const uint8_t*>(scales), gs_log2, partial);
    if (launch_status() != AMX_OK) return AMX_ERR_CUDA;
    quant_error_final_kernel<<<1, kThreads, 0, st>>>(partial, (int)blocks, out);
    return launch_status();
}
}  // namespace

extern "C" int amx_quant_error(const void* x, int64_t rows, int64_t K, int64_t ld_x, const uint8_t* codes,
                               const uint8_t* scales, int group_size, double* out, void* workspace,
                               size_t workspace_bytes, void* stream) {
    return quant_error(x, rows, K, ld_x, codes, scales, false, group_size, out, workspace, workspace_bytes, stream);
}

extern "C" int amx_quant_error_f16s(const void* x, int64_t rows, int64_t K, int64_t ld_x, const uint8_t* codes,
                                    const uint16_t* scales, int group_size, double* out, void* workspace,
                                    size_t workspace_bytes, void* stream) {
    return quant_error(x, rows, K, ld_x, codes, scales, true, group_size, out, workspace, workspace_bytes, stream);
}
