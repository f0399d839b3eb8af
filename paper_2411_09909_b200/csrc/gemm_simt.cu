// AMXFP4 x AMXFP4 -> fp32 matrix product on CUDA cores (any shape, any supported group size).
// C[m,n] = sum_k Ahat[m,k] * What[n,k]: every factor is decoded with the shared scale its own
// sign selects (arXiv 2411.09909, Section 4.3), products and sums in fp32.
// This is the general-shape path and the on-device cross-check for the tensor-core kernel.
// The same kernel takes binary16 shared scales (ScaleT = uint16_t, the scale-encoding ablation of the appendix):
// an E2M1 magnitude times a binary16 scale has at most 13 significant bits, exact in fp32.
#include <cuda_fp16.h>

#include "amx_common.cuh"
#include "gemm.cuh"

namespace amx {
namespace {

constexpr int BM = 64, BN = 64, BK = 32, PAD = 4;

__device__ __forceinline__ float scale_value(uint8_t b) { return e5m2_to_float(b); }
__device__ __forceinline__ float scale_value(uint16_t h) { return __half2float(__ushort_as_half(h)); }

// Decodes 8 codes of one row (one 32-bit word) into column `r` of a [BK][B + PAD] tile.
template <typename ScaleT>
__device__ __forceinline__ void decode_word(const uint8_t* __restrict__ codes,
                                            const ScaleT* __restrict__ scales, int64_t row,
                                            int64_t rows, int64_t K, int gs, int64_t k,
                                            float (*tile)[BM + PAD], int r, int kk) {
    uint32_t nib = 0;
    float sp = 0.f, sn = 0.f;
    if (row < rows && k < K) {
        nib = *reinterpret_cast<const uint32_t*>(codes + row * (K / 2) + k / 2);
        const ScaleT* sc = scales + (row * (K / gs) + k / gs) * 2;
        sp = scale_value(sc[0]);
        sn = scale_value(sc[1]);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t c = (nib >> (4 * i)) & 15u;
        const float mag = e2m1_mag_to_float(c & 7u);
        tile[kk + i][r] = (c & 8u) ? -(mag * sn) : mag * sp;
    }
}

template <typename ScaleT>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const uint8_t* __restrict__ a_codes, const ScaleT* __restrict__ a_scales,
                 const uint8_t* __restrict__ w_codes, const ScaleT* __restrict__ w_scales,
                 int64_t M, int64_t N, int64_t K, int gs, float* __restrict__ C, int64_t ld_c) {
    __shared__ __align__(16) float As[BK][BM + PAD];
    __shared__ __align__(16) float Ws[BK][BN + PAD];
    const int t = threadIdx.x, tx = t % 16, ty = t / 16;
    const int64_t m0 = (int64_t)blockIdx.y * BM, n0 = (int64_t)blockIdx.x * BN;
    float acc[4][4] = {};
    for (int64_t k0 = 0; k0 < K; k0 += BK) {
        const int r = t / 4, kk = (t % 4) * 8;
        decode_word(a_codes, a_scales, m0 + r, M, K, gs, k0 + kk, As, r, kk);
        decode_word(w_codes, w_scales, n0 + r, N, K, gs, k0 + kk, Ws, r, kk);
        __syncthreads();
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            const float4 a = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            const float4 w = *reinterpret_cast<const float4*>(&Ws[k][tx * 4]);
            const float av[4] = {a.x, a.y, a.z, a.w}, wv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], wv[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t m = m0 + ty * 4 + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t n = n0 + tx * 4 + j;
            if (n < N) C[m * ld_c + n] = acc[i][j];
        }
    }
}

}  // namespace

int gemm_simt(const uint8_t* a_codes, const uint8_t* a_scales, const uint8_t* w_codes,
              const uint8_t* w_scales, int64_t M, int64_t N, int64_t K, int gs, float* C,
              int64_t ld_c, cudaStream_t st) {
    dim3 grid((unsigned)((N + BN - 1) / BN), (unsigned)((M + BM - 1) / BM));
    if (grid.y > 65535) return AMX_ERR_SHAPE;
    gemm_simt_kernel<uint8_t><<<grid, 256, 0, st>>>(a_codes, a_scales, w_codes, w_scales, M, N, K, gs, C, ld_c);
    return launch_status();
}

int gemm_simt_f16s(const uint8_t* a_codes, const uint16_t* a_scales, const uint8_t* w_codes,
                   const uint16_t* w_scales, int64_t M, int64_t N, int64_t K, int gs, float* C,
                   int64_t ld_c, cudaStream_t st) {
    dim3 grid((unsigned)((N + BN - 1) / BN), (unsigned)((M + BM - 1) / BM));
    if (grid.y > 65535) return AMX_ERR_SHAPE;
    gemm_simt_kernel<uint16_t><<<grid, 256, 0, st>>>(a_codes, a_scales, w_codes, w_scales, M, N, K, gs, C, ld_c);
    return launch_status();
}

}  // namespace amx
