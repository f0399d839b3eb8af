// Quantize-dequantize in one pass ("fake quantization"): xhat = decode(cast(x)) written back as bf16, for AMXFP4
// and the comparison formats of amx_quantize_fmt.  This is what the paper's emulation does to every tensor
// (arXiv 2411.09909, Algorithm 1 is exactly this routine for the MX power-of-two scale; Sections 4.2-4.3 for the
// FP8 and asymmetric scales): accuracy studies need the decoded tensor, not the codes.  Same arithmetic as the cast
// kernels (cast_math.cuh) and the exact bf16 decode (decode_math.cuh), so the result equals amx_quantize_fmt
// followed by amx_dequantize bit for bit, without the codes ever reaching memory: 4 bytes per element instead of
// 2.56 + 2.56.
//
// Each thread owns EPT = min(gs, 32) consecutive elements, a group is TPG = gs / EPT consecutive lanes (as in the
// cast kernel); the whole row as one group (group_size == K) is not offered here.
#include "cast_math.cuh"
#include "decode_math.cuh"

namespace amx {
namespace {

constexpr int kThreads = 256;

template <int EPT, int TPG, int FMT>
__global__ void __launch_bounds__(kThreads)
fake_quantize_kernel(const uint4* __restrict__ x, int64_t n_items, int64_t items_per_row, int64_t ld_vec,
                     uint4* __restrict__ out, int64_t ld_out_vec) {
    constexpr int NV = EPT / 8;
    const int64_t v = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    const bool live = v < n_items;
    const int64_t row = live ? v / items_per_row : 0, col = live ? v % items_per_row : 0;
    uint32_t w[NV * 4];
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        uint4 q = make_uint4(0, 0, 0, 0);
        if (live) q = __ldg(x + row * ld_vec + col * NV + j);
        w[4 * j] = q.x; w[4 * j + 1] = q.y; w[4 * j + 2] = q.z; w[4 * j + 3] = q.w;
    }
    uint32_t c = cast::side_maxima<NV * 4>(w);
#pragma unroll
    for (int d = 1; d < TPG; d <<= 1) c = __vmaxs2(c, __shfl_xor_sync(0xFFFFFFFFu, c, d));
    float inv_p, inv_n;
    const uint32_t sc = cast::group_scales_fmt<FMT>(c, inv_p, inv_n);
    const decode::GroupTables tb = decode::make_tables(sc);
    if (!live) return;
#pragma unroll
    for (int j = 0; j < NV; ++j)
        out[row * ld_out_vec + col * NV + j] = decode::decode_word(cast::encode8(w + 4 * j, inv_p, inv_n), tb);
}

template <int EPT, int TPG, int FMT>
int launch(const void* x, int64_t rows, int64_t K, int64_t ld_x, void* out, int64_t ld_out, cudaStream_t st) {
    const int64_t items_per_row = K / EPT, n_items = rows * items_per_row, blocks = (n_items + kThreads - 1) / kThreads;
    if (blocks > 0x7FFFFFFF) return AMX_ERR_SHAPE;
    fake_quantize_kernel<EPT, TPG, FMT><<<(unsigned)blocks, kThreads, 0, st>>>(
        static_cast<const uint4*>(x), n_items, items_per_row, ld_x / 8, static_cast<uint4*>(out), ld_out / 8);
    return launch_status();
}

template <int FMT>
int launch_gs(const void* x, int64_t rows, int64_t K, int64_t ld_x, int gs, void* out, int64_t ld_out, cudaStream_t st) {
    switch (gs) {
        case 16: return launch<16, 1, FMT>(x, rows, K, ld_x, out, ld_out, st);
        case 32: return launch<32, 1, FMT>(x, rows, K, ld_x, out, ld_out, st);
        case 64: return launch<32, 2, FMT>(x, rows, K, ld_x, out, ld_out, st);
        default: return launch<32, 4, FMT>(x, rows, K, ld_x, out, ld_out, st);
    }
}

}  // namespace
}  // namespace amx

extern "C" int amx_fake_quantize(const void* x, int64_t rows, int64_t K, int64_t ld_x, int group_size, int format,
                                 void* out, int64_t ld_out, void* stream) {
    using namespace amx;
    if (format < AMX_FMT_AMXFP4 || format > AMX_FMT_AMXFP4_POT_ROUND) return AMX_ERR_FLAGS;
    if (!fixed_group_size(group_size) || rows < 0 || K <= 0 || K % group_size || ld_x < K || ld_out < K) return AMX_ERR_SHAPE;
    if (rows == 0) return AMX_OK;
    if (!x || !out) return AMX_ERR_NULL;
    if (!aligned(x, 16) || ld_x % 8 || !aligned(out, 16) || ld_out % 8) return AMX_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    switch (format) {
        case AMX_FMT_SYM_FP8: return launch_gs<1>(x, rows, K, ld_x, group_size, out, ld_out, st);
        case AMX_FMT_MXFP4: return launch_gs<2>(x, rows, K, ld_x, group_size, out, ld_out, st);
        case AMX_FMT_AMXFP4_POT: return launch_gs<3>(x, rows, K, ld_x, group_size, out, ld_out, st);
        case AMX_FMT_MXFP4_POT_ROUND: return launch_gs<4>(x, rows, K, ld_x, group_size, out, ld_out, st);
        case AMX_FMT_AMXFP4_POT_ROUND: return launch_gs<5>(x, rows, K, ld_x, group_size, out, ld_out, st);
        default: return launch_gs<0>(x, rows, K, ld_x, group_size, out, ld_out, st);
    }
}
