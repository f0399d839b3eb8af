// C-ABI entry points that combine kernels: GEMM dispatch, quantize+GEMM, the host-buffer
// layer call, workspace sizing and status strings.
#include <cmath>
#include <vector>

#include "gemm.cuh"

namespace amx {
namespace {

constexpr size_t kAlign = 256;
inline size_t round_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

bool gemm_shape_ok(int64_t M, int64_t N, int64_t K, int gs) {
    return valid_group_size(gs, K) && M >= 0 && N >= 0 && K > 0 && K % gs == 0 && K % 8 == 0;
}

constexpr uint32_t kKernelMask = AMX_GEMM_SIMT | AMX_GEMM_TC | AMX_GEMM_FP4 | AMX_GEMM_ROWS;

// The kernel to run (one AMX_GEMM_* bit), or 0 when the flags cannot be honoured for this shape.
uint32_t pick_kernel(int64_t M, int64_t N, int64_t K, int gs, uint32_t flags) {
    const uint32_t want = flags & kKernelMask;
    if (want & (want - 1)) return 0;                                   // more than one kernel asked for
    if (want == AMX_GEMM_FP4) return gemm_fp4_supported(M, N, K, gs) ? AMX_GEMM_FP4 : 0;
    const bool tc = gemm_tc_supported(M, N, K, gs);
    if (want == AMX_GEMM_TC) return tc ? AMX_GEMM_TC : 0;
    if (want == AMX_GEMM_SIMT) return AMX_GEMM_SIMT;
    const bool rows = gemm_rows_supported(M, N, K, gs);
    if (want == AMX_GEMM_ROWS) return rows ? AMX_GEMM_ROWS : 0;
    // AMX_GEMM_AUTO: the FP4-pipe kernel for anything that fills the machine (it is about twice as fast as
    // the bf16-decode kernel); the exact bf16-decode kernel for small products (below 2^28 multiply-adds), where
    // launch count matters more than throughput - the FP4 route costs two launches more: one preparation per
    // operand, and under AUTO the gated exact kernel behind it; the SIMT kernel for group sizes the tensor-core kernels do not take.
    // A few token rows against a big weight (decode-like): too few 128 x 256 tiles to fill the machine, and the
    // FP4 kernel would have to prepare the whole weight for them; the bf16-decode kernel slices K over CTAs.
    // At most 64 token rows: the weight-streaming kernel reads the canonical weight once.
    if (rows && K >= 512) return AMX_GEMM_ROWS;
    const int64_t tiles = ((M + 127) / 128) * ((N + 255) / 256);
    if (tc && M <= 64 && tiles < 148 && K >= 1024) return AMX_GEMM_TC;      // K not a multiple of 128
    if (gemm_fp4_supported(M, N, K, gs) && (double)M * (double)N * (double)K >= 256.0 * 1024.0 * 1024.0) return AMX_GEMM_FP4;
    return tc ? AMX_GEMM_TC : AMX_GEMM_SIMT;
}

// AMX_GEMM_AUTO on the FP4 kernel: when preparing the operands flushed a scale (see to_ue4m3), the FP4 kernel
// returns at once and the exact bf16-decode kernel runs instead - decided on the device, from the count in the
// workspace's second word.  That kernel's scratch follows the FP4 kernel's.
bool auto_fallback(uint32_t flags, uint32_t kernel) { return (flags & kKernelMask) == AMX_GEMM_AUTO && kernel == AMX_GEMM_FP4; }

size_t kernel_workspace(uint32_t kernel, int64_t M, int64_t N, int64_t K, bool fallback = false) {
    if (kernel == AMX_GEMM_TC) return round_up(gemm_tc_workspace_bytes(M, N, K));
    if (kernel == AMX_GEMM_FP4)
        return round_up(gemm_fp4_workspace_bytes(M, N, K)) + (fallback ? round_up(gemm_tc_workspace_bytes(M, N, K)) : 0);
    if (kernel == AMX_GEMM_ROWS) return round_up(gemm_rows_workspace_bytes(M, K));
    return 0;
}

struct QuantSizes {
    size_t codes, scales;
};
QuantSizes quant_sizes(int64_t rows, int64_t K, int gs) {
    return {round_up((size_t)rows * (size_t)(K / 2)), round_up((size_t)rows * (size_t)(K / gs) * 2)};
}

constexpr uint32_t kQuantGemmFlags = kKernelMask | AMX_GEMM_CAST_IN_KERNEL | AMX_WEIGHT_BF16;

}  // namespace
}  // namespace amx

using namespace amx;

extern "C" uint32_t amx_gemm_kernel_for(int64_t M, int64_t N, int64_t K, int group_size, uint32_t flags) {
    if (!gemm_shape_ok(M, N, K, group_size)) return 0;
    return pick_kernel(M, N, K, group_size, flags);
}

extern "C" size_t amx_workspace_bytes(int64_t M, int64_t N, int64_t K, int group_size, uint32_t flags) {
    if (!gemm_shape_ok(M, N, K, group_size)) return 0;
    const uint32_t kernel = pick_kernel(M, N, K, group_size, flags);
    return kernel_workspace(kernel, M, N, K, auto_fallback(flags, kernel));
}

extern "C" size_t amx_quant_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K, int group_size, uint32_t flags) {
    if (!gemm_shape_ok(M, N, K, group_size)) return 0;
    const QuantSizes a = quant_sizes(M, K, group_size), w = quant_sizes(N, K, group_size);
    // the first 256 bytes always hold the status word and the flushed-scale count, whichever kernel runs
    size_t gemm_ws = amx_workspace_bytes(M, N, K, group_size, flags & kKernelMask);
    if (gemm_ws < 256) gemm_ws = 256;
    return gemm_ws + a.codes + a.scales + ((flags & AMX_WEIGHT_BF16) ? w.codes + w.scales : 0);
}

extern "C" size_t amx_linear_host_workspace_bytes(int64_t M, int64_t N, int64_t K, int group_size, uint32_t flags) {
    if (!gemm_shape_ok(M, N, K, group_size)) return 0;
    return amx_quant_gemm_workspace_bytes(M, N, K, group_size, (flags & kKernelMask) | AMX_WEIGHT_BF16) +
           round_up((size_t)M * K * 2) + round_up((size_t)N * K * 2) + round_up((size_t)M * N * 4);
}

extern "C" int amx_gemm(const uint8_t* a_codes, const uint8_t* a_scales, const uint8_t* w_codes,
                        const uint8_t* w_scales, int64_t M, int64_t N, int64_t K, int group_size,
                        uint32_t flags, float* C, int64_t ld_c, void* workspace, size_t workspace_bytes,
                        void* stream) {
    if (flags & ~kKernelMask) return AMX_ERR_FLAGS;
    if (!gemm_shape_ok(M, N, K, group_size) || ld_c < N) return AMX_ERR_SHAPE;
    uint32_t kernel = pick_kernel(M, N, K, group_size, flags);
    if (!kernel) return ((flags & kKernelMask) & ((flags & kKernelMask) - 1)) ? AMX_ERR_FLAGS : AMX_ERR_SHAPE;
    if (M == 0 || N == 0) return AMX_OK;
    if (!a_codes || !a_scales || !w_codes || !w_scales || !C) return AMX_ERR_NULL;
    if (!aligned(a_codes, 4) || !aligned(w_codes, 4) || !aligned(a_scales, 2) || !aligned(w_scales, 2) ||
        !aligned(C, 4))
        return AMX_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (kernel == AMX_GEMM_SIMT)
        return gemm_simt(a_codes, a_scales, w_codes, w_scales, M, N, K, group_size, C, ld_c, st);
    if (!aligned(a_codes, 16) || !aligned(w_codes, 16)) return AMX_ERR_ALIGN;
    // AUTO picked the weight-streaming kernel but the weight's scales miss its alignment (4-byte asynchronous
    // copies): the plain kernel takes any 2-byte aligned scales and needs no scratch
    if (kernel == AMX_GEMM_ROWS && !aligned(w_scales, 4)) {
        if ((flags & kKernelMask) == AMX_GEMM_ROWS) return AMX_ERR_ALIGN;
        return gemm_simt(a_codes, a_scales, w_codes, w_scales, M, N, K, group_size, C, ld_c, st);
    }
    const bool fallback = auto_fallback(flags, kernel);
    const size_t need = kernel_workspace(kernel, M, N, K, fallback);
    if (need && (!workspace || workspace_bytes < need)) return AMX_ERR_WORKSPACE;
    if (need && !aligned(workspace, kAlign)) return AMX_ERR_ALIGN;
    if (kernel == AMX_GEMM_FP4) {
        int rc = gemm_fp4(a_codes, a_scales, w_codes, w_scales, M, N, K, C, ld_c, workspace, st, fallback);
        if (rc != AMX_OK || !fallback) return rc;
        int* words = static_cast<int*>(workspace);       // [0] status, [1] flushed scales
        return gemm_tc(a_codes, a_scales, w_codes, w_scales, M, N, K, C, ld_c,
                       static_cast<uint8_t*>(workspace) + round_up(gemm_fp4_workspace_bytes(M, N, K)), st, words + 1, words);
    }
    if (kernel == AMX_GEMM_ROWS)
        return gemm_rows(a_codes, a_scales, w_codes, w_scales, M, N, K, C, ld_c, workspace, st);
    return gemm_tc(a_codes, a_scales, w_codes, w_scales, M, N, K, C, ld_c, workspace, st);
}

extern "C" size_t amx_prepared_bytes(int64_t rows, int64_t K, int group_size, int is_weight) {
    if (rows <= 0 || !gemm_fp4_supported(rows, rows, K, group_size)) return 0;
    return round_up(gemm_fp4_prepared_bytes(rows, K, is_weight != 0));
}

extern "C" int amx_prepare(const uint8_t* codes, const uint8_t* scales, int64_t rows, int64_t K, int group_size,
                           int is_weight, void* prepared, size_t prepared_bytes, void* stream) {
    if (rows <= 0 || !gemm_fp4_supported(rows, rows, K, group_size)) return AMX_ERR_SHAPE;
    if (!codes || !scales || !prepared) return AMX_ERR_NULL;
    if (prepared_bytes < amx_prepared_bytes(rows, K, group_size, is_weight)) return AMX_ERR_WORKSPACE;
    if (!aligned(codes, 16) || !aligned(scales, 2) || !aligned(prepared, kAlign)) return AMX_ERR_ALIGN;
    return gemm_fp4_prepare(codes, scales, rows, K, is_weight != 0, prepared, static_cast<cudaStream_t>(stream));
}

extern "C" int amx_quantize_prepared(const void* x, int64_t rows, int64_t K, int group_size, int is_weight,
                                     uint8_t* codes, uint8_t* scales, void* prepared, size_t prepared_bytes,
                                     void* stream) {
    return amx_quantize_prepared_fmt(x, rows, K, group_size, is_weight, AMX_FMT_AMXFP4, codes, scales, prepared,
                                     prepared_bytes, stream);
}

extern "C" int amx_quantize_prepared_fmt(const void* x, int64_t rows, int64_t K, int group_size, int is_weight,
                                         int format, uint8_t* codes, uint8_t* scales, void* prepared,
                                         size_t prepared_bytes, void* stream) {
    if (format != AMX_FMT_AMXFP4 && format != AMX_FMT_SYM_FP8 && format != AMX_FMT_MXFP4) return AMX_ERR_FLAGS;
    if (rows <= 0 || !gemm_fp4_supported(rows, rows, K, group_size)) return AMX_ERR_SHAPE;
    if (!x || !scales || !prepared) return AMX_ERR_NULL;       // codes may be NULL: they are then not written
    if (prepared_bytes < amx_prepared_bytes(rows, K, group_size, is_weight)) return AMX_ERR_WORKSPACE;
    if (!aligned(x, 16) || !aligned(codes, 16) || !aligned(scales, 2) || !aligned(prepared, kAlign)) return AMX_ERR_ALIGN;
    return gemm_fp4_quantize_prepared(x, rows, K, is_weight != 0, codes, scales, prepared, static_cast<cudaStream_t>(stream),
                                      0, format);
}

extern "C" size_t amx_gemm_prepared_workspace_bytes(int64_t M, int64_t N, int64_t K, int group_size) {
    if (M <= 0 || N <= 0 || !gemm_fp4_supported(M, N, K, group_size)) return 0;
    return round_up(gemm_fp4_prepared_workspace_bytes(M, N, K));
}

namespace {
int gemm_prepared_checked(const void* a_prepared, const void* w_prepared, int64_t M, int64_t N, int64_t K, int group_size,
                          void* C, int64_t ld_c, void* workspace, size_t workspace_bytes, void* stream, bool one_plane,
                          bool out_bf16) {
    if (M <= 0 || N <= 0 || !gemm_fp4_supported(M, N, K, group_size) || ld_c < N) return AMX_ERR_SHAPE;
    if (!a_prepared || !w_prepared || !C) return AMX_ERR_NULL;
    if (!workspace || workspace_bytes < 256) return AMX_ERR_WORKSPACE;
    if (!aligned(a_prepared, kAlign) || !aligned(w_prepared, kAlign) || !aligned(workspace, kAlign) ||
        !aligned(C, out_bf16 ? 2 : 4))
        return AMX_ERR_ALIGN;
    return gemm_fp4_prepared_at({a_prepared, M, M, 0}, {w_prepared, N, N, 0}, M, N, K, static_cast<float*>(C), ld_c, workspace,
                                static_cast<cudaStream_t>(stream), workspace_bytes, nullptr, nullptr, nullptr, one_plane,
                                out_bf16);
}
}  // namespace

extern "C" int amx_gemm_prepared(const void* a_prepared, const void* w_prepared, int64_t M, int64_t N, int64_t K,
                                 int group_size, float* C, int64_t ld_c, void* workspace, size_t workspace_bytes,
                                 void* stream) {
    return gemm_prepared_checked(a_prepared, w_prepared, M, N, K, group_size, C, ld_c, workspace, workspace_bytes, stream,
                                 false, false);
}

extern "C" int amx_gemm_prepared_sym(const void* a_prepared, const void* w_prepared, int64_t M, int64_t N, int64_t K,
                                     int group_size, float* C, int64_t ld_c, void* workspace, size_t workspace_bytes,
                                     void* stream) {
    return gemm_prepared_checked(a_prepared, w_prepared, M, N, K, group_size, C, ld_c, workspace, workspace_bytes, stream,
                                 true, false);
}

extern "C" int amx_gemm_prepared_ex(const void* a_prepared, const void* w_prepared, int64_t M, int64_t N, int64_t K,
                                    int group_size, uint32_t flags, void* C, int64_t ld_c, void* workspace,
                                    size_t workspace_bytes, void* stream) {
    if (flags & ~(AMX_PREP_ONE_PLANE | AMX_PREP_OUT_BF16)) return AMX_ERR_FLAGS;
    return gemm_prepared_checked(a_prepared, w_prepared, M, N, K, group_size, C, ld_c, workspace, workspace_bytes, stream,
                                 flags & AMX_PREP_ONE_PLANE, flags & AMX_PREP_OUT_BF16);
}

extern "C" int amx_quant_gemm(const void* A, int64_t ld_a, const uint8_t* w_codes, const uint8_t* w_scales,
                              const void* W_bf16, int64_t ld_w, int64_t M, int64_t N, int64_t K, int group_size,
                              uint32_t flags, float* C, int64_t ld_c, void* workspace, size_t workspace_bytes,
                              void* stream) {
    if (flags & ~kQuantGemmFlags) return AMX_ERR_FLAGS;
    const bool cast_in_kernel = flags & AMX_GEMM_CAST_IN_KERNEL;
    const bool w_is_bf16 = W_bf16 != nullptr;
    flags &= kKernelMask;
    if (cast_in_kernel && flags != AMX_GEMM_TC) return AMX_ERR_FLAGS;
    if (!gemm_shape_ok(M, N, K, group_size) || ld_a < K || ld_c < N || (w_is_bf16 && ld_w < K)) return AMX_ERR_SHAPE;
    const uint32_t kernel = pick_kernel(M, N, K, group_size, flags);
    if (!kernel) return (flags & (flags - 1)) ? AMX_ERR_FLAGS : AMX_ERR_SHAPE;
    if (M == 0 || N == 0) return AMX_OK;
    // exactly one form of the weight
    if (!A || !C || (w_is_bf16 ? (w_codes || w_scales) : (!w_codes || !w_scales))) return AMX_ERR_NULL;
    const size_t need = amx_quant_gemm_workspace_bytes(M, N, K, group_size, flags | (w_is_bf16 ? AMX_WEIGHT_BF16 : 0));
    if (!workspace || workspace_bytes < need) return AMX_ERR_WORKSPACE;
    const int code_align = kernel == AMX_GEMM_SIMT ? 4 : 16;
    if (!aligned(workspace, kAlign) || !aligned(A, 16) || ld_a % 8 || !aligned(C, 4) ||
        (w_is_bf16 ? (!aligned(W_bf16, 16) || ld_w % 8) : (!aligned(w_codes, code_align) || !aligned(w_scales, 2))))
        return AMX_ERR_ALIGN;
    if (kernel == AMX_GEMM_ROWS && !w_is_bf16 && !aligned(w_scales, 4)) return AMX_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool fallback = auto_fallback(flags, kernel);
    size_t gemm_ws = kernel_workspace(kernel, M, N, K, fallback);
    if (gemm_ws < 256) gemm_ws = 256;                       // the plain kernel has no scratch of its own: header only
    const QuantSizes a = quant_sizes(M, K, group_size), w = quant_sizes(N, K, group_size);
    uint8_t* base = static_cast<uint8_t*>(workspace);
    if (kernel == AMX_GEMM_SIMT && cudaMemsetAsync(base, 0, 8, st) != cudaSuccess) return AMX_ERR_CUDA;
    uint8_t* a_codes = base + gemm_ws;
    uint8_t* a_scales = a_codes + a.codes;
    uint8_t* wq_codes = a_scales + a.scales;               // only with a bf16 weight
    uint8_t* wq_scales = wq_codes + w.codes;
    int rc = AMX_OK;
    if (kernel == AMX_GEMM_FP4) {
        // Both casts write the kernel's operands themselves where the rows are contiguous (one launch per operand,
        // the codes are not read again); workspace: status word and flushed-scale count, prepared A, prepared W
        uint8_t* pa = base + 256;
        uint8_t* pw = pa + gemm_fp4_prepared_bytes(M, K, false);
        int* words = reinterpret_cast<int*>(base);
        if (cudaMemsetAsync(words, 0, 8, st) != cudaSuccess) return AMX_ERR_CUDA;
        if (ld_a == K) rc = gemm_fp4_quantize_prepared(A, M, K, false, a_codes, a_scales, pa, st, 0, AMX_FMT_AMXFP4, words + 1);
        else {
            rc = amx_quantize(A, M, K, ld_a, group_size, a_codes, a_scales, stream);
            if (rc == AMX_OK) rc = gemm_fp4_prepare(a_codes, a_scales, M, K, false, pa, st, 0, words + 1);
        }
        if (rc != AMX_OK) return rc;
        if (w_is_bf16 && ld_w == K)
            rc = gemm_fp4_quantize_prepared(W_bf16, N, K, true, wq_codes, wq_scales, pw, st, 0, AMX_FMT_AMXFP4, words + 1);
        else {
            if (w_is_bf16) rc = amx_quantize(W_bf16, N, K, ld_w, group_size, wq_codes, wq_scales, stream);
            if (rc == AMX_OK)
                rc = gemm_fp4_prepare(w_is_bf16 ? wq_codes : w_codes, w_is_bf16 ? wq_scales : w_scales, N, K, true, pw, st, 0,
                                      words + 1);
        }
        if (rc != AMX_OK) return rc;
        rc = gemm_fp4_prepared(pa, pw, M, N, K, C, ld_c, base, st, 256, fallback ? words + 1 : nullptr);
        if (rc != AMX_OK || !fallback) return rc;
        return gemm_tc(a_codes, a_scales, w_is_bf16 ? wq_codes : w_codes, w_is_bf16 ? wq_scales : w_scales, M, N, K, C, ld_c,
                       base + round_up(gemm_fp4_workspace_bytes(M, N, K)), st, words + 1, words);
    }
    if (w_is_bf16) {
        rc = amx_quantize(W_bf16, N, K, ld_w, group_size, wq_codes, wq_scales, stream);
        if (rc != AMX_OK) return rc;
        w_codes = wq_codes;
        w_scales = wq_scales;
    }
    if (cast_in_kernel)
        // one launch: the kernel's producers cast the activation tile in registers (same arithmetic as
        // amx_quantize, so the result is bit-identical to the two-call sequence)
        return gemm_tc_cast(A, ld_a, w_codes, w_scales, M, N, K, C, ld_c, base, st);
    if (kernel == AMX_GEMM_ROWS)
        // the cast of the few rows writes the decoded operand of the weight-streaming kernel directly: two launches
        return gemm_rows_cast(A, ld_a, w_codes, w_scales, M, N, K, C, ld_c, base, st);
    rc = amx_quantize(A, M, K, ld_a, group_size, a_codes, a_scales, stream);
    if (rc != AMX_OK) return rc;
    return amx_gemm(a_codes, a_scales, w_codes, w_scales, M, N, K, group_size, kernel, C, ld_c, base, gemm_ws, stream);
}

extern "C" int amx_linear_host(const void* A_host, const void* W_host, int64_t M, int64_t N, int64_t K,
                               int group_size, uint32_t flags, float* C_host, void* workspace,
                               size_t workspace_bytes, void* stream) {
    const bool no_sync = flags & AMX_HOST_NO_SYNC;
    flags &= ~AMX_HOST_NO_SYNC;
    if (flags & ~kKernelMask) return AMX_ERR_FLAGS;
    if (!gemm_shape_ok(M, N, K, group_size)) return AMX_ERR_SHAPE;
    if (!pick_kernel(M, N, K, group_size, flags)) return (flags & (flags - 1)) ? AMX_ERR_FLAGS : AMX_ERR_SHAPE;
    if (M == 0 || N == 0) return AMX_OK;
    if (!A_host || !W_host || !C_host) return AMX_ERR_NULL;
    const size_t need = amx_linear_host_workspace_bytes(M, N, K, group_size, flags);
    if (!workspace || workspace_bytes < need) return AMX_ERR_WORKSPACE;
    if (!aligned(workspace, kAlign)) return AMX_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // everything is validated: from here on only a failing CUDA call can stop the sequence
    const size_t qg_ws = amx_quant_gemm_workspace_bytes(M, N, K, group_size, flags | AMX_WEIGHT_BF16);
    uint8_t* p = static_cast<uint8_t*>(workspace);
    uint8_t* qg_base = p;              p += qg_ws;
    uint8_t* a_dev = p;                p += round_up((size_t)M * K * 2);
    uint8_t* w_dev = p;                p += round_up((size_t)N * K * 2);
    float* c_dev = reinterpret_cast<float*>(p);
    if (cudaMemcpyAsync(a_dev, A_host, (size_t)M * K * 2, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(w_dev, W_host, (size_t)N * K * 2, cudaMemcpyHostToDevice, st) != cudaSuccess) {
        cudaGetLastError();
        return AMX_ERR_CUDA;
    }
    const int rc = amx_quant_gemm(a_dev, K, nullptr, nullptr, w_dev, K, M, N, K, group_size, flags, c_dev, N, qg_base, qg_ws,
                                  stream);
    if (rc != AMX_OK) return rc;
    if (cudaMemcpyAsync(C_host, c_dev, (size_t)M * N * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) {
        cudaGetLastError();
        return AMX_ERR_CUDA;
    }
    if (no_sync) return AMX_OK;
    return cudaStreamSynchronize(st) == cudaSuccess ? AMX_OK : AMX_ERR_CUDA;
}

// ---- the same layer as a pipeline over three caller-owned streams
namespace {
constexpr int kHostChunksMax = 16;                       // status slots at the start of the workspace
// Rows of A per chunk: about 2048, a multiple of 128 (so that every chunk but the last fills whole tiles), at most
// kHostChunksMax chunks.
int64_t host_chunk_rows(int64_t M) {
    int64_t n = (M + 2047) / 2048;
    if (n > kHostChunksMax) n = kHostChunksMax;
    if (n < 1) n = 1;
    const int64_t rows = ((M + n - 1) / n + 127) / 128 * 128;
    return rows < M ? rows : M;
}
struct HostLayout {
    size_t w_dev, w_codes, w_scales, a_dev, c_dev, qg, total;
    size_t qg_bytes;
};
HostLayout host_layout(int64_t M, int64_t N, int64_t K, int gs, uint32_t kernel_flags) {
    HostLayout h{};
    const QuantSizes w = quant_sizes(N, K, gs);
    size_t off = 256;                                    // kHostChunksMax status slots of 8 bytes (+ padding)
    h.w_dev = off;    off += round_up((size_t)N * K * 2);
    h.w_codes = off;  off += round_up(w.codes);
    h.w_scales = off; off += round_up(w.scales);
    h.a_dev = off;    off += round_up((size_t)M * K * 2);
    h.c_dev = off;    off += round_up((size_t)M * N * 4);
    h.qg = off;
    const int64_t mc = host_chunk_rows(M), last = M % mc ? M % mc : mc;     // the last chunk may pick another kernel
    const size_t q_full = amx_quant_gemm_workspace_bytes(mc, N, K, gs, kernel_flags);
    const size_t q_last = amx_quant_gemm_workspace_bytes(last, N, K, gs, kernel_flags);
    h.qg_bytes = q_full > q_last ? q_full : q_last;
    h.total = off + h.qg_bytes;
    return h;
}
}  // namespace

extern "C" size_t amx_linear_host_pipelined_workspace_bytes(int64_t M, int64_t N, int64_t K, int group_size,
                                                            uint32_t flags) {
    flags &= ~AMX_HOST_NO_SYNC;
    if ((flags & ~kKernelMask) || !gemm_shape_ok(M, N, K, group_size) || M == 0 || N == 0) return 0;
    return host_layout(M, N, K, group_size, flags).total;
}

extern "C" int amx_linear_host_pipelined(const void* A_host, const void* W_host, int64_t M, int64_t N, int64_t K,
                                         int group_size, uint32_t flags, float* C_host, void* workspace,
                                         size_t workspace_bytes, void* stream_in, void* stream_compute,
                                         void* stream_out) {
    const bool no_sync = flags & AMX_HOST_NO_SYNC;
    flags &= ~AMX_HOST_NO_SYNC;
    if (flags & ~kKernelMask) return AMX_ERR_FLAGS;
    if (!gemm_shape_ok(M, N, K, group_size)) return AMX_ERR_SHAPE;
    const int64_t mc = host_chunk_rows(M);
    // every chunk must find a kernel under these flags (an explicit kernel choice binds every chunk)
    if (!pick_kernel(M, N, K, group_size, flags)) return (flags & (flags - 1)) ? AMX_ERR_FLAGS : AMX_ERR_SHAPE;
    if (M == 0 || N == 0) return AMX_OK;
    for (int64_t m0 = 0; m0 < M; m0 += mc)
        if (!pick_kernel(M - m0 < mc ? M - m0 : mc, N, K, group_size, flags)) return AMX_ERR_SHAPE;
    if (!A_host || !W_host || !C_host) return AMX_ERR_NULL;
    if (stream_in == stream_compute || stream_out == stream_compute || stream_in == stream_out) return AMX_ERR_FLAGS;
    const HostLayout h = host_layout(M, N, K, group_size, flags);
    if (!workspace || workspace_bytes < h.total) return AMX_ERR_WORKSPACE;
    if (!aligned(workspace, kAlign)) return AMX_ERR_ALIGN;
    cudaStream_t s_in = static_cast<cudaStream_t>(stream_in), s_cmp = static_cast<cudaStream_t>(stream_compute),
                 s_out = static_cast<cudaStream_t>(stream_out);
    uint8_t* base = static_cast<uint8_t*>(workspace);
    uint8_t* w_dev = base + h.w_dev;
    uint8_t* a_dev = base + h.a_dev;
    float* c_dev = reinterpret_cast<float*>(base + h.c_dev);
    // One event per hand-over between two streams; destroying an event that is still pending is allowed (its
    // resources are released when it completes), so nothing outlives the call.
    cudaEvent_t ev = nullptr;
    auto hand_over = [&](cudaStream_t from, cudaStream_t to) -> bool {
        if (cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) != cudaSuccess) return false;
        const bool ok = cudaEventRecord(ev, from) == cudaSuccess && cudaStreamWaitEvent(to, ev, 0) == cudaSuccess;
        cudaEventDestroy(ev);
        return ok;
    };
    auto fail = [&]() { cudaGetLastError(); return AMX_ERR_CUDA; };
    // weight: in, then cast once to canonical codes and scales
    if (cudaMemsetAsync(base, 0, 256, s_cmp) != cudaSuccess) return fail();
    if (cudaMemcpyAsync(w_dev, W_host, (size_t)N * K * 2, cudaMemcpyHostToDevice, s_in) != cudaSuccess) return fail();
    if (!hand_over(s_in, s_cmp)) return fail();
    int rc = amx_quantize(w_dev, N, K, K, group_size, base + h.w_codes, base + h.w_scales, stream_compute);
    if (rc != AMX_OK) return rc;
    // activation rows in chunks: copy in | cast + multiply | copy out, each on its stream
    int slot = 0;
    for (int64_t m0 = 0; m0 < M; m0 += mc, ++slot) {
        const int64_t rows = M - m0 < mc ? M - m0 : mc;
        uint8_t* a_rows = a_dev + (size_t)m0 * K * 2;
        float* c_rows = c_dev + (size_t)m0 * N;
        if (cudaMemcpyAsync(a_rows, static_cast<const uint8_t*>(A_host) + (size_t)m0 * K * 2, (size_t)rows * K * 2,
                            cudaMemcpyHostToDevice, s_in) != cudaSuccess || !hand_over(s_in, s_cmp))
            return fail();
        rc = amx_quant_gemm(a_rows, K, base + h.w_codes, base + h.w_scales, nullptr, 0, rows, N, K, group_size, flags, c_rows,
                            N, base + h.qg, h.qg_bytes, stream_compute);
        if (rc != AMX_OK) return rc;
        // the chunk's status word and flushed-scale count, kept past the next chunk's use of the same scratch
        if (cudaMemcpyAsync(base + 8 * slot, base + h.qg, 8, cudaMemcpyDeviceToDevice, s_cmp) != cudaSuccess ||
            !hand_over(s_cmp, s_out) ||
            cudaMemcpyAsync(C_host + (size_t)m0 * N, c_rows, (size_t)rows * N * 4, cudaMemcpyDeviceToHost, s_out) != cudaSuccess)
            return fail();
    }
    if (no_sync) return AMX_OK;
    return cudaStreamSynchronize(s_out) == cudaSuccess ? AMX_OK : AMX_ERR_CUDA;
}

extern "C" int amx_linear_host_pipelined_status(const void* workspace, void* stream) {
    if (!workspace) return AMX_ERR_NULL;
    int words[2 * kHostChunksMax] = {};
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(words, workspace, sizeof(words), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return AMX_ERR_CUDA;
    }
    for (int i = 0; i < kHostChunksMax; ++i)
        if (words[2 * i] != 0) return words[2 * i];
    return AMX_OK;
}

extern "C" int amx_softmax_quantize(const float* S, int64_t rows, int64_t cols, int64_t ld_s, float alpha,
                                    uint8_t* codes, uint8_t* scales, int is_weight, void* prepared,
                                    size_t prepared_bytes, void* stream) {
    if (rows < 0 || cols <= 0 || cols % 32 || ld_s < cols) return AMX_ERR_SHAPE;
    if (rows == 0) return AMX_OK;
    if (!S || !codes || !scales) return AMX_ERR_NULL;
    if (!aligned(S, 4) || !aligned(codes, 16) || !aligned(scales, 2)) return AMX_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!prepared) return softmax_cast_rows(S, rows, cols, ld_s, alpha, codes, scales, nullptr, nullptr, nullptr, nullptr,
                                            nullptr, 0, rows, st);
    if (!gemm_fp4_supported(rows, rows, cols, 32)) return AMX_ERR_SHAPE;
    if (prepared_bytes < amx_prepared_bytes(rows, cols, 32, is_weight)) return AMX_ERR_WORKSPACE;
    if (!aligned(prepared, kAlign)) return AMX_ERR_ALIGN;
    return gemm_fp4_softmax_prepared(S, rows, cols, ld_s, alpha, is_weight != 0, codes, scales, prepared, st);
}

namespace {
// Workspace of amx_attention.  Heads are taken in chunks: the casts of Q, K and V (small per head) run once per
// chunk on the stacked heads, the two products and the softmax once per head.  Holds the canonical codes and
// scales of the chunk's Q, K and V^T and of one head's P, the logits S of one head, then either the prepared
// operands of the FP4 kernel (Q and P as left-hand, K and V^T as right-hand operands) or the other kernels' own
// scratch, and the status word.
constexpr int64_t kAttnChunk = 8, kAttnChunkFused = 16;
int64_t attn_chunk(int64_t L, int64_t d) {
    if (attn_fused_supported(L, d)) return kAttnChunkFused;   // 16 x (L / 128) items: an even load for 148 persistent CTAs
    return (L % 128 == 0 && d % 128 == 0) ? kAttnChunk : 1;
}

struct AttnLayout {
    size_t qc, qs, kc, ks, vc, vs, pc, ps, S, pq, pk, pv, pp, stats, gemm, total;
};
// fused_only: the fused kernel will run (both products on the FP4 kernel, attn_fused_supported): no room for one
// head's logits, cast map and prepared map, nor for the other kernels' scratch.
AttnLayout attn_layout(int64_t L, int64_t d, bool fused_only = false) {
    AttnLayout a;
    const int64_t hc = attn_chunk(L, d);
    const QuantSizes qd = quant_sizes(hc * L, d, 32), ql = quant_sizes(L, L, 32), qv = quant_sizes(hc * d, L, 32);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += round_up(bytes); return o; };
    a.qc = take(qd.codes); a.qs = take(qd.scales); a.kc = take(qd.codes); a.ks = take(qd.scales);
    a.vc = take(qv.codes); a.vs = take(qv.scales);
    a.pc = take(fused_only ? 0 : ql.codes); a.ps = take(fused_only ? 0 : ql.scales);
    a.S = take(fused_only ? 0 : (size_t)L * L * 4);
    // right-hand operands are laid out for 128 rows more: the last head's 256-row tiles may reach past the stack
    a.pq = take(gemm_fp4_prepared_bytes(hc * L, d, false));
    a.pk = take(gemm_fp4_prepared_bytes(hc * L + 128, d, true));
    a.pv = take(gemm_fp4_prepared_bytes(hc * d + 128, L, true));
    a.pp = take(fused_only ? 0 : gemm_fp4_prepared_bytes(L, L, false));
    a.stats = take(attn_fused_supported(L, d) ? attn_fused_scratch_bytes(hc, L) : 0);
    a.gemm = off;
    const size_t g1 = fused_only ? 0 : amx_workspace_bytes(L, L, d, 32, AMX_GEMM_TC);
    const size_t g2 = fused_only ? 0 : amx_workspace_bytes(L, d, L, 32, AMX_GEMM_TC);
    a.total = off + (g1 > g2 ? g1 : g2) + 256;
    return a;
}
}  // namespace

extern "C" size_t amx_attention_workspace_bytes(int64_t L, int64_t d) {
    if (L <= 0 || d <= 0 || L % 32 || d % 32) return 0;
    return attn_layout(L, d).total;
}

namespace {
// Whether a call with these flags runs the fused kernel.
bool attn_runs_fused(int64_t L, int64_t d, uint32_t flags) {
    flags &= ~AMX_ATTN_CAUSAL;
    if (flags & ~kKernelMask) return false;
    return attn_fused_supported(L, d) && pick_kernel(L, L, d, 32, flags) == AMX_GEMM_FP4 &&
           pick_kernel(L, d, L, 32, flags) == AMX_GEMM_FP4;
}
}  // namespace

extern "C" size_t amx_attention_workspace_bytes_for(int64_t L, int64_t d, uint32_t flags) {
    if (L <= 0 || d <= 0 || L % 32 || d % 32) return 0;
    return attn_layout(L, d, attn_runs_fused(L, d, flags)).total;
}

extern "C" int amx_attention(const void* q, const void* k, const void* v, int64_t heads, int64_t L, int64_t d,
                             uint32_t flags, float* o, void* workspace, size_t workspace_bytes, void* stream) {
    return amx_attention_gqa(q, k, v, heads, heads, L, d, flags, o, workspace, workspace_bytes, stream);
}

extern "C" int amx_attention_gqa(const void* q, const void* k, const void* v, int64_t heads, int64_t kv_heads, int64_t L,
                                 int64_t d, uint32_t flags, float* o, void* workspace, size_t workspace_bytes,
                                 void* stream) {
    const int causal = (flags & AMX_ATTN_CAUSAL) ? 1 : 0;
    flags &= ~AMX_ATTN_CAUSAL;
    if (flags & ~kKernelMask) return AMX_ERR_FLAGS;
    if (heads < 0 || L <= 0 || d <= 0 || L % 32 || d % 32) return AMX_ERR_SHAPE;
    if (heads > 0 && (kv_heads <= 0 || heads % kv_heads)) return AMX_ERR_SHAPE;
    const int64_t group = heads > 0 ? heads / kv_heads : 1;        // query heads per head of keys and values
    const uint32_t k_qk = pick_kernel(L, L, d, 32, flags), k_pv = pick_kernel(L, d, L, 32, flags);
    if (!k_qk || !k_pv) return ((flags & kKernelMask) & ((flags & kKernelMask) - 1)) ? AMX_ERR_FLAGS : AMX_ERR_SHAPE;
    if (heads == 0) return AMX_OK;
    if (!q || !k || !v || !o) return AMX_ERR_NULL;
    const AttnLayout a = attn_layout(L, d, attn_runs_fused(L, d, flags));
    if (!workspace || workspace_bytes < a.total) return AMX_ERR_WORKSPACE;
    if (!aligned(workspace, kAlign) || !aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(o, 4))
        return AMX_ERR_ALIGN;
    uint8_t* w = static_cast<uint8_t*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t gemm_bytes = a.total - a.gemm;
    const float alpha = 1.0f / sqrtf((float)d);
    float* S = reinterpret_cast<float*>(w + a.S);
    const int64_t chunk_max = attn_chunk(L, d);
    // a chunk holds whole groups of query heads (or, when a group is larger than a chunk, part of one group)
    const int64_t chunk = group >= chunk_max ? chunk_max : (chunk_max / group) * group;
    // both products on the FP4 kernel at head dimension 128: one fused kernel, logits and attention map stay on chip
    const bool fused = k_qk == AMX_GEMM_FP4 && k_pv == AMX_GEMM_FP4 && attn_fused_supported(L, d);
    const size_t head_in = (size_t)L * d * 2;                       // bytes of one head of q, k or v
    const size_t qk_codes = (size_t)L * d / 2, qk_scales = (size_t)L * (d / 32) * 2;   // one head of Q or K, canonical
    const size_t v_codes = (size_t)d * L / 2, v_scales = (size_t)d * (L / 32) * 2;     // one head of V^T
    for (int64_t h0 = 0; h0 < heads;) {
        // query heads h0 .. h0 + hc - 1 and the heads of keys and values they use, kv0 .. kv0 + kvc - 1
        const int64_t left_in_group = group - h0 % group;
        int64_t hc = heads - h0 < chunk ? heads - h0 : chunk;
        if (group >= chunk_max && hc > left_in_group) hc = left_in_group;      // never across two large groups
        const int64_t kv0 = h0 / group, kvc = (h0 + hc - 1) / group - kv0 + 1;
        const int64_t h_off = h0 - kv0 * group;                     // first query head's place inside its group
        const uint8_t* qh = static_cast<const uint8_t*>(q) + h0 * head_in;
        const uint8_t* kh = static_cast<const uint8_t*>(k) + kv0 * head_in;
        const uint8_t* vh = static_cast<const uint8_t*>(v) + kv0 * head_in;
        // casts of the chunk's heads, stacked row-wise: Q and K along head_dim, V along the sequence (V^T)
        int rc;
        if (k_qk == AMX_GEMM_FP4) {
            rc = gemm_fp4_quantize_prepared(qh, hc * L, d, false, nullptr, w + a.qs, w + a.pq, st, chunk_max * L);
            if (rc == AMX_OK)
                rc = gemm_fp4_quantize_prepared(kh, kvc * L, d, true, nullptr, w + a.ks, w + a.pk, st, chunk_max * L + 128);
        } else {
            rc = amx_quantize(qh, hc * L, d, d, 32, w + a.qc, w + a.qs, stream);
            if (rc == AMX_OK) rc = amx_quantize(kh, kvc * L, d, d, 32, w + a.kc, w + a.ks, stream);
        }
        if (rc == AMX_OK) rc = quantize_cols_batched(vh, kvc, L, d, w + a.vc, w + a.vs, st);
        if (rc == AMX_OK && k_pv == AMX_GEMM_FP4)
            rc = gemm_fp4_prepare(w + a.vc, w + a.vs, kvc * d, L, true, w + a.pv, st, chunk_max * d + 128);
        if (rc != AMX_OK) return rc;
        if (fused) {
            // head dimension 128: both products and the softmax of all the chunk's heads in two launches.  The chunk
            // starts at a group boundary unless the group is larger than a chunk, in which case it lies inside one
            // group (every head maps to the chunk's one head of keys and values either way).
            rc = attn_fused({w + a.pq, hc * L, chunk_max * L, 0}, {w + a.pk, kvc * L, chunk_max * L + 128, 0},
                            {w + a.pv, kvc * d, chunk_max * d + 128, 0}, (int)hc, L, alpha, causal, w + a.stats,
                            o + (size_t)h0 * L * d, w + a.gemm, st, nullptr, nullptr, nullptr, nullptr,
                            (int)(group >= chunk_max ? chunk_max : group));
            if (rc != AMX_OK) return rc;
            h0 += hc;
            continue;
        }
        for (int64_t i = 0; i < hc; ++i) {
            const int64_t kv = (h_off + i) / group;                 // this head's keys and values inside the chunk
            float* oh = o + (size_t)(h0 + i) * L * d;
            // S = AMX(Q) AMX(K)^T
            if (k_qk == AMX_GEMM_FP4)
                rc = gemm_fp4_prepared_at({w + a.pq, hc * L, chunk_max * L, i * L},
                                          {w + a.pk, kvc * L, chunk_max * L + 128, kv * L}, L, L, d, S, L, w + a.gemm, st);
            else
                rc = amx_gemm(w + a.qc + i * qk_codes, w + a.qs + i * qk_scales, w + a.kc + kv * qk_codes,
                              w + a.ks + kv * qk_scales, L, L, d, 32, k_qk, S, L, w + a.gemm, gemm_bytes, stream);
            if (rc != AMX_OK) return rc;
            // softmax, rounding to bf16 and the cast of P in one kernel; O = AMX(P) AMX(V)
            if (k_pv == AMX_GEMM_FP4) {
                rc = gemm_fp4_softmax_prepared(S, L, L, L, alpha, false, w + a.pc, w + a.ps, w + a.pp, st, causal);
                if (rc == AMX_OK)
                    rc = gemm_fp4_prepared_at({w + a.pp, L, L, 0}, {w + a.pv, kvc * d, chunk_max * d + 128, kv * d}, L, d, L, oh,
                                              d, w + a.gemm, st);
            } else {
                rc = softmax_cast_rows(S, L, L, L, alpha, w + a.pc, w + a.ps, nullptr, nullptr, nullptr, nullptr, nullptr, 0, L,
                                       st, causal);
                if (rc == AMX_OK)
                    rc = amx_gemm(w + a.pc, w + a.ps, w + a.vc + kv * v_codes, w + a.vs + kv * v_scales, L, d, L, 32, k_pv, oh,
                                  d, w + a.gemm, gemm_bytes, stream);
            }
            if (rc != AMX_OK) return rc;
        }
        h0 += hc;
    }
    return AMX_OK;
}

extern "C" int amx_attention_map(const void* q, const void* k, const void* v, int64_t L, int64_t d, uint32_t flags,
                                 float* o, void* p_bf16, uint8_t* p_codes, uint8_t* p_scales, void* p_prepared,
                                 size_t prepared_bytes, void* workspace, size_t workspace_bytes, void* stream) {
    const int causal = (flags & AMX_ATTN_CAUSAL) ? 1 : 0;
    if (flags & ~AMX_ATTN_CAUSAL) return AMX_ERR_FLAGS;
    if (L <= 0 || d <= 0 || !attn_fused_supported(L, d)) return AMX_ERR_SHAPE;
    if (!q || !k || !v || !o || !p_prepared) return AMX_ERR_NULL;
    const AttnLayout a = attn_layout(L, d);
    if (!workspace || workspace_bytes < a.total || prepared_bytes < amx_prepared_bytes(L, L, 32, 0)) return AMX_ERR_WORKSPACE;
    if (!aligned(workspace, kAlign) || !aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(o, 16) ||
        !aligned(p_prepared, kAlign) || !aligned(p_bf16, 16) || !aligned(p_codes, 16) || !aligned(p_scales, 2))
        return AMX_ERR_ALIGN;
    uint8_t* w = static_cast<uint8_t*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (causal) {
        // blocks of keys that lie entirely after their queries are never visited: their entries are +0
        if ((p_bf16 && cudaMemsetAsync(p_bf16, 0, (size_t)L * L * 2, st) != cudaSuccess) ||
            (p_codes && cudaMemsetAsync(p_codes, 0, (size_t)L * L / 2, st) != cudaSuccess) ||
            (p_scales && cudaMemsetAsync(p_scales, 0, (size_t)L * (L / 32) * 2, st) != cudaSuccess))
            return AMX_ERR_CUDA;
    }
    // one head through the launch sequence of amx_attention: casts of Q, K (along head_dim) and V (along the
    // sequence), then the two passes
    int rc = gemm_fp4_quantize_prepared(q, L, d, false, nullptr, w + a.qs, w + a.pq, st);
    if (rc == AMX_OK) rc = gemm_fp4_quantize_prepared(k, L, d, true, nullptr, w + a.ks, w + a.pk, st);
    if (rc == AMX_OK) rc = quantize_cols_batched(v, 1, L, d, w + a.vc, w + a.vs, st);
    if (rc == AMX_OK) rc = gemm_fp4_prepare(w + a.vc, w + a.vs, d, L, true, w + a.pv, st);
    if (rc != AMX_OK) return rc;
    return attn_fused({w + a.pq, L, L, 0}, {w + a.pk, L, L, 0}, {w + a.pv, d, d, 0}, 1, L, 1.0f / sqrtf((float)d), causal,
                      w + a.stats, o, w + a.gemm, st, p_bf16, p_codes, p_scales, p_prepared);
}

extern "C" int amx_gemm_status(const void* workspace, void* stream) {
    return gemm_tc_status(workspace, static_cast<cudaStream_t>(stream));
}

extern "C" int64_t amx_gemm_flushed_scales(const void* workspace, void* stream) {
    if (!workspace) return AMX_ERR_NULL;
    int v = 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&v, static_cast<const int*>(workspace) + 1, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return AMX_ERR_CUDA;
    }
    return v;
}

extern "C" int64_t amx_prepared_flushed_scales(const void* prepared, int64_t rows, int64_t K, int group_size, int is_weight,
                                               void* stream) {
    if (rows <= 0 || !gemm_fp4_supported(rows, rows, K, group_size)) return AMX_ERR_SHAPE;
    if (!prepared) return AMX_ERR_NULL;
    // diagnostic, off the hot path: the per-row counts sit in the operand's row words; they are summed on the host
    std::vector<int> words((size_t)rows);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(words.data(), gemm_fp4_row_words(prepared, rows, K, is_weight != 0), (size_t)rows * sizeof(int),
                        cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return AMX_ERR_CUDA;
    }
    int64_t total = 0;
    for (int w : words) total += row_word_flushed(w);
    return total;
}

extern "C" const char* amx_status_string(int status) {
    switch (status) {
        case AMX_OK: return "ok";
        case AMX_ERR_NULL: return "null pointer";
        case AMX_ERR_SHAPE: return "unsupported shape or group size";
        case AMX_ERR_ALIGN: return "misaligned pointer or leading dimension";
        case AMX_ERR_WORKSPACE: return "workspace missing or too small";
        case AMX_ERR_FLAGS: return "bad flags";
        case AMX_ERR_CUDA: return "CUDA runtime error";
        case AMX_ERR_DEVICE: return "device is not sm_100";
        case AMX_ERR_TIMEOUT: return "device-side wait timed out";
        case AMX_ERR_TOO_LARGE: return "problem exceeds the fixed scratch capacity";
        default: return "unknown status";
    }
}
