// Internal launchers of the two GEMM kernels.
#pragma once

#include "amx_common.cuh"

namespace amx {

int gemm_simt(const uint8_t* a_codes, const uint8_t* a_scales, const uint8_t* w_codes,
              const uint8_t* w_scales, int64_t M, int64_t N, int64_t K, int gs, float* C,
              int64_t ld_c, cudaStream_t st);

// The same kernel on operands with binary16 shared scales ([rows, K/gs, 2] uint16).
int gemm_simt_f16s(const uint8_t* a_codes, const uint16_t* a_scales, const uint8_t* w_codes,
                   const uint16_t* w_scales, int64_t M, int64_t N, int64_t K, int gs, float* C,
                   int64_t ld_c, cudaStream_t st);

// Tensor-core (tcgen05) kernel: shapes it accepts, scratch it needs, launcher.
bool gemm_tc_supported(int64_t M, int64_t N, int64_t K, int gs);
size_t gemm_tc_workspace_bytes(int64_t M, int64_t N, int64_t K);
// run_if_nonzero (optional, device word): the launch does nothing when that word is zero.  status_word
// (optional): a status word the caller has cleared, used instead of the workspace's first word.
int gemm_tc(const uint8_t* a_codes, const uint8_t* a_scales, const uint8_t* w_codes,
            const uint8_t* w_scales, int64_t M, int64_t N, int64_t K, float* C, int64_t ld_c,
            void* workspace, cudaStream_t st, const int* run_if_nonzero = nullptr, int* status_word = nullptr);
// The same product with the cast of the bf16 activation X [M, ld_a] done inside the kernel.
int gemm_tc_cast(const void* x, int64_t ld_a, const uint8_t* w_codes, const uint8_t* w_scales, int64_t M,
                 int64_t N, int64_t K, float* C, int64_t ld_c, void* workspace, cudaStream_t st);
int gemm_tc_status(const void* workspace, cudaStream_t st);

// Weight-streaming kernel for at most 64 rows of A (mma.sync on exactly decoded bf16, K ranges over a cluster):
// the workspace holds the decoded rows; gemm_rows_cast casts the bf16 rows X [M, ld_x] itself.
bool gemm_rows_supported(int64_t M, int64_t N, int64_t K, int gs);
size_t gemm_rows_workspace_bytes(int64_t M, int64_t K);
int gemm_rows(const uint8_t* a_codes, const uint8_t* a_scales, const uint8_t* w_codes, const uint8_t* w_scales,
              int64_t M, int64_t N, int64_t K, float* C, int64_t ld_c, void* workspace, cudaStream_t st);
int gemm_rows_cast(const void* x, int64_t ld_x, const uint8_t* w_codes, const uint8_t* w_scales, int64_t M, int64_t N,
                   int64_t K, float* C, int64_t ld_c, void* workspace, cudaStream_t st);

// FP4-pipe kernel (four block-scaled MMAs per tile pair): same contract; the workspace also holds
// the prepared operands (sign planes, UE4M3 scale-factor blocks, row offsets).
bool gemm_fp4_supported(int64_t M, int64_t N, int64_t K, int gs);
size_t gemm_fp4_workspace_bytes(int64_t M, int64_t N, int64_t K);
int gemm_fp4(const uint8_t* a_codes, const uint8_t* a_scales, const uint8_t* w_codes,
             const uint8_t* w_scales, int64_t M, int64_t N, int64_t K, float* C, int64_t ld_c,
             void* workspace, cudaStream_t st, bool gate_on_flushed = false);
// The same in two phases, so that an operand (typically the weight) is prepared once and reused.
size_t gemm_fp4_prepared_bytes(int64_t rows, int64_t K, bool is_weight);
// flushed_total (optional, device): incremented by the number of nonzero scales that fell below the UE4M3 range
// of their row and were flushed; the per-row counts are in the row words either way.
int gemm_fp4_prepare(const uint8_t* codes, const uint8_t* scales, int64_t rows, int64_t K, bool is_weight,
                     void* prepared, cudaStream_t st, int64_t layout_rows = 0 /* 0: rows */, int* flushed_total = nullptr);
int gemm_fp4_quantize_prepared(const void* x, int64_t rows, int64_t K, bool is_weight, uint8_t* codes,
                               uint8_t* scales, void* prepared, cudaStream_t st, int64_t layout_rows = 0,
                               int format = AMX_FMT_AMXFP4, int* flushed_total = nullptr);
int quantize_rows_prepared(const void* x, int64_t rows, int64_t K, uint8_t* codes, uint8_t* scales, void* pos,
                           void* neg, uint8_t* sf_pos, uint8_t* sf_neg, int* row_exp, int nk64, int64_t padded_rows,
                           cudaStream_t st, int format = AMX_FMT_AMXFP4, int* flushed_total = nullptr);
const int* gemm_fp4_row_words(const void* prepared, int64_t rows, int64_t K, bool is_weight);
// Softmax of the rows of S, rounded to bf16 and cast in one launch (cols % 32 == 0); pos == nullptr: canonical
// output only.  gemm_fp4_softmax_prepared lays the prepared operand out like gemm_fp4_quantize_prepared.
int softmax_cast_rows(const float* S, int64_t rows, int64_t cols, int64_t ld_s, float alpha, uint8_t* codes,
                      uint8_t* scales, void* pos, void* neg, uint8_t* sf_pos, uint8_t* sf_neg, int* row_exp, int nk64,
                      int64_t padded_rows, cudaStream_t st, int causal = 0);
int gemm_fp4_softmax_prepared(const float* S, int64_t rows, int64_t cols, int64_t ld_s, float alpha, bool is_weight,
                              uint8_t* codes, uint8_t* scales, void* prepared, cudaStream_t st, int causal = 0);
// A prepared operand that stacks several matrices row-wise (rows_total rows, laid out for layout_rows >=
// rows_total rows) and the first row of the one to multiply; row0 % 128 == 0.  A right-hand operand whose 256-row
// tiles can reach past rows_total needs layout_rows >= rows_total + 128.
struct Fp4Operand {
    const void* prepared;
    int64_t rows_total, layout_rows, row0;
};
int gemm_fp4_prepared_at(const Fp4Operand& a, const Fp4Operand& w, int64_t M, int64_t N, int64_t K, float* C,
                         int64_t ld_c, void* workspace, cudaStream_t st, size_t workspace_bytes = 256,
                         const int* gate = nullptr /* device word: the kernel does nothing when it is nonzero */,
                         const float* scale_a = nullptr, const float* scale_w = nullptr /* device: one factor per
                         operand; every result is multiplied by their product (NVFP4 tensor scales) */,
                         bool one_plane = false /* the caller states that neither operand has a second sign plane:
                         full-width tiles run the deeper one-plane pipeline, which reports AMX_ERR_FLAGS in the status
                         word when a tile has a second plane after all */,
                         bool out_bf16 = false /* C points to bf16 [M, ld_c]: results rounded to nearest even */);
// workspace that lets the kernel cut K into ranges for products with few output tiles (256 bytes otherwise)
size_t gemm_fp4_prepared_workspace_bytes(int64_t M, int64_t N, int64_t K);
// C[m][n] = sum over `slices` partial products [slices][M][N], in slice order (defined with the bf16-decode kernel)
int reduce_slices(const float* part, int slices, int64_t M, int64_t N, float* C, int64_t ld_c, cudaStream_t st,
                  const int* run_if_nonzero = nullptr);
// Fused attention for head dimension 128 (attention_fp4.cu): both products and the softmax in two launches, logits
// and attention map never in global memory.  Operands prepared ahead, heads stacked row-wise.
bool attn_fused_supported(int64_t L, int64_t d);
size_t attn_fused_scratch_bytes(int64_t heads, int64_t L);
int attn_fused(const Fp4Operand& q, const Fp4Operand& k, const Fp4Operand& vt, int heads, int64_t L, float alpha, int causal,
               void* scratch, float* O, void* workspace /* 256 B: status word */, cudaStream_t st, void* dbg_bits = nullptr,
               uint8_t* dbg_codes = nullptr, uint8_t* dbg_scales = nullptr, void* dbg_prepared = nullptr,
               int kv_group = 1 /* query heads per head of keys and values; k and vt then stack heads / kv_group heads */);
int quantize_cols_batched(const void* x, int64_t batch, int64_t R, int64_t C, uint8_t* codes, uint8_t* scales,
                          cudaStream_t st);
int gemm_fp4_prepared(const void* a_prepared, const void* w_prepared, int64_t M, int64_t N, int64_t K,
                      float* C, int64_t ld_c, void* workspace /* 256 B: status word */, cudaStream_t st,
                      size_t workspace_bytes = 256, const int* gate = nullptr);

}  // namespace amx
