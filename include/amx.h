/*
 * amx.h - C ABI of the AMXFP4 quantize + GEMM library for NVIDIA B200 (sm_100a).
 *
 * AMXFP4 (arXiv 2411.09909, Sections 4.2-4.3, Eq. 1): FP4 E2M1 elements in groups
 * of 32 along the reduction axis; each group carries two shared FP8 E5M2 scales,
 * one applied to the elements whose sign bit is 0 and one to those whose sign
 * bit is 1.  Decoded value = (-1)^s * E2M1 * scale_s.
 *
 * Conventions for every entry point
 *   - Pointers are DEVICE pointers owned by the caller unless the name of the
 *     argument ends in _host.  The library allocates no device memory and keeps
 *     no state between calls; scratch comes from the caller as `workspace`.
 *     (One exception, stated at its declaration: amx_quant_gemm_static keeps its
 *     scratch in a fixed array inside the library image.)
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Work is enqueued on it; calls return without synchronising
 *     unless stated otherwise.
 *   - Return value: AMX_OK (0) or a negative amx_status; on error nothing was
 *     launched.  amx_status_string() names the code.
 *   - Quantized tensor layout ("canonical"), for a logical [rows, K] operand:
 *       codes   uint8 [rows, K/2]      byte j of a row holds element 2j in its low
 *                                      nibble and element 2j+1 in its high nibble;
 *                                      a nibble is sign<<3 | E2M1 magnitude code
 *       scales  uint8 [rows, K/gs, 2]  E5M2 bytes: [..][0] positive-side scale,
 *                                      [..][1] negative-side scale
 *     That is 4.5 bits per element at gs = 32.
 *   - group_size (gs) must be 16, 32, 64 or 128 and divide K; or gs == K (K % 8 == 0): the whole row is
 *     one group, the grouping of the worked example in Appendix B.3 (`group_size=-1` there).  Whole-row
 *     groups are taken by amx_quantize / amx_quantize_fmt, amx_dequantize and the plain GEMM kernel
 *     (amx_gemm / amx_quant_gemm pick it by themselves); the tensor-core kernels need gs = 32.
 *   - NaN / Inf inputs are outside the format's definition; results for them are
 *     unspecified (no fault).
 */
#ifndef AMX_H_
#define AMX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum amx_status {
    AMX_OK = 0,
    AMX_ERR_NULL = -1,       /* a required pointer is NULL */
    AMX_ERR_SHAPE = -2,      /* bad sizes: non-positive, K % gs != 0, unsupported gs, ld too small */
    AMX_ERR_ALIGN = -3,      /* pointer or leading dimension not aligned as documented */
    AMX_ERR_WORKSPACE = -4,  /* workspace missing or smaller than amx_workspace_bytes() */
    AMX_ERR_FLAGS = -5,      /* unknown or contradictory flags */
    AMX_ERR_CUDA = -6,       /* a CUDA runtime call failed (launch or copy) */
    AMX_ERR_DEVICE = -7,     /* the device is not compute capability 10.x */
    AMX_ERR_TIMEOUT = -8,    /* a bounded device-side wait expired (reported by amx_gemm_status) */
    AMX_ERR_TOO_LARGE = -9   /* the problem needs more scratch than a fixed-capacity entry point holds */
} amx_status;

/* formats for amx_quantize_fmt / amx_quantize_prepared_fmt.  The two symmetric ones are the formats the
 * paper compares AMXFP4 with; they are stored in AMXFP4's layout with the one shared scale of a group in both
 * scale bytes, so every other entry point (dequantize, GEMMs, attention) takes them unchanged. */
#define AMX_FMT_AMXFP4 0    /* two E5M2 scales per group, selected by the element's sign (Section 4.3) */
#define AMX_FMT_SYM_FP8 1   /* one E5M2 scale per group, nearest to max|x| / 6 (Section 4.2 without the split) */
#define AMX_FMT_MXFP4 2     /* Algorithm 1: scale 2^(floor(log2 max|x|) - 2), stored as the E5M2 byte of that power
                             * of two; exponents above 15 are stored as 2^15, below -16 as a zero scale */
/* power-of-two scale variants of the shared-scale ablation (amx_quantize_fmt only; for the FP4 GEMM follow with
 * amx_prepare, which finds rows whose two scales agree by itself) */
#define AMX_FMT_AMXFP4_POT 3        /* per-sign scales, each Algorithm 1's power of two ("AMXFP4, shared scale PoT"
                                     * of the worked example in Appendix B.3) */
#define AMX_FMT_MXFP4_POT_ROUND 4   /* one scale per group, exponent rounded instead of floored (appendix
                                     * "Determining PoT Shared Scale: Floor vs. Round"): 2^(round(log2 max|x|) - 2) */
#define AMX_FMT_AMXFP4_POT_ROUND 5  /* the same per sign */

/* flags for amx_dequantize: output element type (default bf16) */
#define AMX_OUT_BF16 0x0u
#define AMX_OUT_F32 0x1u
/* flags for amx_gemm / amx_quant_gemm: kernel choice.  Default (AMX_GEMM_AUTO): group size 32 runs on
 * the tensor cores - the FP4 kernel when M*N*K >= 2^28, the exact bf16-decode kernel below that and for
 * at most 64 rows of A against a large weight (decode-like shapes: that kernel then cuts K into slices over
 * CTAs and adds the partial products in slice order) - except that at most 64 rows of A with K >= 512 and
 * K % 128 == 0 go to the weight-streaming kernel (AMX_GEMM_ROWS); other group sizes run on the SIMT kernel.
 * AUTO never loses a scale: where it picks the FP4 kernel and preparing the operands had to flush one (see
 * AMX_GEMM_FP4), the FP4 kernel returns at once and the exact bf16-decode kernel computes the product instead.
 * The decision is taken on the device, from the count amx_gemm_flushed_scales() reports; it costs one empty
 * launch per call and the bf16-decode kernel's scratch on top of the FP4 kernel's. */
#define AMX_GEMM_AUTO 0x0u
#define AMX_GEMM_SIMT 0x10u  /* plain CUDA-core kernel: any shape, any supported gs */
#define AMX_GEMM_TC 0x20u    /* tcgen05 kernel, exact bf16 decode: AMX_ERR_SHAPE if the shape does not fit */
#define AMX_GEMM_FP4 0x40u   /* tcgen05 block-scaled FP4 kernel (four sign-pair MMAs per tile).  The kernel's
                              * scale type (UE4M3) spans 15 binades, E5M2 spans 32: per operand row the scales
                              * are shifted so that the row's largest lands in the top binade, and a nonzero
                              * scale 15 or more binades below it is FLUSHED to zero - its group then contributes
                              * nothing.  One flushed group is below 2^-14 of the row's largest group, but a row
                              * can hold K/32 - 1 of them: the error of an output is bounded by
                              * (number of flushed groups) * 2^-14 of its dominant term, i.e. up to K * 2^-19
                              * (1.6 % at K = 8192) for adversarial rows; rows whose scales span less than 15
                              * binades (all of the benchmark's data) lose nothing and the result then equals
                              * the other kernels' up to fp32 summation order.  Flushed scales are counted:
                              * amx_gemm_flushed_scales / amx_prepared_flushed_scales.  Needs the larger
                              * workspace amx_workspace_bytes() reports. */
#define AMX_GEMM_ROWS 0x100u /* weight-streaming kernel for M <= 64 rows of A (decode phase): reads the canonical
                              * weight once, exact bf16 decode, K ranges added in a fixed order; gs = 32,
                              * K % 128 == 0, else AMX_ERR_SHAPE; w_scales 4-byte aligned, else AMX_ERR_ALIGN
                              * (also when AMX_GEMM_AUTO picked this kernel) */
/* extra flag for amx_quant_gemm, only together with AMX_GEMM_TC: one launch, the GEMM's operand-staging
 * warps cast each activation tile to AMXFP4 in registers instead of reading codes a separate cast launch
 * wrote.  Bit-identical result.  The tile is cast once per column of output tiles, and the staging warps
 * are what bounds that kernel, so this is slower than the default two launches (measured 1.05x at
 * 128 x 1024 x 1024, 1.25x at 2048 x 12288 x 4096); it is for callers that must not hold the codes. */
#define AMX_GEMM_CAST_IN_KERNEL 0x80u
/* flag for amx_quant_gemm_workspace_bytes: size the scratch for a bf16 weight (amx_quant_gemm called with W_bf16) */
#define AMX_WEIGHT_BF16 0x200u
/* extra flag for amx_attention / amx_attention_map: causal mask */
#define AMX_ATTN_CAUSAL 0x1000u
/* extra flag for amx_linear_host: return after enqueueing everything, without synchronising `stream` */
#define AMX_HOST_NO_SYNC 0x2000u

/*
 * amx_quantize - direct cast of a bf16 matrix to AMXFP4 (Sections 4.2-4.3; procedure per
 * Algorithm 1 applied to each sign with the FP8 scale of Section 4.2, as in the worked example
 * of Appendix B.3).
 * Per group of gs consecutive elements of a row:
 *   pmax = largest element with sign bit 0, nmax = largest magnitude with sign bit 1;
 *   scale_side = E5M2 nearest (ties to even, saturating at 57344) to max_side / 6;
 *   magnitude  = E2M1 nearest (ties to even) to |x| / scale_side, clamped at 6 (0 if the scale is 0);
 *   the sign bit of a code is the sign bit of x.
 *   x       bf16 [rows, ld_x] row-major, ld_x >= K in elements; 16-byte aligned, ld_x % 8 == 0
 *   codes   out, [rows, K/2], 16-byte aligned (8-byte for gs = 16)
 *   scales  out, [rows, K/gs, 2], 2-byte aligned
 * K % 8 == 0 is required.  rows == 0 is a no-op.  With gs == K (whole-row groups) scales is [rows, 1, 2] and
 * codes need 4-byte alignment only.
 */
int amx_quantize(const void* x, int64_t rows, int64_t K, int64_t ld_x, int group_size,
                 uint8_t* codes, uint8_t* scales, void* stream);
/* amx_quantize for one of the AMX_FMT_* formats (AMX_ERR_FLAGS for an unknown one); AMX_FMT_AMXFP4 is
 * amx_quantize itself.  Element rounding, sign bit and zero-scale rules are the same for all formats. */
int amx_quantize_fmt(const void* x, int64_t rows, int64_t K, int64_t ld_x, int group_size, int format,
                     uint8_t* codes, uint8_t* scales, void* stream);

/*
 * amx_fake_quantize - quantize and dequantize in one pass: out[r, k] = the value amx_dequantize would return for
 * the codes and scales amx_quantize_fmt produces (any AMX_FMT_* format), as bf16, without the codes reaching memory.
 * This is the operation the paper's emulation applies to every tensor (Algorithm 1 is this routine for the MX
 * power-of-two scale; Sections 4.2-4.3 give the FP8 and the asymmetric scales).  Bit-identical to the two calls.
 *   x, out   device, bf16 [rows, ld], 16-byte aligned, ld % 8 == 0, ld >= K; out may be x (in place)
 *   group_size 16, 32, 64 or 128; K % group_size == 0
 * One launch on `stream`; nothing is synchronised; on error nothing was launched.
 */
int amx_fake_quantize(const void* x, int64_t rows, int64_t K, int64_t ld_x, int group_size, int format,
                      void* out, int64_t ld_out, void* stream);

/*
 * amx_quantize_t - the same cast with the groups running DOWN the rows of x (the strided axis):
 * x is bf16 [R, C] row-major (ld_x >= C), groups are gs consecutive rows of one column, and the
 * result is laid out as the canonical quantization of x transposed:
 *   codes [C, R/2], scales [C, R/gs, 2].
 * This is how V enters the P*V product with groups along the sequence (Appendix C: Value and the
 * self-attention map are quantized too).  R % gs == 0; gs is 16, 32 or 64 here; x 2-byte aligned.
 */
int amx_quantize_t(const void* x, int64_t R, int64_t C, int64_t ld_x, int group_size,
                   uint8_t* codes, uint8_t* scales, void* stream);

/*
 * amx_dequantize - Eq. 1 evaluated: out[r,k] = (-1)^s * E2M1 * (s ? scale_neg : scale_pos).
 * Every result has at most 5 significant bits and is exact in bf16 and in fp32.
 *   out  bf16 or fp32 (flags) [rows, ld_out], ld_out >= K; 16-byte aligned, ld_out % 8 == 0
 */
int amx_dequantize(const uint8_t* codes, const uint8_t* scales, int64_t rows, int64_t K,
                   int group_size, uint32_t flags, void* out, int64_t ld_out, void* stream);

/*
 * amx_gemm - C[m,n] = sum_k Ahat[m,k] * What[n,k] with Ahat, What the decoded operands
 * (Section 4.3: each factor uses the shared scale its own sign selects), fp32 accumulation.
 *   a_codes/a_scales  canonical [M, K];  w_codes/w_scales canonical [N, K] (both K-major)
 *   C   out fp32 [M, ld_c], ld_c >= N
 *   alignment: codes 4 bytes (16 bytes for the tensor-core kernel), scales 2 bytes, C 4 bytes
 *   (the tensor-core kernel stores vectors when C is 16-byte aligned and ld_c % 4 == 0)
 *   workspace  device scratch of at least amx_workspace_bytes(M, N, K, gs, flags) bytes,
 *              256-byte aligned (may be NULL when that size is 0)
 * M == 0 or N == 0 is a no-op.
 */
int amx_gemm(const uint8_t* a_codes, const uint8_t* a_scales,
             const uint8_t* w_codes, const uint8_t* w_scales,
             int64_t M, int64_t N, int64_t K, int group_size, uint32_t flags,
             float* C, int64_t ld_c, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Two-phase form of the AMX_GEMM_FP4 kernel, for operands that are reused (the quantized weight of a
 * layer, across calls).  amx_gemm with AMX_GEMM_FP4 prepares both operands on every call; here
 *   amx_prepare        turns one canonical operand [rows, K] (gs = 32) into its "prepared" form - the two
 *                      sign planes, the UE4M3 scale factors in the tensor cores' layout and a power-of-two
 *                      offset per row - in a caller-owned buffer of amx_prepared_bytes() bytes
 *                      (256-byte aligned).  is_weight selects the padding of the W (right-hand) operand.
 *   amx_gemm_prepared  multiplies a prepared A [M, K] with a prepared W [N, K]; same result as amx_gemm
 *                      with AMX_GEMM_FP4.  workspace: 256 bytes (status word, see amx_gemm_status) always
 *                      suffice; with amx_gemm_prepared_workspace_bytes() bytes a product with few output tiles
 *                      and a long K (a few token rows against a big weight) is cut into K ranges that run as
 *                      separate CTAs, their partial products added in range order (same result up to fp32
 *                      summation order, run-to-run identical).
 *   amx_quantize_prepared  amx_quantize (x bf16 [rows, K], contiguous rows, gs = 32) and amx_prepare in one
 *                      go: the cast kernel itself writes the sign planes, so the codes are not read again.
 *                      Writes the canonical scales too, and the canonical codes unless `codes` is NULL (a caller
 *                      that only multiplies does not need them: 0.5 of 3.7 bytes per element less to write).
 * This is how Section 4.3's product runs when the weights were cast once ahead of time.
 */
int amx_quantize_prepared(const void* x, int64_t rows, int64_t K, int group_size, int is_weight,
                          uint8_t* codes, uint8_t* scales, void* prepared, size_t prepared_bytes, void* stream);
/* The same for one of the AMX_FMT_* formats.  A symmetric format needs no split by sign: its prepared form
 * holds the signed codes as one plane, and amx_gemm_prepared issues one product per tile pair instead of four
 * (amx_prepare and amx_gemm detect operand rows whose two scales agree in every group and do the same). */
int amx_quantize_prepared_fmt(const void* x, int64_t rows, int64_t K, int group_size, int is_weight, int format,
                              uint8_t* codes, uint8_t* scales, void* prepared, size_t prepared_bytes,
                              void* stream);
size_t amx_prepared_bytes(int64_t rows, int64_t K, int group_size, int is_weight);
int amx_prepare(const uint8_t* codes, const uint8_t* scales, int64_t rows, int64_t K, int group_size,
                int is_weight, void* prepared, size_t prepared_bytes, void* stream);
size_t amx_gemm_prepared_workspace_bytes(int64_t M, int64_t N, int64_t K, int group_size);
int amx_gemm_prepared(const void* a_prepared, const void* w_prepared, int64_t M, int64_t N, int64_t K,
                      int group_size, float* C, int64_t ld_c, void* workspace, size_t workspace_bytes,
                      void* stream);
/* amx_gemm_prepared for two operands that the caller knows to be single planes: each prepared in a symmetric
 * format (AMX_FMT_SYM_FP8 or AMX_FMT_MXFP4 through amx_quantize_prepared_fmt; any canonical operand whose two
 * scales agree in every group through amx_prepare), or with all its values non-negative.  Same arguments and result.  With one product per K step the tensor cores wait for the operand loads, so this form
 * keeps twice as many K blocks in flight, in the shared memory the second planes would have taken.  The promise
 * is checked on the device, per output tile, against the operands' row words: if a tile has a second plane,
 * amx_gemm_status(workspace) returns AMX_ERR_FLAGS and C is not the product (the kernel still runs to its end
 * and touches nothing outside C).  Products narrower than 129 columns, or cut into K ranges, run the general
 * kernel, where the promise changes nothing. */
int amx_gemm_prepared_sym(const void* a_prepared, const void* w_prepared, int64_t M, int64_t N, int64_t K,
                          int group_size, float* C, int64_t ld_c, void* workspace, size_t workspace_bytes,
                          void* stream);
/* amx_gemm_prepared with options.  flags: AMX_PREP_ONE_PLANE = the promise of amx_gemm_prepared_sym;
 * AMX_PREP_OUT_BF16 = C is bf16 [M, ld_c] (2-byte aligned; 32-byte stores when C is 32-byte aligned and
 * ld_c % 16 == 0): every result is the fp32 accumulator value - what amx_gemm_prepared stores - rounded to bf16,
 * ties to even, in the epilogue.  For layers whose output feeds the next cast: half the bytes written, and no
 * separate conversion pass (Section 5 casts bf16 activations).  The K ranges of amx_gemm_prepared are not used
 * with a bf16 result (their partial sums are fp32).  Other flag bits: AMX_ERR_FLAGS. */
#define AMX_PREP_ONE_PLANE 0x1u
#define AMX_PREP_OUT_BF16 0x2u
int amx_gemm_prepared_ex(const void* a_prepared, const void* w_prepared, int64_t M, int64_t N, int64_t K,
                         int group_size, uint32_t flags, void* C, int64_t ld_c, void* workspace,
                         size_t workspace_bytes, void* stream);

/*
 * amx_quant_gemm - the fully quantized linear layer of Section 5 (the evaluation setting there casts both
 * inputs of every matrix multiplication of a decoder layer): quantizes the bf16 activation A[M, ld_a] and
 * multiplies it with the weight, which comes in exactly one of two forms:
 *   w_codes / w_scales   an already quantized weight, canonical [N, K] (then W_bf16 must be NULL), or
 *   W_bf16, ld_w         a bf16 weight [N, ld_w] that this call casts as well (then w_codes and w_scales must
 *                        be NULL): both operands of the layer are cast per call, the direct-cast setting of
 *                        Section 5 with nothing prepared ahead
 * Same result as amx_quantize (of each bf16 operand) followed by amx_gemm.  How it runs: on the FP4 kernel each
 * bf16 operand with contiguous rows is cast by one launch that also writes the kernel's operand form; on the
 * weight-streaming kernel the few rows of A are cast and decoded in one launch; otherwise amx_quantize per bf16
 * operand, then the GEMM; AMX_GEMM_TC | AMX_GEMM_CAST_IN_KERNEL asks for the kernel that casts A inside
 * (with any other kernel choice: AMX_ERR_FLAGS).  The workspace additionally holds the quantized operands:
 * amx_quant_gemm_workspace_bytes(flags | AMX_WEIGHT_BF16) with a bf16 weight.
 * A (and W_bf16) 16-byte aligned, ld_a % 8 == 0 (ld_w % 8 == 0).
 */
int amx_quant_gemm(const void* A, int64_t ld_a,
                   const uint8_t* w_codes, const uint8_t* w_scales,
                   const void* W_bf16, int64_t ld_w,
                   int64_t M, int64_t N, int64_t K, int group_size, uint32_t flags,
                   float* C, int64_t ld_c, void* workspace, size_t workspace_bytes, void* stream);

/*
 * amx_softmax_bf16 - the step between the two attention products: P = softmax(alpha * S) per
 * row in fp32, rounded to bf16 (the quantizer's input type) so that the normalised
 * self-attention map can be quantized along the key axis (Appendix C).
 *   S  fp32 [rows, ld_s];  P  out bf16 [rows, ld_p];  cols <= ld_s, ld_p
 */
int amx_softmax_bf16(const float* S, int64_t rows, int64_t cols, int64_t ld_s, float alpha,
                     void* P, int64_t ld_p, void* stream);

/*
 * amx_softmax_quantize - the same step and the cast that follows it in one kernel (Appendix C: the
 * self-attention map is quantized): per row P = softmax(alpha * S) in fp32, rounded to bf16, then cast to
 * AMXFP4 with groups of 32 along the row, exactly as amx_softmax_bf16 followed by amx_quantize would (same
 * bits), but the map never reaches memory as fp32 or bf16.
 *   S  fp32 [rows, ld_s], cols % 32 == 0;  codes u8 [rows, cols/2], scales u8 [rows, cols/32, 2]
 *   prepared  NULL, or a buffer of amx_prepared_bytes(rows, cols, 32, is_weight) bytes (256-aligned) that also
 *             receives the operand in the form amx_gemm_prepared reads (as amx_quantize_prepared writes it)
 */
int amx_softmax_quantize(const float* S, int64_t rows, int64_t cols, int64_t ld_s, float alpha,
                         uint8_t* codes, uint8_t* scales, int is_weight, void* prepared, size_t prepared_bytes,
                         void* stream);

/*
 * amx_attention - fully quantized attention, one call for all heads (Appendix C: Query, Key, the
 * self-attention map and Value are all quantized; Section 1: these are the products rotation methods
 * leave in 16 bits).  Per head h:
 *   S = AMX(Q_h) AMX(K_h)^T          groups along head_dim
 *   P = softmax(S / sqrt(d)) per row, fp32, rounded to bf16; no mask.  P itself is never stored.  When both
 *       products run on the FP4 kernel, d == 128 and L % 128 == 0, S is not stored either: one fused kernel does both
 *       products and the softmax in two launches - the first pass over Q K^T keeps per-row softmax statistics, the
 *       second recomputes each tile, normalises and casts it in registers and multiplies it with V on the tensor
 *       cores (row sums are taken tile by tile, so single elements of P may round to the neighbouring bf16 value
 *       compared with amx_softmax_quantize on a stored S; O agrees to ~1e-5 relative).  Other shapes and kernels
 *       store one head's S in the workspace.
 *   O_h = AMX(P) AMX(V_h)            groups along the key axis (V is quantized down its rows)
 *   flags    AMX_GEMM_* kernel choice for both products, optionally | AMX_ATTN_CAUSAL: query i sees keys 0..i only
 *            (the mask is applied to the logits before the softmax; masked entries of P are exactly 0).  In the
 *            fused kernel the blocks of keys that lie entirely after their queries are not visited at all.
 *   q, k, v  bf16 [heads, L, d] contiguous;  o  out fp32 [heads, L, d]
 *   d % 32 == 0, L % 32 == 0 (group size 32 on both axes)
 *   workspace  at least amx_attention_workspace_bytes_for(L, d, flags) bytes (reused head after head), 256-aligned.
 *            amx_attention_workspace_bytes(L, d) is the size that suffices for every flag: it includes one head's
 *            logits and attention map (L x L x 4.6 bytes), which the fused kernel does not need - at long
 *            sequences ask with the flags of the call (32768 tokens: 5 GB against 40 MB).
 * The heads are processed one after another on `stream`.
 */
int amx_attention(const void* q, const void* k, const void* v, int64_t heads, int64_t L, int64_t d,
                  uint32_t flags, float* o, void* workspace, size_t workspace_bytes, void* stream);
size_t amx_attention_workspace_bytes(int64_t L, int64_t d);
size_t amx_attention_workspace_bytes_for(int64_t L, int64_t d, uint32_t flags);
/*
 * amx_attention_gqa - the same with grouped queries: k and v hold kv_heads heads [kv_heads, L, d] and query head h
 * attends to head h / (heads / kv_heads) of them (heads % kv_heads == 0, else AMX_ERR_SHAPE); keys and values are
 * cast once per head of theirs.  kv_heads == heads is amx_attention; the results are those of amx_attention on
 * keys and values repeated heads / kv_heads times, bit for bit.  Same workspace.
 */
int amx_attention_gqa(const void* q, const void* k, const void* v, int64_t heads, int64_t kv_heads, int64_t L, int64_t d,
                      uint32_t flags, float* o, void* workspace, size_t workspace_bytes, void* stream);

/*
 * amx_attention_map - ONE head through the launch sequence amx_attention uses at head dimension 128 (both products
 * on the FP4 kernel, logits and attention map never stored), with the intermediate the library otherwise never
 * writes: the cast attention map.  P = softmax(Q K^T / sqrt(d)) per row, rounded to bf16 and cast to AMXFP4 in
 * registers inside the second pass over Q K^T (Appendix C: the self-attention map is quantized), then multiplied
 * with the cast V on the tensor cores in the same kernel.  Same kernels and launch sequence as amx_attention; in
 * addition the second pass stores, so that the cast can be checked against a reference:
 *   q, k, v     bf16 [L, d], d == 128, L % 128 == 0 (else AMX_ERR_SHAPE)
 *   o           out fp32 [L, d]: the head's attention output, as amx_attention computes it
 *   p_bf16      out, nullable: bf16 [L, L], the normalised map as rounded to bf16 - the cast's input
 *   p_codes     out, nullable: canonical codes [L, L/2] of that map;  p_scales  out, nullable: [L, L/32, 2]
 *   p_prepared  out: P in the FP4 kernels' operand form as the kernel feeds it to the tensor cores (positive
 *               plane, UE4M3 scale factors, row words), amx_prepared_bytes(L, L, 32, 0) bytes, 256-aligned
 *   flags       0 or AMX_ATTN_CAUSAL (blocks of 128 keys entirely after their block of 128 queries are not visited;
 *               their entries of the optional outputs are zero, those of p_prepared are not written)
 *   workspace   amx_attention_workspace_bytes(L, d) bytes
 */
int amx_attention_map(const void* q, const void* k, const void* v, int64_t L, int64_t d, uint32_t flags, float* o,
                      void* p_bf16, uint8_t* p_codes, uint8_t* p_scales, void* p_prepared, size_t prepared_bytes,
                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * amx_linear_host - one whole layer from HOST memory: copies the bf16 activation A_host[M,K] and
 * weight W_host[N,K] to the device, quantizes both, multiplies, and copies C back to
 * C_host[M,N] (fp32).  All copies and kernels are enqueued on `stream`; the call returns after
 * synchronising it - unless flags carry AMX_HOST_NO_SYNC: then it returns once everything is enqueued, the
 * caller synchronises, and calls on different streams with different workspaces overlap their copies in both
 * directions.  Host buffers should be page-locked for the copies to be asynchronous.  Runs as amx_quant_gemm
 * with a bf16 weight.  All arguments are checked before the first copy is enqueued.
 *   flags      AMX_GEMM_* kernel choice, optionally | AMX_HOST_NO_SYNC
 *   workspace  device scratch, at least amx_linear_host_workspace_bytes(M, N, K, gs, flags) bytes
 */
int amx_linear_host(const void* A_host, const void* W_host, int64_t M, int64_t N, int64_t K,
                    int group_size, uint32_t flags, float* C_host,
                    void* workspace, size_t workspace_bytes, void* stream);
/*
 * amx_linear_host_pipelined - the same layer as a pipeline over THREE streams of the caller (no hidden streams):
 * W_host goes in on stream_in and is cast once on stream_compute; the rows of A_host then go through in chunks
 * of about 2048 rows (a multiple of 128) - chunk i is copied in on stream_in, cast and multiplied on
 * stream_compute (amx_quant_gemm with the quantized weight), and its rows of C are copied out on stream_out while
 * chunk i + 1 is copied in and chunk i + 2... follow; events recorded between the streams (created and destroyed
 * inside the call) carry the dependencies.  Host-to-device and device-to-host copies so run at the same time
 * within one layer, and consecutive calls on the same three streams (each with its own workspace) keep both copy
 * directions busy across layers.  Same C as amx_linear_host, bit for bit when the chunks run the same kernel as
 * the whole product would (a chunk is a smaller product: under AMX_GEMM_AUTO it may pick another kernel, whose fp32
 * summation order differs).
 *   flags      AMX_GEMM_* kernel choice (binds every chunk: AMX_ERR_SHAPE if a chunk does not fit it),
 *              optionally | AMX_HOST_NO_SYNC (return once everything is enqueued; without it the call returns after
 *              synchronising stream_out, when C_host is complete)
 *   workspace  device scratch, amx_linear_host_pipelined_workspace_bytes() bytes, 256-aligned.  It may be used by
 *              another call only after this call's work has completed on all three streams.
 *   streams    three different streams (two equal ones: AMX_ERR_FLAGS)
 * amx_linear_host_pipelined_status: the first nonzero status word of the call's chunks (see amx_gemm_status; each
 * chunk's word is kept at the start of the workspace), or AMX_OK.  Synchronises `stream` (pass stream_compute).
 */
size_t amx_linear_host_pipelined_workspace_bytes(int64_t M, int64_t N, int64_t K, int group_size, uint32_t flags);
int amx_linear_host_pipelined(const void* A_host, const void* W_host, int64_t M, int64_t N, int64_t K,
                              int group_size, uint32_t flags, float* C_host, void* workspace,
                              size_t workspace_bytes, void* stream_in, void* stream_compute, void* stream_out);
int amx_linear_host_pipelined_status(const void* workspace, void* stream);

/*
 * amx_quant_gemm_static - amx_quant_gemm (quantized-weight form) without a workspace argument, for callers
 * that cannot allocate device memory: processes that gave the whole GPU to their own memory pool at start-up,
 * plug-ins that must not touch the allocator, and latency-critical loops that cannot afford an
 * allocation's implicit synchronisation.  (The paper has no counterpart; this is a deployment
 * convenience of this library.)  Same result as amx_quant_gemm with the same kernel choice.
 *   - flags: AMX_GEMM_AUTO, AMX_GEMM_SIMT or AMX_GEMM_TC only.  AMX_GEMM_FP4, AMX_GEMM_ROWS and
 *     AMX_GEMM_CAST_IN_KERNEL are rejected with AMX_ERR_FLAGS; AUTO may still pick any kernel.
 *   - The scratch is a fixed 16 MiB array that is part of the library image: every GPU that loads the
 *     library holds it until the process exits.  It holds whatever amx_quant_gemm would keep in its
 *     workspace: the status word, the quantized activation and, when AUTO picks the FP4 kernel, both
 *     operands in that kernel's form.  amx_quant_gemm_static_capacity() returns its size; a problem for which
 *     amx_quant_gemm_workspace_bytes() exceeds it is rejected with AMX_ERR_TOO_LARGE and nothing runs.
 *   - The entry point calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - The first call on each device looks up the array's device address, which is also when the CUDA
 *     runtime loads this part of the library onto the device and the array starts to occupy memory there:
 *     make that first call outside any stream capture and BEFORE the application's own pool takes the rest of
 *     the device, or the call fails with AMX_ERR_CUDA (nothing was launched; the error is cleared).
 *   - amx_quant_gemm_static_status() reads the status word the way amx_gemm_status does for a caller-owned
 *     workspace (AMX_ERR_TIMEOUT after a bounded device-side wait expired); it synchronises `stream`.
 *   - All calls share the one array, which keeps whatever the previous call left in it.  The
 *     call itself re-initialises what it needs; but two calls whose work overlaps on the GPU
 *     (different streams or host threads) race on the array - serialise them.
 */
int amx_quant_gemm_static(const void* A, int64_t ld_a,
                          const uint8_t* w_codes, const uint8_t* w_scales,
                          int64_t M, int64_t N, int64_t K, int group_size, uint32_t flags,
                          float* C, int64_t ld_c, void* stream);
size_t amx_quant_gemm_static_capacity(void);
int amx_quant_gemm_static_status(void* stream);

/*
 * NVFP4 and ANVFP4 - the format the paper compares AMXFP4 with in Section 5 (its table of NVFP4 / ANVFP4 results):
 * E2M1 elements in groups of 16, one FP8 E4M3 scale per group - ANVFP4: one per sign, as in AMXFP4 - and one fp32
 * scale for the whole tensor.  The paper names the parts, not the arithmetic; implemented (every step an IEEE fp32
 * operation, in this order, so that the CPU reference takes the same decisions):
 *   t = max|x| / 2688 (1 for an all-zero tensor);  group scale byte = E4M3 nearest (ties to even, saturating at 448)
 *   to (max_side * fl(1/6)) * (1/t);  element = E2M1 nearest (ties to even, clamped at 6) to x * (1 / (E4M3(byte) * t)),
 *   sign bit = sign of x;  decoded value = (-1)^s * E2M1 * E4M3(scale_s) * t.
 * amx_quantize_nvfp4  two launches (the tensor maximum, then the cast).
 *   x             bf16 [rows, ld_x], 16-byte aligned, ld_x % 8 == 0, K % 64 == 0
 *   flags         0 (NVFP4: the group's one scale is stored in both scale bytes) or AMX_NV_ASYMMETRIC (ANVFP4)
 *   codes         out, nullable: [rows, K/2] as for AMXFP4;  scales  out, nullable: E4M3 bytes [rows, K/16, 2]
 *   tensor_scale  out: TWO floats, 8-byte aligned: [0] = t, [1] = max|x|
 *   prepared      out, nullable: the operand in the FP4 tensor-core kernel's form (amx_nvfp4_prepared_bytes() bytes,
 *                 256-aligned; is_weight selects the right-hand operand's padding).  Group size 16 and E4M3 are that
 *                 kernel's native scale block and type: the scale bytes go in as they are, nothing is shifted or
 *                 flushed, and a symmetric operand is one plane.
 * amx_dequantize_nvfp4  the decoded values, fp32 (AMX_OUT_F32) or bf16 (the fp32 value rounded to nearest even).
 * amx_gemm_nvfp4  C = decoded A x decoded W^T for two prepared operands; fp32 accumulation, every result multiplied by
 *   the product of the two tensor scales.  NVFP4 x NVFP4 issues one block-scaled MMA per tile pair, ANVFP4 four.
 *   workspace: 256 bytes (status word, see amx_gemm_status).
 */
#define AMX_NV_ASYMMETRIC 0x1u
int amx_quantize_nvfp4(const void* x, int64_t rows, int64_t K, int64_t ld_x, uint32_t flags, uint8_t* codes,
                       uint8_t* scales, float* tensor_scale, int is_weight, void* prepared, size_t prepared_bytes,
                       void* stream);
size_t amx_nvfp4_prepared_bytes(int64_t rows, int64_t K, int is_weight);
int amx_dequantize_nvfp4(const uint8_t* codes, const uint8_t* scales, const float* tensor_scale, int64_t rows, int64_t K,
                         uint32_t flags, void* out, int64_t ld_out, void* stream);
int amx_gemm_nvfp4(const void* a_prepared, const void* w_prepared, int64_t M, int64_t N, int64_t K, float* C,
                   int64_t ld_c, void* workspace, size_t workspace_bytes, void* stream);
/* The same for two operands cast without AMX_NV_ASYMMETRIC (see amx_gemm_prepared_sym: the deeper one-plane
 * pipeline, AMX_ERR_FLAGS in the status word if an operand has a second plane after all). */
int amx_gemm_nvfp4_sym(const void* a_prepared, const void* w_prepared, int64_t M, int64_t N, int64_t K, float* C,
                       int64_t ld_c, void* workspace, size_t workspace_bytes, void* stream);

/*
 * FP4 with binary16 shared scales - the "FP16" row of the paper's ablation of the shared-scale encoding (appendix
 * "Ablation Study on Shared-Scale Bit-Encoding"): the quantizer of Sections 4.2-4.3 with "nearest E5M2" replaced by
 * "nearest binary16" (ties to even, subnormals kept, saturating at 65504; a quotient that rounds to zero gives a
 * zero scale and zero magnitudes).  flags: AMX_F16S_ASYMMETRIC = one scale per sign (AMXFP4 with FP16 scales),
 * 0 = one scale per group from max|x| / 6, stored in both slots; AMX_F16S_SCALE_E4M3 = the same table's "FP8
 * 1-4-3" row: the scale is the nearest FP8 E4M3 value (ties to even, subnormals kept, saturating at 448), stored as
 * the binary16 pattern of that value, so that dequantize, product and error report take it unchanged.
 *   x        device, bf16 [rows, ld_x], 16-byte aligned, ld_x % 8 == 0
 *   codes    device out/in, [rows, K/2], 4-byte aligned (layout as amx_quantize)
 *   scales   device out/in, uint16 [rows, K/group_size, 2]: binary16 bit patterns {positive side, negative side},
 *            4-byte aligned
 *   group_size 16, 32, 64 or 128; K % group_size == 0
 * amx_dequantize_f16s writes fp32 [rows, ld_out] (a decoded value has up to 13 significant bits: exact in fp32, not
 * in bf16; out 16-byte aligned, ld_out % 4 == 0).  amx_gemm_f16s: C[m, n] = sum_k Ahat[m, k] What[n, k] on the
 * CUDA cores, fp32 products (exact) and fp32 accumulation - no tensor-core type holds 13-bit operands exactly;
 * C fp32 [M, ld_c].  amx_quant_error_f16s: amx_quant_error (below) for this layout.
 * One launch each (the error report two) on `stream`; nothing is synchronised; on error nothing was launched.
 */
#define AMX_F16S_ASYMMETRIC 0x1u
#define AMX_F16S_SCALE_E4M3 0x2u
int amx_quantize_f16s(const void* x, int64_t rows, int64_t K, int64_t ld_x, int group_size, uint32_t flags,
                      uint8_t* codes, uint16_t* scales, void* stream);
int amx_dequantize_f16s(const uint8_t* codes, const uint16_t* scales, int64_t rows, int64_t K, int group_size,
                        float* out, int64_t ld_out, void* stream);
int amx_gemm_f16s(const uint8_t* a_codes, const uint16_t* a_scales, const uint8_t* w_codes, const uint16_t* w_scales,
                  int64_t M, int64_t N, int64_t K, int group_size, float* C, int64_t ld_c, void* stream);
int amx_quant_error_f16s(const void* x, int64_t rows, int64_t K, int64_t ld_x, const uint8_t* codes,
                         const uint16_t* scales, int group_size, double* out, void* workspace,
                         size_t workspace_bytes, void* stream);

/*
 * amx_quant_error - squared error of a quantized tensor against its bf16 source, split as the appendix
 * "Determining PoT Shared Scale: Floor vs. Round" splits the error of a shared scale: elements whose magnitude
 * exceeds the largest value their side represents (|x| > 6 * scale of the element's side) make up the
 * max-clamping error, all others the rounding error.
 *   x, codes, scales   as for amx_quantize / amx_quantize_fmt (any of the formats, group size 16..128);
 *                      x 16-byte aligned with ld_x % 8 == 0, codes 8-byte aligned
 *   out        device, 4 doubles: sum x^2, sum (x - xhat)^2, the part of the latter from clamped elements,
 *              the number of clamped elements (exact).  Squares are added in fp32 within chunks of 16 consecutive
 *              elements and in fp64 above (relative error of a sum < 2^-20), in a fixed order: the same bits on
 *              every run.
 *   workspace  device scratch of amx_quant_error_workspace_bytes() bytes, 8-byte aligned
 * Two launches on `stream`; nothing is synchronised.  rows == 0 writes zeros.
 */
int amx_quant_error(const void* x, int64_t rows, int64_t K, int64_t ld_x, const uint8_t* codes,
                    const uint8_t* scales, int group_size, double* out, void* workspace, size_t workspace_bytes,
                    void* stream);
size_t amx_quant_error_workspace_bytes(void);

/* Scratch sizes (bytes; 0 is possible).  Return 0 for invalid shapes. */
size_t amx_workspace_bytes(int64_t M, int64_t N, int64_t K, int group_size, uint32_t flags);
size_t amx_quant_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K, int group_size, uint32_t flags);
size_t amx_linear_host_workspace_bytes(int64_t M, int64_t N, int64_t K, int group_size, uint32_t flags);

/* Which kernel amx_gemm would run for this shape and flags: one AMX_GEMM_* kernel bit, or 0 when the flags
 * cannot be honoured for the shape. */
uint32_t amx_gemm_kernel_for(int64_t M, int64_t N, int64_t K, int group_size, uint32_t flags);

/*
 * Status word of the most recent amx_gemm / amx_quant_gemm / amx_gemm_prepared that used `workspace` (its
 * first word, for every kernel that takes a workspace): AMX_OK, or AMX_ERR_TIMEOUT when a bounded wait inside
 * a tensor-core kernel expired (the kernel then stopped issuing work, released its resources and returned; C is
 * not valid), or AMX_ERR_FLAGS after amx_gemm_prepared_sym / amx_gemm_nvfp4_sym on an operand with two planes.  The weight-streaming kernel has no such wait and always leaves AMX_OK.  Synchronises `stream`.
 */
int amx_gemm_status(const void* workspace, void* stream);

/*
 * Flushed scales (see AMX_GEMM_FP4).  amx_gemm_flushed_scales: how many nonzero scales of the two operands the
 * most recent amx_gemm / amx_quant_gemm that used `workspace` flushed while preparing them for the FP4 kernel
 * (the workspace's second word; 0 for the other kernels); under AMX_GEMM_AUTO a nonzero count means the exact
 * bf16-decode kernel computed the product.  amx_prepared_flushed_scales: the same count for one prepared operand
 * (amx_prepare, amx_quantize_prepared[_fmt], amx_softmax_quantize), read from its per-row words.
 * Both synchronise `stream` and return the count, or a negative amx_status.
 */
int64_t amx_gemm_flushed_scales(const void* workspace, void* stream);
int64_t amx_prepared_flushed_scales(const void* prepared, int64_t rows, int64_t K, int group_size, int is_weight,
                                    void* stream);

/*
 * amx_selftest_wait_timeout - exercises the bounded-wait protocol of the tensor-core kernels without a GEMM:
 * one CTA allocates tensor memory, starts a bulk copy, then waits on an mbarrier nothing arrives at.  After
 * `polls` polls (1..65536) the waiting role gives up, records AMX_ERR_TIMEOUT in the status word
 * (amx_gemm_status(workspace) returns it), the other roles leave through the abort flag, the copy is drained,
 * tensor memory is released and the kernel returns; the context stays usable.  (No counterpart in the paper: a
 * check of this library's failure handling.)
 *   workspace  at least 2048 bytes, 256-aligned.  After the kernel, int words 8..11 tell how warps 0..3 left
 *              their wait (2 = gave up at its own limit, 3 = left through the abort flag, 1 = the wait
 *              completed, which must not happen) and word 12 is 1 when the copy in flight was seen to land.
 */
int amx_selftest_wait_timeout(void* workspace, size_t workspace_bytes, uint32_t polls, void* stream);

const char* amx_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* AMX_H_ */
