// Host-side description of a prepared operand of the FP4 tensor-core kernels, shared by the GEMM and the attention
// kernel: where its parts lie, and the TMA tensor map over its sign planes.
//
// A prepared operand [rows, K] (group size 32) consists of, in this order, each part padded to 256 bytes:
//   the two sign planes, [rows][K/2] bytes each (positive first): every 4-bit code in the plane of its sign bit,
//     zero in the other (a symmetric format keeps its signed codes in the first plane);
//   the UE4M3 scale factors of the two planes: chunks of 512 bytes per [128 rows x 64 elements], the chunks of a
//     128-row block consecutive along K (nk64 of them, K padded to whole 256-element blocks); inside a chunk byte
//     (r % 32) * 16 + (r / 32) * 4 + (k16 % 4), one scale per 16 elements - what the MMA reads once copied to TMEM;
//   one word per row: the power-of-two offset, which sides occur, how many scales were flushed (row_word()).
#pragma once
#include <cuda.h>

#include <mutex>

#include "amx_common.cuh"

namespace amx {
namespace fp4 {

constexpr int kSfChunk = kSfChunkBytes;

inline size_t up256(size_t v) { return (v + 255) / 256 * 256; }

struct OperandLayout {      // offsets inside the buffer of one prepared operand
    size_t plane, sf, exps, total;
    int64_t row_blocks;     // blocks of 128 rows the scale factors are laid out for
    int nk64;
};
// rows_per_tile: 128 for a left-hand operand, 256 for a right-hand one (rows padded to whole tiles).
inline OperandLayout operand_layout(int64_t rows, int64_t K, int rows_per_tile) {
    OperandLayout o;
    o.row_blocks = (rows + rows_per_tile - 1) / rows_per_tile * (rows_per_tile / 128);
    o.nk64 = (int)((K + 255) / 256) * 4;    // padded to whole 256-element blocks
    o.plane = up256((size_t)rows * (K / 2));
    o.sf = up256((size_t)o.row_blocks * o.nk64 * kSfChunk);
    o.exps = up256((size_t)rows * 4);      // row words
    o.total = 2 * o.plane + 2 * o.sf + o.exps;
    return o;
}

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(f);
    });
    return fn;
}

// Both sign planes of an operand as one 3-D tensor [2][rows][K/2] of bytes (plane_stride bytes apart);
// box = {row_bytes, box_rows, planes}, 128- or 64-byte swizzle, zero fill outside.
inline bool make_map(CUtensorMap* map, const void* base, int64_t rows, int64_t K, size_t plane_stride, int box_rows,
                     int row_bytes, int planes = 2) {
    EncodeTiledFn fn = encode_tiled();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)(K / 2), (cuuint64_t)rows, 2};
    const cuuint64_t strides[2] = {(cuuint64_t)(K / 2), (cuuint64_t)plane_stride};
    const cuuint32_t box[3] = {(cuuint32_t)row_bytes, (cuuint32_t)box_rows, (cuuint32_t)planes};   // 1: positive plane only
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace fp4
}  // namespace amx
