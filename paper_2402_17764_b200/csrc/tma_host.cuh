// Host side of the TMA tensor maps the GEMM kernels use: the driver's encoder, looked up through the runtime
// (the library does not link against libcuda), and the two maps every form of the GEMM needs.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "internal.cuh"

namespace bitlinear {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// cuTensorMapEncodeTiled, or null if the driver does not offer it.
inline EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// int8 activations [rows][K bytes], row-major; box = 128 bytes x box_rows rows, 128-byte swizzle; rows and columns
// past the end read 0.
inline bool encode_activation_map(CUtensorMap *map, const int8_t *Xq, int64_t rows, int64_t K, int box_rows)
{
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K};
    const cuuint32_t box[2] = {128u, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t *>(Xq), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Packed weights as [row blocks][column tiles][256 words]; box = box_row_blocks row blocks x 2 column tiles (one
// 128-wide k block).  Tiles past the end read as zero; the activations there are zero too (columns >= K), and
// output rows >= N are never stored.
inline bool encode_packed_weight_map(CUtensorMap *map, const void *packed, int64_t N, int64_t K, int box_row_blocks)
{
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return false;
    const cuuint64_t tiles_k = (cuuint64_t)((K + kTileCols - 1) / kTileCols);
    const cuuint64_t tiles_n = (cuuint64_t)((N + kTileRows - 1) / kTileRows);
    const cuuint64_t dims[3] = {kTileBytes / 4, tiles_k, tiles_n};
    const cuuint64_t strides[2] = {(cuuint64_t)kTileBytes, tiles_k * kTileBytes};
    const cuuint32_t box[3] = {kTileBytes / 4, 2u, (cuuint32_t)box_row_blocks};
    const cuuint32_t estr[3] = {1, 1, 1};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<void *>(packed), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same packed weights as rows of 128 bytes (eight per tile) with the 128-byte swizzle: the box (two column tiles
// x four row blocks = 8 KiB) lands with the byte order of the plain map above, except that the 16-byte piece at offset o
// stands at o ^ (((o >> 7) & 7) << 4).  A warp that reads the pieces (slab s, slot 4 g + tq) of the eight g at once then
// touches eight different bank groups (decode_tc.cu).
inline bool encode_packed_weight_map_swizzled(CUtensorMap *map, const void *packed, int64_t N, int64_t K, int box_row_blocks)
{
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return false;
    const cuuint64_t tiles_k = (cuuint64_t)((K + kTileCols - 1) / kTileCols);
    const cuuint64_t tiles_n = (cuuint64_t)((N + kTileRows - 1) / kTileRows);
    const cuuint64_t dims[3] = {128u, tiles_k * (kTileBytes / 128), tiles_n};
    const cuuint64_t strides[2] = {128u, tiles_k * kTileBytes};
    const cuuint32_t box[3] = {128u, 2u * (kTileBytes / 128), (cuuint32_t)box_row_blocks};
    const cuuint32_t estr[3] = {1, 1, 1};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void *>(packed), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

} // namespace bitlinear
