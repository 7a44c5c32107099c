// Host side of the TMA loads: tensor maps for the [B*H, L, d] bf16 operand tensors.
// cuTensorMapEncodeTiled is reached through the runtime's driver entry point
// query, so the library does not link against libcuda.
#include "ap_common.cuh"

namespace ap {

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

}  // namespace

// [B*H, L, d] bf16 tensor, boxes of box_rows rows x 64 elements, 128-byte swizzle, zero fill outside.
bool make_tile_map_bf16(CUtensorMap *m, const void *base, int BH, int L, int d, int box_rows) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)L, (cuuint64_t)BH};
  cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)L * d * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  cuuint32_t elem_strides[3] = {1, 1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, elem_strides,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// [B*H, L, 128] bf16 tensor seen as [B*H][L/8][half][8 rows][64 elements]: one box brings box_rows rows of
// both 64-element halves and lays them out as [8-row group][half][8 rows][128 bytes] (128-byte swizzle), so
// that a 128-wide operand tile is one copy and rows stay contiguous whatever the box height.  Needs
// L % 8 == 0 (a ragged last group of eight rows would read past the tensor).
bool make_split_map_bf16_d128(CUtensorMap *m, const void *base, int BH, int L, int box_rows) {
  EncodeTiledFn enc = encode_fn();
  if (!enc || L % 8 != 0 || box_rows % 8 != 0) return false;
  cuuint64_t dims[5] = {64, 8, 2, (cuuint64_t)(L / 8), (cuuint64_t)BH};
  cuuint64_t strides[4] = {256, 128, 2048, (cuuint64_t)L * 256};
  cuuint32_t box[5] = {64, 8, 2, (cuuint32_t)(box_rows / 8), 1};
  cuuint32_t elem_strides[5] = {1, 1, 1, 1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(base), dims, strides, box, elem_strides,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// [H, Lq, Lk] fp32 tensor, boxes of 128 rows x 32 columns (128 bytes), 128-byte swizzle, zero fill outside.
// Needs Lk % 4 == 0 (row pitch a multiple of 16 bytes).
bool make_tile_map_f32(CUtensorMap *m, const void *base, int H, int Lq, int Lk, int box_rows) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  cuuint64_t dims[3] = {(cuuint64_t)Lk, (cuuint64_t)Lq, (cuuint64_t)H};
  cuuint64_t strides[2] = {(cuuint64_t)Lk * 4, (cuuint64_t)Lq * Lk * 4};
  cuuint32_t box[3] = {32, (cuuint32_t)box_rows, 1};
  cuuint32_t elem_strides[3] = {1, 1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void *>(base), dims, strides, box, elem_strides,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace ap
