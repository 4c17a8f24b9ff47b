// Host helper: TMA tensor maps over [unit or page][token][channel] bf16 arrays.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include "common.cuh"

namespace spectra {

// Tensor map over the bf16 input of a bulk encode: dimensions (channel, token, unit), box 8 channels x 128 tokens, no
// swizzle, zeros outside.  The driver's encoder is looked up through the runtime (no link against the driver library).
inline bool make_token_map(CUtensorMap* map, const void* x, int64_t n_tokens, int64_t n_units, int64_t stride_token,
                    int64_t stride_unit, bool swizzle128 = false) {
  typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                               const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static EncodeFn fn = nullptr;
  if (!fn) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess || !sym ||
        q != cudaDriverEntryPointSuccess)
      return false;
    fn = reinterpret_cast<EncodeFn>(sym);
  }
  if (n_tokens < 1 || n_units < 1) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)n_tokens, (cuuint64_t)n_units};
  // a single unit or token leaves its stride unused; the encoder still wants a legal value
  const cuuint64_t strides[2] = {(cuuint64_t)(stride_token > 0 ? stride_token : kD) * 2,
                                 (cuuint64_t)(stride_unit > 0 ? stride_unit : n_tokens * kD) * 2};
  // plain: 8 channels (one 16-byte column of core matrices) per copy; 128-byte swizzle: 64 channels per copy, the
  // 16-byte pieces of a token's 128-byte row XOR-ed with the row index modulo 8
  const cuuint32_t box[3] = {swizzle128 ? 64u : 8u, (cuuint32_t)kTile, 1}, estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(x), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


}  // namespace spectra
