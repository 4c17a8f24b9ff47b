// Pieces shared by the tensor-core codec kernels: the argument block of the bulk bf16 encode and the row stride of
// a byte code tile.  A fp32 matrix enters the tensor cores as a sum of bf16 parts, W = W1 + W2 (+ W3),
// W1 = bf16(W), W2 = bf16(W - W1), W3 = bf16(W - W1 - W2); with bf16 inputs the products are exact, so three parts
// keep fp32-level accuracy.
#pragma once
#include "common.cuh"

namespace spectra {

constexpr int kLdCode = kD + 4;  // row stride of a byte code tile

struct EncodeTcArgs {
  const __nv_bfloat16* x; int side; int64_t n_param_sets; const int32_t* pos0; int32_t n_new;
  int64_t stride_unit, stride_token; const float* w_enc; const float* mean_rot; const uint8_t* widths;
  uint8_t* cache; const int64_t* unit_offset; int32_t* status;
};

}  // namespace spectra
