// Pieces shared by the tensor-core codec kernels: the argument block of the bulk bf16 encode, shared-memory row
// strides, and the ldmatrix / mma.sync (bf16, fp32 accumulate) wrappers the reconstruction kernel uses.
// A fp32 matrix enters the tensor cores as a sum of bf16 parts, W = W1 + W2 (+ W3), W1 = bf16(W),
// W2 = bf16(W - W1), W3 = bf16(W - W1 - W2); with bf16 inputs the products are exact, so three parts keep
// fp32-level accuracy.
#pragma once
#include "common.cuh"

namespace spectra {

constexpr int kLdB16 = kD + 8;   // bf16 row stride of staged tiles (272 bytes: conflict-free ldmatrix)
constexpr int kLdCode = kD + 4;  // row stride of a byte code tile

struct EncodeTcArgs {
  const __nv_bfloat16* x; int side; int64_t n_param_sets; const int32_t* pos0; int32_t n_new;
  int64_t stride_unit, stride_token; const float* w_enc; const float* mean_rot; const uint8_t* widths;
  uint8_t* cache; const int64_t* unit_offset; int32_t* status;
};

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* p) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* p) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

}  // namespace spectra
