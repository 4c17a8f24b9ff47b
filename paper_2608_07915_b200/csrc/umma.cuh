// Wrappers around the 5th-generation tensor-core instructions (tcgen05) and bounded mbarrier waits, shared by the
// kernels that run dense products: shared-memory operand descriptors without swizzle (a core matrix is 8 rows of 16
// bytes), MMA issue with both operands in shared memory, tensor-memory loads and stores, commit.
#pragma once
#include <cuda.h>
#include "common.cuh"

namespace spectra {

__device__ __forceinline__ uint32_t um_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint64_t um_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  // shared-memory matrix descriptor, no swizzle: start address, leading (K direction) and stride (M/N direction)
  // byte offsets between core matrices, all in 16-byte units
  return (uint64_t)((saddr >> 4) & 0x3FFF) | ((uint64_t)((lbo >> 4) & 0x3FFF) << 16) |
         ((uint64_t)((sbo >> 4) & 0x3FFF) << 32) | ((uint64_t)1 << 46);
}
// D (tensor memory) (+)= A (shared) x B (shared); M = 128, N = 128, K = 16; bf16 in, fp32 out
__device__ __forceinline__ void um_mma_ss(uint32_t d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile("{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p; }" ::"r"(d),
               "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
               : "memory");
}
__device__ __forceinline__ void um_ld16(uint32_t a, float* r) {
  uint32_t v[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(a));
#pragma unroll
  for (int i = 0; i < 16; i++) r[i] = __uint_as_float(v[i]);
}
// bf16 A and B, fp32 D, A K-major, B MN-major, N = 128, M = 128
constexpr uint32_t kUmIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

// Bounded wait for a phase of an mbarrier.  Each poll may suspend the thread for up to about a microsecond (the hint),
// so a warp that waits long (the producer) does not spend issue slots on polling.
__device__ __forceinline__ bool um_wait(uint32_t bar, uint32_t parity) {
  uint32_t done = 0;
#ifdef UM_WAIT_SPIN
  for (int it = 0; it < (1 << 26) && !done; ++it)
    asm volatile("{ .reg .pred p; mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
#else
#ifndef UM_WAIT_HINT
#define UM_WAIT_HINT 1000u
#endif
  for (int it = 0; it < (1 << 21) && !done; ++it)
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3; selp.u32 %0, 1, 0, p; }"
                 : "=r"(done) : "r"(bar), "r"(parity), "r"(UM_WAIT_HINT) : "memory");
#endif
  return done != 0;
}

// shared-memory matrix descriptor, 128-byte swizzle: rows of 128 bytes in groups of 8 (1024 bytes, sbo apart); lbo is
// the distance between 64-element blocks along M/N of an MN-major operand (unused for K-major)
__device__ __forceinline__ uint64_t um_desc_sw128(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((saddr >> 4) & 0x3FFF) | ((uint64_t)((lbo >> 4) & 0x3FFF) << 16) | ((uint64_t)((sbo >> 4) & 0x3FFF) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
__device__ __forceinline__ void um_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

}  // namespace spectra
