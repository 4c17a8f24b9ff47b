// Second moments of spectra_fit_basis on the 5th-generation tensor cores (tcgen05), for bf16 inputs:
// S = sum_t x_t^T x_t as X^T X with both operands taken from the same token tile, and s = sum_t x_t.
//
// One CTA per unit-side walks that unit's tokens 128 at a time.  A tile [128 tokens][128 channels] arrives by TMA
// in the 128-byte swizzled form (two blocks of 64 channels); read with the tokens as the contraction index it is
// an MN-major operand, and it serves as A (M = channels) and as B (N = channels) of the same MMA.  Products of bf16
// values are exact in fp32; a chunk of 256 tokens (16 MMAs of K = 16) is accumulated in fp32 in tensor memory, then
// added in fp64 to the running totals, chunk after chunk in token order: the sums do not depend on how the launch was
// scheduled (no atomics), so a fit is reproducible bit for bit.  Tokens past the end read as zeros.
// Six warps: 0..3 add finished chunks to the fp64 totals (thread r owns row r of S; the totals live in shared memory
// column by column, so that a warp's accesses are conflict-free) and sum the columns of each tile for s; warp 4 (one
// lane) issues the copies through a ring of three slots, warp 5 (one lane) the MMAs into two accumulator tiles.
// All waits are bounded; after a timeout the unit's moments are written as NaN (and `flag`, if given, gets
// SPECTRA_STATUS_WAIT_TIMEOUT): every output fitted from them is then NaN.
#pragma once
#include "umma.cuh"

namespace spectra {

constexpr int kMuThreads = 192;
constexpr int kMuSlots = 3;
constexpr int kMuChunkTiles = 2;                          // tiles (of 128 tokens) per fp32 chunk
// bf16 A and B, fp32 D, both operands MN-major, M = N = 128
constexpr uint32_t kMuIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

struct MomentsSmem {
  alignas(1024) uint8_t x[kMuSlots][kTile * kD * 2];
  double S[kD * kD];                                      // entry (r, c) at c * 128 + r
  alignas(8) uint64_t full[kMuSlots], free_[kMuSlots], acc_full[2], acc_free[2];
  uint32_t tmem_base;
};
static_assert(sizeof(MomentsSmem) + 1024 <= 227 * 1024, "the moments kernel's shared memory must fit one SM");

__global__ void __launch_bounds__(kMuThreads, 1) moments_umma_kernel(const __grid_constant__ CUtensorMap xmap, int64_t n_tokens,
                                                                     double* S_out, double* s_out, int64_t out_stride,
                                                                     int32_t* flag) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned char* smem_al = smem_raw + ((1024u - (um_smem_u32(smem_raw) & 1023u)) & 1023u);
  MomentsSmem& M = *reinterpret_cast<MomentsSmem*>(smem_al);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int u = blockIdx.x;
  const int n_tiles = (int)((n_tokens + kTile - 1) / kTile);
  const int n_chunks = (n_tiles + kMuChunkTiles - 1) / kMuChunkTiles;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kMuSlots; s++) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(um_smem_u32(&M.full[s])) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 5;" ::"r"(um_smem_u32(&M.free_[s])) : "memory");   // MMAs + four warps
    }
    for (int b = 0; b < 2; b++) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(um_smem_u32(&M.acc_full[b])) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 4;" ::"r"(um_smem_u32(&M.acc_free[b])) : "memory");
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(um_smem_u32(&M.tmem_base)), "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  for (int i = threadIdx.x; i < kD * kD; i += kMuThreads) M.S[i] = 0.0;
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tb = M.tmem_base;
  bool ok = true;

  if (warp == 4) {
    if (lane == 0) {
#pragma unroll 1
      for (int t = 0; t < n_tiles && ok; t++) {
        const int s = t % kMuSlots;
        if (t >= kMuSlots) ok = um_wait(um_smem_u32(&M.free_[s]), (uint32_t)((t / kMuSlots - 1) & 1));
        if (!ok) break;
        const uint32_t bar = um_smem_u32(&M.full[s]), dst = um_smem_u32(M.x[s]);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(kTile * kD * 2) : "memory");
#pragma unroll 1
        for (int c = 0; c < 2; c++)
          asm volatile(
              "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
                  dst + 16384u * c),
              "l"(&xmap), "r"(64 * c), "r"(t * kTile), "r"(u), "r"(bar)
              : "memory");
      }
    }
  } else if (warp == 5) {
    if (lane == 0) {
#pragma unroll 1
      for (int c = 0; c < n_chunks && ok; c++) {
        const int b = c & 1;
        if (c >= 2) ok = um_wait(um_smem_u32(&M.acc_free[b]), (uint32_t)(((c >> 1) - 1) & 1));
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
        for (int tt = 0; tt < kMuChunkTiles && ok; tt++) {
          const int t = c * kMuChunkTiles + tt;
          if (t >= n_tiles) break;
          const int s = t % kMuSlots;
          ok = um_wait(um_smem_u32(&M.full[s]), (uint32_t)((t / kMuSlots) & 1));
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          // A and B are the same bytes: channels along M / N in two blocks of 64 (16 KB apart), 8 tokens per 1 KB
          const uint64_t d0 = um_desc_sw128(um_smem_u32(M.x[s]), 16384, 1024);
#pragma unroll
          for (int ks = 0; ks < kTile / 16; ks++)
            um_mma_ss(tb + 128u * b, d0 + (uint64_t)(128 * ks), d0 + (uint64_t)(128 * ks), kMuIdesc, (tt | ks) != 0);
          um_commit(um_smem_u32(&M.free_[s]));
        }
        if (ok) um_commit(um_smem_u32(&M.acc_full[b]));
      }
    }
  } else {
    const int r = threadIdx.x;                            // row of S, and the channel whose column sum this thread keeps
    const uint32_t lane_base = tb + ((uint32_t)(warp * 32) << 16);
    auto wait_w = [&](const uint64_t* bar, uint32_t parity) { return __all_sync(0xffffffffu, um_wait(um_smem_u32(bar), parity)) != 0; };
    double col = 0.0;
#pragma unroll 1
    for (int c = 0; c < n_chunks && ok; c++) {
      // ---- s: this thread's channel over the tokens of the chunk's tiles (fp32 inside a tile, fp64 across tiles)
#pragma unroll 1
      for (int tt = 0; tt < kMuChunkTiles && ok; tt++) {
        const int t = c * kMuChunkTiles + tt;
        if (t >= n_tiles) break;
        const int s = t % kMuSlots;
        ok = wait_w(&M.full[s], (uint32_t)((t / kMuSlots) & 1));
        if (!ok) break;
        const uint8_t* blk = M.x[s] + (r >> 6) * 16384;
        const int c16 = (r & 63) >> 3, e = r & 7;
        float part[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 8
        for (int tok = 0; tok < kTile; tok++)
          part[tok & 3] += __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(blk + tok * 128 + ((c16 ^ (tok & 7)) << 4) + 2 * e));
        col += (double)((part[0] + part[1]) + (part[2] + part[3]));
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(um_smem_u32(&M.free_[s])) : "memory");
      }
      if (!ok) break;
      // ---- S: the chunk's fp32 products into the fp64 totals
      const int b = c & 1;
      ok = wait_w(&M.acc_full[b], (uint32_t)((c >> 1) & 1));
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
      for (int q = 0; q < 4; q++) {
        float v[32];
        um_ld16(lane_base + 128u * b + 32 * q, v);
        um_ld16(lane_base + 128u * b + 32 * q + 16, v + 16);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int e = 0; e < 32; e++) M.S[(32 * q + e) * kD + r] += (double)v[e];
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(um_smem_u32(&M.acc_free[b])) : "memory");
    }
    // a wait that gave up leaves no usable sums: the unit's moments become NaN, and so does everything fitted from them
    double* So = S_out + (int64_t)u * out_stride;
    const double bad = __longlong_as_double(0x7ff8000000000000LL);
    for (int c = 0; c < kD; c++) So[(int64_t)r * kD + c] = ok ? M.S[c * kD + r] : bad;
    s_out[(int64_t)u * out_stride + r] = ok ? col : bad;
  }
  if (!ok && flag) atomicOr(flag, SPECTRA_STATUS_WAIT_TIMEOUT);
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(M.tmem_base), "r"(256u) : "memory");
}

}  // namespace spectra
