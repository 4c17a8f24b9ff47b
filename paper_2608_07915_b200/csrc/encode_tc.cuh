// Bulk path of spectra_encode for bf16 inputs and scale_group 64: the 128 x 128 rotation of a tile runs on the
// tensor cores (mma.sync bf16, fp32 accumulate) with W_enc held as a three-way bf16 split
//     W = W1 + W2 + W3,  W1 = bf16(W), W2 = bf16(W - W1), W3 = bf16(W - W1 - W2)
// so that, with bf16 inputs (exact products), the rotated coordinates keep fp32-level accuracy: a code only flips
// against the fp64 reference when it sits on a rounding tie.  One CTA of 512 threads walks several consecutive
// tiles of one unit-side and converts W once; its two halves (8 warps each) take alternate tiles with buffers of
// their own, so that one half's scalar phases overlap the other's MMAs.  Warp (wm, wn) of a half owns tokens
// [32 wm, 32 wm + 32) and the 64 channels
// of scale group wn, so the per-token group minimum and maximum are a reduction over the warp's own accumulators
// plus two shuffles; codes go to shared memory and are packed exactly like in the CUDA-core kernel.
#pragma once
#include "common.cuh"

namespace spectra {

constexpr int kTcThreads = 512;      // two halves of 256
constexpr int kTcTilesPerCta = 8;
constexpr int kLdB16 = kD + 8;   // bf16 row stride of the staged tiles (272 bytes: conflict-free ldmatrix)
constexpr int kLdCode = kD + 4;

struct EncodeTcSmem {
  StripTable tab;
  alignas(16) __nv_bfloat16 w[3][kD * kLdB16];     // the three parts of W_enc, [k][n]
  struct Half {
    alignas(16) __nv_bfloat16 x[kTile * kLdB16];   // tokens of the tile, [token][k]
    alignas(16) uint8_t codes[kTile * kLdCode];
    uint16_t lo16[2][kTile], r16[2][kTile];
  } half[2];
  float mean_rot[kD];
};

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

__global__ void __launch_bounds__(kTcThreads, 1) encode_tc_kernel(EncodeTcArgs p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  EncodeTcSmem& S = *reinterpret_cast<EncodeTcSmem*>(smem_raw);
  const int u = blockIdx.y;
  const int ps = (int)(u % p.n_param_sets);
  const int hf = threadIdx.x >> 8;                       // which half of the CTA
  const int tid = threadIdx.x & 255, lane = tid & 31, warp = tid >> 5;
  const int gid = lane >> 2, tig = lane & 3;
  const int wm = warp & 3, wn = warp >> 2;
  const int pos_first = p.pos0[u];
  const int pos_end = pos_first + p.n_new;
  const int tile_first = pos_first / kTile + blockIdx.x * kTcTilesPerCta;
  if (tile_first * kTile >= pos_end) return;

  build_strip_table(S.tab, p.widths + (int64_t)ps * kD, 64);
  const StripTable& T = S.tab;
  // W_enc -> three bf16 parts
  const float* wsrc = p.w_enc + (int64_t)ps * kD * kD;
  for (int idx = threadIdx.x; idx < kD * kD; idx += kTcThreads) {
    const int k = idx / kD, n = idx - k * kD;
    const float v = wsrc[idx];
    const __nv_bfloat16 w1 = __float2bfloat16_rn(v);
    const float r1 = v - __bfloat162float(w1);
    const __nv_bfloat16 w2 = __float2bfloat16_rn(r1);
    const __nv_bfloat16 w3 = __float2bfloat16_rn(r1 - __bfloat162float(w2));
    S.w[0][k * kLdB16 + n] = w1; S.w[1][k * kLdB16 + n] = w2; S.w[2][k * kLdB16 + n] = w3;
  }
  if (threadIdx.x < kD) S.mean_rot[threadIdx.x] = p.mean_rot[(int64_t)ps * kD + threadIdx.x];
  const bool group_active = T.meta_off[wn] >= 0;
  int status = 0;
  EncodeTcSmem::Half& Hs = S.half[hf];
  __syncthreads();                                       // W and the rotated mean are in place
  auto half_sync = [&]() { asm volatile("bar.sync %0, 256;" ::"r"(1 + hf) : "memory"); };

  for (int tt = hf; tt < kTcTilesPerCta; tt += 2) {
    const int tile = tile_first + tt;
    const int tile_pos = tile * kTile;
    if (tile_pos >= pos_end) break;
    const int slot_lo = max(pos_first - tile_pos, 0);
    const int slot_hi = min(pos_end - tile_pos, kTile);
    half_sync();                                         // previous tile's pack has finished with codes / metadata
    // stage the tile's tokens (16-byte chunks); rows outside [slot_lo, slot_hi) are zero
    const __nv_bfloat16* xsrc = p.x + (int64_t)u * p.stride_unit + (int64_t)(tile_pos - pos_first) * p.stride_token;
    for (int idx = tid; idx < kTile * (kD / 8); idx += 256) {
      const int t = idx / (kD / 8), c = idx - t * (kD / 8);
      uint4 v = make_uint4(0, 0, 0, 0);
      if (t >= slot_lo && t < slot_hi) v = *reinterpret_cast<const uint4*>(xsrc + (int64_t)t * p.stride_token + 8 * c);
      *reinterpret_cast<uint4*>(&Hs.x[t * kLdB16 + 8 * c]) = v;
    }
    half_sync();
    // ---- y = x W_enc on the tensor cores
    float acc[2][8][4];
#pragma unroll
    for (int mb = 0; mb < 2; mb++)
#pragma unroll
      for (int nb = 0; nb < 8; nb++)
#pragma unroll
        for (int e = 0; e < 4; e++) acc[mb][nb][e] = 0.f;
#pragma unroll 1
    for (int ks = 0; ks < kD / 16; ks++) {
      uint32_t a[2][4];
#pragma unroll
      for (int mb = 0; mb < 2; mb++)
        ldmatrix_x4(a[mb], &Hs.x[(32 * wm + 16 * mb + (lane & 7) + ((lane >> 3) & 1) * 8) * kLdB16 + 16 * ks + (lane >> 4) * 8]);
#pragma unroll
      for (int part = 0; part < 3; part++) {
#pragma unroll
        for (int np = 0; np < 4; np++) {               // two 8-channel blocks per ldmatrix
          uint32_t b[4];
          ldmatrix_x4_trans(b, &S.w[part][(16 * ks + (lane & 7) + ((lane >> 3) & 1) * 8) * kLdB16 + 64 * wn + 16 * np + (lane >> 4) * 8]);
#pragma unroll
          for (int mb = 0; mb < 2; mb++) {
            mma_bf16(acc[mb][2 * np], a[mb], b[0], b[1]);
            mma_bf16(acc[mb][2 * np + 1], a[mb], b[2], b[3]);
          }
        }
      }
    }
    // ---- centre, per-token group range, quantise (this warp: tokens 32 wm + .., channels 64 wn + ..)
#pragma unroll
    for (int mb = 0; mb < 2; mb++) {
#pragma unroll
      for (int half = 0; half < 2; half++) {
        const int t = 32 * wm + 16 * mb + gid + 8 * half;
        float lo = INFINITY, hi = -INFINITY;
#pragma unroll
        for (int nb = 0; nb < 8; nb++) {
#pragma unroll
          for (int e = 0; e < 2; e++) {
            const int j = 64 * wn + 8 * nb + 2 * tig + e;
            const float y = __fsub_rn(acc[mb][nb][2 * half + e], S.mean_rot[j]);
            acc[mb][nb][2 * half + e] = y;
            if (T.width[j]) {
              if (!isfinite(y)) status |= SPECTRA_STATUS_NONFINITE;
              lo = fminf(lo, y); hi = fmaxf(hi, y);
            }
          }
        }
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, 1)); hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, 1));
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, 2)); hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, 2));
        const bool live = group_active && t >= slot_lo && t < slot_hi;
        if (live) {
          float lo_c = lo;
          if (lo_c < -65504.f) { lo_c = -65504.f; status |= SPECTRA_STATUS_F16_RANGE; }
          if (lo_c > 65504.f) { lo_c = 65504.f; status |= SPECTRA_STATUS_F16_RANGE; }
          const __half lo16 = __float2half_rd(lo_c);
          const float lo_f = __half2float(lo16);
          float R = __fsub_rn(hi, lo_f);
          if (!(R <= 65504.f)) { R = 65504.f; status |= SPECTRA_STATUS_F16_RANGE; }
          if (R < 0.f) R = 0.f;
          const __half r16 = __float2half_ru(R);
          const float R_f = __half2float(r16);
          if (tig == 0) { Hs.lo16[wn][t] = __half_as_ushort(lo16); Hs.r16[wn][t] = __half_as_ushort(r16); }
#pragma unroll
          for (int nb = 0; nb < 8; nb++) {
            unsigned pair = 0;
#pragma unroll
            for (int e = 0; e < 2; e++) {
              const int j = 64 * wn + 8 * nb + 2 * tig + e;
              const int b = T.width[j];
              float r = 0.f;
              if (b && R_f != 0.f) {
                const float L = (float)((1 << b) - 1);
                r = rintf(__fmul_rn(__fsub_rn(acc[mb][nb][2 * half + e], lo_f), __fdiv_rn(L, R_f)));
                if (!(r >= 0.f)) r = 0.f;
                if (r > L) r = L;
              }
              pair |= (unsigned)r << (8 * e);
            }
            *reinterpret_cast<uint16_t*>(&Hs.codes[t * kLdCode + 64 * wn + 8 * nb + 2 * tig]) = (uint16_t)pair;
          }
        }
      }
    }
    half_sync();
    // ---- pack: one half-word of the payload at a time, in storage order
    uint8_t* tile_ptr = p.cache + p.unit_offset[u] + (int64_t)tile * T.tile_bytes;
    const int payload = T.class_off[4];
    if (slot_lo == 0 && slot_hi == kTile) pack_full_tile(T, p.side, Hs.codes, kLdCode, tile_ptr, tid, 256);
    else
    for (int off = 2 * tid; off < payload; off += 2 * 256) {
      int w, first;
      const int k = halfword_owner(T, p.side, off, w, first);
      const int chan = T.chan[k], shift = T.shift[k];
      const int per = 16 / w;
      const unsigned fmask = (1u << w) - 1u;
      unsigned hw = 0, keep = 0;
      for (int e = 0; e < per; e++) {
        const int tok = first + e;
        if (tok < slot_lo) keep |= fmask << (e * w);
        else if (tok < slot_hi) hw |= (((unsigned)Hs.codes[tok * kLdCode + chan] >> shift) & fmask) << (e * w);
      }
      uint16_t* dst = reinterpret_cast<uint16_t*>(tile_ptr + off);
      if (keep) hw |= (unsigned)(*dst) & keep;
      *dst = (uint16_t)hw;
    }
    for (int idx = tid; idx < 2 * kTile; idx += 256) {
      const int g = idx / kTile, t = idx - g * kTile;
      if (T.meta_off[g] < 0 || t < slot_lo) continue;
      uint16_t* dst = reinterpret_cast<uint16_t*>(tile_ptr + T.meta_off[g]) + t;
      const bool written = t < slot_hi;
      dst[0] = written ? Hs.lo16[g][t] : (uint16_t)0;
      dst[kTile] = written ? Hs.r16[g][t] : (uint16_t)0;
    }
  }
  if (status && p.status) atomicOr(p.status, status);
}

}  // namespace spectra
