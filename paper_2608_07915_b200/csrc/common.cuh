// Shared device/host helpers of libspectra: configuration checks, the per-unit strip table that
// describes a packed tile, and the mapping between (strip, token) and storage bits.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/spectra.h"

namespace spectra {

constexpr int kD = 128;          // head_dim
constexpr int kTile = 128;       // tokens per tile
constexpr int kMaxStrips = 384;  // 128 channels x at most 3 sub-fields
constexpr int kMaxGroups = 4;    // scale groups per token (scale_group >= 32)

inline int check_config(const spectra_config* c) {
  if (!c) return SPECTRA_INVALID_ARG;
  if (c->head_dim != kD || c->tile_tokens != kTile || c->layout_version != 2) return SPECTRA_UNSUPPORTED;
  if (c->scale_group != 32 && c->scale_group != 64 && c->scale_group != 128) return SPECTRA_UNSUPPORTED;
  if (c->b_max < 1 || c->b_max > 8) return SPECTRA_INVALID_ARG;
  int wg = c->width_group;
  if (wg < 1 || wg > c->scale_group || (wg & (wg - 1))) return SPECTRA_INVALID_ARG;
  if (c->gain_mode < 0 || c->gain_mode > 2) return SPECTRA_INVALID_ARG;
  return SPECTRA_OK;
}

inline int launch_status() { return cudaGetLastError() == cudaSuccess ? SPECTRA_OK : SPECTRA_CUDA_ERROR; }

// Description of one unit-side's tile, built in shared memory from the 128 widths.
// Strips are numbered in storage order: class 8 first, then 4, 2, 1; ascending channel inside a class.
struct StripTable {
  int n_strips;
  int class_first[5];             // first strip index of class c (w = 8 >> c); class_first[4] = n_strips
  int class_off[5];               // byte offset of the class region; class_off[4] = payload bytes
  int n_groups;                   // d / scale_group
  int n_act;                      // active scale groups
  int meta_off[kMaxGroups];       // byte offset of lo16[128] of group g (R16 follows 256 bytes later), -1 if inactive
  int tile_bytes;
  uint8_t chan[kMaxStrips];
  uint8_t shift[kMaxStrips];
  uint8_t width[kD];
};

// The scan itself, run by one full warp after T.width has been filled.
__device__ inline void strip_table_scan(StripTable& T, int scale_group, int lane) {
  {
    int count = 0, off = 0;
#pragma unroll
    for (int c = 0; c < 4; c++) {
      const int w = 8 >> c;
      if (lane == 0) { T.class_first[c] = count; T.class_off[c] = off; }
      int first = count;
      for (int word = 0; word < kD / 32; word++) {
        const int j = word * 32 + lane;
        const int b = T.width[j];
        const bool present = (b & w) != 0;
        const unsigned m = __ballot_sync(0xffffffffu, present);
        if (present) {
          const int k = count + __popc(m & ((1u << lane) - 1u));
          T.chan[k] = (uint8_t)j;
          T.shift[k] = (uint8_t)(b & (w - 1));
        }
        count += __popc(m);
      }
      off += 16 * w * (count - first);
    }
    int n_groups = kD / scale_group;
    int n_act = 0;
    for (int g = 0; g < n_groups; g++) {
      bool any = false;
      for (int j = g * scale_group + lane; j < (g + 1) * scale_group; j += 32) any |= T.width[j] != 0;
      const bool act = __any_sync(0xffffffffu, any);
      if (lane == 0) T.meta_off[g] = act ? off + 512 * n_act : -1;
      n_act += act ? 1 : 0;
    }
    if (lane == 0) {
      T.n_strips = count; T.class_first[4] = count; T.class_off[4] = off;
      T.n_groups = n_groups; T.n_act = n_act; T.tile_bytes = off + 512 * n_act;
      for (int g = n_groups; g < kMaxGroups; g++) T.meta_off[g] = -1;
    }
  }
}

// Called by all threads of a CTA (at least one full warp); includes the closing __syncthreads().
__device__ inline void build_strip_table(StripTable& T, const uint8_t* __restrict__ widths_global, int scale_group) {
  const int tid = threadIdx.x;
  if (tid < kD) T.width[tid] = widths_global[tid];
  __syncthreads();
  if (tid < 32) strip_table_scan(T, scale_group, tid);
  __syncthreads();
}

// Two tables at once (at least 256 threads): warp 0 scans the first, warp 1 the second.
__device__ inline void build_strip_tables(StripTable& A, const uint8_t* __restrict__ wa, StripTable& B,
                                          const uint8_t* __restrict__ wb, int scale_group) {
  const int tid = threadIdx.x;
  if (tid < kD) A.width[tid] = wa[tid];
  else if (tid < 2 * kD) B.width[tid - kD] = wb[tid - kD];
  __syncthreads();
  if (tid < 32) strip_table_scan(A, scale_group, tid);
  else if (tid < 64) strip_table_scan(B, scale_group, tid - 32);
  __syncthreads();
}

__device__ inline int strip_class(const StripTable& T, int k) {
  return (k >= T.class_first[1]) + (k >= T.class_first[2]) + (k >= T.class_first[3]);
}

// ---- storage positions (tile bit n = bit n%8 of byte n/8)
// K side, token-major: the fields of a token in strip order form its token string of B bits; string bits
// [32 i, 32 i + 32), i < F = B / 32, are the 32-bit word at byte 4 * (128 i + t); the last r = B % 32 string bits of
// the 128 tokens are packed densely behind the words (token t at tile bit 4096 F + r t).
// V side, strip-major: strip k is 16 w bytes; tokens t and t + 16 sit 16 bits apart in a 32-bit word.

__device__ inline int string_bits(const StripTable& T) { return T.class_off[4] >> 4; }

// Offset of strip k's field inside a token string (K side).
__device__ inline int string_offset(const StripTable& T, int k) {
  const int c = strip_class(T, k);
  return (T.class_off[c] >> 4) + (k - T.class_first[c]) * (8 >> c);
}

// Tile bit offset of the field of token t of strip k; its w bits are consecutive tile bits.
__device__ inline int field_bit(const StripTable& T, int side, int k, int t) {
  const int c = strip_class(T, k);
  const int w = 8 >> c;
  const int i_in = k - T.class_first[c];
  if (side == SPECTRA_SIDE_V) {
    const int a = t >> 5, h = (t >> 4) & 1, i = t & 15;
    return 8 * (T.class_off[c] + 16 * w * i_in + 4 * (a * w + ((i * w) >> 4)) + 2 * h) + ((i * w) & 15);
  }
  const int B = string_bits(T), F = B >> 5, r = B & 31;
  const int o = (T.class_off[c] >> 4) + i_in * w;
  if (o < 32 * F) return 32 * (kTile * (o >> 5) + t) + (o & 31);
  return 4096 * F + r * t + (o - 32 * F);
}

// A field of w <= 8 bits at tile bit `bit` (any alignment).  Reads the byte behind the field's first byte, which
// is inside the tile (the metadata follows the payload).
__device__ inline unsigned read_field(const uint8_t* tile, int bit, int w) {
  const unsigned two = (unsigned)tile[bit >> 3] | ((unsigned)tile[(bit >> 3) + 1] << 8);
  return (two >> (bit & 7)) & ((1u << w) - 1u);
}

// Inverse map of the V side: the half-word at payload byte offset `off` (even) belongs to strip k and holds the
// 16/w consecutive tokens from first_token on: returns k, sets w and first_token.
__device__ inline int halfword_owner_v(const StripTable& T, int off, int& w, int& first_token) {
  int c = (off >= T.class_off[1]) + (off >= T.class_off[2]) + (off >= T.class_off[3]);
  w = 8 >> c;
  const int rel = off - T.class_off[c];
  const int per = 16 / w;  // tokens per half-word
  const int i_in = rel / (16 * w);
  const int r = rel - i_in * 16 * w;
  const int q = r >> 2, h = (r >> 1) & 1;
  const int a = q / w, m = q - a * w;
  first_token = 32 * a + 16 * h + m * per;
  return T.class_first[c] + i_in;
}

// String bits [lo, hi) (hi - lo <= 32) of the token whose codes are `codes` (one byte per channel), at bit 0 up.
__device__ inline unsigned string_window(const StripTable& T, const uint8_t* __restrict__ codes, int lo, int hi) {
  unsigned word = 0;
#pragma unroll
  for (int c = 0; c < 4; c++) {
    const int w = 8 >> c;
    const int cb = T.class_off[c] >> 4, ce = T.class_off[c + 1] >> 4;
    const int o0 = max(lo, cb), o1 = min(hi, ce);
    for (int o = o0; o < o1; o += w) {
      const int k = T.class_first[c] + (o - cb) / w;
      word |= (((unsigned)codes[T.chan[k]] >> T.shift[k]) & ((1u << w) - 1u)) << (o - lo);
    }
  }
  return word;
}

// Write the payload of one tile from a shared-memory code array (codes[t * ld + channel], one byte each) for the
// token slots [slot_lo, slot_hi); slots before slot_lo keep their bits, slots from slot_hi on are cleared.
// Called by all `nthreads` threads of the CTA that owns the tile.
__device__ inline void pack_tile_payload(const StripTable& T, int side, const uint8_t* __restrict__ codes, int ld,
                                         int slot_lo, int slot_hi, uint8_t* __restrict__ tile_ptr, int tid,
                                         int nthreads) {
  if (side == SPECTRA_SIDE_V) {
    const int payload = T.class_off[4];
    for (int off = 2 * tid; off < payload; off += 2 * nthreads) {
      int w, first;
      const int k = halfword_owner_v(T, off, w, first);
      const int chan = T.chan[k], shift = T.shift[k];
      const int per = 16 / w;
      const unsigned fmask = (1u << w) - 1u;
      unsigned hw = 0, keep = 0;
      for (int e = 0; e < per; e++) {
        const int tok = first + e;
        if (tok < slot_lo) keep |= fmask << (e * w);
        else if (tok < slot_hi) hw |= (((unsigned)codes[tok * ld + chan] >> shift) & fmask) << (e * w);
      }
      uint16_t* dst = reinterpret_cast<uint16_t*>(tile_ptr + off);
      if (keep) hw |= (unsigned)(*dst) & keep;
      *dst = (uint16_t)hw;
    }
    return;
  }
  const int B = string_bits(T), F = B >> 5, r = B & 31;
  for (int idx = tid; idx < F * kTile; idx += nthreads) {
    const int i = idx >> 7, t = idx & (kTile - 1);
    if (t < slot_lo) continue;
    const unsigned word = t < slot_hi ? string_window(T, codes + t * ld, 32 * i, 32 * i + 32) : 0u;
    reinterpret_cast<uint32_t*>(tile_ptr)[idx] = word;
  }
  if (r) {
    uint32_t* tail = reinterpret_cast<uint32_t*>(tile_ptr + 512 * F);
    for (int q = tid; q < 4 * r; q += nthreads) {          // 32-bit words of the dense remainder region
      const int t0 = (32 * q) / r, t1 = min((32 * q + 31) / r, kTile - 1);
      unsigned word = 0, keep = 0;
      for (int t = t0; t <= t1; t++) {
        const int rel = r * t - 32 * q;                     // bit of the word where the token's remainder starts
        const unsigned full = r == 32 ? 0xffffffffu : ((1u << r) - 1u);
        const unsigned m = rel >= 0 ? full << rel : full >> (-rel);
        if (t < slot_lo) keep |= m;
        else if (t < slot_hi) {
          const unsigned v = string_window(T, codes + t * ld, 32 * F, B);
          word |= rel >= 0 ? v << rel : v >> (-rel);
        }
      }
      if (keep) word |= tail[q] & keep;
      tail[q] = word;
    }
  }
}

__device__ inline float load_as_float(const void* p, int dtype, int64_t idx) {
  if (dtype == SPECTRA_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[idx]);
  return reinterpret_cast<const float*>(p)[idx];
}

__device__ inline void store_from_float(void* p, int dtype, int64_t idx, float v) {
  if (dtype == SPECTRA_BF16) reinterpret_cast<__nv_bfloat16*>(p)[idx] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(p)[idx] = v;
}

}  // namespace spectra
