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
  if (c->head_dim != kD || c->tile_tokens != kTile || c->layout_version != 1) return SPECTRA_UNSUPPORTED;
  if (c->scale_group != 32 && c->scale_group != 64 && c->scale_group != 128) return SPECTRA_UNSUPPORTED;
  if (c->b_max < 1 || c->b_max > 8) return SPECTRA_INVALID_ARG;
  int wg = c->width_group;
  if (wg < 1 || wg > c->scale_group || (wg & (wg - 1))) return SPECTRA_INVALID_ARG;
  if (c->gain_mode < 0 || c->gain_mode > 2) return SPECTRA_INVALID_ARG;
  return SPECTRA_OK;
}

// SMs of the current device (0 if the query fails).
inline int sm_count() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  return sms;
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
  alignas(16) uint8_t width[kD];   // read four and eight at a time
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

// Two tables at once, by the first eight warps of the CTA (at least 256 threads): warp (side, class) counts its class,
// the counts are exchanged through shared memory, then every warp places the strips of its own class.  Same result as
// strip_table_scan, a quarter of its dependent chain (for callers whose whole run is a few microseconds).
__device__ inline void build_strip_tables(StripTable& A, const uint8_t* __restrict__ wa, StripTable& B,
                                          const uint8_t* __restrict__ wb, int scale_group) {
  __shared__ int cnt[2][4];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid < kD) A.width[tid] = wa[tid];
  else if (tid < 2 * kD) B.width[tid - kD] = wb[tid - kD];
  __syncthreads();
  const int side = warp >> 2, c = warp & 3, w = 8 >> c;
  StripTable& T = side ? B : A;
  unsigned m[kD / 32];
  int bw[kD / 32];
  if (warp < 8) {
    int n = 0;
#pragma unroll
    for (int word = 0; word < kD / 32; word++) {
      bw[word] = T.width[word * 32 + lane];
      m[word] = __ballot_sync(0xffffffffu, (bw[word] & w) != 0);
      n += __popc(m[word]);
    }
    if (lane == 0) cnt[side][c] = n;
  }
  __syncthreads();
  if (warp < 8) {
    int first = 0, off = 0;
    for (int cc = 0; cc < c; cc++) { first += cnt[side][cc]; off += 16 * (8 >> cc) * cnt[side][cc]; }
    if (lane == 0) { T.class_first[c] = first; T.class_off[c] = off; }
    int k0 = first;
#pragma unroll
    for (int word = 0; word < kD / 32; word++) {
      if ((bw[word] & w) != 0) {
        const int k = k0 + __popc(m[word] & ((1u << lane) - 1u));
        T.chan[k] = (uint8_t)(word * 32 + lane);
        T.shift[k] = (uint8_t)(bw[word] & (w - 1));
      }
      k0 += __popc(m[word]);
    }
    if (c == 3) {                       // the last class also closes the table: totals and the metadata offsets
      const int count = k0, payload = off + 16 * w * cnt[side][3];
      const int n_groups = kD / scale_group;
      int n_act = 0;
      for (int g = 0; g < n_groups; g++) {
        bool any = false;
        for (int j = g * scale_group + lane; j < (g + 1) * scale_group; j += 32) any |= T.width[j] != 0;
        const bool act = __any_sync(0xffffffffu, any);
        if (lane == 0) T.meta_off[g] = act ? payload + 512 * n_act : -1;
        n_act += act ? 1 : 0;
      }
      if (lane == 0) {
        T.n_strips = count; T.class_first[4] = count; T.class_off[4] = payload;
        T.n_groups = n_groups; T.n_act = n_act; T.tile_bytes = payload + 512 * n_act;
        for (int g = n_groups; g < kMaxGroups; g++) T.meta_off[g] = -1;
      }
    }
  }
  __syncthreads();
}

__device__ inline int strip_class(const StripTable& T, int k) {
  return (k >= T.class_first[1]) + (k >= T.class_first[2]) + (k >= T.class_first[3]);
}

// Storage position of the field of token t in strip k: byte offset of its half-word and the bit inside it.
__device__ inline void locate_field(const StripTable& T, int side, int k, int t, int& byte_off, int& bit) {
  const int c = strip_class(T, k);
  const int w = 8 >> c;
  const int i_in = k - T.class_first[c];
  const int cnt = T.class_first[c + 1] - T.class_first[c];
  if (side == SPECTRA_SIDE_V) {
    const int a = t >> 5, h = (t >> 4) & 1, i = t & 15;
    byte_off = T.class_off[c] + 16 * w * i_in + 4 * (a * w + ((i * w) >> 4)) + 2 * h;
    bit = (i * w) & 15;
  } else {
    const int n = (t * w) >> 4;
    bit = (t * w) & 15;
    if ((i_in | 1) < cnt) byte_off = T.class_off[c] + 32 * w * (i_in >> 1) + 4 * n + 2 * (i_in & 1);
    else byte_off = T.class_off[c] + 16 * w * i_in + 2 * n;
  }
}

// Inverse map: the half-word at payload byte offset `off` (even) belongs to strip k and holds the
// 16/w tokens first_token + e * token_step... (always consecutive tokens): returns k (or -1), sets w and first token.
__device__ inline int halfword_owner(const StripTable& T, int side, int off, int& w, int& first_token) {
  int c = (off >= T.class_off[1]) + (off >= T.class_off[2]) + (off >= T.class_off[3]);
  w = 8 >> c;
  const int rel = off - T.class_off[c];
  const int cnt = T.class_first[c + 1] - T.class_first[c];
  const int per = 16 / w;  // tokens per half-word
  if (side == SPECTRA_SIDE_V) {
    const int i_in = rel / (16 * w);
    const int r = rel - i_in * 16 * w;
    const int q = r >> 2, h = (r >> 1) & 1;
    const int a = q / w, m = q - a * w;
    first_token = 32 * a + 16 * h + m * per;
    return T.class_first[c] + i_in;
  }
  const int paired_bytes = 32 * w * (cnt >> 1);
  if (rel < paired_bytes) {
    const int p = rel / (32 * w);
    const int r = rel - p * 32 * w;
    first_token = (r >> 2) * per;
    return T.class_first[c] + 2 * p + ((r >> 1) & 1);
  }
  first_token = ((rel - paired_bytes) >> 1) * per;
  return T.class_first[c] + cnt - 1;
}

// Packs the payload of a completely written tile (all 128 slots) from a shared-memory code array
// (codes[t * ld + channel], one byte each), one 32-bit word per step, with shifts only.  Called by all `nthreads`
// threads of the CTA that owns the tile; stores are coalesced 4-byte words in storage order.
__device__ inline void pack_full_tile(const StripTable& T, int side, const uint8_t* __restrict__ codes, int ld,
                                      uint8_t* __restrict__ tile_ptr, int tid, int nthreads) {
#pragma unroll
  for (int c = 0; c < 4; c++) {
    const int w = 8 >> c, lw = 3 - c;                       // field width and its log2
    const int per = 16 >> lw;                               // tokens per half-word
    const int first = T.class_first[c], n = T.class_first[c + 1] - first;
    if (n == 0) continue;
    uint32_t* dst = reinterpret_cast<uint32_t*>(tile_ptr + T.class_off[c]);
    const unsigned fmask = (1u << w) - 1u;
    const int words = 4 * w * n;                            // 32-bit words of the class region
    for (int W = tid; W < words; W += nthreads) {
      int k_lo, k_hi, t_lo, t_hi;                           // strip and first token of the low / high half-word
      if (side == SPECTRA_SIDE_V) {
        const int i_in = W >> (2 + lw), q = W & (4 * w - 1);
        const int a = q >> lw, m = q & (w - 1);
        k_lo = k_hi = first + i_in;
        t_lo = 32 * a + m * per; t_hi = t_lo + 16;
      } else {
        const int paired_words = 8 * w * (n >> 1);          // words of the interleaved pairs
        if (W < paired_words) {
          const int p = W >> (3 + lw), nn = W & (8 * w - 1);
          k_lo = first + 2 * p; k_hi = k_lo + 1;
          t_lo = t_hi = nn * per;
        } else {                                            // the odd last strip: half-words in order
          const int j = W - paired_words;
          k_lo = k_hi = first + n - 1;
          t_lo = 2 * j * per; t_hi = t_lo + per;
        }
      }
      const int c_lo = T.chan[k_lo], s_lo = T.shift[k_lo], c_hi = T.chan[k_hi], s_hi = T.shift[k_hi];
      unsigned word = 0;
      for (int e = 0; e < per; e++) {
        word |= (((unsigned)codes[(t_lo + e) * ld + c_lo] >> s_lo) & fmask) << (e * w);
        word |= (((unsigned)codes[(t_hi + e) * ld + c_hi] >> s_hi) & fmask) << (16 + e * w);
      }
      dst[W] = word;
    }
  }
}

// Inverse of pack_full_tile: scatters the fields of a tile's payload into a shared-memory code array
// (codes[t * ld + channel], zeroed by the caller), one 32-bit word per step and one class after the other, so that
// a code byte is touched by one thread at a time.  Called by all `nthreads` threads; ends with a barrier.
__device__ inline void unpack_tile(const StripTable& T, int side, const uint8_t* __restrict__ tile_ptr,
                                   uint8_t* __restrict__ codes, int ld, int tid, int nthreads) {
#pragma unroll
  for (int c = 0; c < 4; c++) {
    const int w = 8 >> c, lw = 3 - c;
    const int per = 16 >> lw;
    const int first = T.class_first[c], n = T.class_first[c + 1] - first;
    if (n) {
      const uint32_t* src = reinterpret_cast<const uint32_t*>(tile_ptr + T.class_off[c]);
      const unsigned fmask = (1u << w) - 1u;
      const int words = 4 * w * n;
      for (int W = tid; W < words; W += nthreads) {
        int k_lo, k_hi, t_lo, t_hi;
        if (side == SPECTRA_SIDE_V) {
          const int i_in = W >> (2 + lw), q = W & (4 * w - 1);
          const int a = q >> lw, m = q & (w - 1);
          k_lo = k_hi = first + i_in;
          t_lo = 32 * a + m * per; t_hi = t_lo + 16;
        } else {
          const int paired_words = 8 * w * (n >> 1);
          if (W < paired_words) {
            const int p = W >> (3 + lw), nn = W & (8 * w - 1);
            k_lo = first + 2 * p; k_hi = k_lo + 1;
            t_lo = t_hi = nn * per;
          } else {
            const int j = W - paired_words;
            k_lo = k_hi = first + n - 1;
            t_lo = 2 * j * per; t_hi = t_lo + per;
          }
        }
        const int c_lo = T.chan[k_lo], s_lo = T.shift[k_lo], c_hi = T.chan[k_hi], s_hi = T.shift[k_hi];
        const unsigned word = src[W];
        for (int e = 0; e < per; e++) {
          codes[(t_lo + e) * ld + c_lo] |= (uint8_t)(((word >> (e * w)) & fmask) << s_lo);
          codes[(t_hi + e) * ld + c_hi] |= (uint8_t)(((word >> (16 + e * w)) & fmask) << s_hi);
        }
      }
    }
    __syncthreads();
  }
}

// Where the tiles of a unit-side live.  Contiguous caches (table == NULL): tile t of unit u starts t tile sizes after
// the unit's offset.  Paged caches: the unit's offset is the base of a pool of tile-sized pages and logical tile t
// sits in page table[u * stride + t] of that pool (the append-only streaming cache of Sec. 3.3 grows a page at a time).
struct TileMap {
  const int32_t* table; int64_t stride;
  __device__ __forceinline__ int64_t page(int64_t u, int t) const { return table ? (int64_t)table[u * stride + t] : (int64_t)t; }
};

// Asks the L2 for the 128-byte line that holds p; a later load then pays the L2's latency instead of the DRAM's.
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

__device__ inline float load_as_float(const void* p, int dtype, int64_t idx) {
  if (dtype == SPECTRA_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[idx]);
  return reinterpret_cast<const float*>(p)[idx];
}

__device__ inline void store_from_float(void* p, int dtype, int64_t idx, float v) {
  if (dtype == SPECTRA_BF16) reinterpret_cast<__nv_bfloat16*>(p)[idx] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(p)[idx] = v;
}

}  // namespace spectra
