// Generic (CUDA-core) coded-cache decode attention: any GQA group size up to 8 and any supported
// scale group.  One CTA of 128 threads per (unit, sequence split); a second kernel merges the
// splits and lifts the result out of the rotated value space.
#pragma once
#include "common.cuh"

namespace spectra {

constexpr int kMaxGqa = 8;
constexpr int kMaxTileBytes = 16 * 8 * kD + 512 * kMaxGroups;
constexpr int kPartialStride = kD + 4;  // per (unit, split, head): o'[128], m, l, qconst, pad

struct AttnArgs {
  const void* q; int q_dtype; int batch, n_kv, n_q, gqa; const int32_t* seq_len; int scale_group;
  const uint8_t* cache_k; const int64_t* off_k; const uint8_t* cache_v; const int64_t* off_v;
  int64_t n_param_sets;
  const float* w_dec_k; const float* mean_rot_k; const uint8_t* widths_k;
  const float* w_dec_v; const float* mean_rot_v; const uint8_t* widths_v;
  float scale; void* out; int out_dtype; float* lse; float* partials; int n_splits; int32_t* status;
  TileMap map_k, map_v;
  int max_seq_len;   // capacity of every sequence's buffers in tokens: a longer seq_len is reported and attends to nothing
};

// Tokens sequence b attends to: its length, or 0 when the length exceeds what the buffers hold (the caller learns
// of it through SPECTRA_STATUS_CAPACITY; nothing past a buffer's end is ever read or written).
__device__ __forceinline__ int attended_tokens(const AttnArgs& p, int b) {
  const int n = p.seq_len[b];
  return n > p.max_seq_len ? 0 : n;
}

struct GenericSmem {
  StripTable tk, tv;
  __align__(16) uint8_t tile_k[kMaxTileBytes];
  __align__(16) uint8_t tile_v[kMaxTileBytes];
  alignas(16) float qrot[kMaxGqa][kD];              // q' = scale * W_dec,K q
  float qs[kMaxGqa][kMaxStrips];        // q'_chan * 2^shift / L_chan per K strip
  float qsum[kMaxGqa][kMaxGroups];      // sum of q' over the active channels of a scale group
  alignas(16) float pr[kMaxGqa][kMaxGroups][kTile]; // p_t * R^V_{g,t}
  float red[kMaxGqa][4];
  float o[kMaxGqa][kD];
  float plo[kMaxGqa][kMaxGroups];
  float lsum[kMaxGqa];
  alignas(16) float qraw[kMaxGqa][kD];
};

__global__ void __launch_bounds__(128) attention_generic_kernel(AttnArgs p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  GenericSmem& S = *reinterpret_cast<GenericSmem*>(smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int u = blockIdx.y, split = blockIdx.x;
  const int b = u / p.n_kv, hk = u - b * p.n_kv;
  const int ps = (int)(u % p.n_param_sets);
  const int G = p.gqa, gs = p.scale_group;
  const int n = attended_tokens(p, b);
  if (split == 0 && hk == 0 && tid == 0 && p.seq_len[b] > p.max_seq_len && p.status) atomicOr(p.status, SPECTRA_STATUS_CAPACITY);
  const int n_tiles = (n + kTile - 1) / kTile;
  const int per = (n_tiles + p.n_splits - 1) / p.n_splits;
  const int tile_begin = split * per, tile_end = min(tile_begin + per, n_tiles);

  build_strip_table(S.tk, p.widths_k + (int64_t)ps * kD, gs);
  build_strip_table(S.tv, p.widths_v + (int64_t)ps * kD, gs);
  const StripTable& TK = S.tk;
  const StripTable& TV = S.tv;
  const int n_groups = TK.n_groups;

  // ---- fold the up-projection into the query: q'_j = scale * sum_i W_dec,K[j][i] q_i
  for (int idx = tid; idx < G * kD; idx += blockDim.x) {
    const int h = idx / kD, i = idx - h * kD;
    S.qraw[h][i] = load_as_float(p.q, p.q_dtype, ((int64_t)b * p.n_q + hk * G + h) * kD + i);
    S.o[h][i] = 0.f;
  }
  __syncthreads();
  const float* wk = p.w_dec_k + (int64_t)ps * kD * kD;
  for (int j = warp; j < kD; j += 4) {
    const float4 wrow = *reinterpret_cast<const float4*>(wk + j * kD + lane * 4);
    for (int h = 0; h < G; h++) {
      const float4 qv = *reinterpret_cast<const float4*>(&S.qraw[h][lane * 4]);
      float acc = wrow.x * qv.x + wrow.y * qv.y + wrow.z * qv.z + wrow.w * qv.w;
#pragma unroll
      for (int s = 16; s; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
      if (lane == 0) S.qrot[h][j] = acc * p.scale;
    }
  }
  __syncthreads();
  float qconst = 0.f;  // q' . m'_K, valid in warp h lane 0.. computed by every thread of head loop below
  for (int idx = tid; idx < G * TK.n_strips; idx += blockDim.x) {
    const int h = idx / TK.n_strips, k = idx - h * TK.n_strips;
    const int c = TK.chan[k];
    S.qs[h][k] = S.qrot[h][c] * (float)(1 << TK.shift[k]) / (float)((1 << TK.width[c]) - 1);
  }
  if (tid < G * n_groups) {
    const int h = tid / n_groups, g = tid - h * n_groups;
    float acc = 0.f;
    for (int j = g * gs; j < (g + 1) * gs; j++) if (TK.width[j]) acc += S.qrot[h][j];
    S.qsum[h][g] = acc;
  }
  if (tid < G && p.mean_rot_k) {
    for (int j = 0; j < kD; j++) qconst += S.qrot[tid][j] * p.mean_rot_k[(int64_t)ps * kD + j];
  }
  __syncthreads();

  float m_run[kMaxGqa], l_run[kMaxGqa], plo_run[kMaxGqa][kMaxGroups];
  float acc_v[3][kMaxGqa];
#pragma unroll
  for (int h = 0; h < kMaxGqa; h++) {
    m_run[h] = -INFINITY; l_run[h] = 0.f;
#pragma unroll
    for (int g = 0; g < kMaxGroups; g++) plo_run[h][g] = 0.f;
#pragma unroll
    for (int s = 0; s < 3; s++) acc_v[s][h] = 0.f;
  }

  const uint8_t* base_k = p.cache_k + p.off_k[u];
  const uint8_t* base_v = p.cache_v + p.off_v[u];
  for (int tile = tile_begin; tile < tile_end; tile++) {
    __syncthreads();
    {
      const uint4* sk = reinterpret_cast<const uint4*>(base_k + p.map_k.page(u, tile) * TK.tile_bytes);
      const uint4* sv = reinterpret_cast<const uint4*>(base_v + p.map_v.page(u, tile) * TV.tile_bytes);
      for (int i = tid; i < TK.tile_bytes / 16; i += blockDim.x) reinterpret_cast<uint4*>(S.tile_k)[i] = sk[i];
      for (int i = tid; i < TV.tile_bytes / 16; i += blockDim.x) reinterpret_cast<uint4*>(S.tile_v)[i] = sv[i];
    }
    __syncthreads();
    // ---- scores: thread t owns token t of the tile
    const int t = tid;
    const bool valid = tile * kTile + t < n;
    float sc[kMaxGqa];
    {
      float acc[kMaxGroups][kMaxGqa];
#pragma unroll
      for (int g = 0; g < kMaxGroups; g++)
#pragma unroll
        for (int h = 0; h < kMaxGqa; h++) acc[g][h] = 0.f;
      for (int k = 0; k < TK.n_strips; k++) {
        int bo, bit;
        locate_field(TK, SPECTRA_SIDE_K, k, t, bo, bit);
        const int w = 8 >> strip_class(TK, k);
        const unsigned hw = *reinterpret_cast<const uint16_t*>(S.tile_k + bo);
        const float f = (float)((hw >> bit) & ((1u << w) - 1u));
        const int g = TK.chan[k] / gs;
#pragma unroll
        for (int gg = 0; gg < kMaxGroups; gg++)
          if (gg == g) {
#pragma unroll
            for (int h = 0; h < kMaxGqa; h++)
              if (h < G) acc[gg][h] = fmaf(S.qs[h][k], f, acc[gg][h]);
          }
      }
#pragma unroll
      for (int h = 0; h < kMaxGqa; h++) sc[h] = 0.f;
#pragma unroll
      for (int g = 0; g < kMaxGroups; g++) {
        if (g < n_groups && TK.meta_off[g] >= 0) {
          const uint16_t* mm = reinterpret_cast<const uint16_t*>(S.tile_k + TK.meta_off[g]) + t;
          const float lo = __half2float(__ushort_as_half(mm[0]));
          const float R = __half2float(__ushort_as_half(mm[kTile]));
#pragma unroll
          for (int h = 0; h < kMaxGqa; h++)
            if (h < G) sc[h] += R * acc[g][h] + lo * S.qsum[h][g];
        }
      }
    }
    // ---- online softmax across the tile
    float alpha[kMaxGqa], pt[kMaxGqa];
#pragma unroll
    for (int h = 0; h < kMaxGqa; h++) {
      if (h < G) {
        float v = valid ? sc[h] : -INFINITY;
#pragma unroll
        for (int s = 16; s; s >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, s));
        if (lane == 0) S.red[h][warp] = v;
      }
    }
    __syncthreads();
#pragma unroll
    for (int h = 0; h < kMaxGqa; h++) {
      alpha[h] = 1.f; pt[h] = 0.f;
      if (h < G) {
        const float tmax = fmaxf(fmaxf(S.red[h][0], S.red[h][1]), fmaxf(S.red[h][2], S.red[h][3]));
        const float m_new = fmaxf(m_run[h], tmax);
        alpha[h] = m_run[h] == -INFINITY ? 0.f : __expf(m_run[h] - m_new);
        pt[h] = valid ? __expf(sc[h] - m_new) : 0.f;
        m_run[h] = m_new;
        l_run[h] = l_run[h] * alpha[h] + pt[h];
      }
    }
#pragma unroll
    for (int g = 0; g < kMaxGroups; g++) {
      if (g < n_groups) {
        float lo = 0.f, R = 0.f;
        if (TV.meta_off[g] >= 0) {
          const uint16_t* mm = reinterpret_cast<const uint16_t*>(S.tile_v + TV.meta_off[g]) + t;
          lo = __half2float(__ushort_as_half(mm[0]));
          R = __half2float(__ushort_as_half(mm[kTile]));
        }
#pragma unroll
        for (int h = 0; h < kMaxGqa; h++)
          if (h < G) {
            S.pr[h][g][t] = pt[h] * R;
            plo_run[h][g] = plo_run[h][g] * alpha[h] + pt[h] * lo;
          }
      }
    }
    __syncthreads();
    // ---- P.V in the rotated value space: thread owns V strips tid, tid+128, tid+256
#pragma unroll
    for (int s = 0; s < 3; s++) {
      const int k = tid + s * 128;
      if (k < TV.n_strips) {
        const int c = strip_class(TV, k);
        const int w = 8 >> c;
        const int g = TV.chan[k] / gs;
        const int perhw = 16 / w;
        const unsigned fmask = (1u << w) - 1u;
        const uint8_t* sp = S.tile_v + TV.class_off[c] + 16 * w * (k - TV.class_first[c]);
        float acc[kMaxGqa];
#pragma unroll
        for (int h = 0; h < kMaxGqa; h++) acc[h] = acc_v[s][h] * alpha[h];
        for (int qw = 0; qw < 4 * w; qw++) {
          const unsigned word = *reinterpret_cast<const uint32_t*>(sp + 4 * qw);
          const int a = qw / w, mword = qw - a * w;
          const int tok0 = 32 * a + mword * perhw;
          for (int e = 0; e < perhw; e++) {
            const float f_lo = (float)((word >> (e * w)) & fmask);
            const float f_hi = (float)((word >> (16 + e * w)) & fmask);
#pragma unroll
            for (int h = 0; h < kMaxGqa; h++)
              if (h < G) {
                acc[h] = fmaf(S.pr[h][g][tok0 + e], f_lo, acc[h]);
                acc[h] = fmaf(S.pr[h][g][tok0 + e + 16], f_hi, acc[h]);
              }
          }
        }
#pragma unroll
        for (int h = 0; h < kMaxGqa; h++) acc_v[s][h] = acc[h];
      }
    }
  }
  __syncthreads();
  // ---- fold strips back to channels, reduce the per-thread partial sums
#pragma unroll
  for (int s = 0; s < 3; s++) {
    const int k = tid + s * 128;
    if (k < TV.n_strips) {
      const int c = TV.chan[k];
      const float wgt = (float)(1 << TV.shift[k]) / (float)((1 << TV.width[c]) - 1);
#pragma unroll
      for (int h = 0; h < kMaxGqa; h++)
        if (h < G) atomicAdd(&S.o[h][c], acc_v[s][h] * wgt);
    }
  }
  if (tid < kMaxGqa) S.lsum[tid] = 0.f;
  if (tid < kMaxGqa * kMaxGroups) S.plo[tid / kMaxGroups][tid % kMaxGroups] = 0.f;
  __syncthreads();
#pragma unroll
  for (int h = 0; h < kMaxGqa; h++) {
    if (h < G) {
      float v = l_run[h];
#pragma unroll
      for (int s = 16; s; s >>= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
      if (lane == 0) atomicAdd(&S.lsum[h], v);
#pragma unroll
      for (int g = 0; g < kMaxGroups; g++) {
        if (g < n_groups) {
          float x = plo_run[h][g];
#pragma unroll
          for (int s = 16; s; s >>= 1) x += __shfl_xor_sync(0xffffffffu, x, s);
          if (lane == 0) atomicAdd(&S.plo[h][g], x);
        }
      }
    }
  }
  __syncthreads();
  float* part = p.partials + ((int64_t)u * p.n_splits + split) * G * kPartialStride;
  for (int idx = tid; idx < G * kD; idx += blockDim.x) {
    const int h = idx / kD, j = idx - h * kD;
    float v = S.o[h][j];
    if (TV.width[j]) v += S.plo[h][j / gs];
    part[h * kPartialStride + j] = v;
  }
  if (tid < G) {
    part[tid * kPartialStride + kD] = m_run[tid];
    part[tid * kPartialStride + kD + 1] = S.lsum[tid];
    part[tid * kPartialStride + kD + 2] = qconst;
  }
}

// Merge the sequence splits (log-sum-exp), add the rotated value mean and lift: out = (o'/l + m'_V) W_dec,V.
__global__ void __launch_bounds__(128) attention_combine_kernel(AttnArgs p) {
  __shared__ float orot[kD];
  const int tid = threadIdx.x;
  const int u = blockIdx.x;
  const int b = u / p.n_kv, hk = u - b * p.n_kv;
  const int ps = (int)(u % p.n_param_sets);
  const int G = p.gqa;
  const float* wv = p.w_dec_v + (int64_t)ps * kD * kD;
  for (int h = 0; h < G; h++) {
    const float* part = p.partials + ((int64_t)u * p.n_splits) * G * kPartialStride + h * kPartialStride;
    const int64_t sstride = (int64_t)G * kPartialStride;
    float M = -INFINITY;
    for (int s = 0; s < p.n_splits; s++) M = fmaxf(M, part[s * sstride + kD]);
    float L = 0.f, acc = 0.f;
    for (int s = 0; s < p.n_splits; s++) {
      const float ms = part[s * sstride + kD];
      const float wgt = ms == -INFINITY ? 0.f : __expf(ms - M);
      L += wgt * part[s * sstride + kD + 1];
      acc += wgt * part[s * sstride + tid];
    }
    __syncthreads();
    orot[tid] = L > 0.f ? acc / L + p.mean_rot_v[(int64_t)ps * kD + tid] : 0.f;
    __syncthreads();
    float outv = 0.f;
    for (int j = 0; j < kD; j++) outv = fmaf(orot[j], wv[j * kD + tid], outv);
    const int64_t oidx = ((int64_t)b * p.n_q + hk * G + h) * kD + tid;
    store_from_float(p.out, p.out_dtype, oidx, L > 0.f ? outv : 0.f);
    if (p.lse && tid == 0)
      p.lse[(int64_t)b * p.n_q + hk * G + h] = L > 0.f ? M + logf(L) + part[kD + 2] : -INFINITY;
  }
}

}  // namespace spectra
