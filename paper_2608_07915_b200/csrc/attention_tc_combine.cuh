// Combine kernel of the tensor-core decode attention: one CTA of 128 threads per (unit of the tensor path, head slot).
// Merges the partial records the worker warps wrote for the unit (log-sum-exp over the sequence split), folds the
// per-strip accumulators back into channels of the rotated value space, adds the rotated mean and lifts the result
// once through W_dec,V:  out = (o' / l + m'_V) W_dec,V.
#pragma once
#include "attention_tc_common.cuh"

namespace spectra {

constexpr int kCombineBatch = 32;   // records merged per batch (one per lane)
constexpr int kCombineDynSmem = kD * kD * 4 + 16;   // W_dec,V and the barrier of its copy

// A worker without tiles writes no record (only when there are fewer tiles than workers).
__device__ __noinline__ bool worker_has_tiles(long long gw, long long total, int W) {
  return (gw + 1) * total / W > gw * total / W;
}

// The CTA's work is a chain of dependent global reads, each costing a full memory latency, and it starts on a cold
// instruction cache (straight-line code costs far more per instruction than a loop that is fetched once).  So the
// reads are issued in two groups and rare cases are kept out of the main path: (1) everything whose address is
// known at launch - W_dec,V (one bulk copy into shared memory), the tile prefix, the descriptor fields, the rotated
// mean; (2) the unit's partial records, up to 32 at a time, headers and accumulators together, before any of them
// is used.  Records are merged with a running maximum; every warp computes the weights of a batch redundantly
// (lane i = record i), so the merge needs no cross-warp exchange.
__global__ void __launch_bounds__(128) attention_mma_combine_kernel(AttnArgs p, FastArgs f) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* s_w = reinterpret_cast<float*>(smem_raw);                    // W_dec,V [j][channel]
  const uint32_t wbar = smem_u32(smem_raw + kD * kD * 4);
  __shared__ float s_o[kD];
  const int tid = threadIdx.x, lane = tid & 31;
  const int vu = blockIdx.x / kFastGqa, h = blockIdx.x - vu * kFastGqa;   // unit of the tensor path, head slot of its pass
  const int u = vu / f.npass, h0 = kFastGqa * (vu - u * f.npass);
  if (h0 + h >= p.gqa) return;
  const int b = u / p.n_kv, hk = u - b * p.n_kv;
  const int ps = (int)(u % p.n_param_sets);
  const UnitDesc& D = f.desc[vu];
  // ---- first group of reads
  if (tid == 0) {
    mbar_init(wbar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    mbar_expect_tx(wbar, kD * kD * 4);
    bulk_load(smem_u32(s_w), p.w_dec_v + (int64_t)ps * kD * kD, kD * kD * 4, wbar);
  }
  const long long total = f.tile_prefix[f.n_units];
  const long long ta = f.tile_prefix[vu], tb = f.tile_prefix[vu + 1];
  const int ns = D.n_vstrips;
  const int vf1 = (int)D.vfirst[1], vf2 = (int)D.vfirst[2], vf3 = (int)D.vfirst[3];
  constexpr int kPerThread = kMaxStrips / 128;      // strips tid, tid + 128, tid + 256
  int chan[kPerThread];
  float coef[kPerThread];
#pragma unroll
  for (int q = 0; q < kPerThread; q++) { chan[q] = D.vchan[tid + 128 * q]; coef[q] = D.vcoef[tid + 128 * q]; }
  const bool has_width = p.widths_v[(int64_t)ps * kD + tid] != 0;
  const float mean_rot = p.mean_rot_v[(int64_t)ps * kD + tid];
  const float qconst = D.qconst[h];
  const int64_t hidx = (int64_t)b * p.n_q + hk * p.gqa + h0 + h;         // query head in the caller's order
  const int64_t oidx = hidx * kD + tid;
  s_o[tid] = 0.f;
  asm volatile("griddepcontrol.wait;" ::: "memory");         // from here on the main kernel's records are read
  __syncthreads();                                           // the barrier's initialisation is visible to all
  if (tb <= ta) {                                            // empty sequence
    store_from_float(p.out, p.out_dtype, oidx, 0.f);
    if (p.lse && tid == 0) p.lse[hidx] = -INFINITY;
    mbar_wait(wbar, 0);                                      // the copy must land before the shared memory is released
    return;
  }
  // workers whose tile ranges intersect this unit: the largest gw with floor(gw * total / W) <= tile
  const int W = f.total_warps;
  const int gw_first = (int)(((ta + 1) * W + total - 1) / total) - 1;
  const int gw_last = (int)((tb * W + total - 1) / total) - 1;
  const int nrec = gw_last - gw_first + 1;
  const float* rec0 = f.records + (int64_t)(gw_first + vu) * f.rec_stride + (int64_t)h * (kRecHead + f.vs_max);
  // ---- second group of reads
  float M = -INFINITY, L = 0.f, P0 = 0.f, P1 = 0.f;
  float acc[kPerThread];
#pragma unroll
  for (int q = 0; q < kPerThread; q++) acc[q] = 0.f;
  if (total >= W) {
    // every worker has tiles, so every record exists
#pragma unroll 1
    for (int r0 = 0; r0 < nrec; r0 += kCombineBatch) {
      const int nb = min(kCombineBatch, nrec - r0);
      const float* rb = rec0 + (int64_t)r0 * f.rec_stride;
      float hd[4] = {-INFINITY, 0.f, 0.f, 0.f};
      if (lane < nb) {
#pragma unroll
        for (int i = 0; i < 4; i++) hd[i] = rb[(int64_t)lane * f.rec_stride + i];
      }
      float v[kCombineBatch][2];
#pragma unroll
      for (int i = 0; i < kCombineBatch; i++) {
        const float* rv = rb + (int64_t)i * f.rec_stride + kRecHead + tid;
        v[i][0] = (i < nb && tid < ns) ? rv[0] : 0.f;
        v[i][1] = (i < nb && tid + 128 < ns) ? rv[128] : 0.f;
      }
      float mb = hd[0];
#pragma unroll
      for (int s = 16; s; s >>= 1) mb = fmaxf(mb, __shfl_xor_sync(0xffffffffu, mb, s));
      const float Mn = fmaxf(M, mb);
      const float alpha = M == -INFINITY ? 0.f : exp2f(M - Mn);
      const float e = hd[0] == -INFINITY ? 0.f : exp2f(hd[0] - Mn);
      float dl = e * hd[1], d0 = e * hd[2], d1 = e * hd[3];
#pragma unroll
      for (int s = 16; s; s >>= 1) {
        dl += __shfl_xor_sync(0xffffffffu, dl, s);
        d0 += __shfl_xor_sync(0xffffffffu, d0, s);
        d1 += __shfl_xor_sync(0xffffffffu, d1, s);
      }
      L = fmaf(L, alpha, dl); P0 = fmaf(P0, alpha, d0); P1 = fmaf(P1, alpha, d1);
#pragma unroll
      for (int q = 0; q < kPerThread; q++) acc[q] *= alpha;
#pragma unroll
      for (int i = 0; i < kCombineBatch; i++) {
        const float ei = __shfl_sync(0xffffffffu, e, i);
        acc[0] = fmaf(ei, v[i][0], acc[0]);
        acc[1] = fmaf(ei, v[i][1], acc[1]);
      }
      if (ns > 256) {                                        // third strip of a thread: widths rarely ask for it
#pragma unroll 1
        for (int i = 0; i < nb; i++) {
          const float ei = __shfl_sync(0xffffffffu, e, i);
          if (tid + 256 < ns) acc[2] = fmaf(ei, rb[(int64_t)i * f.rec_stride + kRecHead + tid + 256], acc[2]);
        }
      }
      M = Mn;
    }
  } else {
    // fewer tiles than workers (tiny calls): some workers wrote nothing; one record at a time
#pragma unroll 1
    for (int r = 0; r < nrec; r++) {
      if (!worker_has_tiles(gw_first + r, total, W)) continue;
      const float* rec = rec0 + (int64_t)r * f.rec_stride;
      const float mr = rec[0];
      if (mr == -INFINITY) continue;
      const float Mn = fmaxf(M, mr);
      const float alpha = M == -INFINITY ? 0.f : exp2f(M - Mn);
      const float e = exp2f(mr - Mn);
      L = fmaf(L, alpha, e * rec[1]); P0 = fmaf(P0, alpha, e * rec[2]); P1 = fmaf(P1, alpha, e * rec[3]);
#pragma unroll
      for (int q = 0; q < kPerThread; q++)
        acc[q] = fmaf(acc[q], alpha, tid + 128 * q < ns ? e * rec[kRecHead + tid + 128 * q] : 0.f);
      M = Mn;
    }
  }
  // strips of one class belong to distinct channels: adding class by class needs no atomics and has a fixed order
#pragma unroll 1
  for (int c = 0; c < 4; c++) {
#pragma unroll
    for (int q = 0; q < kPerThread; q++) {
      const int k = tid + 128 * q;
      if (k < ns && (k >= vf1) + (k >= vf2) + (k >= vf3) == c) s_o[chan[q]] += acc[q] * coef[q];
    }
    __syncthreads();
  }
  // ---- normalise, add the group offsets and the rotated mean, lift
  const bool live = L > 0.f;
  float val = 0.f;
  if (live) {
    val = s_o[tid];
    if (has_width) val += tid < 64 ? P0 : P1;
    val = val / L + mean_rot;
  }
  __syncthreads();
  s_o[tid] = val;
  __syncthreads();
  const bool ok = mbar_wait(wbar, 0);
  if (!ok && tid == 0 && p.status) atomicOr(p.status, SPECTRA_STATUS_WAIT_TIMEOUT);
  float o0 = 0.f, o1 = 0.f, o2 = 0.f, o3 = 0.f;
#pragma unroll 4
  for (int j = 0; j < kD; j += 4) {
    o0 = fmaf(s_o[j], s_w[j * kD + tid], o0);
    o1 = fmaf(s_o[j + 1], s_w[(j + 1) * kD + tid], o1);
    o2 = fmaf(s_o[j + 2], s_w[(j + 2) * kD + tid], o2);
    o3 = fmaf(s_o[j + 3], s_w[(j + 3) * kD + tid], o3);
  }
  store_from_float(p.out, p.out_dtype, oidx, live && ok ? (o0 + o1) + (o2 + o3) : 0.f);
  if (p.lse && tid == 0)
    p.lse[hidx] = live ? (M + log2f(L)) / kLog2e + qconst : -INFINITY;
}

}  // namespace spectra
