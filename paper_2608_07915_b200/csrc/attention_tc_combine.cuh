// Combine kernel of the tensor-core decode attention: one CTA of 128 threads per (unit of the tensor path, head slot).
// Merges the partial records the worker warps wrote for the unit (log-sum-exp over the sequence split), folds the
// per-strip accumulators back into channels of the rotated value space, adds the rotated mean and lifts the result
// once through W_dec,V:  out = (o' / l + m'_V) W_dec,V.
#pragma once
#include "attention_tc_common.cuh"

namespace spectra {

constexpr int kMaxRecSmem = 2048;   // record headers kept in shared memory; longer lists are re-read from global

__global__ void __launch_bounds__(128) attention_mma_combine_kernel(AttnArgs p, FastArgs f) {
  __shared__ float s_e[kMaxRecSmem];       // exp2(m_r - M), 0 for workers that wrote nothing
  __shared__ float s_red[4][4];
  __shared__ float s_o[kD];
  __shared__ float s_part[4][kMaxStrips];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int vu = blockIdx.x / kFastGqa, h = blockIdx.x - vu * kFastGqa;   // unit of the tensor path, head slot of its pass
  const int u = vu / f.npass, h0 = kFastGqa * (vu - u * f.npass);
  if (h0 + h >= p.gqa) return;
  const int b = u / p.n_kv, hk = u - b * p.n_kv;
  const int ps = (int)(u % p.n_param_sets);
  const UnitDesc& D = f.desc[vu];
  {  // the tail of this CTA's dependent chain reads W_dec,V, the rotated mean and the strip tables: ask for them now
    const float* wv = p.w_dec_v + (int64_t)ps * kD * kD;
#pragma unroll
    for (int i = 0; i < 4; i++) prefetch_l2(wv + (tid * 4 + i) * 32);
    if (tid < 4) prefetch_l2(p.mean_rot_v + (int64_t)ps * kD + tid * 32);
    if (tid >= 32 && tid < 32 + kMaxStrips * 4 / 128) prefetch_l2(D.vcoef + (tid - 32) * 32);
    if (tid >= 64 && tid < 64 + kMaxStrips / 128) prefetch_l2(D.vchan + (tid - 64) * 128);
    if (tid == 96) prefetch_l2(p.widths_v + (int64_t)ps * kD);
  }
  const long long total = f.tile_prefix[f.n_units];
  const long long ta = f.tile_prefix[vu], tb = f.tile_prefix[vu + 1];
  const int64_t hidx = (int64_t)b * p.n_q + hk * p.gqa + h0 + h;         // query head in the caller's order
  const int64_t oidx = hidx * kD + tid;
  if (tb <= ta) {                                            // empty sequence
    store_from_float(p.out, p.out_dtype, oidx, 0.f);
    if (p.lse && tid == 0) p.lse[hidx] = -INFINITY;
    return;
  }
  // workers whose tile ranges intersect this unit: the largest gw with floor(gw * total / W) <= tile
  const int W = f.total_warps;
  const int gw_first = (int)(((ta + 1) * W + total - 1) / total) - 1;
  const int gw_last = (int)((tb * W + total - 1) / total) - 1;
  const int nrec = gw_last - gw_first + 1;
  const int64_t hoff = (int64_t)h * (kRecHead + f.vs_max);
  auto rec_ptr = [&](int r) { return f.records + (int64_t)(gw_first + r + vu) * f.rec_stride + hoff; };
  auto nonempty = [&](int r) {
    const long long gw = gw_first + r;
    return (gw + 1) * total / W > gw * total / W;
  };
  // ---- running maximum over the records
  float m = -INFINITY;
  for (int r = tid; r < nrec; r += 128)
    if (nonempty(r)) m = fmaxf(m, rec_ptr(r)[0]);
#pragma unroll
  for (int s = 16; s; s >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, s));
  if (lane == 0) s_red[0][warp] = m;
  __syncthreads();
  const float M = fmaxf(fmaxf(s_red[0][0], s_red[0][1]), fmaxf(s_red[0][2], s_red[0][3]));
  __syncthreads();
  // ---- weights of the records, softmax denominator, offset sums
  float L = 0.f, P0 = 0.f, P1 = 0.f;
  for (int r = tid; r < nrec; r += 128) {
    float e = 0.f;
    if (nonempty(r)) {
      const float* rec = rec_ptr(r);
      const float mr = rec[0];
      e = mr == -INFINITY ? 0.f : exp2f(mr - M);
      L += e * rec[1]; P0 += e * rec[2]; P1 += e * rec[3];
    }
    if (r < kMaxRecSmem) s_e[r] = e;
  }
#pragma unroll
  for (int s = 16; s; s >>= 1) {
    L += __shfl_xor_sync(0xffffffffu, L, s);
    P0 += __shfl_xor_sync(0xffffffffu, P0, s);
    P1 += __shfl_xor_sync(0xffffffffu, P1, s);
  }
  if (lane == 0) { s_red[1][warp] = L; s_red[2][warp] = P0; s_red[3][warp] = P1; }
  s_o[tid] = 0.f;
  __syncthreads();
  L = s_red[1][0] + s_red[1][1] + s_red[1][2] + s_red[1][3];
  P0 = s_red[2][0] + s_red[2][1] + s_red[2][2] + s_red[2][3];
  P1 = s_red[3][0] + s_red[3][1] + s_red[3][2] + s_red[3][3];
  // ---- per-strip sums: warp w takes records w, w + 4, ..; lanes take strips lane, lane + 32, ..
  const int ns = D.n_vstrips;
  constexpr int kPerLane = kMaxStrips / 32;
  float acc[kPerLane];
#pragma unroll
  for (int i = 0; i < kPerLane; i++) acc[i] = 0.f;
  for (int r = warp; r < nrec; r += 4) {
    float e;
    if (r < kMaxRecSmem) e = s_e[r];
    else { e = 0.f; if (nonempty(r)) { const float mr = rec_ptr(r)[0]; e = mr == -INFINITY ? 0.f : exp2f(mr - M); } }
    if (e == 0.f) continue;
    const float* rec = rec_ptr(r) + kRecHead;
#pragma unroll
    for (int i = 0; i < kPerLane; i++) {
      const int k = lane + 32 * i;
      if (k < ns) acc[i] = fmaf(e, rec[k], acc[i]);
    }
  }
#pragma unroll
  for (int i = 0; i < kPerLane; i++) s_part[warp][lane + 32 * i] = acc[i];
  __syncthreads();
  for (int k = tid; k < ns; k += 128) {
    const float v = s_part[0][k] + s_part[1][k] + s_part[2][k] + s_part[3][k];
    atomicAdd(&s_o[D.vchan[k]], v * D.vcoef[k]);
  }
  __syncthreads();
  // ---- normalise, add the group offsets and the rotated mean, lift
  const bool live = L > 0.f;
  float v = 0.f;
  if (live) {
    v = s_o[tid];
    if (p.widths_v[(int64_t)ps * kD + tid]) v += tid < 64 ? P0 : P1;
    v = v / L + p.mean_rot_v[(int64_t)ps * kD + tid];
  }
  __syncthreads();
  s_o[tid] = v;
  __syncthreads();
  const float* wv = p.w_dec_v + (int64_t)ps * kD * kD;
  float o0 = 0.f, o1 = 0.f, o2 = 0.f, o3 = 0.f;
#pragma unroll 8
  for (int j = 0; j < kD; j += 4) {
    o0 = fmaf(s_o[j], wv[j * kD + tid], o0);
    o1 = fmaf(s_o[j + 1], wv[(j + 1) * kD + tid], o1);
    o2 = fmaf(s_o[j + 2], wv[(j + 2) * kD + tid], o2);
    o3 = fmaf(s_o[j + 3], wv[(j + 3) * kD + tid], o3);
  }
  store_from_float(p.out, p.out_dtype, oidx, live ? (o0 + o1) + (o2 + o3) : 0.f);
  if (p.lse && tid == 0)
    p.lse[hidx] = live ? (M + log2f(L)) / kLog2e + D.qconst[h] : -INFINITY;
}

}  // namespace spectra
