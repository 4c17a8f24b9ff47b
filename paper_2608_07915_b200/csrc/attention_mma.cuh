// Fused coded-cache decode attention for GQA groups of up to 4 query heads and scale_group 64.
//
// Three kernels per call:
//   prep    (one CTA per unit)  folds W_dec,K and the softmax scale into the query (q'), turns it into
//           tensor-core B fragments per 16-strip chunk of the K tile, and lays out the per-unit descriptor;
//           one extra CTA builds the tile prefix sums and each warp's starting unit.
//   main    persistent, one warp = one worker.  The (unit, tile) space is flattened and cut into equal
//           contiguous ranges, one per warp.  A warp streams its K and V tiles into its own shared-memory
//           ring with 1-D bulk copies (cp.async.bulk + mbarrier), and per 64-token half tile
//             - unpacks K codes straight into mma.sync A fragments (rows = tokens, k = strips), multiplies by
//               the q' fragments (columns = head x {hi, lo} halves of an fp16 split), applies the per-token
//               group scales, runs the online softmax with warp shuffles,
//             - transposes the probabilities (times the V group ranges) with movmatrix into B fragments,
//             - unpacks V codes into A fragments (rows = strips, k = tokens) and accumulates the output in the
//               rotated value space in registers.
//           At the end of a unit the warp writes one partial record (max, sum, accumulators per V strip).
//   combine (one CTA per unit)  merges the records (log-sum-exp), folds strips back into channels, adds the
//           rotated mean and lifts the result once with W_dec,V.
//
// Codes enter the MMA as fp16 numbers 2^w + code, built with one shift and one logic op per pair: the field is
// moved to the top of the fp16 mantissa and OR-ed with the exponent of 2^w.  The constant 2^w is removed
// analytically (K: precomputed per head and group; V: an extra all-ones MMA row sum).
#pragma once
#include "attention_generic.cuh"

namespace spectra {

constexpr int kFastGqa = 4;
constexpr int kKcMax = 28;       // upper bound of 16-strip chunks in a K tile (384 strips in 4 classes)
constexpr int kFastWarps = 4;    // warps per CTA of the main kernel
constexpr int kRecHead = 4;      // floats of a record's per-head header: m, l, plo0, plo1
constexpr float kLog2e = 1.4426950408889634f;

struct alignas(16) UnitDesc {
  int32_t tbk, tbv;
  int32_t kmeta[2], vmeta[2];   // byte offset of lo16[128] of scale group g (R16 256 bytes later), -1 if inactive
  uint32_t kcls[4], vcls[4];    // per class: strips | strips of scale group 0 << 8 | (byte offset / 16) << 16
  uint32_t vfirst[4];           // index of the first V strip of each class
  int32_t n_vstrips, pad0;
  float kscale[4];              // 2^-e_h
  float kcorr[4][2];            // sum_k 2^w_k (B_hi + B_lo) per head and scale group
  float qlo[4][2];              // sum of q' over the active channels of a scale group
  float qconst[4];              // q' . m'_K (natural-log units)
  uint2 kB[kKcMax][2][32];      // [chunk][scale group][lane] -> (b0, b1)
};

struct FastArgs {
  UnitDesc* desc; int32_t* tile_prefix; int32_t* warp_unit; float* records;
  int total_warps; int rec_stride; int vs_max; int n_units;
  int depth; int slot_k, slot_v;
};

// ------------------------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after a fixed number of polls (each poll itself blocks for a bounded hardware interval).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (int it = 0; it < (1 << 20); ++it)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t lds32(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ uint32_t lds16(uint32_t a) {
  uint16_t v;
  asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t a) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
  return v;
}
__device__ __forceinline__ uint4 lds128(uint32_t a) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
  return v;
}

__device__ __forceinline__ float2 h2f2(uint32_t x) {
  __half2 h;
  *reinterpret_cast<uint32_t*>(&h) = x;
  return __half22float2(h);
}

// ------------------------------------------------------------------------------------------------ unpacking
// Words a thread needs for its 8 tokens of one 64-token half tile, per class width W.
template <int W> struct WordsPerPass { static constexpr int n = W == 8 ? 4 : (W == 4 ? 2 : 1); };

// fp16 pair (2^W + field_lo, 2^W + field_hi): the fields of in-pass token `ii` in the two half-words of a word.
template <int W>
__device__ __forceinline__ uint32_t extract(const uint32_t (&wd)[WordsPerPass<W>::n], int ii) {
  constexpr int per = 16 / W;                              // tokens per half-word
  const int wi = W == 1 ? 0 : ii / per;
  const int pos = (W == 1 ? ii : (ii % per)) * W;
  constexpr int top = 10 - W;                              // field goes to mantissa bits [10-W, 10)
  constexpr uint32_t mask = (((1u << W) - 1u) << top) * 0x00010001u;
  constexpr uint32_t magic = ((uint32_t)(15 + W) << 10) * 0x00010001u;
  const uint32_t x = pos >= top ? (wd[wi] >> (pos - top)) : (wd[wi] << (top - pos));
  return (x & mask) | magic;
}

// Loads the words of one K pair slot (two strips interleaved at 16 bits) for tokens gid*16 + 8*hp + [0, 8).
// `ns` strips of the chunk exist; slot ps holds strips 2ps and 2ps+1; an odd last strip is stored alone.
template <int W>
__device__ __forceinline__ void load_k_words(uint32_t chunk_base, int ps, int gid, int hp, int ns,
                                             uint32_t (&wd)[WordsPerPass<W>::n]) {
  constexpr int NW = WordsPerPass<W>::n;
#pragma unroll
  for (int i = 0; i < NW; i++) wd[i] = 0u;
  if (2 * ps + 1 < ns) {
    const uint32_t a = chunk_base + 32 * W * ps + 4 * W * gid + (W == 1 ? 0 : 4 * NW * hp);
    if constexpr (W == 8) { const uint4 v = lds128(a); wd[0] = v.x; wd[1] = v.y; wd[2] = v.z; wd[3] = v.w; }
    else if constexpr (W == 4) { const uint2 v = lds64(a); wd[0] = v.x; wd[1] = v.y; }
    else wd[0] = lds32(a);
  } else if (2 * ps < ns) {
    const uint32_t a = chunk_base + 32 * W * ps + 2 * W * gid + (W == 1 ? 0 : 2 * NW * hp);
    if constexpr (W == 8) { const uint2 v = lds64(a); wd[0] = v.x & 0xffffu; wd[1] = v.x >> 16; wd[2] = v.y & 0xffffu; wd[3] = v.y >> 16; }
    else if constexpr (W == 4) { const uint32_t v = lds32(a); wd[0] = v & 0xffffu; wd[1] = v >> 16; }
    else wd[0] = lds16(a);
  }
  if constexpr (W == 1) wd[0] >>= 8 * hp;
}

// Loads the words of V strip `row` of a class (n strips) for token pairs (32 tig + i, 32 tig + 16 + i), i in the pass.
template <int W>
__device__ __forceinline__ void load_v_words(uint32_t class_base, int row, int n, int tig, int hp,
                                             uint32_t (&wd)[WordsPerPass<W>::n]) {
  constexpr int NW = WordsPerPass<W>::n;
#pragma unroll
  for (int i = 0; i < NW; i++) wd[i] = 0u;
  if (row < n) {
    const uint32_t a = class_base + 16 * W * row + 4 * W * tig + (W == 1 ? 0 : 4 * NW * hp);
    if constexpr (W == 8) { const uint4 v = lds128(a); wd[0] = v.x; wd[1] = v.y; wd[2] = v.z; wd[3] = v.w; }
    else if constexpr (W == 4) { const uint2 v = lds64(a); wd[0] = v.x; wd[1] = v.y; }
    else wd[0] = lds32(a);
  }
  if constexpr (W == 1) wd[0] >>= 8 * hp;
}

// Scores of one class of the K tile for one half tile: acc[g][u] += A(chunk) x B(chunk, g).
template <int W>
__device__ __forceinline__ void k_class(uint32_t ktile, uint32_t cls, const uint2* __restrict__ kB, int& chunk_id,
                                        int hp, int gid, int tig, int lane, float (&acc)[2][4][4]) {
  const int n = cls & 0xff, n_g0 = (cls >> 8) & 0xff;
  const uint32_t base = ktile + (cls >> 16) * 16;
  constexpr int NW = WordsPerPass<W>::n;
  for (int ci = 0; ci * 16 < n; ci++, chunk_id++) {
    const int ns = min(16, n - 16 * ci);
    const bool has0 = 16 * ci < n_g0, has1 = 16 * ci + ns > n_g0;
    uint2 b0 = make_uint2(0u, 0u), b1 = make_uint2(0u, 0u);
    if (has0) b0 = __ldg(kB + (chunk_id * 2 + 0) * 32 + lane);
    if (has1) b1 = __ldg(kB + (chunk_id * 2 + 1) * 32 + lane);
    uint32_t wa[NW], wb[NW];
    load_k_words<W>(base + 256 * W * ci, tig, gid, hp, ns, wa);
    load_k_words<W>(base + 256 * W * ci, tig + 4, gid, hp, ns, wb);
#pragma unroll
    for (int u = 0; u < 4; u++) {
      const uint32_t a0 = extract<W>(wa, 2 * u), a1 = extract<W>(wa, 2 * u + 1);
      const uint32_t a2 = extract<W>(wb, 2 * u), a3 = extract<W>(wb, 2 * u + 1);
      if (has0) mma16816(acc[0][u], a0, a1, a2, a3, b0.x, b0.y);
      if (has1) mma16816(acc[1][u], a0, a1, a2, a3, b1.x, b1.y);
    }
  }
}

// One 16-strip block of the V tile for one half tile: acc += A(block) x P~.
template <int W>
__device__ __forceinline__ void v_block(uint32_t vtile, uint32_t cls, int bi, int hp, int gid, int tig,
                                        const uint32_t (&pb)[8], float (&acc)[4]) {
  const int n = cls & 0xff;
  const uint32_t base = vtile + (cls >> 16) * 16;
  constexpr int NW = WordsPerPass<W>::n;
  uint32_t wa[NW], wb[NW];
  load_v_words<W>(base, 16 * bi + gid, n, tig, hp, wa);
  load_v_words<W>(base, 16 * bi + gid + 8, n, tig, hp, wb);
#pragma unroll
  for (int u = 0; u < 4; u++) {
    const uint32_t a0 = extract<W>(wa, 2 * u), a1 = extract<W>(wb, 2 * u);
    const uint32_t a2 = extract<W>(wa, 2 * u + 1), a3 = extract<W>(wb, 2 * u + 1);
    mma16816(acc, a0, a1, a2, a3, pb[2 * u], pb[2 * u + 1]);
  }
}

// ------------------------------------------------------------------------------------------------ prep kernel
struct PrepSmem {
  StripTable tk, tv;
  alignas(16) float qraw[kFastGqa][kD];
  alignas(16) float qrot[kFastGqa][kD];
  __half bhi[kFastGqa][kMaxStrips];
  __half blo[kFastGqa][kMaxStrips];
  float red[kFastGqa][4];
  int escale[kFastGqa];
  int scan[128];
};

__device__ inline uint32_t pack_cls(const StripTable& T, int c) {
  const int first = T.class_first[c], n = T.class_first[c + 1] - first;
  int n_g0 = 0;
  for (int k = first; k < first + n; k++) n_g0 += T.chan[k] < 64;
  return (uint32_t)n | ((uint32_t)n_g0 << 8) | ((uint32_t)(T.class_off[c] / 16) << 16);
}

__global__ void __launch_bounds__(128) attention_prep_kernel(AttnArgs p, FastArgs f) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  PrepSmem& S = *reinterpret_cast<PrepSmem*>(smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if ((int)blockIdx.x == f.n_units) {
    // ---- tile prefix sums over units and each worker warp's first unit
    const int n_units = f.n_units;
    const int per = (n_units + 127) / 128;
    int local = 0;
    for (int i = tid * per; i < min((tid + 1) * per, n_units); i++) local += (p.seq_len[i / p.n_kv] + kTile - 1) / kTile;
    S.scan[tid] = local;
    __syncthreads();
    if (tid == 0) {
      int run = 0;
      for (int i = 0; i < 128; i++) { const int v = S.scan[i]; S.scan[i] = run; run += v; }
      f.tile_prefix[n_units] = run;
    }
    __syncthreads();
    int run = S.scan[tid];
    for (int i = tid * per; i < min((tid + 1) * per, n_units); i++) {
      f.tile_prefix[i] = run;
      run += (p.seq_len[i / p.n_kv] + kTile - 1) / kTile;
    }
    __syncthreads();
    __threadfence_block();
    const long long total = f.tile_prefix[n_units];
    for (int gw = tid; gw < f.total_warps; gw += 128) {
      const long long g0 = (long long)gw * total / f.total_warps;
      int lo = 0, hi = n_units;             // first unit whose end is beyond g0
      while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (f.tile_prefix[mid + 1] > g0) hi = mid; else lo = mid + 1;
      }
      f.warp_unit[gw] = lo;
    }
    return;
  }
  const int u = blockIdx.x;
  const int b = u / p.n_kv, hk = u - b * p.n_kv;
  const int ps = (int)(u % p.n_param_sets);
  const int G = p.gqa;
  build_strip_table(S.tk, p.widths_k + (int64_t)ps * kD, 64);
  build_strip_table(S.tv, p.widths_v + (int64_t)ps * kD, 64);
  const StripTable& TK = S.tk;
  const StripTable& TV = S.tv;
  UnitDesc& D = f.desc[u];
  for (int idx = tid; idx < kFastGqa * kD; idx += 128) {
    const int h = idx / kD, i = idx - h * kD;
    S.qraw[h][i] = h < G ? load_as_float(p.q, p.q_dtype, ((int64_t)b * p.n_q + hk * G + h) * kD + i) : 0.f;
  }
  __syncthreads();
  const float* wk = p.w_dec_k + (int64_t)ps * kD * kD;
  for (int j = warp; j < kD; j += 4) {
    const float4 wrow = *reinterpret_cast<const float4*>(wk + j * kD + lane * 4);
#pragma unroll
    for (int h = 0; h < kFastGqa; h++) {
      const float4 qv = *reinterpret_cast<const float4*>(&S.qraw[h][lane * 4]);
      float acc = wrow.x * qv.x + wrow.y * qv.y + wrow.z * qv.z + wrow.w * qv.w;
#pragma unroll
      for (int s = 16; s; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
      if (lane == 0) S.qrot[h][j] = acc * p.scale * kLog2e;   // scores live in the log2 domain
    }
  }
  __syncthreads();
  // per-head power-of-two normalisation so that the fp16 hi/lo split of q'' = q' 2^shift / L is well conditioned
  const int nk = TK.n_strips;
  {
    const int h = warp;  // one warp per head
    float mx = 0.f;
    for (int k = lane; k < nk; k += 32) {
      const int c = TK.chan[k];
      mx = fmaxf(mx, fabsf(S.qrot[h][c] * (float)(1 << TK.shift[k]) / (float)((1 << TK.width[c]) - 1)));
    }
#pragma unroll
    for (int s = 16; s; s >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, s));
    int e = 0;
    if (mx > 0.f && isfinite(mx)) { int ex; frexpf(mx, &ex); e = 10 - ex; }
    e = max(-100, min(100, e));
    if (lane == 0) { S.escale[h] = e; D.kscale[h] = ldexpf(1.f, -e); }
    float corr0 = 0.f, corr1 = 0.f;
    for (int k = lane; k < nk; k += 32) {
      const int c = TK.chan[k];
      const float v = ldexpf(S.qrot[h][c] * (float)(1 << TK.shift[k]) / (float)((1 << TK.width[c]) - 1), e);
      const __half hi = __float2half_rn(v);
      const __half lo = __float2half_rn(v - __half2float(hi));
      S.bhi[h][k] = hi; S.blo[h][k] = lo;
      const float off = (float)(1 << (8 >> strip_class(TK, k)));    // 2^w
      const float t = off * (__half2float(hi) + __half2float(lo));
      if (c < 64) corr0 += t; else corr1 += t;
    }
    float q0 = 0.f, q1 = 0.f, qc = 0.f;
    for (int j = lane; j < kD; j += 32) {
      const float v = S.qrot[h][j];
      if (TK.width[j]) { if (j < 64) q0 += v; else q1 += v; }
      if (p.mean_rot_k) qc += v * p.mean_rot_k[(int64_t)ps * kD + j];
    }
#pragma unroll
    for (int s = 16; s; s >>= 1) {
      corr0 += __shfl_xor_sync(0xffffffffu, corr0, s); corr1 += __shfl_xor_sync(0xffffffffu, corr1, s);
      q0 += __shfl_xor_sync(0xffffffffu, q0, s); q1 += __shfl_xor_sync(0xffffffffu, q1, s);
      qc += __shfl_xor_sync(0xffffffffu, qc, s);
    }
    if (lane == 0) {
      D.kcorr[h][0] = corr0; D.kcorr[h][1] = corr1; D.qlo[h][0] = q0; D.qlo[h][1] = q1;
      D.qconst[h] = qc / kLog2e;
    }
  }
  __syncthreads();
  // B fragments: chunk = 16 consecutive strips of a class; column n = head (n >> 1), hi (n & 1 == 0) or lo half
  int chunk0 = 0;
  for (int c = 0; c < 4; c++) {
    const int first = TK.class_first[c], n = TK.class_first[c + 1] - first;
    const int nch = (n + 15) / 16;
    for (int idx = tid; idx < nch * 2 * 32; idx += 128) {
      const int ci = idx / 64, g = (idx >> 5) & 1, ln = idx & 31;
      const int gid = ln >> 2, tg = ln & 3, h = gid >> 1, part = gid & 1;
      uint32_t r[2];
#pragma unroll
      for (int half = 0; half < 2; half++) {
        uint32_t v = 0;
#pragma unroll
        for (int e = 0; e < 2; e++) {
          const int krow = 2 * tg + 8 * half + e;
          const int k = first + 16 * ci + krow;
          uint16_t bits = 0;
          if (16 * ci + krow < n && h < G && (TK.chan[k] >= 64 ? 1 : 0) == g)
            bits = __half_as_ushort(part ? S.blo[h][k] : S.bhi[h][k]);
          v |= (uint32_t)bits << (16 * e);
        }
        r[half] = v;
      }
      if (chunk0 + ci < kKcMax) D.kB[chunk0 + ci][g][ln] = make_uint2(r[0], r[1]);
    }
    chunk0 += nch;
  }
  if (tid < 4) {
    D.kcls[tid] = pack_cls(TK, tid);
    D.vcls[tid] = pack_cls(TV, tid);
    D.vfirst[tid] = TV.class_first[tid];
  }
  if (tid == 0) {
    D.tbk = TK.tile_bytes; D.tbv = TV.tile_bytes;
    D.kmeta[0] = TK.meta_off[0]; D.kmeta[1] = TK.meta_off[1];
    D.vmeta[0] = TV.meta_off[0]; D.vmeta[1] = TV.meta_off[1];
    D.n_vstrips = TV.n_strips; D.pad0 = 0;
  }
}

// ------------------------------------------------------------------------------------------------ main kernel
struct TileCursor {   // walks the flattened (unit, tile) space; all fields are warp-uniform
  int u, t, nt;
  __device__ __forceinline__ void seek_unit(const FastArgs& f) {
    while (u < f.n_units) {
      nt = f.tile_prefix[u + 1] - f.tile_prefix[u];
      if (t < nt) break;
      u++; t = 0;
    }
  }
  __device__ __forceinline__ void next(const FastArgs& f) {
    t++;
    if (t >= nt) { u++; t = 0; seek_unit(f); }
  }
};

template <int NVB>
__global__ void __launch_bounds__(kFastWarps * 32, 2) attention_mma_kernel(AttnArgs p, FastArgs f) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int gid = lane >> 2, tig = lane & 3;
  const int gw = blockIdx.x * kFastWarps + warp;
  const int D = f.depth;
  const uint32_t warp_bytes = (uint32_t)D * (f.slot_k + f.slot_v);
  const uint32_t ring = smem_u32(smem_raw) + warp * warp_bytes;
  const uint32_t ring_v = ring + D * f.slot_k;
  const uint32_t bars = smem_u32(smem_raw) + kFastWarps * warp_bytes + warp * (2 * 4 * 8);  // [K slots 0..3][V slots 0..3]
  if (lane == 0)
    for (int s = 0; s < 2 * 4; s++) mbar_init(bars + 8 * s, 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  __syncwarp();

  const long long total = f.tile_prefix[f.n_units];
  const long long g0 = (long long)gw * total / f.total_warps;
  const long long g1 = (long long)(gw + 1) * total / f.total_warps;
  const int count = (int)(g1 - g0);
  if (count <= 0) return;

  TileCursor cons, prod;
  cons.u = f.warp_unit[gw]; cons.t = (int)(g0 - f.tile_prefix[cons.u]); cons.seek_unit(f);
  prod = cons;
  int issued_k = 0, issued_v = 0;
  const uint8_t* prod_v_src = nullptr; uint32_t prod_v_bytes = 0;

  auto issue_k = [&]() {   // lane 0 only: K tile of the producer's current position, then remember its V tile
    const UnitDesc& d = f.desc[prod.u];
    const int slot = issued_k % D;
    const uint32_t tbk = d.tbk, tbv = d.tbv;
    const uint8_t* src = p.cache_k + p.off_k[prod.u] + (int64_t)prod.t * tbk;
    mbar_expect_tx(bars + 8 * slot, tbk);
    bulk_load(ring + slot * f.slot_k, src, tbk, bars + 8 * slot);
    prod_v_src = p.cache_v + p.off_v[prod.u] + (int64_t)prod.t * tbv; prod_v_bytes = tbv;
    issued_k++;
    prod.next(f);
  };
  auto issue_v = [&]() {
    const int slot = issued_v % D;
    mbar_expect_tx(bars + 8 * (4 + slot), prod_v_bytes);
    bulk_load(ring_v + slot * f.slot_v, prod_v_src, prod_v_bytes, bars + 8 * (4 + slot));
    issued_v++;
  };
  if (lane == 0) {
    for (int j = 0; j < min(D, count); j++) { issue_k(); issue_v(); }
  }

  // per-unit state
  float acc_o[NVB][4];
  float acc_one[4];
  float m_run = -INFINITY, l_run = 0.f, plo0 = 0.f, plo1 = 0.f;
  uint32_t kcls[4], vcls[4];
  int kmeta0 = -1, kmeta1 = -1, vmeta0 = -1, vmeta1 = -1;
  float kscale = 0.f, kcorr0 = 0.f, kcorr1 = 0.f, qlo0 = 0.f, qlo1 = 0.f;
  const uint2* kB = nullptr;
  int n_seq = 0;
  bool fresh = true, ok = true;

  for (int j = 0; j < count && ok; j++) {
    const int slot = j % D;
    const uint32_t parity = (uint32_t)(j / D) & 1u;
    const uint32_t ktile = ring + slot * f.slot_k, vtile = ring_v + slot * f.slot_v;
    if (fresh) {
      const UnitDesc& d = f.desc[cons.u];
#pragma unroll
      for (int c = 0; c < 4; c++) { kcls[c] = d.kcls[c]; vcls[c] = d.vcls[c]; }
      kmeta0 = d.kmeta[0]; kmeta1 = d.kmeta[1]; vmeta0 = d.vmeta[0]; vmeta1 = d.vmeta[1];
      kscale = d.kscale[tig]; kcorr0 = d.kcorr[tig][0]; kcorr1 = d.kcorr[tig][1];
      qlo0 = d.qlo[tig][0]; qlo1 = d.qlo[tig][1];
      kB = &d.kB[0][0][0];
      n_seq = p.seq_len[cons.u / p.n_kv];
#pragma unroll
      for (int mb = 0; mb < NVB; mb++)
#pragma unroll
        for (int e = 0; e < 4; e++) acc_o[mb][e] = 0.f;
#pragma unroll
      for (int e = 0; e < 4; e++) acc_one[e] = 0.f;
      m_run = -INFINITY; l_run = 0.f; plo0 = 0.f; plo1 = 0.f;
      fresh = false;
    }
    const int nb0 = ((vcls[0] & 0xff) + 15) >> 4, nb1 = nb0 + (((vcls[1] & 0xff) + 15) >> 4);
    const int nb2 = nb1 + (((vcls[2] & 0xff) + 15) >> 4), nb3 = nb2 + (((vcls[3] & 0xff) + 15) >> 4);

    for (int hp = 0; hp < 2; hp++) {
      // ------------------------------------------------------------ scores of 64 tokens
      if (hp == 0) ok = mbar_wait(bars + 8 * slot, parity);
      float acc[2][4][4];
#pragma unroll
      for (int u4 = 0; u4 < 4; u4++) {
        acc[0][u4][0] = -kcorr0; acc[0][u4][1] = 0.f; acc[0][u4][2] = -kcorr0; acc[0][u4][3] = 0.f;
        acc[1][u4][0] = -kcorr1; acc[1][u4][1] = 0.f; acc[1][u4][2] = -kcorr1; acc[1][u4][3] = 0.f;
      }
      int chunk_id = 0;
      k_class<8>(ktile, kcls[0], kB, chunk_id, hp, gid, tig, lane, acc);
      k_class<4>(ktile, kcls[1], kB, chunk_id, hp, gid, tig, lane, acc);
      k_class<2>(ktile, kcls[2], kB, chunk_id, hp, gid, tig, lane, acc);
      k_class<1>(ktile, kcls[3], kB, chunk_id, hp, gid, tig, lane, acc);

      // per-token group ranges of the K tile (fp16 lo, R), this thread's 8 tokens
      const uint32_t tok_off = 2 * (gid * 16 + 8 * hp);
      uint4 klo0 = make_uint4(0, 0, 0, 0), kr0 = klo0, klo1 = klo0, kr1 = klo0;
      if (kmeta0 >= 0) { klo0 = lds128(ktile + kmeta0 + tok_off); kr0 = lds128(ktile + kmeta0 + 256 + tok_off); }
      if (kmeta1 >= 0) { klo1 = lds128(ktile + kmeta1 + tok_off); kr1 = lds128(ktile + kmeta1 + 256 + tok_off); }
      if (hp == 1) {           // the K slot is free: refill it with the tile D positions ahead
        __syncwarp();
        if (lane == 0 && issued_k < count) { fence_async_smem(); issue_k(); }
      }
      if (hp == 0) ok = ok && mbar_wait(bars + 8 * (4 + slot), parity);
      uint4 vlo0 = make_uint4(0, 0, 0, 0), vr0 = vlo0, vlo1 = vlo0, vr1 = vlo0;
      if (vmeta0 >= 0) { vlo0 = lds128(vtile + vmeta0 + tok_off); vr0 = lds128(vtile + vmeta0 + 256 + tok_off); }
      if (vmeta1 >= 0) { vlo1 = lds128(vtile + vmeta1 + tok_off); vr1 = lds128(vtile + vmeta1 + 256 + tok_off); }

      float s[8];
      float mx = -INFINITY;
      const int tok0 = cons.t * kTile + gid * 16 + 8 * hp;
      const uint32_t klo0w[4] = {klo0.x, klo0.y, klo0.z, klo0.w}, kr0w[4] = {kr0.x, kr0.y, kr0.z, kr0.w};
      const uint32_t klo1w[4] = {klo1.x, klo1.y, klo1.z, klo1.w}, kr1w[4] = {kr1.x, kr1.y, kr1.z, kr1.w};
#pragma unroll
      for (int ii = 0; ii < 8; ii++) {
        const int u4 = ii >> 1, cb = (ii & 1) * 2;
        const float a0 = acc[0][u4][cb] + acc[0][u4][cb + 1];
        const float a1 = acc[1][u4][cb] + acc[1][u4][cb + 1];
        const float2 lo0 = h2f2(klo0w[ii >> 1]), r0 = h2f2(kr0w[ii >> 1]);
        const float2 lo1 = h2f2(klo1w[ii >> 1]), r1 = h2f2(kr1w[ii >> 1]);
        const float l0 = (ii & 1) ? lo0.y : lo0.x, rr0 = (ii & 1) ? r0.y : r0.x;
        const float l1 = (ii & 1) ? lo1.y : lo1.x, rr1 = (ii & 1) ? r1.y : r1.x;
        float v = kscale * (rr0 * a0 + rr1 * a1) + l0 * qlo0 + l1 * qlo1;
        if (tok0 + ii >= n_seq) v = -INFINITY;
        s[ii] = v;
        mx = fmaxf(mx, v);
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
      if (mx > m_run) {        // new running maximum for this thread's head: rescale what has been accumulated
        const float alpha = fast_exp2(m_run - mx);   // exp2(-inf) = 0 on the first tile
        m_run = mx;
        l_run *= alpha; plo0 *= alpha; plo1 *= alpha;
#pragma unroll
        for (int e = 0; e < 4; e++) acc_one[e] *= alpha;
#pragma unroll
        for (int mb = 0; mb < NVB; mb++)
#pragma unroll
          for (int e = 0; e < 4; e++) acc_o[mb][e] *= alpha;
      }
      // probabilities, times the V group ranges, as fp16 pairs (group 0, group 1); transposed into B fragments
      uint32_t pb[8];
      const uint32_t vlo0w[4] = {vlo0.x, vlo0.y, vlo0.z, vlo0.w}, vr0w[4] = {vr0.x, vr0.y, vr0.z, vr0.w};
      const uint32_t vlo1w[4] = {vlo1.x, vlo1.y, vlo1.z, vlo1.w}, vr1w[4] = {vr1.x, vr1.y, vr1.z, vr1.w};
#pragma unroll
      for (int ii = 0; ii < 8; ii++) {
        const float pr = m_run == -INFINITY ? 0.f : fast_exp2(s[ii] - m_run);
        const float2 lo0 = h2f2(vlo0w[ii >> 1]), r0 = h2f2(vr0w[ii >> 1]);
        const float2 lo1 = h2f2(vlo1w[ii >> 1]), r1 = h2f2(vr1w[ii >> 1]);
        l_run += pr;
        plo0 = fmaf(pr, (ii & 1) ? lo0.y : lo0.x, plo0);
        plo1 = fmaf(pr, (ii & 1) ? lo1.y : lo1.x, plo1);
        const __half2 pk = __floats2half2_rn(pr * ((ii & 1) ? r0.y : r0.x), pr * ((ii & 1) ? r1.y : r1.x));
        pb[ii] = movmatrix_trans(*reinterpret_cast<const uint32_t*>(&pk));
      }
      // ------------------------------------------------------------ P~ x V codes
#pragma unroll
      for (int u4 = 0; u4 < 4; u4++)
        mma16816(acc_one, 0x3C003C00u, 0x3C003C00u, 0x3C003C00u, 0x3C003C00u, pb[2 * u4], pb[2 * u4 + 1]);
#pragma unroll
      for (int mb = 0; mb < NVB; mb++) {
        if (mb < nb0) v_block<8>(vtile, vcls[0], mb, hp, gid, tig, pb, acc_o[mb]);
        else if (mb < nb1) v_block<4>(vtile, vcls[1], mb - nb0, hp, gid, tig, pb, acc_o[mb]);
        else if (mb < nb2) v_block<2>(vtile, vcls[2], mb - nb1, hp, gid, tig, pb, acc_o[mb]);
        else if (mb < nb3) v_block<1>(vtile, vcls[3], mb - nb2, hp, gid, tig, pb, acc_o[mb]);
      }
      if (hp == 1) {
        __syncwarp();
        if (lane == 0 && issued_v < count && issued_v < issued_k) { fence_async_smem(); issue_v(); }
      }
    }
    // ------------------------------------------------------------ end of this warp's share of the unit?
    const bool last_of_unit = (cons.t + 1 >= cons.nt) || (j + 1 >= count);
    if (last_of_unit) {
      float l = l_run, q0 = plo0, q1 = plo1;
#pragma unroll
      for (int sft = 4; sft <= 16; sft <<= 1) {
        l += __shfl_xor_sync(0xffffffffu, l, sft);
        q0 += __shfl_xor_sync(0xffffffffu, q0, sft);
        q1 += __shfl_xor_sync(0xffffffffu, q1, sft);
      }
      float* rec = f.records + (int64_t)(gw + cons.u) * f.rec_stride + tig * (kRecHead + f.vs_max);
      if (gid == 0) { rec[0] = m_run; rec[1] = l; rec[2] = q0; rec[3] = q1; }
      const UnitDesc& d = f.desc[cons.u];
#pragma unroll
      for (int mb = 0; mb < NVB; mb++) {
        if (mb < nb3) {
          const int c = (mb >= nb0) + (mb >= nb1) + (mb >= nb2);
          const int bi = mb - (c == 0 ? 0 : (c == 1 ? nb0 : (c == 2 ? nb1 : nb2)));
          const uint32_t cls = vcls[c];
          const int n = cls & 0xff, n_g0 = (cls >> 8) & 0xff;
          const float off = (float)(1 << (8 >> c));   // 2^w
          const int first = d.vfirst[c];
#pragma unroll
          for (int half = 0; half < 2; half++) {
            const int r = 16 * bi + gid + 8 * half;
            if (r < n) {
              const bool g1 = r >= n_g0;
              const float av = g1 ? acc_o[mb][2 * half + 1] : acc_o[mb][2 * half];
              rec[kRecHead + first + r] = av - off * (g1 ? acc_one[1] : acc_one[0]);
            }
          }
        }
      }
      fresh = true;
    }
    cons.next(f);
  }
  if (!ok) {
    if (lane == 0 && p.status) atomicOr(p.status, SPECTRA_STATUS_WAIT_TIMEOUT);
    // give copies that may still be in flight a bounded time to land before the shared memory is released
    for (int s = 0; s < D; s++) { mbar_wait(bars + 8 * s, 0); mbar_wait(bars + 8 * (4 + s), 0); }
  }
}

// ------------------------------------------------------------------------------------------------ combine kernel
struct CombineSmem {
  StripTable tv;
  float o[kD];
  float orot[kD];
};

__global__ void __launch_bounds__(128) attention_mma_combine_kernel(AttnArgs p, FastArgs f) {
  __shared__ CombineSmem S;
  const int tid = threadIdx.x;
  const int u = blockIdx.x;
  const int b = u / p.n_kv, hk = u - b * p.n_kv;
  const int ps = (int)(u % p.n_param_sets);
  const int G = p.gqa;
  build_strip_table(S.tv, p.widths_v + (int64_t)ps * kD, 64);
  const StripTable& TV = S.tv;
  const long long total = f.tile_prefix[f.n_units];
  const long long ta = f.tile_prefix[u], tb = f.tile_prefix[u + 1];
  const float* wv = p.w_dec_v + (int64_t)ps * kD * kD;
  // workers whose ranges intersect this unit: the largest gw with floor(gw * total / W) <= tile
  int gw_first = 0, gw_last = -1;
  if (tb > ta) {
    gw_first = (int)(((ta + 1) * f.total_warps + total - 1) / total) - 1;
    gw_last = (int)(((tb - 1 + 1) * (long long)f.total_warps + total - 1) / total) - 1;
  }
  // a worker whose range is empty wrote no record
  auto nonempty = [&](int gw) {
    return (long long)(gw + 1) * total / f.total_warps > (long long)gw * total / f.total_warps;
  };
  for (int h = 0; h < G; h++) {
    const int64_t hoff = (int64_t)h * (kRecHead + f.vs_max);
    float M = -INFINITY;
    for (int gw = gw_first; gw <= gw_last; gw++)
      if (nonempty(gw)) M = fmaxf(M, f.records[(int64_t)(gw + u) * f.rec_stride + hoff]);
    float L = 0.f, P0 = 0.f, P1 = 0.f;
    for (int gw = gw_first; gw <= gw_last; gw++) {
      if (!nonempty(gw)) continue;
      const float* rec = f.records + (int64_t)(gw + u) * f.rec_stride + hoff;
      const float e = rec[0] == -INFINITY ? 0.f : exp2f(rec[0] - M);
      L += e * rec[1]; P0 += e * rec[2]; P1 += e * rec[3];
    }
    __syncthreads();
    S.o[tid] = 0.f;
    __syncthreads();
    for (int k = tid; k < TV.n_strips; k += 128) {
      float acc = 0.f;
      for (int gw = gw_first; gw <= gw_last; gw++) {
        if (!nonempty(gw)) continue;
        const float* rec = f.records + (int64_t)(gw + u) * f.rec_stride + hoff;
        const float e = rec[0] == -INFINITY ? 0.f : exp2f(rec[0] - M);
        acc += e * rec[kRecHead + k];
      }
      const int c = TV.chan[k];
      atomicAdd(&S.o[c], acc * (float)(1 << TV.shift[k]) / (float)((1 << TV.width[c]) - 1));
    }
    __syncthreads();
    const bool live = L > 0.f;
    float v = 0.f;
    if (live) {
      v = S.o[tid];
      if (TV.width[tid]) v += tid < 64 ? P0 : P1;
      v = v / L + p.mean_rot_v[(int64_t)ps * kD + tid];
    }
    S.orot[tid] = v;
    __syncthreads();
    float outv = 0.f;
    for (int j = 0; j < kD; j++) outv = fmaf(S.orot[j], wv[j * kD + tid], outv);
    const int64_t oidx = ((int64_t)b * p.n_q + hk * G + h) * kD + tid;
    store_from_float(p.out, p.out_dtype, oidx, live ? outv : 0.f);
    if (p.lse && tid == 0)
      p.lse[(int64_t)b * p.n_q + hk * G + h] = live ? (M + log2f(L)) / kLog2e + f.desc[u].qconst[h] : -INFINITY;
  }
}

}  // namespace spectra
