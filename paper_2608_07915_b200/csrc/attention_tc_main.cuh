// Main kernel of the tensor-core decode attention: see attention_tc_common.cuh for the overall scheme.
//
// One CTA of 512 threads per SM (the 512 tensor-memory columns are all taken, so CTAs never share an SM).
//   warps 0-3    token warps: thread = token of the tile = accumulator row of the score MMA
//   warps 4-9    strip warps: thread = V strip = accumulator row of the value MMA (rows 0-127: warps 4-7, 128-191: 8-9)
//   warps 10-11  score-MMA issuers (each takes half of the k-steps, own score columns)
//   warps 12-14  value-MMA issuers (contiguous slices of the (group, k-step) job list, own accumulator sets)
//   warp 15      producer: unit contexts and K/V tiles into shared memory with 1-D bulk copies
// Issuing a tcgen05.mma costs one thread about 56 cycles whatever its shape, and the MMAs here are small
// (128 x 16 x 16), so several threads issue side by side.
//
// Tensor-memory columns: [0,112) score A operand (K codes, one buffer: it is rewritten only after the score MMAs
// that read it have completed), [112,176) scores (2 buffers x 2 issuers x 16), [176,256) value accumulators (5 sets
// x 16), [256,512) value A operand (2 buffers x 2 row blocks x 64).
//
// Every wait is bounded: a wait that gives up sets SPECTRA_STATUS_WAIT_TIMEOUT and a CTA-wide flag that makes all
// later waits return at once; the CTA then drains its copies, frees its tensor memory and returns.
#pragma once
#include "attention_tc_common.cuh"

namespace spectra {

constexpr int kMainThreads = 512;
constexpr int kMaxStages = 8;
constexpr uint32_t kColAK = 0, kColDS = 112, kColDO = 176, kColAV = 256, kTmemCols = 512;

struct MainSmem {
  UnitCtx ctx[2];
  alignas(128) uint8_t pbuf[2][4][4096];     // B operand of the value MMA: [buffer][class][128 tokens x 16 columns fp16]
  float rec[kFastGqa][kVRowsMax];            // flush staging: per head and strip
  float red[2][4][4];                        // tile maxima: [tile parity][token warp][head]
  float fsum[4][12];                         // flush: per token warp l[4], plo[4][2]
  alignas(8) uint64_t kfull[kMaxStages], vfull[kMaxStages], kempty[kMaxStages], vempty[kMaxStages];
  alignas(8) uint64_t ak_ready, s_ready[2][2], p_ready[2], av_ready[2], pv_done[2], ctx_full[2], ctx_empty[2];
  uint32_t tmem_base;
  volatile int dead;
};

// Position of this worker in the flattened (unit, tile) space.
struct Walk {
  const int32_t* prefix; int n_units;
  long long g, g_end;
  int u, tile, tiles_u, it, useq;
  bool ufirst;
  __device__ void init(const FastArgs& f, int worker) {
    prefix = f.tile_prefix; n_units = f.n_units;
    const long long total = prefix[n_units];
    g = (long long)worker * total / f.total_warps;
    g_end = (long long)(worker + 1) * total / f.total_warps;
    it = 0; useq = 0; ufirst = true;
    u = f.worker_unit[worker];
    if (g < g_end) { tile = (int)(g - prefix[u]); tiles_u = prefix[u + 1] - prefix[u]; } else { tile = 0; tiles_u = 0; }
  }
  __device__ bool done() const { return g >= g_end; }
  __device__ bool ulast() const { return tile == tiles_u - 1 || g == g_end - 1; }
  __device__ void next() {
    g++; it++; tile++; ufirst = false;
    if (tile == tiles_u && g < g_end) {
      do { u++; } while (prefix[u + 1] == prefix[u]);
      tile = 0; tiles_u = prefix[u + 1] - prefix[u]; useq++; ufirst = true;
    }
  }
};

__device__ __forceinline__ bool wait_bar(MainSmem& S, uint64_t* bar, uint32_t parity, int32_t* status) {
  const uint32_t a = smem_u32(bar);
  for (int it = 0; it < (1 << 20); ++it) {
    if (mbar_try_wait(a, parity)) return true;
    if ((it & 63) == 63 && S.dead) return false;
  }
  S.dead = 1;
  if (status) atomicOr(status, SPECTRA_STATUS_WAIT_TIMEOUT);
  return false;
}

// ---- K side: one word of a token string -> operand registers -> tensor memory
template <int SHAPE>
__device__ __forceinline__ void k_word_store(uint32_t word, uint32_t mask_addr, uint32_t taddr) {
  constexpr int NU = shape_u(SHAPE), NS = shape_s(SHAPE), N = NU + NS;
  uint32_t m[16], r[16];
#pragma unroll
  for (int i = 0; i < (N + 3) / 4; i++) {
    const uint4 v = lds128(mask_addr + 16 * i);
    m[4 * i] = v.x; m[4 * i + 1] = v.y; m[4 * i + 2] = v.z; m[4 * i + 3] = v.w;
  }
  const uint32_t ws = word >> 6;
#pragma unroll
  for (int e = 0; e < NU; e++) r[e] = word & m[e];
#pragma unroll
  for (int e = 0; e < NS; e++) r[NU + e] = ws & m[NU + e];
  if constexpr (N == 2) tc_st2(taddr, r[0], r[1]);
  else if constexpr (N == 4) tc_st4(taddr, r);
  else if constexpr (N == 8) tc_st8(taddr, r);
  else tc_st16(taddr, r);
}

// ---- V side: the 128 fields of one strip of class W -> 64 operand registers (register q * (16 / W) + e holds
// the e-th field of the low and of the high half of word q: tokens 16 bits apart)
template <int W>
__device__ __forceinline__ void v_unpack(uint32_t saddr, uint32_t (&r)[64]) {
  constexpr int PER = 16 / W;
  constexpr uint32_t M = ((1u << W) - 1u) * 0x00010001u;
#pragma unroll
  for (int q4 = 0; q4 < W; q4++) {
    const uint4 v = lds128(saddr + 16 * q4);
    const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int x = 0; x < 4; x++) {
      const uint32_t word = w4[x], ws = word >> 6;
#pragma unroll
      for (int e = 0; e < PER; e++) {
        const int p = e * W;
        r[(4 * q4 + x) * PER + e] = (p + W <= 10) ? (word & (M << p)) : (ws & (M << (p - 6)));
      }
    }
  }
}

// Where token t sits in the k order of the value MMA for class c, and the effective bit position of its field.
__device__ __forceinline__ void v_token_slot(int t, int c, int& k, int& peff) {
  const int w = 8 >> c, per = 16 >> (3 - c);          // fields per half-word = 16 / w
  const int a = t >> 5, h = (t >> 4) & 1, i = t & 15;
  const int q = a * w + ((i * w) >> 4), e = i & (per - 1);
  k = 2 * (q * per + e) + h;
  const int p = e * w;
  peff = p + w <= 10 ? p : p - 6;
}

__device__ __forceinline__ float h2f_bits(uint32_t bits) { return __half2float(__ushort_as_half((unsigned short)bits)); }

__device__ __forceinline__ uint32_t ordered_bits(float v) {
  const uint32_t b = __float_as_uint(v);
  return b ^ ((b >> 31) ? 0xffffffffu : 0x80000000u);
}
__device__ __forceinline__ float from_ordered_bits(uint32_t o) {
  return __uint_as_float(o ^ ((o >> 31) ? 0x80000000u : 0xffffffffu));
}

__global__ void __launch_bounds__(kMainThreads, 1) attention_umma_kernel(AttnArgs p, FastArgs f) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned char* smem_al = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);     // operands want 128-byte alignment
  MainSmem& S = *reinterpret_cast<MainSmem*>(smem_al);
  uint8_t* ring = smem_al + ((sizeof(MainSmem) + 127) & ~(size_t)127);   // [stage][K slot | V slot]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int NS = f.depth;
  const uint32_t stage_bytes = (uint32_t)(f.slot_k + f.slot_v);
  const int worker = blockIdx.x;

  if (tid == 0) {
    for (int s = 0; s < kMaxStages; s++) {
      mbar_init(smem_u32(&S.kfull[s]), 1); mbar_init(smem_u32(&S.vfull[s]), 1);
      mbar_init(smem_u32(&S.kempty[s]), 4); mbar_init(smem_u32(&S.vempty[s]), 10);
    }
    mbar_init(smem_u32(&S.ak_ready), 4);
    for (int b = 0; b < 2; b++) {
      mbar_init(smem_u32(&S.s_ready[b][0]), 1); mbar_init(smem_u32(&S.s_ready[b][1]), 1);
      mbar_init(smem_u32(&S.p_ready[b]), 4); mbar_init(smem_u32(&S.av_ready[b]), 6);
      mbar_init(smem_u32(&S.pv_done[b]), kVIssuers);
      mbar_init(smem_u32(&S.ctx_full[b]), 1); mbar_init(smem_u32(&S.ctx_empty[b]), 15);
    }
    S.dead = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 15) tmem_alloc(smem_u32(&S.tmem_base), kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tb = S.tmem_base;

  Walk wk;
  wk.init(f, worker);

  if (warp == 15) {
    // ================================================================ producer
    if (lane == 0) {
      int issued = 0;
      uint32_t tbk = 0, tbv = 0;
      const uint8_t* src_k = nullptr;
      const uint8_t* src_v = nullptr;
      for (; !wk.done(); wk.next()) {
        if (wk.ufirst) {
          const UnitCtx* gctx = f.ctx + wk.u;
          const int cb = wk.useq & 1;
          if (wk.useq >= 2 && !wait_bar(S, &S.ctx_empty[cb], ((wk.useq >> 1) - 1) & 1, p.status)) break;
          mbar_expect_tx(smem_u32(&S.ctx_full[cb]), (uint32_t)sizeof(UnitCtx));
          bulk_load(smem_u32(&S.ctx[cb]), gctx, (uint32_t)sizeof(UnitCtx), smem_u32(&S.ctx_full[cb]));
          tbk = (uint32_t)gctx->tbk; tbv = (uint32_t)gctx->tbv;
          src_k = p.cache_k + p.off_k[wk.u]; src_v = p.cache_v + p.off_v[wk.u];
        }
        const int s = wk.it % NS;
        const uint32_t par = ((wk.it / NS) - 1) & 1;
        if (wk.it >= NS && !wait_bar(S, &S.kempty[s], par, p.status)) break;
        mbar_expect_tx(smem_u32(&S.kfull[s]), tbk);
        bulk_load(smem_u32(ring + s * stage_bytes), src_k + (int64_t)wk.tile * tbk, tbk, smem_u32(&S.kfull[s]));
        if (wk.it >= NS && !wait_bar(S, &S.vempty[s], par, p.status)) break;
        mbar_expect_tx(smem_u32(&S.vfull[s]), tbv);
        bulk_load(smem_u32(ring + s * stage_bytes + f.slot_k), src_v + (int64_t)wk.tile * tbv, tbv, smem_u32(&S.vfull[s]));
        issued = wk.it + 1;
      }
      if (S.dead) {
        // drain: copies already issued must land before the CTA may exit (bounded polls, no flag checks)
        for (int i = max(issued - NS, 0); i < issued; i++) {
          const int s = i % NS;
          for (int n = 0; n < (1 << 16) && !mbar_try_wait(smem_u32(&S.kfull[s]), (i / NS) & 1); n++) {}
          for (int n = 0; n < (1 << 16) && !mbar_try_wait(smem_u32(&S.vfull[s]), (i / NS) & 1); n++) {}
        }
      }
    }
  } else if (warp >= 10 && warp < 12) {
    // ================================================================ score-MMA issuers
    if (lane == 0) {
      const int j = warp - 10;
      for (; !wk.done(); wk.next()) {
        const int cb = wk.useq & 1, b = wk.it & 1;
        if (wk.ufirst && !wait_bar(S, &S.ctx_full[cb], (wk.useq >> 1) & 1, p.status)) break;
        const UnitCtx& C = S.ctx[cb];
        if (!wait_bar(S, &S.ak_ready, wk.it & 1, p.status)) break;
        tc_fence_after();
        const int mid = C.k_steps >> 1;
        const int k0 = j ? mid : 0, k1 = j ? C.k_steps : mid;
        const uint32_t d = tb + kColDS + (uint32_t)(2 * b + j) * 16;
        const uint32_t kb = smem_u32(C.kb);
        for (int ks = k0; ks < k1; ks++)
          tc_mma(d, tb + kColAK + 8 * ks, smem_desc(kb + 512 * ks, 128, 256), kIdescKMajor, ks != k0);
        tc_commit(smem_u32(&S.s_ready[b][j]));
        if (wk.ulast()) mbar_arrive(smem_u32(&S.ctx_empty[cb]));
      }
    }
  } else if (warp >= 12 && warp < 15) {
    // ================================================================ value-MMA issuers
    if (lane == 0) {
      const int j = warp - 12;
      int ja = 0, jb = 0, set0 = 0;
      for (; !wk.done(); wk.next()) {
        const int cb = wk.useq & 1, b = wk.it & 1;
        if (wk.ufirst && !wait_bar(S, &S.ctx_full[cb], (wk.useq >> 1) & 1, p.status)) break;
        const UnitCtx& C = S.ctx[cb];
        if (wk.ufirst) {
          const int J = 8 * C.n_vgroups;
          ja = j * J / kVIssuers; jb = (j + 1) * J / kVIssuers;
          int sg[kVSetsMax + 3], si[kVSetsMax + 3];
          const int ns = v_sets(C.n_vgroups, sg, si);
          set0 = 0;
          for (int s = 0; s < ns; s++) if (si[s] < j) set0++;
        }
        if (!wait_bar(S, &S.p_ready[b], (wk.it >> 1) & 1, p.status)) break;
        if (!wait_bar(S, &S.av_ready[b], (wk.it >> 1) & 1, p.status)) break;
        tc_fence_after();
        int prev_g = -1, set = set0 - 1;
        for (int job = ja; job < jb; job++) {
          const int g = job >> 3, ks = job & 7;
          const bool first = g != prev_g;
          if (first) { set++; prev_g = g; }
          const int rb = C.vgroup[g] & 0xff, cls = C.vgroup[g] >> 8;
          tc_mma(tb + kColDO + 16 * set, tb + kColAV + (uint32_t)(2 * b + rb) * 64 + 8 * ks,
                 smem_desc(smem_u32(&S.pbuf[b][cls][0]) + 256 * ks, 128, 2048), kIdescMnMajor, !(wk.ufirst && first));
        }
        tc_commit(smem_u32(&S.pv_done[b]));
        if (wk.ulast()) mbar_arrive(smem_u32(&S.ctx_empty[cb]));
      }
    }
  } else if (warp >= 4) {
    // ================================================================ strip warps (value A operand)
    const int rb = (warp - 4) >> 2, quarter = warp & 3;
    const int row = rb * 128 + quarter * 32 + lane;
    uint32_t entry = 0;
    for (; !wk.done(); wk.next()) {
      const int cb = wk.useq & 1, b = wk.it & 1, s = wk.it % NS;
      if (wk.ufirst) {
        if (!wait_bar(S, &S.ctx_full[cb], (wk.useq >> 1) & 1, p.status)) break;
        entry = S.ctx[cb].vrow[row];
      }
      if (!wait_bar(S, &S.vfull[s], (wk.it / NS) & 1, p.status)) break;
      if (wk.it >= 2 && !wait_bar(S, &S.pv_done[b], ((wk.it - 2) >> 1) & 1, p.status)) break;
      tc_fence_after();
      if (rb * 128 < S.ctx[cb].n_vrows) {
        uint32_t r[64];
        const uint32_t src = smem_u32(ring + s * stage_bytes + f.slot_k) + ((entry & 0xfffu) << 4);
        const int cls = (entry >> 12) & 3;
        if (!(entry >> 31)) {
#pragma unroll
          for (int i = 0; i < 64; i++) r[i] = 0u;
        } else if (cls == 2) v_unpack<2>(src, r);
        else if (cls == 3) v_unpack<1>(src, r);
        else if (cls == 1) v_unpack<4>(src, r);
        else v_unpack<8>(src, r);
        __syncwarp();
        const uint32_t dst = tb + ((uint32_t)(quarter * 32) << 16) + kColAV + (uint32_t)(2 * b + rb) * 64;
        tc_st16(dst, r); tc_st16(dst + 16, r + 16); tc_st16(dst + 32, r + 32); tc_st16(dst + 48, r + 48);
        tc_wait_st();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(smem_u32(&S.av_ready[b]));
        mbar_arrive(smem_u32(&S.vempty[s]));
        if (wk.ulast()) mbar_arrive(smem_u32(&S.ctx_empty[cb]));
      }
    }
  } else {
    // ================================================================ token warps
    const int t = tid;
    const uint32_t lane_base = tb + ((uint32_t)(warp * 32) << 16);
    // where this token sits in the k order of each V class, and the power of two that undoes its field position
    uint32_t prow[4], pscale[4];
#pragma unroll
    for (int c = 0; c < 4; c++) {
      int k, peff;
      v_token_slot(t, c, k, peff);
      prow[c] = (uint32_t)((k >> 3) * 128 + (k & 7) * 16);
      const uint32_t hs = (uint32_t)(15 - peff) << 10;           // fp16 bits of 2^-peff
      pscale[c] = hs | (hs << 16);
    }
    float m_run[4], l_run[4], plo[4][2];
#pragma unroll
    for (int h = 0; h < 4; h++) { m_run[h] = -INFINITY; l_run[h] = 0.f; plo[h][0] = 0.f; plo[h][1] = 0.f; }

    Walk wu = wk;          // cursor of the unpack stage (one tile ahead of the softmax stage)
    bool ok = true;

    auto unpack_k = [&](const Walk& w) -> bool {
      const int cb = w.useq & 1, s = w.it % NS;
      if (w.ufirst && !wait_bar(S, &S.ctx_full[cb], (w.useq >> 1) & 1, p.status)) return false;
      const UnitCtx& C = S.ctx[cb];
      if (!wait_bar(S, &S.kfull[s], (w.it / NS) & 1, p.status)) return false;
      if (w.it >= 1) {   // the score MMAs of the previous tile have read the operand buffer
        const int pb = (w.it - 1) & 1;
        const uint32_t pp = ((w.it - 1) >> 1) & 1;
        if (!wait_bar(S, &S.s_ready[pb][0], pp, p.status)) return false;
        if (!wait_bar(S, &S.s_ready[pb][1], pp, p.status)) return false;
      }
      tc_fence_after();
      const uint32_t ktile = smem_u32(ring + s * stage_bytes);
      const int F = C.k_full, n_words = C.k_words;
      for (int i = 0; i < n_words; i++) {
        uint32_t word;
        if (i < F) word = lds32(ktile + 4 * (kTile * i + t));
        else {
          const int r = C.k_rem, bit = r * t;
          const uint32_t a = ktile + 512 * F + 4 * (bit >> 5);
          word = __funnelshift_r(lds32(a), lds32(a + 4), bit & 31) & ((1u << r) - 1u);
        }
        const uint32_t ma = smem_u32(&C.kmask[i][0]);
        const uint32_t dst = lane_base + kColAK + C.kcol[i];
        switch (C.kshape[i]) {
          case 0: k_word_store<0>(word, ma, dst); break;
          case 1: k_word_store<1>(word, ma, dst); break;
          case 2: k_word_store<2>(word, ma, dst); break;
          default: k_word_store<3>(word, ma, dst); break;
        }
      }
      for (int c = C.k_cols; c < 8 * C.k_steps; c += 2) tc_st2(lane_base + kColAK + c, 0u, 0u);   // pad of the last k-step
      tc_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&S.ak_ready));
      return true;
    };

    if (!wk.done()) ok = unpack_k(wu);
    for (; ok && !wk.done(); wk.next()) {
      wu.next();
      if (!wu.done() && !(ok = unpack_k(wu))) break;
      // ------------------------------------------------------------ scores, softmax, probabilities of tile wk
      const int cb = wk.useq & 1, b = wk.it & 1, s = wk.it % NS;
      const UnitCtx& C = S.ctx[cb];
      const uint32_t par = (wk.it >> 1) & 1;
      if (!wait_bar(S, &S.s_ready[b][0], par, p.status) || !wait_bar(S, &S.s_ready[b][1], par, p.status) ||
          !wait_bar(S, &S.vfull[s], (wk.it / NS) & 1, p.status)) { ok = false; break; }
      tc_fence_after();
      const int mid = C.k_steps >> 1;
      float d[16];
      {
        uint32_t r0[16], r1[16];
        tc_ld16(lane_base + kColDS + (uint32_t)(2 * b) * 16, r0);
        tc_ld16(lane_base + kColDS + (uint32_t)(2 * b + 1) * 16, r1);
        tc_wait_ld();
#pragma unroll
        for (int n = 0; n < 16; n++)
          d[n] = (mid > 0 ? __uint_as_float(r0[n]) : 0.f) + (C.k_steps > mid ? __uint_as_float(r1[n]) : 0.f);
      }
      const uint32_t ktile = smem_u32(ring + s * stage_bytes), vtile = ktile + f.slot_k;
      const int n_seq = p.seq_len[wk.u / p.n_kv];
      const bool valid = wk.tile * kTile + t < n_seq;
      float klo[2] = {0.f, 0.f}, kr[2] = {0.f, 0.f}, vlo[2] = {0.f, 0.f}, vr[2] = {0.f, 0.f};
#pragma unroll
      for (int g = 0; g < 2; g++) {
        if (C.kmeta[g] >= 0) { klo[g] = h2f_bits(lds16(ktile + C.kmeta[g] + 2 * t)); kr[g] = h2f_bits(lds16(ktile + C.kmeta[g] + 256 + 2 * t)); }
        if (C.vmeta[g] >= 0 && valid) { vlo[g] = h2f_bits(lds16(vtile + C.vmeta[g] + 2 * t)); vr[g] = h2f_bits(lds16(vtile + C.vmeta[g] + 256 + 2 * t)); }
      }
      float sc[4];
      uint32_t wmax[4];
#pragma unroll
      for (int h = 0; h < 4; h++) {
        const float x = kr[0] * (d[4 * h] + d[4 * h + 1]) + kr[1] * (d[4 * h + 2] + d[4 * h + 3]);
        sc[h] = valid ? fmaf(C.kscale[h], x, fmaf(klo[0], C.qlo[h][0], klo[1] * C.qlo[h][1])) : -INFINITY;
        wmax[h] = redux_max_u32(ordered_bits(sc[h]));
      }
      if (lane == 0) {
#pragma unroll
        for (int h = 0; h < 4; h++) S.red[b][warp][h] = from_ordered_bits(wmax[h]);
      }
      named_barrier(1, 128);
      float m_new[4], fac[4];
      bool grew = false;
#pragma unroll
      for (int h = 0; h < 4; h++) {
        const float mt = fmaxf(fmaxf(S.red[b][0][h], S.red[b][1][h]), fmaxf(S.red[b][2][h], S.red[b][3][h]));
        m_new[h] = fmaxf(m_run[h], mt);
        grew |= m_new[h] > m_run[h];
        fac[h] = m_run[h] == -INFINITY ? 0.f : fast_exp2(m_run[h] - m_new[h]);
      }
      if (grew) {      // uniform over the four token warps
#pragma unroll
        for (int h = 0; h < 4; h++) { l_run[h] *= fac[h]; plo[h][0] *= fac[h]; plo[h][1] *= fac[h]; m_run[h] = m_new[h]; }
        if (!wk.ufirst) {
          // rescale the value accumulators once the value MMAs of the previous tile have completed
          if (!wait_bar(S, &S.pv_done[(wk.it - 1) & 1], ((wk.it - 1) >> 1) & 1, p.status)) { ok = false; break; }
          tc_fence_after();
          int sg[kVSetsMax + 3], si[kVSetsMax + 3];
          const int ns = v_sets(C.n_vgroups, sg, si);
          for (int st = 0; st < ns; st++) {
            uint32_t r[16];
            tc_ld16(lane_base + kColDO + 16 * st, r);
            tc_wait_ld();
#pragma unroll
            for (int n = 0; n < 16; n++) r[n] = __float_as_uint(__uint_as_float(r[n]) * fac[n >> 2]);
            tc_st16(lane_base + kColDO + 16 * st, r);
          }
          tc_wait_st();
        }
      }
      // probabilities; the B operand of the value MMA carries p R^V 2^(9 - p_eff) as an fp16 hi/lo pair
      float pr[4];
#pragma unroll
      for (int h = 0; h < 4; h++) {
        pr[h] = valid ? fast_exp2(sc[h] - m_run[h]) : 0.f;
        l_run[h] += pr[h];
        plo[h][0] = fmaf(pr[h], vlo[0], plo[h][0]);
        plo[h][1] = fmaf(pr[h], vlo[1], plo[h][1]);
      }
      uint32_t base[8];
#pragma unroll
      for (int h = 0; h < 4; h++)
#pragma unroll
        for (int g = 0; g < 2; g++) {
          const float x = pr[h] * vr[g] * 512.f;
          const __half hi = __float2half_rn(fminf(x, 65504.f));
          const __half lo = __float2half_rn(fminf(x - __half2float(hi), 65504.f));
          base[2 * h + g] = (uint32_t)__half_as_ushort(hi) | ((uint32_t)__half_as_ushort(lo) << 16);
        }
      if (wk.it >= 2 && !wait_bar(S, &S.pv_done[b], ((wk.it - 2) >> 1) & 1, p.status)) { ok = false; break; }
      for (int gi = 0; gi < C.n_vgroups; gi++) {
        const int cls = C.vgroup[gi] >> 8;
        if (gi > 0 && (C.vgroup[gi - 1] >> 8) == cls) continue;       // one copy per class
        uint32_t sv[8];
#pragma unroll
        for (int i = 0; i < 8; i++) {
          const __half2 v = __hmul2(*reinterpret_cast<const __half2*>(&base[i]), *reinterpret_cast<const __half2*>(&pscale[cls]));
          sv[i] = *reinterpret_cast<const uint32_t*>(&v);
        }
        const uint32_t dst = smem_u32(&S.pbuf[b][cls][0]) + prow[cls];
        sts128(dst, make_uint4(sv[0], sv[1], sv[2], sv[3]));
        sts128(dst + 2048, make_uint4(sv[4], sv[5], sv[6], sv[7]));
      }
      fence_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(smem_u32(&S.p_ready[b]));
        mbar_arrive(smem_u32(&S.kempty[s]));
        mbar_arrive(smem_u32(&S.vempty[s]));
      }
      if (wk.ulast()) {
        // ---------------------------------------------------------- end of this worker's share of the unit: one record
        if (!wait_bar(S, &S.pv_done[b], par, p.status)) { ok = false; break; }
        tc_fence_after();
        for (int i = t; i < kFastGqa * kVRowsMax; i += 128) (&S.rec[0][0])[i] = 0.f;
        float sums[12];
#pragma unroll
        for (int h = 0; h < 4; h++) { sums[h] = l_run[h]; sums[4 + 2 * h] = plo[h][0]; sums[5 + 2 * h] = plo[h][1]; }
#pragma unroll
        for (int i = 0; i < 12; i++) {
#pragma unroll
          for (int sft = 16; sft; sft >>= 1) sums[i] += __shfl_xor_sync(0xffffffffu, sums[i], sft);
          if (lane == 0) S.fsum[warp][i] = sums[i];
        }
        named_barrier(1, 128);
        int sg[kVSetsMax + 3], si[kVSetsMax + 3];
        const int ns = v_sets(C.n_vgroups, sg, si);
        for (int st = 0; st < ns; st++) {
          const int rbk = C.vgroup[sg[st]] & 0xff, cls = C.vgroup[sg[st]] >> 8;
          uint32_t r[16];
          tc_ld16(lane_base + kColDO + 16 * st, r);
          tc_wait_ld();
          const uint32_t e = C.vrow[rbk * 128 + t];
          if ((e >> 31) && (int)((e >> 12) & 3) == cls) {
            const int k = (e >> 16) & 0x1ff;
            const bool g1 = (e >> 30) & 1;
#pragma unroll
            for (int h = 0; h < 4; h++) {
              const float a = g1 ? __uint_as_float(r[4 * h + 2]) + __uint_as_float(r[4 * h + 3])
                                 : __uint_as_float(r[4 * h]) + __uint_as_float(r[4 * h + 1]);
              S.rec[h][k] += a * 0.001953125f;      // 2^-9: the record holds 2^-24 sum_t p R field
            }
          }
        }
        named_barrier(1, 128);
        float* rec = f.records + (int64_t)(worker + wk.u) * f.rec_stride;
        const int nvs = C.n_vstrips, hstride = kRecHead + f.vs_max;
        if (t < 4) {
          float* hd = rec + t * hstride;
          float mh = -INFINITY;
#pragma unroll
          for (int h = 0; h < 4; h++) if (h == t) mh = m_run[h];
          hd[0] = mh;
          hd[1] = S.fsum[0][t] + S.fsum[1][t] + S.fsum[2][t] + S.fsum[3][t];
          hd[2] = S.fsum[0][4 + 2 * t] + S.fsum[1][4 + 2 * t] + S.fsum[2][4 + 2 * t] + S.fsum[3][4 + 2 * t];
          hd[3] = S.fsum[0][5 + 2 * t] + S.fsum[1][5 + 2 * t] + S.fsum[2][5 + 2 * t] + S.fsum[3][5 + 2 * t];
        }
        for (int idx = t; idx < kFastGqa * nvs; idx += 128) {
          const int h = idx / nvs, k = idx - h * nvs;
          rec[h * hstride + kRecHead + k] = S.rec[h][k];
        }
#pragma unroll
        for (int h = 0; h < 4; h++) { m_run[h] = -INFINITY; l_run[h] = 0.f; plo[h][0] = 0.f; plo[h][1] = 0.f; }
        named_barrier(1, 128);
        tc_fence_before();
        if (lane == 0) mbar_arrive(smem_u32(&S.ctx_empty[cb]));
      }
    }
  }
  // ---- all roles meet here; the warp that allocated the tensor memory frees it
  tc_fence_before();
  __syncthreads();
  if (warp == 15) tmem_dealloc(tb, kTmemCols);
}

}  // namespace spectra
