// Main kernel of the tensor-core coded-cache decode attention (see attention_tc_common.cuh for the overview).
//
// Unpacking.  A w-bit code left in place inside a 16-bit half-word, with every other bit masked off, is a
// subnormal (or lowest-binade) fp16 number equal to code * 2^(p - 24), p = bit position of the field, as long as
// p + w <= 10; mma.sync handles fp16 subnormals exactly.  So one logic op per register (two values) turns packed
// codes into A fragments; fields above bit 10 are first brought down by one shift of the whole word.  The
// position-dependent power of two is folded into the B operand (exact): on the K side the four MMAs of a chunk
// take the tokens whose fields share a position, on the V side the probabilities get one scaled copy per class.
//
// The V accumulators live in registers, one 16-strip block per accumulator.  Their number and their class must be
// compile-time facts, so the kernel is instantiated for a few "quota" tuples (blocks per class 8, 4, 2, 1); the
// host picks the smallest tuple that covers the widths of the call.
#pragma once
#include "attention_tc_common.cuh"

namespace spectra {

// In-pass token ii (0..7) of a thread: which word of the pass, whether the >>8 (>>4 for w = 1) copy is used,
// and the effective bit position p_eff; tokens ii and ii + 4 always share p_eff.
template <int W> struct Unpack;
template <> struct Unpack<8> {   // 4 words, 2 tokens each (bits 0 and 8)
  static constexpr int NW = 4;
  static __device__ __forceinline__ uint32_t get(const uint32_t (&w)[NW], const uint32_t (&ws)[NW], int ii) {
    return ((ii & 1) ? ws[ii >> 1] : w[ii >> 1]) & 0x00FF00FFu;
  }
  static __device__ __forceinline__ void shifted(const uint32_t (&w)[NW], uint32_t (&ws)[NW]) {
#pragma unroll
    for (int i = 0; i < NW; i++) ws[i] = w[i] >> 8;
  }
  static __host__ __device__ constexpr int peff(int u) { return 0 * u; }
};
template <> struct Unpack<4> {   // 2 words, 4 tokens each (bits 0, 4, 8, 12)
  static constexpr int NW = 2;
  static __device__ __forceinline__ uint32_t get(const uint32_t (&w)[NW], const uint32_t (&ws)[NW], int ii) {
    const int j = ii >> 2, q = ii & 3;
    return ((q & 2) ? ws[j] : w[j]) & ((q & 1) ? 0x00F000F0u : 0x000F000Fu);
  }
  static __device__ __forceinline__ void shifted(const uint32_t (&w)[NW], uint32_t (&ws)[NW]) {
#pragma unroll
    for (int i = 0; i < NW; i++) ws[i] = w[i] >> 8;
  }
  static __host__ __device__ constexpr int peff(int u) { return 4 * (u & 1); }
};
template <> struct Unpack<2> {   // 1 word, 8 tokens (bits 0, 2, .., 14)
  static constexpr int NW = 1;
  static __device__ __forceinline__ uint32_t get(const uint32_t (&w)[NW], const uint32_t (&ws)[NW], int ii) {
    return ((ii & 4) ? ws[0] : w[0]) & (0x00030003u << (2 * (ii & 3)));
  }
  static __device__ __forceinline__ void shifted(const uint32_t (&w)[NW], uint32_t (&ws)[NW]) { ws[0] = w[0] >> 8; }
  static __host__ __device__ constexpr int peff(int u) { return 2 * (u & 3); }
};
template <> struct Unpack<1> {   // 1 word (already shifted right by 8 * pass), 8 tokens at bits 0..7
  static constexpr int NW = 1;
  static __device__ __forceinline__ uint32_t get(const uint32_t (&w)[NW], const uint32_t (&ws)[NW], int ii) {
    return ((ii & 4) ? ws[0] : w[0]) & (0x00010001u << (ii & 3));
  }
  static __device__ __forceinline__ void shifted(const uint32_t (&w)[NW], uint32_t (&ws)[NW]) { ws[0] = w[0] >> 4; }
  static __host__ __device__ constexpr int peff(int u) { return u & 3; }
};

__device__ __forceinline__ uint32_t hmul2_pow2(uint32_t x, int neg_exp) {   // x * 2^-neg_exp on both halves (exact)
  if (neg_exp == 0) return x;
  const uint32_t s = (uint32_t)((15 - neg_exp) << 10) * 0x00010001u;
  __half2 a, b;
  *reinterpret_cast<uint32_t*>(&a) = x;
  *reinterpret_cast<uint32_t*>(&b) = s;
  const __half2 r = __hmul2(a, b);
  return *reinterpret_cast<const uint32_t*>(&r);
}

// Plain loads of n words from shared memory (the compiler may schedule them freely between barrier waits).
template <int NW>
__device__ __forceinline__ void ld_words(const unsigned char* p, uint32_t (&w)[NW]) {
  if constexpr (NW == 4) { const uint4 v = *reinterpret_cast<const uint4*>(p); w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w; }
  else if constexpr (NW == 2) { const uint2 v = *reinterpret_cast<const uint2*>(p); w[0] = v.x; w[1] = v.y; }
  else w[0] = *reinterpret_cast<const uint32_t*>(p);
}
// Same for a strip stored alone (half-words in order): each half-word becomes the low half of a word.
template <int NW>
__device__ __forceinline__ void ld_halfwords(const unsigned char* p, uint32_t (&w)[NW]) {
  if constexpr (NW == 4) { const uint2 v = *reinterpret_cast<const uint2*>(p); w[0] = v.x & 0xffffu; w[1] = v.x >> 16; w[2] = v.y & 0xffffu; w[3] = v.y >> 16; }
  else if constexpr (NW == 2) { const uint32_t v = *reinterpret_cast<const uint32_t*>(p); w[0] = v & 0xffffu; w[1] = v >> 16; }
  else w[0] = *reinterpret_cast<const uint16_t*>(p);
}

// Four MMAs of one chunk into one scale group's accumulators: MMA u takes tokens u (row gid) and u + 4 (row
// gid + 8) of the pass, pair slots tig and tig + 4 as its k columns, and B variant u (scaled by 2^-p_eff(u); rows
// of strips that belong to the other scale group, or lie past the end of the class, are zero).
template <int W>
__device__ __forceinline__ void k_chunk(const uint32_t (&wa)[Unpack<W>::NW], const uint32_t (&wb)[Unpack<W>::NW],
                                        const uint2* __restrict__ kb, float (&acc)[4][4]) {
  using U = Unpack<W>;
  constexpr int NW = U::NW;
  uint32_t was[NW], wbs[NW];
  U::shifted(wa, was);
  U::shifted(wb, wbs);
#pragma unroll
  for (int u = 0; u < 4; u++) {
    const uint2 b = __ldg(kb + u * 32);
    mma16816(acc[u], U::get(wa, was, u), U::get(wa, was, u + 4), U::get(wb, wbs, u), U::get(wb, wbs, u + 4), b.x, b.y);
  }
}

// The chunk that holds strips of both scale groups: the A fragments are unpacked once and multiplied with both
// groups' B entries (consecutive in the table).
template <int W>
__device__ __forceinline__ void k_chunk_both(const uint32_t (&wa)[Unpack<W>::NW], const uint32_t (&wb)[Unpack<W>::NW],
                                             const uint2* __restrict__ kb, float (&acc)[2][4][4]) {
  using U = Unpack<W>;
  constexpr int NW = U::NW;
  uint32_t was[NW], wbs[NW];
  U::shifted(wa, was);
  U::shifted(wb, wbs);
#pragma unroll
  for (int u = 0; u < 4; u++) {
    const uint2 b0 = __ldg(kb + u * 32), b1 = __ldg(kb + (4 + u) * 32);
    const uint32_t a0 = U::get(wa, was, u), a1 = U::get(wa, was, u + 4), a2 = U::get(wb, wbs, u), a3 = U::get(wb, wbs, u + 4);
    mma16816(acc[0][u], a0, a1, a2, a3, b0.x, b0.y);
    mma16816(acc[1][u], a0, a1, a2, a3, b1.x, b1.y);
  }
}

// One class of the K tile for one half tile.  Chunks of 16 strips = 8 interleaved pairs, in storage order; the
// strips of scale group 0 come first (n_g0 of them), so at most one chunk per class holds strips of both groups: it
// is multiplied twice, once per group, each time with the other group's rows zeroed in B.  The B table is walked in
// the same order (chunk-major, group-minor).  An odd last strip of the class is stored alone (half-words in order).
template <int W>
__device__ __forceinline__ void k_class(const unsigned char* ktile, uint32_t cls, const uint2* __restrict__& kb,
                                        int hp, int gid, int tig, float (&acc)[2][4][4]) {
  using U = Unpack<W>;
  constexpr int NW = U::NW;
  const int n = cls & 0xff, n_g0 = (cls >> 8) & 0xff;
  if (n == 0) return;
  const unsigned char* cbase = ktile + (cls >> 16) * 16;
  const int thr = 4 * W * gid + (W == 1 ? 0 : 4 * NW * hp);    // this thread's token block inside a pair
  const unsigned char* pa = cbase + 32 * W * tig + thr;
  int s = 0;
#pragma unroll 1
  for (; s + 16 <= (n & ~1); s += 16, pa += 256 * W) {          // complete chunks
    uint32_t wa[NW], wb[NW];
    ld_words<NW>(pa, wa);
    ld_words<NW>(pa + 128 * W, wb);
    if constexpr (W == 1) { wa[0] >>= 8 * hp; wb[0] >>= 8 * hp; }
    if (s + 16 <= n_g0) { k_chunk<W>(wa, wb, kb, acc[0]); kb += 4 * 32; }
    else if (s >= n_g0) { k_chunk<W>(wa, wb, kb, acc[1]); kb += 4 * 32; }
    else { k_chunk_both<W>(wa, wb, kb, acc); kb += 8 * 32; }
  }
  if (s < n) {                                                  // the last, incomplete chunk of the class
    const int avail = n - s;                                    // strips stored from s on (B rows past them are zero)
    const unsigned char* cb = cbase + 16 * W * s;
    uint32_t wa[NW], wb[NW];
    if (!(avail & 1)) {
      // whole pairs only: slots past the end re-read the last pair
      const int last = (avail >> 1) - 1;
      ld_words<NW>(cb + 32 * W * min(tig, last) + thr, wa);
      ld_words<NW>(cb + 32 * W * min(tig + 4, last) + thr, wb);
    } else {
      // the class has an odd number of strips: its last strip is stored alone, half-words in order
#pragma unroll
      for (int i = 0; i < NW; i++) { wa[i] = 0u; wb[i] = 0u; }
      const int thr_h = 2 * W * gid + (W == 1 ? 0 : 2 * NW * hp);
#pragma unroll
      for (int half = 0; half < 2; half++) {
        const int ps = tig + 4 * half;
        uint32_t (&wd)[NW] = half ? wb : wa;
        if (2 * ps + 1 < avail) ld_words<NW>(cb + 32 * W * ps + thr, wd);
        else if (2 * ps < avail) ld_halfwords<NW>(cb + 32 * W * ps + thr_h, wd);
      }
    }
    if constexpr (W == 1) { wa[0] >>= 8 * hp; wb[0] >>= 8 * hp; }
    if (n <= n_g0) { k_chunk<W>(wa, wb, kb, acc[0]); kb += 4 * 32; }
    else if (s >= n_g0) { k_chunk<W>(wa, wb, kb, acc[1]); kb += 4 * 32; }
    else { k_chunk_both<W>(wa, wb, kb, acc); kb += 8 * 32; }
  }
}

// One class of the V tile for one half tile, at most Q blocks of 16 strips, accumulators acc_o[OFF .. OFF + Q).
// The probabilities first get the class's position scales; MMA u of a block contracts the token pairs of B
// fragments u and u + 4.
template <int W, int Q, int OFF, int NACC>
__device__ __forceinline__ void v_class(const unsigned char* vtile, uint32_t cls, int hp, int gid, int tig,
                                        const uint32_t (&pb)[8], float (&acc_o)[NACC][4]) {
  if constexpr (Q > 0) {
    using U = Unpack<W>;
    constexpr int NW = U::NW;
    const int n = cls & 0xff;
    if (n == 0) return;
    uint32_t pw[8];
#pragma unroll
    for (int ii = 0; ii < 8; ii++) pw[ii] = hmul2_pow2(pb[ii], U::peff(ii));
    const unsigned char* cbase = vtile + (cls >> 16) * 16 + 4 * W * tig + (W == 1 ? 0 : 4 * NW * hp);
#pragma unroll
    for (int bi = 0; bi < Q; bi++) {
      if (16 * bi < n) {
        uint32_t wa[NW], wb[NW], was[NW], wbs[NW];
        if (16 * bi + 16 <= n) {
          ld_words<NW>(cbase + 16 * W * (16 * bi + gid), wa);
          ld_words<NW>(cbase + 16 * W * (16 * bi + gid + 8), wb);
        } else {                               // rows past the end repeat the last strip; their results are unused
          ld_words<NW>(cbase + 16 * W * min(16 * bi + gid, n - 1), wa);
          ld_words<NW>(cbase + 16 * W * min(16 * bi + gid + 8, n - 1), wb);
        }
        if constexpr (W == 1) { wa[0] >>= 8 * hp; wb[0] >>= 8 * hp; }
        U::shifted(wa, was);
        U::shifted(wb, wbs);
#pragma unroll
        for (int u = 0; u < 4; u++)
          mma16816(acc_o[OFF + bi], U::get(wa, was, u), U::get(wb, wbs, u), U::get(wa, was, u + 4),
                   U::get(wb, wbs, u + 4), pw[u], pw[u + 4]);
      }
    }
  }
}

// Writes one class's accumulators into a partial record: row r of the class goes to strip index first + r, taking
// the column of the scale group the strip belongs to.
template <int Q, int OFF, int NACC>
__device__ __forceinline__ void store_class(float* rec, uint32_t cls, int first, int gid, const float (&acc_o)[NACC][4]) {
  const int n = cls & 0xff, n_g0 = (cls >> 8) & 0xff;
#pragma unroll
  for (int bi = 0; bi < Q; bi++) {
#pragma unroll
    for (int half = 0; half < 2; half++) {
      const int r = 16 * bi + gid + 8 * half;
      if (r < n) rec[kRecHead + first + r] = r >= n_g0 ? acc_o[OFF + bi][2 * half + 1] : acc_o[OFF + bi][2 * half];
    }
  }
}

// Two floats to packed fp16 (low = a), saturating at the largest finite value instead of producing infinity.
__device__ __forceinline__ uint32_t pack_half2_sat(float a, float b) {
  uint32_t d;
  asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(b), "f"(a));
  return d;
}

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

template <int Q8, int Q4, int Q2, int Q1>
__global__ void __launch_bounds__(kFastWarps * 32, 3) attention_mma_kernel(AttnArgs p, FastArgs f) {
  constexpr int NACC = Q8 + Q4 + Q2 + Q1;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int gid = lane >> 2, tig = lane & 3;
  const int gw = blockIdx.x * kFastWarps + warp;
  const int D = f.depth;
  const uint32_t warp_bytes = (uint32_t)D * (f.slot_k + f.slot_v);
  unsigned char* ring_k = smem_raw + warp * warp_bytes;
  unsigned char* ring_v = ring_k + D * f.slot_k;
  const uint32_t bars = smem_u32(smem_raw) + kFastWarps * warp_bytes + warp * (2 * 4 * 8);  // K slots 0..3, V slots 0..3
  if (lane == 0)
    for (int s = 0; s < 2 * 4; s++) mbar_init(bars + 8 * s, 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  __syncwarp();

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the combine kernel may be scheduled as SMs free up
  const long long total = f.tile_prefix[f.n_units];
  const long long g0 = (long long)gw * total / f.total_warps;
  const long long g1 = (long long)(gw + 1) * total / f.total_warps;
  const int count = (int)(g1 - g0);
  if (count <= 0) return;

  TileCursor cons, prod;
  cons.u = f.warp_unit[gw]; cons.t = (int)(g0 - f.tile_prefix[cons.u]); cons.nt = 0; cons.seek_unit(f);
  prod = cons;
  // Copies are started by lane 0; every lane keeps the same counts of tiles whose K / V copy has been started.
  int issued_k = 0, issued_v = 0;
  const uint8_t* v_src = nullptr;   // V tile that goes with the most recently started K tile (lane 0)
  uint32_t v_bytes = 0;
  auto start_k = [&](int slot) {
    const UnitDesc& d = f.desc[prod.u];
    const uint32_t tbk = d.tbk, tbv = d.tbv;
    mbar_expect_tx(bars + 8 * slot, tbk);
    bulk_load(smem_u32(ring_k + slot * f.slot_k), p.cache_k + p.off_k[prod.u / f.npass] + (int64_t)prod.t * tbk, tbk,
              bars + 8 * slot, l2_evict_first_policy());
    v_src = p.cache_v + p.off_v[prod.u / f.npass] + (int64_t)prod.t * tbv;
    v_bytes = tbv;
    prod.next(f);
  };
  auto start_v = [&](int slot) {
    mbar_expect_tx(bars + 8 * (4 + slot), v_bytes);
    bulk_load(smem_u32(ring_v + slot * f.slot_v), v_src, v_bytes, bars + 8 * (4 + slot),
              l2_evict_first_policy());
  };
  if (lane == 0)
    for (int j = 0; j < min(D, count); j++) { start_k(j); start_v(j); }
  issued_k = issued_v = min(D, count);

  float acc_o[NACC][4];
  float m_run = -INFINITY, l_run = 0.f, plo0 = 0.f, plo1 = 0.f;
  uint32_t kcls[4], vcls[4];
  int kmeta0 = -1, kmeta1 = -1, vmeta0 = -1, vmeta1 = -1;
  float kscale = 0.f, qlo0 = 0.f, qlo1 = 0.f;
  const uint2* kB = nullptr;
  int n_seq = 0;
  bool fresh = true, ok = true;
  float boost = 0.f;          // power-of-two lift of the probabilities (see below); -1 = not chosen yet

  for (int j = 0; j < count && ok; j++) {
    const int slot = j % D;
    const uint32_t parity = (uint32_t)(j / D) & 1u;
    const unsigned char* ktile = ring_k + slot * f.slot_k;
    const unsigned char* vtile = ring_v + slot * f.slot_v;
    if (fresh) {
      const UnitDesc& d = f.desc[cons.u];
#pragma unroll
      for (int c = 0; c < 4; c++) { kcls[c] = d.kcls[c]; vcls[c] = d.vcls[c]; }
      kmeta0 = d.kmeta[0]; kmeta1 = d.kmeta[1]; vmeta0 = d.vmeta[0]; vmeta1 = d.vmeta[1];
      kscale = d.kscale[tig]; qlo0 = d.qlo[tig][0]; qlo1 = d.qlo[tig][1];
      kB = &d.kB[0][0][0];
      n_seq = p.seq_len[(cons.u / f.npass) / p.n_kv];
#pragma unroll
      for (int mb = 0; mb < NACC; mb++)
#pragma unroll
        for (int e = 0; e < 4; e++) acc_o[mb][e] = 0.f;
      m_run = -INFINITY; l_run = 0.f; plo0 = 0.f; plo1 = 0.f;
      fresh = false;
      boost = -1.f;
    }

#pragma unroll 1
    for (int hp = 0; hp < 2; hp++) {
      // ------------------------------------------------------------ scores of 64 tokens
      if (hp == 0) ok = mbar_wait(bars + 8 * slot, parity);
      float acc[2][4][4];
#pragma unroll
      for (int g = 0; g < 2; g++)
#pragma unroll
        for (int u = 0; u < 4; u++)
#pragma unroll
          for (int e = 0; e < 4; e++) acc[g][u][e] = 0.f;
      const uint2* kb = kB + lane;       // walks the B fragment table in chunk order
      k_class<8>(ktile, kcls[0], kb, hp, gid, tig, acc);
      k_class<4>(ktile, kcls[1], kb, hp, gid, tig, acc);
      k_class<2>(ktile, kcls[2], kb, hp, gid, tig, acc);
      k_class<1>(ktile, kcls[3], kb, hp, gid, tig, acc);

      // per-token group minimum and range of the K tile (fp16), this thread's 8 tokens: token ii is MMA u = ii & 3,
      // row gid (ii < 4) or gid + 8; the fp16 pair r holds tokens 2r and 2r + 1
      const int tok_off = 2 * (gid * 16 + 8 * hp);
      uint32_t klo0[4] = {0, 0, 0, 0}, kr0[4] = {0, 0, 0, 0}, klo1[4] = {0, 0, 0, 0}, kr1[4] = {0, 0, 0, 0};
      if (kmeta0 >= 0) { ld_words<4>(ktile + kmeta0 + tok_off, klo0); ld_words<4>(ktile + kmeta0 + 256 + tok_off, kr0); }
      if (kmeta1 >= 0) { ld_words<4>(ktile + kmeta1 + tok_off, klo1); ld_words<4>(ktile + kmeta1 + 256 + tok_off, kr1); }
      if (hp == 1 && issued_k < count) {     // the K slot is free: refill it with the tile D positions ahead
        __syncwarp();
        if (lane == 0) { fence_async_smem(); start_k(issued_k % D); }
        issued_k++;
      }
      float s[8];
      float mx = -INFINITY;
      const int tok0 = cons.t * kTile + gid * 16 + 8 * hp;
#pragma unroll
      for (int r = 0; r < 4; r++) {
        const float2 lo0 = h2f2(klo0[r]), r0 = h2f2(kr0[r]), lo1 = h2f2(klo1[r]), r1 = h2f2(kr1[r]);
#pragma unroll
        for (int e = 0; e < 2; e++) {
          const int ii = 2 * r + e, u = ii & 3, cb = (ii >> 2) * 2;
          const float a0 = acc[0][u][cb] + acc[0][u][cb + 1];   // hi + lo halves of q'
          const float a1 = acc[1][u][cb] + acc[1][u][cb + 1];
          float v = kscale * ((e ? r0.y : r0.x) * a0 + (e ? r1.y : r1.x) * a1) + (e ? lo0.y : lo0.x) * qlo0 +
                    (e ? lo1.y : lo1.x) * qlo1;
          s[ii] = v;
        }
      }
      if ((cons.t + 1) * kTile > n_seq) {                      // only the unit's last tile has slots past the end
#pragma unroll
        for (int ii = 0; ii < 8; ii++)
          if (tok0 + ii >= n_seq) s[ii] = -INFINITY;
      }
#pragma unroll
      for (int ii = 0; ii < 8; ii++) mx = fmaxf(mx, s[ii]);
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
      if (mx > m_run) {        // new running maximum for this thread's head: rescale what has been accumulated
        const float alpha = fast_exp2(m_run - mx);   // exp2(-inf) = 0 on the first tile
        m_run = mx;
        l_run *= alpha; plo0 *= alpha; plo1 *= alpha;
#pragma unroll
        for (int mb = 0; mb < NACC; mb++)
#pragma unroll
          for (int e = 0; e < 4; e++) acc_o[mb][e] *= alpha;
      }
      if (hp == 0) ok = ok && mbar_wait(bars + 8 * (4 + slot), parity);
      uint32_t vlo0[4] = {0, 0, 0, 0}, vr0[4] = {0, 0, 0, 0}, vlo1[4] = {0, 0, 0, 0}, vr1[4] = {0, 0, 0, 0};
      if (vmeta0 >= 0) { ld_words<4>(vtile + vmeta0 + tok_off, vlo0); ld_words<4>(vtile + vmeta0 + 256 + tok_off, vr0); }
      if (vmeta1 >= 0) { ld_words<4>(vtile + vmeta1 + tok_off, vlo1); ld_words<4>(vtile + vmeta1 + 256 + tok_off, vr1); }
      // probabilities times the V group ranges, as fp16 pairs (group 0, group 1), transposed into B fragments
      uint32_t pb[8];
      if (boost < 0.f) {
        // First half tile of this warp's share of the unit.  Probabilities are exp2(s - max) <= 1 and enter the
        // tensor core as fp16 times the V group range; with tens of thousands of tokens the typical probability is
        // far below the fp16 normal range.  Lift everything by 2^boost (the record's maximum is lowered by the same
        // amount, so the merge is unaffected), leaving room for group ranges 8x larger than in this half tile.
        float rmax = 0.f;
#pragma unroll
        for (int r = 0; r < 4; r++) {
          const float2 a = h2f2(vr0[r]), b = h2f2(vr1[r]);
          rmax = fmaxf(rmax, fmaxf(fmaxf(a.x, a.y), fmaxf(b.x, b.y)));
        }
#pragma unroll
        for (int sft = 1; sft <= 16; sft <<= 1) rmax = fmaxf(rmax, __shfl_xor_sync(0xffffffffu, rmax, sft));
        const int e = (int)((__float_as_uint(rmax) >> 23) & 0xff) - 126;     // rmax < 2^e
        boost = (float)max(0, min(13, 13 - e));
      }
      const float m_use = (m_run == -INFINITY ? 0.f : m_run) - boost;
#pragma unroll
      for (int r = 0; r < 4; r++) {
        const float2 lo0 = h2f2(vlo0[r]), r0 = h2f2(vr0[r]), lo1 = h2f2(vlo1[r]), r1 = h2f2(vr1[r]);
#pragma unroll
        for (int e = 0; e < 2; e++) {
          const int ii = 2 * r + e;
          const float pr = fast_exp2(s[ii] - m_use);
          l_run += pr;
          plo0 = fmaf(pr, e ? lo0.y : lo0.x, plo0);
          plo1 = fmaf(pr, e ? lo1.y : lo1.x, plo1);
          pb[ii] = movmatrix_trans(pack_half2_sat(pr * (e ? r0.y : r0.x), pr * (e ? r1.y : r1.x)));
        }
      }
      // ------------------------------------------------------------ P~ x V codes
      v_class<8, Q8, 0, NACC>(vtile, vcls[0], hp, gid, tig, pb, acc_o);
      v_class<4, Q4, Q8, NACC>(vtile, vcls[1], hp, gid, tig, pb, acc_o);
      v_class<2, Q2, Q8 + Q4, NACC>(vtile, vcls[2], hp, gid, tig, pb, acc_o);
      v_class<1, Q1, Q8 + Q4 + Q2, NACC>(vtile, vcls[3], hp, gid, tig, pb, acc_o);
      if (hp == 1 && issued_v < issued_k) {
        __syncwarp();
        if (lane == 0) { fence_async_smem(); start_v(issued_v % D); }
        issued_v++;
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
      if (gid == 0) { rec[0] = m_run - boost; rec[1] = l; rec[2] = q0; rec[3] = q1; }
      const UnitDesc& d = f.desc[cons.u];
      store_class<Q8, 0, NACC>(rec, vcls[0], d.vfirst[0], gid, acc_o);
      store_class<Q4, Q8, NACC>(rec, vcls[1], d.vfirst[1], gid, acc_o);
      store_class<Q2, Q8 + Q4, NACC>(rec, vcls[2], d.vfirst[2], gid, acc_o);
      store_class<Q1, Q8 + Q4 + Q2, NACC>(rec, vcls[3], d.vfirst[3], gid, acc_o);
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

}  // namespace spectra
