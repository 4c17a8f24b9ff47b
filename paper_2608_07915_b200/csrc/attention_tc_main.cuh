// Main kernel of the tensor-core coded-cache decode attention (see attention_tc_common.cuh for the overview).
//
// Unpacking.  A w-bit code left in place inside a 16-bit half-word, with every other bit masked off, is a
// subnormal (or lowest-binade) fp16 number equal to code * 2^(p - 24), p = bit position of the field, as long as
// p + w <= 10; mma.sync handles fp16 subnormals exactly.  So one logic op per register (two values) turns packed
// codes into A fragments; fields above bit 10 are first brought down by one shift of the whole word.  The
// position-dependent power of two is folded into the B operand (exact): on the K side the four MMAs of a chunk
// take the tokens whose fields share a position, on the V side the probabilities get one scaled copy per class.
#pragma once
#include "attention_tc_common.cuh"

namespace spectra {

// In-pass token ii (0..7) of a thread: which word of the pass, whether the >>8 (>>4 for w = 1) copy is used,
// and the effective bit position p_eff; tokens ii and ii + 4 always share p_eff.
template <int W> struct Unpack;
template <> struct Unpack<8> {   // 4 words, 2 tokens each (bits 0 and 8)
  static constexpr int NW = 4;
  static constexpr uint32_t kMask = 0x00FF00FFu;
  static __device__ __forceinline__ uint32_t get(const uint32_t (&w)[NW], const uint32_t (&ws)[NW], int ii) {
    return ((ii & 1) ? ws[ii >> 1] : w[ii >> 1]) & kMask;
  }
  static __device__ __forceinline__ void shifted(const uint32_t (&w)[NW], uint32_t (&ws)[NW]) {
#pragma unroll
    for (int i = 0; i < NW; i++) ws[i] = w[i] >> 8;
  }
  static __host__ __device__ constexpr int peff(int u) { return 0; }
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

// Four MMAs of one 16-strip chunk: MMA u takes tokens u (row gid) and u + 4 (row gid + 8) of the pass.
template <int W, bool G0, bool G1>
__device__ __forceinline__ void k_chunk_mma(const uint32_t (&wa)[Unpack<W>::NW], const uint32_t (&wb)[Unpack<W>::NW],
                                            uint2 b0, uint2 b1, float (&acc)[2][4][4]) {
  using U = Unpack<W>;
  uint32_t was[U::NW], wbs[U::NW];
  U::shifted(wa, was);
  U::shifted(wb, wbs);
#pragma unroll
  for (int u = 0; u < 4; u++) {
    const uint32_t a0 = U::get(wa, was, u), a1 = U::get(wa, was, u + 4);
    const uint32_t a2 = U::get(wb, wbs, u), a3 = U::get(wb, wbs, u + 4);
    if constexpr (G0) mma16816(acc[0][u], a0, a1, a2, a3, hmul2_pow2(b0.x, U::peff(u)), hmul2_pow2(b0.y, U::peff(u)));
    if constexpr (G1) mma16816(acc[1][u], a0, a1, a2, a3, hmul2_pow2(b1.x, U::peff(u)), hmul2_pow2(b1.y, U::peff(u)));
  }
}

// One class of the K tile for one half tile.  Chunks are 16 strips (8 interleaved pairs); chunks whose strips all
// belong to one scale group and that are complete take the straight path, the others the guarded one.
template <int W>
__device__ __forceinline__ void k_class(const unsigned char* ktile, uint32_t cls, const uint2* __restrict__ kB,
                                        int& chunk_id, int hp, int gid, int tig, int lane, float (&acc)[2][4][4]) {
  using U = Unpack<W>;
  constexpr int NW = U::NW;
  const int n = cls & 0xff, n_g0 = (cls >> 8) & 0xff;
  if (n == 0) return;
  const unsigned char* base = ktile + (cls >> 16) * 16 + 32 * W * tig + 4 * W * gid + (W == 1 ? 0 : 4 * NW * hp);
  const int full0 = n_g0 >> 4;                 // complete chunks inside scale group 0
  const int first1 = (n_g0 + 15) >> 4;         // first chunk that lies inside scale group 1
  const int full_end = n >> 4;                 // complete chunks overall
  int ci = 0;
  for (; ci < full0; ci++, chunk_id++) {
    uint32_t wa[NW], wb[NW];
    ld_words<NW>(base + 256 * W * ci, wa);
    ld_words<NW>(base + 256 * W * ci + 128 * W, wb);
    if constexpr (W == 1) { wa[0] >>= 8 * hp; wb[0] >>= 8 * hp; }
    const uint2 b0 = __ldg(kB + (chunk_id * 2 + 0) * 32 + lane);
    k_chunk_mma<W, true, false>(wa, wb, b0, b0, acc);
  }
  for (; ci * 16 < n; ci++, chunk_id++) {
    if (ci >= first1 && ci < full_end) {       // complete chunk inside scale group 1
      uint32_t wa[NW], wb[NW];
      ld_words<NW>(base + 256 * W * ci, wa);
      ld_words<NW>(base + 256 * W * ci + 128 * W, wb);
      if constexpr (W == 1) { wa[0] >>= 8 * hp; wb[0] >>= 8 * hp; }
      const uint2 b1 = __ldg(kB + (chunk_id * 2 + 1) * 32 + lane);
      k_chunk_mma<W, false, true>(wa, wb, b1, b1, acc);
      continue;
    }
    // guarded path: chunk straddles the scale groups and/or is the incomplete last chunk of the class
    const int ns = min(16, n - 16 * ci);
    uint32_t wa[NW], wb[NW];
#pragma unroll
    for (int i = 0; i < NW; i++) { wa[i] = 0u; wb[i] = 0u; }
    const unsigned char* cb = ktile + (cls >> 16) * 16 + 256 * W * ci;
#pragma unroll
    for (int half = 0; half < 2; half++) {
      const int ps = tig + 4 * half;
      uint32_t (&wd)[NW] = half ? wb : wa;
      if (2 * ps + 1 < ns) ld_words<NW>(cb + 32 * W * ps + 4 * W * gid + (W == 1 ? 0 : 4 * NW * hp), wd);
      else if (2 * ps < ns) ld_halfwords<NW>(cb + 32 * W * ps + 2 * W * gid + (W == 1 ? 0 : 2 * NW * hp), wd);
    }
    if constexpr (W == 1) { wa[0] >>= 8 * hp; wb[0] >>= 8 * hp; }
    const bool has0 = 16 * ci < n_g0, has1 = 16 * ci + ns > n_g0;
    uint2 b0 = make_uint2(0u, 0u), b1 = make_uint2(0u, 0u);
    if (has0) b0 = __ldg(kB + (chunk_id * 2 + 0) * 32 + lane);
    if (has1) b1 = __ldg(kB + (chunk_id * 2 + 1) * 32 + lane);
    k_chunk_mma<W, true, true>(wa, wb, b0, b1, acc);   // a group without strips in the chunk has zero B
  }
}

// A fragments of one 16-strip block of the V tile for one half tile (rows gid and gid + 8).
template <int W>
__device__ __forceinline__ void v_block_frags(const unsigned char* cbase, int row0, int n, int hp,
                                              uint32_t (&a)[4][4]) {
  using U = Unpack<W>;
  constexpr int NW = U::NW;
  uint32_t wa[NW], wb[NW], was[NW], wbs[NW];
  ld_words<NW>(cbase + 16 * W * min(row0, n - 1), wa);       // rows past the end repeat the last strip: unused
  ld_words<NW>(cbase + 16 * W * min(row0 + 8, n - 1), wb);
  if constexpr (W == 1) { wa[0] >>= 8 * hp; wb[0] >>= 8 * hp; }
  U::shifted(wa, was);
  U::shifted(wb, wbs);
#pragma unroll
  for (int u = 0; u < 4; u++) {
    a[u][0] = U::get(wa, was, u); a[u][1] = U::get(wb, wbs, u);
    a[u][2] = U::get(wa, was, u + 4); a[u][3] = U::get(wb, wbs, u + 4);
  }
}

template <int NVB>
__device__ __forceinline__ void v_accumulate(float (&acc_o)[NVB][4], int mb, const uint32_t (&a)[4][4],
                                             const uint32_t (&pw)[8]) {
  switch (mb) {
#define SPECTRA_VCASE(K)                                                                        \
  case K:                                                                                       \
    if constexpr (K < NVB) {                                                                    \
      _Pragma("unroll") for (int u = 0; u < 4; u++)                                             \
          mma16816(acc_o[K < NVB ? K : 0], a[u][0], a[u][1], a[u][2], a[u][3], pw[u], pw[u + 4]); \
    }                                                                                           \
    break;
    SPECTRA_VCASE(0) SPECTRA_VCASE(1) SPECTRA_VCASE(2) SPECTRA_VCASE(3) SPECTRA_VCASE(4) SPECTRA_VCASE(5)
    SPECTRA_VCASE(6) SPECTRA_VCASE(7) SPECTRA_VCASE(8) SPECTRA_VCASE(9) SPECTRA_VCASE(10) SPECTRA_VCASE(11)
    SPECTRA_VCASE(12) SPECTRA_VCASE(13) SPECTRA_VCASE(14) SPECTRA_VCASE(15) SPECTRA_VCASE(16) SPECTRA_VCASE(17)
    SPECTRA_VCASE(18) SPECTRA_VCASE(19) SPECTRA_VCASE(20) SPECTRA_VCASE(21) SPECTRA_VCASE(22) SPECTRA_VCASE(23)
#undef SPECTRA_VCASE
    default: break;
  }
}

// One class of the V tile for one half tile: the probabilities get the class's position scales, then every block
// of 16 strips is unpacked and accumulated into its own register accumulator.
template <int W, int NVB>
__device__ __forceinline__ void v_class(const unsigned char* vtile, uint32_t cls, int& mb, int hp, int gid, int tig,
                                        const uint32_t (&pb)[8], float (&acc_o)[NVB][4]) {
  using U = Unpack<W>;
  const int n = cls & 0xff;
  if (n == 0) return;
  uint32_t pw[8];
#pragma unroll
  for (int ii = 0; ii < 8; ii++) pw[ii] = hmul2_pow2(pb[ii], U::peff(ii));
  const unsigned char* cbase = vtile + (cls >> 16) * 16 + 4 * W * tig + (W == 1 ? 0 : 4 * U::NW * hp);
  for (int bi = 0; bi * 16 < n; bi++, mb++) {
    uint32_t a[4][4];
    v_block_frags<W>(cbase, 16 * bi + gid, n, hp, a);
    v_accumulate<NVB>(acc_o, mb, a, pw);
  }
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

template <int NVB>
__global__ void __launch_bounds__(kFastWarps * 32, 2) attention_mma_kernel(AttnArgs p, FastArgs f) {
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
    bulk_load(smem_u32(ring_k + slot * f.slot_k), p.cache_k + p.off_k[prod.u] + (int64_t)prod.t * tbk, tbk,
              bars + 8 * slot);
    v_src = p.cache_v + p.off_v[prod.u] + (int64_t)prod.t * tbv;
    v_bytes = tbv;
    prod.next(f);
  };
  auto start_v = [&](int slot) {
    mbar_expect_tx(bars + 8 * (4 + slot), v_bytes);
    bulk_load(smem_u32(ring_v + slot * f.slot_v), v_src, v_bytes, bars + 8 * (4 + slot));
  };
  if (lane == 0)
    for (int j = 0; j < min(D, count); j++) { start_k(j); start_v(j); }
  issued_k = issued_v = min(D, count);

  float acc_o[NVB][4];
  float m_run = -INFINITY, l_run = 0.f, plo0 = 0.f, plo1 = 0.f;
  uint32_t kcls[4], vcls[4];
  int kmeta0 = -1, kmeta1 = -1, vmeta0 = -1, vmeta1 = -1;
  float kscale = 0.f, qlo0 = 0.f, qlo1 = 0.f;
  const uint2* kB = nullptr;
  int n_seq = 0;
  bool fresh = true, ok = true;

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
      n_seq = p.seq_len[cons.u / p.n_kv];
#pragma unroll
      for (int mb = 0; mb < NVB; mb++)
#pragma unroll
        for (int e = 0; e < 4; e++) acc_o[mb][e] = 0.f;
      m_run = -INFINITY; l_run = 0.f; plo0 = 0.f; plo1 = 0.f;
      fresh = false;
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
      int chunk_id = 0;
      k_class<8>(ktile, kcls[0], kB, chunk_id, hp, gid, tig, lane, acc);
      k_class<4>(ktile, kcls[1], kB, chunk_id, hp, gid, tig, lane, acc);
      k_class<2>(ktile, kcls[2], kB, chunk_id, hp, gid, tig, lane, acc);
      k_class<1>(ktile, kcls[3], kB, chunk_id, hp, gid, tig, lane, acc);

      // per-token group minimum and range of the K tile (fp16), this thread's 8 tokens
      const int tok_off = 2 * (gid * 16 + 8 * hp);
      uint32_t klo0[4] = {0, 0, 0, 0}, kr0[4] = {0, 0, 0, 0}, klo1[4] = {0, 0, 0, 0}, kr1[4] = {0, 0, 0, 0};
      if (kmeta0 >= 0) { ld_words<4>(ktile + kmeta0 + tok_off, klo0); ld_words<4>(ktile + kmeta0 + 256 + tok_off, kr0); }
      if (kmeta1 >= 0) { ld_words<4>(ktile + kmeta1 + tok_off, klo1); ld_words<4>(ktile + kmeta1 + 256 + tok_off, kr1); }
      float s[8];
      float mx = -INFINITY;
      const int tok0 = cons.t * kTile + gid * 16 + 8 * hp;
#pragma unroll
      for (int ii = 0; ii < 8; ii++) {
        const int u = ii & 3, cb = (ii >> 2) * 2;             // token ii: MMA u, row gid (ii < 4) or gid + 8
        const float a0 = acc[0][u][cb] + acc[0][u][cb + 1];   // hi + lo halves of q'
        const float a1 = acc[1][u][cb] + acc[1][u][cb + 1];
        const float2 lo0 = h2f2(klo0[ii >> 1]), r0 = h2f2(kr0[ii >> 1]);
        const float2 lo1 = h2f2(klo1[ii >> 1]), r1 = h2f2(kr1[ii >> 1]);
        const float l0 = (ii & 1) ? lo0.y : lo0.x, rr0 = (ii & 1) ? r0.y : r0.x;
        const float l1 = (ii & 1) ? lo1.y : lo1.x, rr1 = (ii & 1) ? r1.y : r1.x;
        float v = kscale * (rr0 * a0 + rr1 * a1) + l0 * qlo0 + l1 * qlo1;
        if (tok0 + ii >= n_seq) v = -INFINITY;
        s[ii] = v;
        mx = fmaxf(mx, v);
      }
      if (hp == 1) {           // the K slot is free: refill it with the tile D positions ahead
        if (issued_k < count) {
          __syncwarp();
          if (lane == 0) { fence_async_smem(); start_k(issued_k % D); }
          issued_k++;
        }
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
      if (mx > m_run) {        // new running maximum for this thread's head: rescale what has been accumulated
        const float alpha = fast_exp2(m_run - mx);   // exp2(-inf) = 0 on the first tile
        m_run = mx;
        l_run *= alpha; plo0 *= alpha; plo1 *= alpha;
#pragma unroll
        for (int mb = 0; mb < NVB; mb++)
#pragma unroll
          for (int e = 0; e < 4; e++) acc_o[mb][e] *= alpha;
      }
      if (hp == 0) ok = ok && mbar_wait(bars + 8 * (4 + slot), parity);
      uint32_t vlo0[4] = {0, 0, 0, 0}, vr0[4] = {0, 0, 0, 0}, vlo1[4] = {0, 0, 0, 0}, vr1[4] = {0, 0, 0, 0};
      if (vmeta0 >= 0) { ld_words<4>(vtile + vmeta0 + tok_off, vlo0); ld_words<4>(vtile + vmeta0 + 256 + tok_off, vr0); }
      if (vmeta1 >= 0) { ld_words<4>(vtile + vmeta1 + tok_off, vlo1); ld_words<4>(vtile + vmeta1 + 256 + tok_off, vr1); }
      // probabilities times the V group ranges, as fp16 pairs (group 0, group 1), transposed into B fragments
      uint32_t pb[8];
#pragma unroll
      for (int ii = 0; ii < 8; ii++) {
        const float pr = m_run == -INFINITY ? 0.f : fast_exp2(s[ii] - m_run);
        const float2 lo0 = h2f2(vlo0[ii >> 1]), r0 = h2f2(vr0[ii >> 1]);
        const float2 lo1 = h2f2(vlo1[ii >> 1]), r1 = h2f2(vr1[ii >> 1]);
        l_run += pr;
        plo0 = fmaf(pr, (ii & 1) ? lo0.y : lo0.x, plo0);
        plo1 = fmaf(pr, (ii & 1) ? lo1.y : lo1.x, plo1);
        const __half2 pk = __floats2half2_rn(pr * ((ii & 1) ? r0.y : r0.x), pr * ((ii & 1) ? r1.y : r1.x));
        pb[ii] = movmatrix_trans(*reinterpret_cast<const uint32_t*>(&pk));
      }
      // ------------------------------------------------------------ P~ x V codes
      int mb = 0;
      v_class<8, NVB>(vtile, vcls[0], mb, hp, gid, tig, pb, acc_o);
      v_class<4, NVB>(vtile, vcls[1], mb, hp, gid, tig, pb, acc_o);
      v_class<2, NVB>(vtile, vcls[2], mb, hp, gid, tig, pb, acc_o);
      v_class<1, NVB>(vtile, vcls[3], mb, hp, gid, tig, pb, acc_o);
      if (hp == 1) {
        if (issued_v < issued_k) {
          __syncwarp();
          if (lane == 0) { fence_async_smem(); start_v(issued_v % D); }
          issued_v++;
        }
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
      int mbase = 0;
#pragma unroll
      for (int c = 0; c < 4; c++) {
        const uint32_t cls = vcls[c];
        const int n = cls & 0xff, n_g0 = (cls >> 8) & 0xff;
        const int first = d.vfirst[c];
        const int nblk = (n + 15) >> 4;
#pragma unroll
        for (int mb = 0; mb < NVB; mb++) {
          const int bi = mb - mbase;
          if (bi >= 0 && bi < nblk) {
#pragma unroll
            for (int half = 0; half < 2; half++) {
              const int r = 16 * bi + gid + 8 * half;
              if (r < n) rec[kRecHead + first + r] = r >= n_g0 ? acc_o[mb][2 * half + 1] : acc_o[mb][2 * half];
            }
          }
        }
        mbase += nblk;
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

}  // namespace spectra
