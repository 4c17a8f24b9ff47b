// Main kernel of the tensor-core coded-cache decode attention (see attention_tc_common.cuh for the overview).
//
// Unpacking.  A w-bit code left in place inside a 16-bit half-word, with every other bit masked off, is a
// subnormal (or lowest-binade) fp16 number equal to code * 2^(p - 24), p = bit position of the field, as long as
// p + w <= 10; mma.sync handles fp16 subnormals exactly.  So one logic op per register (two values) turns packed
// codes into A fragments; fields above bit 10 are first brought down by one shift of the whole word.  The
// position-dependent power of two is folded into the B operand (exact): on the K side the four MMAs of a chunk
// take the tokens whose fields share a position, on the V side the probabilities get one scaled copy per class.
//
// A warp works on a whole 128-token tile at a time: a thread owns tokens 16 gid .. 16 gid + 15 (two half tiles of
// eight), so one shared-memory load brings both half tiles' words of a strip pair and one B fragment serves both.
// The K tile is walked one scale group at a time (all classes of group 0, then all classes of group 1): a single
// set of score accumulators is live, and each (class, group) run is a short loop whose body is compile-time code.
//
// The V accumulators live in tensor memory, one 16-strip block per 4 columns of the warp's lane quarter: a block is
// fetched, updated and put back, so any number of blocks per class runs through the same code and no register holds
// an accumulator across the score phase.
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
template <> struct Unpack<1> {   // 1 word (already shifted right by 8 * half tile), 8 tokens at bits 0..7
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

// A thread's words of one strip pair (K) or strip (V) for the whole tile: W words of 32 bits, the first half of
// them for half tile 0 and the rest for half tile 1 (W = 1: one word, half tile 1 in the upper byte of each half).
template <int W>
__device__ __forceinline__ void ld_tile_words(const unsigned char* p, uint32_t (&x)[W]) {
  if constexpr (W == 8) {
    const uint4 a = *reinterpret_cast<const uint4*>(p), b = *reinterpret_cast<const uint4*>(p + 16);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
  } else if constexpr (W == 4) {
    const uint4 a = *reinterpret_cast<const uint4*>(p);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
  } else if constexpr (W == 2) {
    const uint2 a = *reinterpret_cast<const uint2*>(p);
    x[0] = a.x; x[1] = a.y;
  } else {
    x[0] = *reinterpret_cast<const uint32_t*>(p);
  }
}
// The same words of a K strip that is stored alone (half-words in order): each half-word becomes the low half of a
// word, the partner strip's half is zero.  p points at the thread's first half-word (2 W gid bytes into the strip).
template <int W>
__device__ __forceinline__ void ld_lone_words(const unsigned char* p, uint32_t (&x)[W]) {
  if constexpr (W == 1) {
    x[0] = *reinterpret_cast<const uint16_t*>(p);
  } else {
    uint32_t h[W / 2];
    ld_tile_words<W / 2>(p, h);
#pragma unroll
    for (int i = 0; i < W / 2; i++) { x[2 * i] = h[i] & 0xffffu; x[2 * i + 1] = h[i] >> 16; }
  }
}
template <int W, int HP>
__device__ __forceinline__ void half_tile_words(const uint32_t (&x)[W], uint32_t (&w)[Unpack<W>::NW]) {
  if constexpr (W == 1) w[0] = HP ? x[0] >> 8 : x[0];
  else {
#pragma unroll
    for (int i = 0; i < Unpack<W>::NW; i++) w[i] = x[Unpack<W>::NW * HP + i];
  }
}

// One chunk (8 strip pairs x 128 tokens) into the score accumulators: per half tile, MMA u takes tokens u (row
// gid) and u + 4 (row gid + 8), pair slots tig and tig + 4 as its k columns, and B variant u (scaled by
// 2^-p_eff(u); rows of strips outside the run's scale group, or past the end of the class, are zero).  The MMAs
// that use variants 0 and 1 come first; then b01 is reloaded with the next chunk's entry while the MMAs of variants
// 2 and 3 run, and b23 after those: the B fragments are fetched half a chunk ahead without a second set of registers.
template <int W>
__device__ __forceinline__ void k_chunk(const uint32_t (&xa)[W], const uint32_t (&xb)[W], uint4& b01, uint4& b23,
                                        const uint4* __restrict__ kb_next, float (&acc)[2][4][4]) {
  using U = Unpack<W>;
  constexpr int NW = U::NW;
  uint32_t wa0[NW], wb0[NW], was0[NW], wbs0[NW], wa1[NW], wb1[NW], was1[NW], wbs1[NW];
  half_tile_words<W, 0>(xa, wa0);
  half_tile_words<W, 0>(xb, wb0);
  half_tile_words<W, 1>(xa, wa1);
  half_tile_words<W, 1>(xb, wb1);
  U::shifted(wa0, was0);
  U::shifted(wb0, wbs0);
  U::shifted(wa1, was1);
  U::shifted(wb1, wbs1);
  mma16816(acc[0][0], U::get(wa0, was0, 0), U::get(wa0, was0, 4), U::get(wb0, wbs0, 0), U::get(wb0, wbs0, 4), b01.x, b01.y);
  mma16816(acc[1][0], U::get(wa1, was1, 0), U::get(wa1, was1, 4), U::get(wb1, wbs1, 0), U::get(wb1, wbs1, 4), b01.x, b01.y);
  mma16816(acc[0][1], U::get(wa0, was0, 1), U::get(wa0, was0, 5), U::get(wb0, wbs0, 1), U::get(wb0, wbs0, 5), b01.z, b01.w);
  mma16816(acc[1][1], U::get(wa1, was1, 1), U::get(wa1, was1, 5), U::get(wb1, wbs1, 1), U::get(wb1, wbs1, 5), b01.z, b01.w);
  b01 = __ldg(kb_next);
  mma16816(acc[0][2], U::get(wa0, was0, 2), U::get(wa0, was0, 6), U::get(wb0, wbs0, 2), U::get(wb0, wbs0, 6), b23.x, b23.y);
  mma16816(acc[1][2], U::get(wa1, was1, 2), U::get(wa1, was1, 6), U::get(wb1, wbs1, 2), U::get(wb1, wbs1, 6), b23.x, b23.y);
  mma16816(acc[0][3], U::get(wa0, was0, 3), U::get(wa0, was0, 7), U::get(wb0, wbs0, 3), U::get(wb0, wbs0, 7), b23.z, b23.w);
  mma16816(acc[1][3], U::get(wa1, was1, 3), U::get(wa1, was1, 7), U::get(wb1, wbs1, 3), U::get(wb1, wbs1, 7), b23.z, b23.w);
  b23 = __ldg(kb_next + 32);
}

// One (class, scale group) run of the K tile: `run` = byte offset / 16 of its first pair | chunks << 16 |
// slot of a strip stored alone in the last chunk << 24 | (such a strip exists) << 27.  A run has at most MAXC chunks
// (64 channels per scale group; a group-1 run may start in the middle of a chunk).  The loop is kept rolled (the
// sixteen warps of an SM run different parts of the kernel: its code has to stay small for the instruction cache)
// and loads the next chunk's words while the current chunk is multiplied.  The B table is walked in the same order; on entry b01, b23 hold the run's first entry and kb points
// at this lane's part of it; on exit they hold the entry after the run (the first of the next run; past the last
// run a spare entry of the table, never used).
template <int W, int MAXC>
__device__ __forceinline__ void k_run(const unsigned char* ktile, uint32_t run, const uint4* __restrict__& kb,
                                      uint4& b01, uint4& b23, int gid, int tig, float (&acc)[2][4][4]) {
  const int nch = (int)(run >> 16) & 0xff;
  if (nch == 0) return;
  const unsigned char* pa = ktile + (run & 0xffffu) * 16 + 32 * W * tig + 4 * W * gid;
  const int lone_i = (run >> 27) & 1u ? nch - 1 : -1;
#pragma unroll 1
  for (int i = 0; i < nch; i++, pa += 256 * W) {
    uint32_t xa[W], xb[W];
    ld_tile_words<W>(pa, xa);
    ld_tile_words<W>(pa + 128 * W, xb);
    kb += 64;
    if (i == lone_i) {
      // the pair in slot `slot` of this chunk is one strip stored alone: the threads of that slot re-read it as
      // half-words (all threads load, a select keeps the result where it belongs)
      const int slot = (int)(run >> 24) & 7;
      uint32_t t[W];
      ld_lone_words<W>(pa - 32 * W * tig - 4 * W * gid + 32 * W * slot + 2 * W * gid, t);
      const bool mine_a = tig == slot, mine_b = tig + 4 == slot;
#pragma unroll
      for (int k = 0; k < W; k++) { xa[k] = mine_a ? t[k] : xa[k]; xb[k] = mine_b ? t[k] : xb[k]; }
    }
    k_chunk<W>(xa, xb, b01, b23, kb, acc);
  }
}

// One half tile of one V block (16 strips x 64 tokens) into the block's accumulators: MMA u contracts the token
// pairs of B fragments u and u + 4.
template <int W, int HP>
__device__ __forceinline__ void v_block_half(const uint32_t (&xa)[W], const uint32_t (&xb)[W], const uint32_t (&pw)[8],
                                             float (&acc)[4]) {
  using U = Unpack<W>;
  constexpr int NW = U::NW;
  uint32_t wa[NW], wb[NW], was[NW], wbs[NW];
  half_tile_words<W, HP>(xa, wa);
  half_tile_words<W, HP>(xb, wb);
  U::shifted(wa, was);
  U::shifted(wb, wbs);
#pragma unroll
  for (int u = 0; u < 4; u++)
    mma16816(acc, U::get(wa, was, u), U::get(wb, wbs, u), U::get(wa, was, u + 4), U::get(wb, wbs, u + 4), pw[u], pw[u + 4]);
}
// The V accumulators (one 16-strip block = 4 registers per thread) live in tensor memory: each warp owns the 32
// lanes of its quarter, a block takes 4 columns.  A block is fetched, updated by its 8 MMAs and put back, so the
// number of blocks and their classes are run-time facts (any width profile runs here) and the registers they would
// occupy through the score phase are free.
__device__ __forceinline__ void tmem_put(uint32_t taddr, const float (&a)[4]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1,%2,%3,%4};" ::"r"(taddr), "f"(a[0]), "f"(a[1]), "f"(a[2]),
               "f"(a[3])
               : "memory");
}
__device__ __forceinline__ void tmem_get(uint32_t taddr, float (&a)[4]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];"
               : "=f"(a[0]), "=f"(a[1]), "=f"(a[2]), "=f"(a[3])
               : "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// One class of the V tile: blocks of 16 strips, accumulators at tensor-memory columns col, col + 4, ...  The
// probabilities first get the class's position scales; per half tile, MMA u of a block contracts the token pairs of
// B fragments u and u + 4.  Rows past the end of the class read whatever follows in shared memory (finite after
// masking); their accumulator rows are never stored.  FRESH: the unit's first tile (accumulators start at zero);
// otherwise what comes back from tensor memory is first multiplied by alpha, the rescaling a new reference owes.
template <int W, bool FRESH>
__device__ __forceinline__ void v_class(const unsigned char* vtile, uint32_t cls, int gid, int tig,
                                        const uint32_t (&pb)[2][8], uint32_t& col, float alpha) {
  using U = Unpack<W>;
  const int n = cls & 0xff;
  if (n == 0) return;
  uint32_t pw[2][8];
#pragma unroll
  for (int hp = 0; hp < 2; hp++)
#pragma unroll
    for (int ii = 0; ii < 8; ii++) pw[hp][ii] = hmul2_pow2(pb[hp][ii], U::peff(ii));
  const unsigned char* px = vtile + (cls >> 16) * 16 + 4 * W * tig + 16 * W * gid;
  const int nb = (n + 15) >> 4;
  const bool rescale = alpha != 1.f;
#pragma unroll 1
  for (int bi = 0; bi < nb; bi++, px += 256 * W, col += 4) {
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    if (!FRESH) tmem_get(col, acc);
    uint32_t xa[W], xb[W];
    ld_tile_words<W>(px, xa);
    ld_tile_words<W>(px + 128 * W, xb);
    if (!FRESH) {
      tmem_wait_ld();
      if (rescale) {
#pragma unroll
        for (int e = 0; e < 4; e++) acc[e] *= alpha;
      }
    }
    v_block_half<W, 0>(xa, xb, pw[0], acc);
    v_block_half<W, 1>(xa, xb, pw[1], acc);
    tmem_put(col, acc);
  }
}
template <bool FRESH>
__device__ __forceinline__ void v_tile(const unsigned char* vtile, const uint4& vc, int gid, int tig,
                                       const uint32_t (&pb)[2][8], uint32_t col, float alpha) {
  v_class<8, FRESH>(vtile, vc.x, gid, tig, pb, col, alpha);
  v_class<4, FRESH>(vtile, vc.y, gid, tig, pb, col, alpha);
  v_class<2, FRESH>(vtile, vc.z, gid, tig, pb, col, alpha);
  v_class<1, FRESH>(vtile, vc.w, gid, tig, pb, col, alpha);
}

// Writes one class's accumulators into a partial record: row r of the class goes to strip index first + r, taking
// the column of the scale group the strip belongs to.
__device__ __forceinline__ void store_class(float* rec, uint32_t cls, int first, int gid, uint32_t& col) {
  const int n = cls & 0xff, n_g0 = (cls >> 8) & 0xff;
#pragma unroll 1
  for (int r0 = 0; r0 < n; r0 += 16, col += 4) {
    float acc[4];
    tmem_get(col, acc);
    tmem_wait_ld();
#pragma unroll
    for (int half = 0; half < 2; half++) {
      const int r = r0 + gid + 8 * half;
      if (r < n) rec[kRecHead + first + r] = r >= n_g0 ? acc[2 * half + 1] : acc[2 * half];
    }
  }
}

// Two floats to packed fp16 (low = a), saturating at the largest finite value instead of producing infinity.
__device__ __forceinline__ uint32_t pack_half2_sat(float a, float b) {
  uint32_t d;
  asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(b), "f"(a));
  return d;
}

// Per-warp state in shared memory: the head of the current unit's descriptor (read as broadcast loads where it is
// used, instead of sitting in registers through the whole tile) and the two producer cursors, which only lane 0
// touches: the next tile to copy is the previous one plus the tile size until the unit's tiles run out.
struct TileProducer {
  uint64_t base;         // global address of the unit's first tile (contiguous cache) or of its page pool (paged)
  uint32_t tb;           // tile bytes of the unit
  int32_t rem;           // tiles of the unit not yet copied
  int32_t unit, t;       // unit of the tensor path, logical index of the next tile to copy
};
struct WarpState {
  alignas(16) uint32_t head[20];   // UnitDesc words 0..5 (tbk, tbv, kmeta[2], vmeta[2]), two spare words, then words
                                   // 6..17 (krun[2][4], vcls[4]) on 16-byte boundaries
  TileProducer k, v;
};
static_assert(sizeof(WarpState) == 128, "WarpState layout");
constexpr int kWarpStateBytes = 128;
constexpr int kAccColumns = 128;       // tensor-memory columns per CTA: 4 per V block of a warp, up to 32 blocks

// Adds one scale group's share to the scores of this thread's 16 tokens, in units of 1 / kscale:
// s'_t += R_t * (hi + lo partial sums) + lo_t * (sum of q' over the group's active channels / kscale).
// meta points at lo16[16 gid] of the group; R16 follows 256 bytes later.
template <bool FIRST>
__device__ __forceinline__ void fold_group(const unsigned char* meta, float qlo, const float (&acc)[2][4][4],
                                           float (&s)[16]) {
#pragma unroll
  for (int half = 0; half < 2; half++) {
    uint32_t lo[4], rg[4];
    ld_tile_words<4>(meta + 16 * half, lo);
    ld_tile_words<4>(meta + 256 + 16 * half, rg);
#pragma unroll
    for (int r = 0; r < 4; r++) {
      const float2 l2 = h2f2(lo[r]), r2 = h2f2(rg[r]);
#pragma unroll
      for (int e = 0; e < 2; e++) {
        const int ii = 2 * r + e, u = ii & 3, cb = (ii >> 2) * 2;
        const float a = acc[half][u][cb] + acc[half][u][cb + 1];            // hi + lo halves of q'
        const float base = FIRST ? (e ? l2.y : l2.x) * qlo : fmaf(e ? l2.y : l2.x, qlo, s[8 * half + ii]);
        s[8 * half + ii] = fmaf(e ? r2.y : r2.x, a, base);
      }
    }
  }
}

template <bool PAGED>
__global__ void __launch_bounds__(kFastWarps * 32, kFastCtasPerSm) attention_mma_kernel(AttnArgs p, FastArgs f) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int gid = lane >> 2, tig = lane & 3;
  const int gw = blockIdx.x * kFastWarps + warp;
  const int D = f.depth;
  const uint32_t warp_bytes = (uint32_t)D * (f.slot_k + f.slot_v);
  unsigned char* ring_k = smem_raw + warp * warp_bytes;
  unsigned char* ring_v = ring_k + D * f.slot_k;
  const uint32_t bars = smem_u32(smem_raw) + kFastWarps * warp_bytes + warp * (2 * 4 * 8);  // K slots 0..3, V slots 0..3
  WarpState& ws = *reinterpret_cast<WarpState*>(smem_raw + kFastWarps * warp_bytes + kFastWarps * 64 + warp * kWarpStateBytes);
  if (lane == 0)
    for (int s = 0; s < 2 * 4; s++) mbar_init(bars + 8 * s, 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  __syncwarp();
  // tensor memory for the V accumulators: kAccColumns columns per CTA, allocated and freed by warp 0
  __shared__ uint32_t tmem_base_s;
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"((uint32_t)kAccColumns) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t acc_base = tmem_base_s + ((uint32_t)(warp & 3) << 21);   // this warp's lanes 32 * (warp % 4), column 0

  // everything above ran beside the preceding launch (descriptors, appended tokens); from here on its results are read
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the combine kernel may be scheduled as SMs free up
  const int4 start = f.warp_start[gw];                 // first unit, first tile in it, tiles of that unit, tiles of the share
  const int count = start.w;
  if (count > 0) {
  int cu = start.x, ct = start.y, cnt = start.z;       // consumer: unit, tile, tiles of the unit
  // Copies are started by lane 0, whose cursors live in shared memory; every lane keeps the same counts of tiles
  // whose K / V copy has been started.  A unit's tiles are contiguous: its next tile is one tile size further.
  // (lane 0 keeps the page of the next tile in a register, looked up one copy ahead, so that a paged cache costs
  // no dependent global read at the time a copy is started)
  int page_k = 0, page_v = 0;
  auto page_of = [&](const TileProducer& q, int side) {
    if constexpr (!PAGED) return q.t;
    else return (int)(side ? p.map_v : p.map_k).page(q.unit / f.npass, q.t);
  };
  auto next_unit = [&](TileProducer& q, int side) {    // the unit's tiles are used up: move to the next unit with tiles
    int u = q.unit + 1, n = 0;
    while (u < f.n_units) {
      n = f.tile_prefix[u + 1] - f.tile_prefix[u];
      if (n > 0) break;
      u++;
    }
    const UnitDesc& d = f.desc[min(u, f.n_units - 1)];
    q.unit = u; q.rem = n; q.t = 0;
    q.tb = side ? d.tbv : d.tbk;
    q.base = (uint64_t)(side ? p.cache_v + d.src_v : p.cache_k + d.src_k);
  };
  auto start_k = [&](int slot) {
    if (ws.k.rem == 0) { next_unit(ws.k, 0); page_k = page_of(ws.k, 0); }
    const uint32_t tb = ws.k.tb;
    mbar_expect_tx(bars + 8 * slot, tb);
    bulk_load(smem_u32(ring_k + slot * f.slot_k), (const void*)(ws.k.base + (uint64_t)page_k * tb), tb, bars + 8 * slot,
              l2_evict_first_policy());
    ws.k.t++;
    if (--ws.k.rem > 0) page_k = page_of(ws.k, 0);
  };
  auto start_v = [&](int slot) {
    if (ws.v.rem == 0) { next_unit(ws.v, 1); page_v = page_of(ws.v, 1); }
    const uint32_t tb = ws.v.tb;
    mbar_expect_tx(bars + 8 * (4 + slot), tb);
    bulk_load(smem_u32(ring_v + slot * f.slot_v), (const void*)(ws.v.base + (uint64_t)page_v * tb), tb,
              bars + 8 * (4 + slot), l2_evict_first_policy());
    ws.v.t++;
    if (--ws.v.rem > 0) page_v = page_of(ws.v, 1);
  };
  int issued_k = min(D, count), issued_v = issued_k;
  int fill_k = issued_k % D, fill_v = fill_k;           // slots the next K / V copies go to
  if (lane == 0) {
    const UnitDesc& d = f.desc[cu];
    ws.k.unit = cu; ws.k.rem = cnt - ct; ws.k.t = ct; ws.k.tb = d.tbk; ws.k.base = (uint64_t)(p.cache_k + d.src_k);
    ws.v.unit = cu; ws.v.rem = cnt - ct; ws.v.t = ct; ws.v.tb = d.tbv; ws.v.base = (uint64_t)(p.cache_v + d.src_v);
    page_k = page_of(ws.k, 0); page_v = page_of(ws.v, 1);
    for (int j = 0; j < issued_k; j++) { start_k(j); start_v(j); }
  }

  float m_ref = -INFINITY, l_run = 0.f, plo0 = 0.f, plo1 = 0.f;
  float alpha_acc = 1.f;      // rescaling the accumulators in tensor memory still owe
  bool acc_fresh = true;      // the unit's first tile: its accumulators start at zero
  float kscale = 0.f, qlo0 = 0.f, qlo1 = 0.f;
  int n_seq = 0;
  bool fresh = true, ok = true;
  int slot = 0;
  uint32_t parity = 0;

  for (int j = 0; j < count && ok; j++) {
    const unsigned char* ktile = ring_k + slot * f.slot_k;
    const unsigned char* vtile = ring_v + slot * f.slot_v;
    if (fresh) {
      const UnitDesc& d = f.desc[cu];
      __syncwarp();
      if (lane < 18) ws.head[lane < 6 ? lane : lane + 2] = reinterpret_cast<const uint32_t*>(&d)[lane];
      kscale = d.kscale[tig];                                  // a power of two: the divisions are exact
      qlo0 = d.qlo[tig][0] / kscale; qlo1 = d.qlo[tig][1] / kscale;
      n_seq = attended_tokens(p, (cu / f.npass) / p.n_kv);
      m_ref = -INFINITY; l_run = 0.f; plo0 = 0.f; plo1 = 0.f;
      alpha_acc = 1.f; acc_fresh = true;
      fresh = false;
      __syncwarp();
    }

    // ------------------------------------------------------------ scores of the tile's 128 tokens, in units of 1 / kscale
    ok = mbar_wait(bars + 8 * slot, parity);
    float s[16];
    {
      const uint4* kb = &f.desc[cu].kB[0][0][0] + lane;   // walks the B fragment table in run order, one entry ahead
      uint4 b01 = __ldg(kb), b23 = __ldg(kb + 32);
      const int kmeta0 = (int)ws.head[2], kmeta1 = (int)ws.head[3];
      float acc[2][4][4];
      if (kmeta0 >= 0) {
        const uint4 runs = *reinterpret_cast<const uint4*>(&ws.head[8]);
#pragma unroll
        for (int hp = 0; hp < 2; hp++)
#pragma unroll
          for (int u = 0; u < 4; u++)
#pragma unroll
            for (int e = 0; e < 4; e++) acc[hp][u][e] = 0.f;
        k_run<8, 4>(ktile, runs.x, kb, b01, b23, gid, tig, acc);
        k_run<4, 4>(ktile, runs.y, kb, b01, b23, gid, tig, acc);
        k_run<2, 4>(ktile, runs.z, kb, b01, b23, gid, tig, acc);
        k_run<1, 4>(ktile, runs.w, kb, b01, b23, gid, tig, acc);
        fold_group<true>(ktile + kmeta0 + 32 * gid, qlo0, acc, s);
      } else {
#pragma unroll
        for (int i = 0; i < 16; i++) s[i] = 0.f;
      }
      if (kmeta1 >= 0) {
        const uint4 runs = *reinterpret_cast<const uint4*>(&ws.head[12]);
#pragma unroll
        for (int hp = 0; hp < 2; hp++)
#pragma unroll
          for (int u = 0; u < 4; u++)
#pragma unroll
            for (int e = 0; e < 4; e++) acc[hp][u][e] = 0.f;
        k_run<8, 5>(ktile, runs.x, kb, b01, b23, gid, tig, acc);
        k_run<4, 5>(ktile, runs.y, kb, b01, b23, gid, tig, acc);
        k_run<2, 5>(ktile, runs.z, kb, b01, b23, gid, tig, acc);
        k_run<1, 5>(ktile, runs.w, kb, b01, b23, gid, tig, acc);
        fold_group<false>(ktile + kmeta1 + 32 * gid, qlo1, acc, s);
      }
    }
    if (issued_k < count) {     // the K slot is free: refill it with the tile D positions ahead
      __syncwarp();
      if (lane == 0) { fence_async_smem(); start_k(fill_k); }
      issued_k++;
      fill_k = fill_k + 1 == D ? 0 : fill_k + 1;
    }
    if ((ct + 1) * kTile > n_seq) {                      // only the unit's last tile has slots past the end
      const int tok0 = ct * kTile + gid * 16;
#pragma unroll
      for (int i = 0; i < 16; i++)
        if (tok0 + i >= n_seq) s[i] = -INFINITY;
    }
    ok = ok && mbar_wait(bars + 8 * (4 + slot), parity);
    // Probabilities enter the tensor core as fp16, multiplied by the V group range of their token: p~ = 2^(s - m_ref) R.
    // The reference exponent m_ref of this warp's share of the unit is kept 13 binades below the largest s + log2 R
    // seen so far (per head), so that no p~ exceeds 2^13 (fp16 holds 65504) while the bulk of them, far smaller with
    // tens of thousands of tokens, stays in fp16's normal range.  Whenever a tile raises it, everything accumulated
    // so far is rescaled: a new maximum score and a token with an unusually large value range are the same event.
    // The record carries m_ref, so the merge of the splits is unaffected.
    uint32_t pb[2][8];
    {
      const int vmeta0 = (int)ws.head[4], vmeta1 = (int)ws.head[5];
      uint32_t vr0[8] = {0, 0, 0, 0, 0, 0, 0, 0}, vr1[8] = {0, 0, 0, 0, 0, 0, 0, 0};
      if (vmeta0 >= 0) ld_tile_words<8>(vtile + vmeta0 + 256 + 32 * gid, vr0);
      if (vmeta1 >= 0) ld_tile_words<8>(vtile + vmeta1 + 256 + 32 * gid, vr1);
      float mx = s[0];
#pragma unroll
      for (int i = 1; i < 16; i++) mx = fmaxf(mx, s[i]);
      __half2 rm = __hmax2(*reinterpret_cast<const __half2*>(&vr0[0]), *reinterpret_cast<const __half2*>(&vr1[0]));
#pragma unroll
      for (int r = 1; r < 8; r++)
        rm = __hmax2(rm, __hmax2(*reinterpret_cast<const __half2*>(&vr0[r]), *reinterpret_cast<const __half2*>(&vr1[r])));
      const float rmax = fmaxf(__low2float(rm), __high2float(rm));          // ranges are non-negative
      // rmax < 2^e; ranges below fp16's normal range (or none at all) count as 2^-14, which keeps 2^(s - m_ref) finite
      const int e = max((int)((__float_as_uint(rmax) >> 23) & 0xff) - 126, -14);
      float need = fmaf(mx, kscale, (float)(e - 13));                       // kscale is a positive power of two
      need = fmaxf(need, __shfl_xor_sync(0xffffffffu, need, 4));
      need = fmaxf(need, __shfl_xor_sync(0xffffffffu, need, 8));
      need = fmaxf(need, __shfl_xor_sync(0xffffffffu, need, 16));
      if (need > m_ref) {      // rescale what has been accumulated (exp2(-inf) = 0 on the first tile)
        const float alpha = fast_exp2(m_ref - need);
        m_ref = need;
        l_run *= alpha; plo0 *= alpha; plo1 *= alpha;
        alpha_acc *= alpha;                                   // applied to the accumulators when they are next fetched
      }
      const float m_use = m_ref == -INFINITY ? 0.f : m_ref;
#pragma unroll
      for (int half = 0; half < 2; half++) {
        uint32_t vlo0[4] = {0, 0, 0, 0}, vlo1[4] = {0, 0, 0, 0};
        if (vmeta0 >= 0) ld_tile_words<4>(vtile + vmeta0 + 32 * gid + 16 * half, vlo0);
        if (vmeta1 >= 0) ld_tile_words<4>(vtile + vmeta1 + 32 * gid + 16 * half, vlo1);
#pragma unroll
        for (int r = 0; r < 4; r++) {
          const float2 lo0 = h2f2(vlo0[r]), r0 = h2f2(vr0[4 * half + r]), lo1 = h2f2(vlo1[r]), r1 = h2f2(vr1[4 * half + r]);
#pragma unroll
          for (int e2 = 0; e2 < 2; e2++) {
            const int ii = 2 * r + e2;
            const float pr = fast_exp2(fmaf(s[8 * half + ii], kscale, -m_use));
            l_run += pr;
            plo0 = fmaf(pr, e2 ? lo0.y : lo0.x, plo0);
            plo1 = fmaf(pr, e2 ? lo1.y : lo1.x, plo1);
            pb[half][ii] = movmatrix_trans(pack_half2_sat(pr * (e2 ? r0.y : r0.x), pr * (e2 ? r1.y : r1.x)));
          }
        }
      }
    }
    // ------------------------------------------------------------ P~ x V codes
    {
      const uint4 vc = *reinterpret_cast<const uint4*>(&ws.head[16]);
      if (acc_fresh) v_tile<true>(vtile, vc, gid, tig, pb, acc_base, 1.f);
      else v_tile<false>(vtile, vc, gid, tig, pb, acc_base, alpha_acc);
      tmem_wait_st();
      alpha_acc = 1.f; acc_fresh = false;
    }
    if (issued_v < issued_k) {
      __syncwarp();
      if (lane == 0) { fence_async_smem(); start_v(fill_v); }
      issued_v++;
      fill_v = fill_v + 1 == D ? 0 : fill_v + 1;
    }
    // ------------------------------------------------------------ end of this warp's share of the unit?
    const bool last_of_unit = (ct + 1 >= cnt) || (j + 1 >= count);
    if (last_of_unit) {
      float l = l_run, q0 = plo0, q1 = plo1;
#pragma unroll
      for (int sft = 4; sft <= 16; sft <<= 1) {
        l += __shfl_xor_sync(0xffffffffu, l, sft);
        q0 += __shfl_xor_sync(0xffffffffu, q0, sft);
        q1 += __shfl_xor_sync(0xffffffffu, q1, sft);
      }
      float* rec = f.records + (int64_t)(gw + cu) * f.rec_stride + tig * (kRecHead + f.vs_max);
      if (gid == 0) { rec[0] = m_ref; rec[1] = l; rec[2] = q0; rec[3] = q1; }
      const UnitDesc& d = f.desc[cu];
      uint32_t col = acc_base;
      store_class(rec, ws.head[16], d.vfirst[0], gid, col);
      store_class(rec, ws.head[17], d.vfirst[1], gid, col);
      store_class(rec, ws.head[18], d.vfirst[2], gid, col);
      store_class(rec, ws.head[19], d.vfirst[3], gid, col);
      fresh = true;
    }
    // next tile of the flattened (unit, tile) space
    ct++;
    if (ct >= cnt) {
      cu++; ct = 0;
      while (cu < f.n_units) {
        cnt = f.tile_prefix[cu + 1] - f.tile_prefix[cu];
        if (cnt > 0) break;
        cu++;
      }
    }
    if (++slot == D) { slot = 0; parity ^= 1u; }
  }
  if (!ok) {
    if (lane == 0 && p.status) atomicOr(p.status, SPECTRA_STATUS_WAIT_TIMEOUT);
    // give copies that may still be in flight a bounded time to land before the shared memory is released
    for (int s = 0; s < D; s++) { mbar_wait(bars + 8 * s, 0); mbar_wait(bars + 8 * (4 + s), 0); }
  }
  }   // count > 0
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base_s), "r"((uint32_t)kAccColumns) : "memory");
}

}  // namespace spectra
