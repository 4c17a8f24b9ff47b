// Many-query (prefill) causal attention over the reconstructed cache: Mode A of Sec. 3.3 (reconstruct, then attend)
// for a chunk of new queries.  The reconstructed keys and values sit in pools of bf16 pages of 128 tokens
// (spectra_decode_paged writes them); query i of a sequence is at position pos0 + i and attends tokens 0 .. pos0 + i.
//
// One CTA takes 256 consecutive queries of one query head as two groups of 128 rows (A, B) and walks the key/value
// tiles up to its diagonal; both groups use every tile that is brought in.  Both products run on the 5th-generation
// tensor cores with fp32 accumulators in tensor memory:
//   S = Q K^T       A = Q   [128 queries x 128 channels], shared memory, K-major;  B = K tile, K-major
//   O += P V        A = P   [128 queries x 128 tokens] bf16 in tensor memory, written over the scores it came from
//                   (two values per 32-bit column);  B = V tile [128 tokens x 128 channels], MN-major
// Operand tiles in shared memory use the 128-byte swizzle: a page [token][channel] arrives by TMA as two blocks of 64
// channels, [128 tokens x 128 bytes] each, which is both layouts at once (K-major with the tokens as rows, MN-major
// with the tokens as the contraction index); Q is stored in the same form by the threads that own its rows.
//
// Twelve warps, three warpgroups; after the set-up the softmax warpgroups take registers from the third one
// (setmaxnreg), so that a thread can hold a whole row of scores and still schedule its arithmetic freely:
//   warps 0..3, 4..7  softmax of group A, B: thread r owns query row r of its group (= its tensor-memory lane): takes
//               its 128 scores into registers, keeps a running reference m and sum l, writes the probabilities as bf16
//               back into the score columns, rescales its row of O when the reference moves (only when it grows by more
//               than 2^8: until then the old one is kept, which is exact as long as numerator and denominator use the
//               same one), and at the end divides and stores;
//   warp 8      (one lane) producer: TMA copies of the K and V tiles through one ring of five slots, keys one tile
//               ahead of the values (K0 K1 V0 K2 V1 ..);
//   warp 9      (one lane) issues the MMAs, group by group: P V of tile j, then the scores of tile j + 1, so that the
//               tensor cores work for one group while the other group's softmax runs.  The sixteen MMAs of a group
//               and tile go out back to back from descriptors computed once: the rate at which one thread can issue
//               them is what bounds the tensor pipe here;
//   warps 10, 11  only give up their registers.
// Tensor memory: columns 0..127 scores / P of A, 128..255 of B, 256..383 O of A, 384..511 O of B.
// Barriers (all waits bounded; a timeout sets SPECTRA_STATUS_WAIT_TIMEOUT and the waiter leaves its loop):
//   full[s], free[s]       ring slot s: the copies have landed / the last MMA that reads it is complete
//   s_full[g]              the scores of group g are complete
//   p_full[g]              the group's four warps have written P (and are done with O)
//   pv_done[g]             the group's P V is complete: O is consistent, the score columns may be overwritten
#pragma once
#include "umma.cuh"

namespace spectra {

struct PrefillArgs {
  const __nv_bfloat16* q; __nv_bfloat16* out; float* lse;
  int64_t q_stride_seq, q_stride_token, q_stride_head;     // elements
  int64_t o_stride_seq, o_stride_token, o_stride_head;
  const int32_t* pos0;       // per sequence: tokens in the cache before this chunk = position of query 0
  int32_t n_new;             // queries per sequence
  int n_seqs, n_kv, gqa;
  float scale_log2;          // softmax scale * log2(e)
  const int32_t* table;      // (unit = sequence * n_kv + kv head, tile) -> page; NULL: page = unit * table_stride + tile
  int64_t table_stride;
  int32_t* status;
  int n_qblocks;
};

constexpr int kPfThreads = 384;
constexpr int kPfRows = 2 * kTile;                       // queries per CTA
constexpr uint32_t kPfTileBytes = kTile * kD * 2;
// bf16 A and B, fp32 D, both operands K-major (scores) / B MN-major (kUmIdesc: P V)
constexpr uint32_t kPfIdescKK = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

constexpr int kPfSlots = 5;
// Ring order: K0, then K(j + 1), V(j) for j = 0, 1, ..: the keys run one tile ahead of the values, because the scores
// of tile j + 1 are issued right behind P V of tile j, whose values are the last thing a tile needs.
__host__ __device__ constexpr int pf_item_k(int j) { return j == 0 ? 0 : 2 * j - 1; }
__host__ __device__ constexpr int pf_item_v(int j) { return 2 * j + 2; }
constexpr bool kPfSwizzle = true;
struct PrefillSmem {
  alignas(1024) uint8_t q[2][kPfTileBytes];
  alignas(1024) uint8_t kv[kPfSlots][kPfTileBytes];
  alignas(8) uint64_t full[kPfSlots], free_[kPfSlots], s_full[2], p_full[2], pv_done[2];
  uint32_t tmem_base;
};
static_assert(sizeof(PrefillSmem) + 1024 <= 227 * 1024, "the prefill kernel's shared memory must fit one SM");

__device__ __forceinline__ void um_st16(uint32_t a, const float* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(a),
      "f"(r[0]), "f"(r[1]), "f"(r[2]), "f"(r[3]), "f"(r[4]), "f"(r[5]), "f"(r[6]), "f"(r[7]), "f"(r[8]), "f"(r[9]),
      "f"(r[10]), "f"(r[11]), "f"(r[12]), "f"(r[13]), "f"(r[14]), "f"(r[15])
      : "memory");
}
__device__ __forceinline__ void um_st16u(uint32_t a, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(a),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
// D (tensor memory) (+)= A (tensor memory: rows = lanes, two bf16 per 32-bit column) x B (shared); M = 128, K = 16
__device__ __forceinline__ void um_mma_ts(uint32_t d, uint32_t a_taddr, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile("{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p; }" ::"r"(d),
               "r"(a_taddr), "l"(bdesc), "r"(idesc), "r"(acc)
               : "memory");
}
__device__ __forceinline__ float pf_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// three-input maximum and packed pairs of fp32 (one instruction for two values)
__device__ __forceinline__ float pf_max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ uint64_t pf_pack2(float a, float b) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(a), "f"(b));
  return d;
}
__device__ __forceinline__ void pf_unpack2(uint64_t v, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v)); }
__device__ __forceinline__ uint64_t pf_fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t pf_add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

__global__ void __launch_bounds__(kPfThreads, 1) prefill_attention_kernel(PrefillArgs p, const __grid_constant__ CUtensorMap kmap,
                                                                          const __grid_constant__ CUtensorMap vmap) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned char* smem_al = smem_raw + ((1024u - (um_smem_u32(smem_raw) & 1023u)) & 1023u);
  PrefillSmem& S = *reinterpret_cast<PrefillSmem*>(smem_al);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // the longest query blocks (the last ones: most tiles under the diagonal) go first; the heads of one KV group are
  // neighbours in the grid, so that they read the same pages at about the same time
  const int heads = p.n_kv * p.gqa;
  const int qb = p.n_qblocks - 1 - (int)(blockIdx.x / (unsigned)(heads * p.n_seqs));
  const int rest = (int)(blockIdx.x % (unsigned)(heads * p.n_seqs));
  const int b = rest / heads, h = rest - b * heads;
  const int unit = b * p.n_kv + h / p.gqa;
  const int pos0 = p.pos0[b];
  const int i0 = qb * kPfRows;                             // first query of the block
  const int kv_len = pos0 + p.n_new;                       // reconstructed tokens of the sequence
  // queries of each group that exist, and the group's tiles: up to its last row's own position (group B may be empty)
  const int rows_a = min(kTile, p.n_new - i0), rows_b = max(0, min(kTile, p.n_new - i0 - kTile));
  const int nt_a = (pos0 + i0 + rows_a - 1) / kTile + 1;
  const int nt_b = rows_b > 0 ? (pos0 + i0 + kTile + rows_b - 1) / kTile + 1 : 0;
  const int n_tiles = max(nt_a, nt_b);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kPfSlots; s++) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(um_smem_u32(&S.full[s])) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(um_smem_u32(&S.free_[s])) : "memory");
    }
    for (int g = 0; g < 2; g++) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(um_smem_u32(&S.s_full[g])) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 4;" ::"r"(um_smem_u32(&S.p_full[g])) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(um_smem_u32(&S.pv_done[g])) : "memory");
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {                                         // warp 0 owns the tensor-memory allocation (512 columns)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(um_smem_u32(&S.tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // Q: every softmax thread copies its row into its group's K-major operand (rows past the chunk's end are zero)
  if (warp < 8) {
    const int g = warp >> 2, r = threadIdx.x & (kTile - 1);
    const int i = i0 + g * kTile + r;
    const uint4* src = reinterpret_cast<const uint4*>(p.q + (int64_t)b * p.q_stride_seq + (int64_t)i * p.q_stride_token +
                                                      (int64_t)h * p.q_stride_head);
#pragma unroll
    for (int c = 0; c < kD / 8; c++)
      *reinterpret_cast<uint4*>(&S.q[g][(c >> 3) * 16384 + r * 128 + (((c & 7) ^ (r & 7)) << 4)]) =
          i < p.n_new ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // Q: generic stores -> tensor-core reads
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tb = S.tmem_base;
  int status = 0;
  // ring item n (pf_item_k, pf_item_v) sits in slot n % kPfSlots, the slot's phase is (n / kPfSlots) & 1

  if (warp >= 8) {
    // the whole warpgroup 8..11 releases registers at one place; 2 x 4 x 232 + 4 x 40 = 12 x 168, the launch's allocation
    asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
  if (warp == 8) {
    // ------------------------------------------------------------------------------------------------ producer
    if (lane == 0) {
      bool ok = true;
#pragma unroll 1
      for (int n = 0; n <= 2 * n_tiles && ok; n++) {
        if (n == 2 * n_tiles - 1) continue;                  // would be the keys of a tile past the last one
        const bool is_v = n >= 2 && !(n & 1);
        const int j = is_v ? (n - 2) >> 1 : (n + 1) >> 1, s = n % kPfSlots;
        const int page = p.table ? p.table[(int64_t)unit * p.table_stride + j] : (int)(unit * p.table_stride + j);
        if (n >= kPfSlots) ok = um_wait(um_smem_u32(&S.free_[s]), (uint32_t)((n / kPfSlots - 1) & 1));
        if (!ok) break;
        const uint32_t bar = um_smem_u32(&S.full[s]), dst = um_smem_u32(S.kv[s]);
        const CUtensorMap* map = is_v ? &vmap : &kmap;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(kPfTileBytes) : "memory");
#pragma unroll 1
        for (int c = 0; c < 2; c++)                          // two blocks of 64 channels, 16 KB each
          asm volatile(
              "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
                  dst + 16384u * c),
              "l"(map), "r"(64 * c), "r"(0), "r"(page), "r"(bar)
              : "memory");
      }
      if (!ok) status |= SPECTRA_STATUS_WAIT_TIMEOUT;
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------------------------------------------ MMA issue
    if (lane == 0) {
      // the last group to use tile j (B whenever it has that tile: it never has fewer tiles than A) releases its slots
      auto last_user = [&](int j, int g) { return g == 1 || j >= nt_b; };
      auto wait_item = [&](int n) { return um_wait(um_smem_u32(&S.full[n % kPfSlots]), (uint32_t)((n / kPfSlots) & 1)); };
      auto issue_scores = [&](int j, int g) -> bool {
        if (!wait_item(pf_item_k(j))) return false;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t qaddr = um_smem_u32(S.q[g]), kaddr = um_smem_u32(S.kv[pf_item_k(j) % kPfSlots]);
        {   // descriptors once, then the eight k-steps back to back: the issuing thread's own instructions are what
            // bounds the MMA rate, so nothing but the low address word changes between them
          const uint64_t a0 = um_desc_sw128(qaddr, 16, 1024), b0 = um_desc_sw128(kaddr, 16, 1024);
#pragma unroll
          for (int ks = 0; ks < kD / 16; ks++) {
            const uint64_t off = (uint64_t)(1024 * (ks >> 2) + 2 * (ks & 3));
            um_mma_ss(tb + 128u * g, a0 + off, b0 + off, kPfIdescKK, ks != 0);
          }
        }
        um_commit(um_smem_u32(&S.s_full[g]));
        if (last_user(j, g)) um_commit(um_smem_u32(&S.free_[pf_item_k(j) % kPfSlots]));
        return true;
      };
      bool ok = issue_scores(0, 0);
      if (ok && nt_b > 0) ok = issue_scores(0, 1);
#pragma unroll 1
      for (int j = 0; j < n_tiles && ok; j++) {
#pragma unroll 1
        for (int g = 0; g < 2 && ok; g++) {
          if (j >= (g ? nt_b : nt_a)) continue;
          ok = um_wait(um_smem_u32(&S.p_full[g]), (uint32_t)(j & 1)) && wait_item(pf_item_v(j));
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t vaddr = um_smem_u32(S.kv[pf_item_v(j) % kPfSlots]);
          {
            const uint64_t b0 = um_desc_sw128(vaddr, 16384, 1024);
            const uint32_t d = tb + 256u + 128u * g, a0 = tb + 128u * g;
            um_mma_ts(d, a0, b0, kUmIdesc, j != 0);
#pragma unroll
            for (int ks = 1; ks < kTile / 16; ks++) um_mma_ts(d, a0 + 8u * ks, b0 + (uint64_t)(128 * ks), kUmIdesc, 1);
          }
          um_commit(um_smem_u32(&S.pv_done[g]));
          if (last_user(j, g)) um_commit(um_smem_u32(&S.free_[pf_item_v(j) % kPfSlots]));
          // the group's score buffer is free (p_full said so): its next scores go out behind this product
          if (j + 1 < (g ? nt_b : nt_a)) ok = issue_scores(j + 1, g);
        }
      }
      if (!ok) status |= SPECTRA_STATUS_WAIT_TIMEOUT;
    }
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 232;");
    // ------------------------------------------------------------------------------------------------ softmax
    const int g = warp >> 2, r = threadIdx.x & (kTile - 1);  // group, query row = tensor-memory lane
    const int rows = g ? rows_b : rows_a, nt = g ? nt_b : nt_a;
    const int ig = i0 + g * kTile;                           // first query of the group
    const uint32_t lane_base = tb + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t s_col = lane_base + 128u * g, o_col = lane_base + 256u + 128u * g;
    const int pos_row = pos0 + ig + min(r, max(rows, 1) - 1);   // rows past the end repeat the last one (never stored)
    float m_use = -INFINITY, l_sum = 0.f;
    bool ok = true;
    // the outcome of a wait is made uniform over the warp: the tensor-memory accesses below are warp-wide
    auto wait_w = [&](const uint64_t* bar, uint32_t parity) { return __all_sync(0xffffffffu, um_wait(um_smem_u32(bar), parity)) != 0; };
#pragma unroll 1
    for (int j = 0; j < nt && ok; j++) {
      const int tok0 = j * kTile;
      if (!wait_w(&S.s_full[g], (uint32_t)(j & 1))) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const bool masked = tok0 + kTile - 1 > pos0 + ig;     // some row of the group cannot see all of this tile
      const int visible = pos_row - tok0 + 1;               // tokens of this tile the row may see (can be <= 0)
      float s[kTile];
#pragma unroll
      for (int c = 0; c < kTile / 16; c++) um_ld16(s_col + 16 * c, s + 16 * c);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      if (masked) {
#pragma unroll
        for (int e = 0; e < kTile; e++) s[e] = e < visible ? s[e] : -INFINITY;
      }
      float mx8[8];
#pragma unroll
      for (int e = 0; e < 8; e++) mx8[e] = fmaxf(s[e], s[e + 8]);
#pragma unroll
      for (int e = 16; e < kTile; e += 16)
#pragma unroll
        for (int k = 0; k < 8; k++) mx8[k] = pf_max3(mx8[k], s[e + k], s[e + 8 + k]);
      const float mx_s = fmaxf(fmaxf(fmaxf(mx8[0], mx8[1]), fmaxf(mx8[2], mx8[3])),
                               fmaxf(fmaxf(mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7]))) * p.scale_log2;   // scale > 0
      // the tile's last tokens may lie past the reconstructed ones: whatever the page holds there must not reach the
      // product as a non-finite value (their probabilities are zero), so those rows of the V tile are cleared; each
      // group does it before it reports its P (both write the same zeros; the slot is not refilled before both
      // groups' products have been issued)
      if (tok0 + kTile > kv_len) {
        const int sv = pf_item_v(j) % kPfSlots;
        if (!wait_w(&S.full[sv], (uint32_t)((pf_item_v(j) / kPfSlots) & 1))) { ok = false; break; }
        if (tok0 + r >= kv_len) {
#pragma unroll
          for (int c = 0; c < kD / 8; c++)
            *reinterpret_cast<uint4*>(&S.kv[sv][(c >> 3) * 16384 + r * 128 + (c & 7) * 16]) = make_uint4(0, 0, 0, 0);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // cleared V rows: generic stores -> tensor-core reads
      }
      if (j > 0) {
        if (!wait_w(&S.pv_done[g], (uint32_t)((j - 1) & 1))) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      }
      // a new reference only when the old one is more than 2^8 too small (or there is none yet)
      const bool grow = mx_s > m_use + 8.f;
      if (__any_sync(0xffffffffu, grow)) {
        const float alpha = grow ? pf_exp2(m_use - mx_s) : 1.f;   // exp2(-inf) = 0 on the first tile
        if (j > 0) {
#pragma unroll 1
          for (int c = 0; c < 4; c++) {
            float o[32];
            um_ld16(o_col + 32 * c, o);
            um_ld16(o_col + 32 * c + 16, o + 16);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
            for (int e = 0; e < 32; e++) o[e] *= alpha;
            um_st16(o_col + 32 * c, o);
            um_st16(o_col + 32 * c + 16, o + 16);
          }
          asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        }
        if (grow) { l_sum *= alpha; m_use = mx_s; }
      }
      // probabilities relative to the reference (masked scores are -inf: zero) as bf16, two per column, over the scores
      uint64_t l2[4] = {0, 0, 0, 0};                          // four running pairs of partial sums
      const uint64_t scale2 = pf_pack2(p.scale_log2, p.scale_log2), negm2 = pf_pack2(-m_use, -m_use);
#pragma unroll
      for (int c = 0; c < kTile / 32; c++) {                 // 32 at a time: independent work for the pipes
        uint32_t w[16];
#pragma unroll
        for (int e2 = 0; e2 < 16; e2++) {
          float x0, x1;
          pf_unpack2(pf_fma2(pf_pack2(s[32 * c + 2 * e2], s[32 * c + 2 * e2 + 1]), scale2, negm2), x0, x1);
          x0 = pf_exp2(x0);
          x1 = pf_exp2(x1);
          l2[e2 & 3] = pf_add2(l2[e2 & 3], pf_pack2(x0, x1));
          const __nv_bfloat162 h2 = __floats2bfloat162_rn(x0, x1);
          w[e2] = *reinterpret_cast<const uint32_t*>(&h2);
        }
        um_st16u(s_col + 16 * c, w);
      }
      float l4[8];
#pragma unroll
      for (int k = 0; k < 4; k++) pf_unpack2(l2[k], l4[2 * k], l4[2 * k + 1]);
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      l_sum += ((l4[0] + l4[1]) + (l4[2] + l4[3])) + ((l4[4] + l4[5]) + (l4[6] + l4[7]));
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(um_smem_u32(&S.p_full[g])) : "memory");
    }
    // ---- the row's output: O / l, and lse = ln 2 * (m + log2 l)
    if (ok && nt > 0) ok = wait_w(&S.pv_done[g], (uint32_t)((nt - 1) & 1));
    if (ok && nt > 0) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const float inv = 1.f / l_sum;
      __nv_bfloat16* dst = p.out + (int64_t)b * p.o_stride_seq + (int64_t)(ig + r) * p.o_stride_token + (int64_t)h * p.o_stride_head;
#pragma unroll 1
      for (int c = 0; c < 4; c++) {
        float o[32];
        um_ld16(o_col + 32 * c, o);
        um_ld16(o_col + 32 * c + 16, o + 16);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (r < rows) {
#pragma unroll
          for (int e8 = 0; e8 < 4; e8++) {
            __nv_bfloat162 h2[4];
#pragma unroll
            for (int e2 = 0; e2 < 4; e2++) h2[e2] = __floats2bfloat162_rn(o[8 * e8 + 2 * e2] * inv, o[8 * e8 + 2 * e2 + 1] * inv);
            *reinterpret_cast<uint4*>(dst + 32 * c + 8 * e8) = *reinterpret_cast<const uint4*>(h2);
          }
        }
      }
      if (p.lse && r < rows) p.lse[((int64_t)b * p.n_new + ig + r) * heads + h] = 0.6931471805599453f * (m_use + log2f(l_sum));
    } else if (!ok) {
      status |= SPECTRA_STATUS_WAIT_TIMEOUT;
    }
  }
  // ---- the warp that allocated the tensor memory frees it
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(S.tmem_base), "r"(512u) : "memory");
  if (status && p.status) atomicOr(p.status, status);
}

}  // namespace spectra
