// Many-query (prefill) causal attention over the reconstructed cache: Mode A of Sec. 3.3 (reconstruct, then attend)
// for a chunk of new queries.  The reconstructed keys and values sit in pools of bf16 pages of 128 tokens
// (spectra_decode_paged writes them); query i of a sequence is at position pos0 + i and attends tokens 0 .. pos0 + i.
//
// One CTA takes 256 consecutive queries of one query head as two groups of 128 rows (A, B) and walks the key/value
// tiles up to its diagonal; both groups use every tile that is brought in.  Both products run on the 5th-generation
// tensor cores with fp32 accumulators in tensor memory:
//   S = Q K^T       A = Q   [128 queries x 128 channels], K-major;  B = K tile [128 tokens x 128 channels], K-major
//   O += P V        A = P   [128 queries x 128 tokens],   K-major;  B = V tile [128 tokens x 128 channels], MN-major
// A page [token][channel] brought in by TMA as sixteen [128 tokens x 16 bytes] columns of core matrices is both
// layouts at once (K-major with the tokens as rows, MN-major with the tokens as the contraction index).
//
// Ten warps:
//   warps 0..3, 4..7  softmax of group A, B: thread r owns query row r of its group (= its tensor-memory lane): takes
//               its 128 scores into registers, keeps a running reference m and sum l, writes the probabilities as bf16
//               into the group's P operand, rescales its row of O when the reference moves (only when it grows by more
//               than 2^8: until then the old one is kept, which is exact as long as numerator and denominator use the
//               same one), and at the end divides and stores;
//   warp 8      (one lane) producer: TMA copies of the K and V tiles through one ring of three slots (K0 V0 K1 V1 ..);
//   warp 9      (one lane) issues the MMAs, group by group: P V of tile j, then the scores of tile j + 1, so that the
//               tensor cores work for one group while the other group's softmax runs.
// Tensor memory: columns 0..127 scores A, 128..255 scores B, 256..383 O of A, 384..511 O of B.
// Barriers (all waits bounded; a timeout sets SPECTRA_STATUS_WAIT_TIMEOUT and the waiter leaves its loop):
//   full[s], free[s]       ring slot s: the copies have landed / the last MMA that reads it is complete
//   s_full[g]              the scores of group g are complete
//   p_full[g]              the group's four warps have written P (and are done with the scores and with O)
//   pv_done[g]             the group's P V is complete: O is consistent, P may be overwritten
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

constexpr int kPfThreads = 320;
constexpr int kPfRows = 2 * kTile;                       // queries per CTA
constexpr uint32_t kPfTileBytes = kTile * kD * 2;
// bf16 A and B, fp32 D, both operands K-major (scores) / B MN-major (kUmIdesc: P V)
constexpr uint32_t kPfIdescKK = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

struct PrefillSmem {
  alignas(128) uint8_t q[2][kPfTileBytes];
  alignas(128) uint8_t kv[3][kPfTileBytes];
  alignas(128) uint8_t p[2][kPfTileBytes];
  alignas(8) uint64_t full[3], free_[3], s_full[2], p_full[2], pv_done[2];
  uint32_t tmem_base;
};
static_assert(sizeof(PrefillSmem) + 128 <= 227 * 1024, "the prefill kernel's shared memory must fit one SM");

__device__ __forceinline__ void um_st16(uint32_t a, const float* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(a),
      "f"(r[0]), "f"(r[1]), "f"(r[2]), "f"(r[3]), "f"(r[4]), "f"(r[5]), "f"(r[6]), "f"(r[7]), "f"(r[8]), "f"(r[9]),
      "f"(r[10]), "f"(r[11]), "f"(r[12]), "f"(r[13]), "f"(r[14]), "f"(r[15])
      : "memory");
}
__device__ __forceinline__ void um_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ float pf_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__global__ void __launch_bounds__(kPfThreads, 1) prefill_attention_kernel(PrefillArgs p, const __grid_constant__ CUtensorMap kmap,
                                                                          const __grid_constant__ CUtensorMap vmap) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned char* smem_al = smem_raw + ((128u - (um_smem_u32(smem_raw) & 127u)) & 127u);
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
    for (int s = 0; s < 3; s++) {
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
      *reinterpret_cast<uint4*>(&S.q[g][c * 2048 + r * 16]) = i < p.n_new ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // Q: generic stores -> tensor-core reads
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tb = S.tmem_base;
  int status = 0;
  // ring items: 2 j = K tile j, 2 j + 1 = V tile j; item n sits in slot n % 3, the slot's phase is (n / 3) & 1

  if (warp == 8) {
    // ------------------------------------------------------------------------------------------------ producer
    if (lane == 0) {
      bool ok = true;
#pragma unroll 1
      for (int n = 0; n < 2 * n_tiles && ok; n++) {
        const int j = n >> 1, s = n % 3;
        const int page = p.table ? p.table[(int64_t)unit * p.table_stride + j] : (int)(unit * p.table_stride + j);
        if (n >= 3) ok = um_wait(um_smem_u32(&S.free_[s]), (uint32_t)((n / 3 - 1) & 1));
        if (!ok) break;
        const uint32_t bar = um_smem_u32(&S.full[s]), dst = um_smem_u32(S.kv[s]);
        const CUtensorMap* map = (n & 1) ? &vmap : &kmap;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(kPfTileBytes) : "memory");
#pragma unroll 1
        for (int c = 0; c < kD / 8; c++)
          asm volatile(
              "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
                  dst + 2048u * c),
              "l"(map), "r"(8 * c), "r"(0), "r"(page), "r"(bar)
              : "memory");
      }
      if (!ok) status |= SPECTRA_STATUS_WAIT_TIMEOUT;
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------------------------------------------ MMA issue
    if (lane == 0) {
      // the last group to use tile j (B whenever it has that tile: it never has fewer tiles than A) releases its slots
      auto last_user = [&](int j, int g) { return g == 1 || j >= nt_b; };
      auto wait_item = [&](int n) { return um_wait(um_smem_u32(&S.full[n % 3]), (uint32_t)((n / 3) & 1)); };
      auto issue_scores = [&](int j, int g) -> bool {
        if (!wait_item(2 * j)) return false;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t qaddr = um_smem_u32(S.q[g]), kaddr = um_smem_u32(S.kv[(2 * j) % 3]);
#pragma unroll 1
        for (int ks = 0; ks < kD / 16; ks++)
          um_mma_ss(tb + 128u * g, um_desc(qaddr + 4096 * ks, 2048, 128), um_desc(kaddr + 4096 * ks, 2048, 128), kPfIdescKK,
                    ks != 0);
        um_commit(um_smem_u32(&S.s_full[g]));
        if (last_user(j, g)) um_commit(um_smem_u32(&S.free_[(2 * j) % 3]));
        return true;
      };
      bool ok = issue_scores(0, 0);
      if (ok && nt_b > 0) ok = issue_scores(0, 1);
#pragma unroll 1
      for (int j = 0; j < n_tiles && ok; j++) {
#pragma unroll 1
        for (int g = 0; g < 2 && ok; g++) {
          if (j >= (g ? nt_b : nt_a)) continue;
          ok = um_wait(um_smem_u32(&S.p_full[g]), (uint32_t)(j & 1)) && wait_item(2 * j + 1);
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t paddr = um_smem_u32(S.p[g]), vaddr = um_smem_u32(S.kv[(2 * j + 1) % 3]);
#pragma unroll 1
          for (int ks = 0; ks < kTile / 16; ks++)
            um_mma_ss(tb + 256u + 128u * g, um_desc(paddr + 4096 * ks, 2048, 128), um_desc(vaddr + 256 * ks, 128, 2048), kUmIdesc,
                      (j | ks) != 0);
          um_commit(um_smem_u32(&S.pv_done[g]));
          if (last_user(j, g)) um_commit(um_smem_u32(&S.free_[(2 * j + 1) % 3]));
          // the group's score buffer is free (p_full said so): its next scores go out behind this product
          if (j + 1 < (g ? nt_b : nt_a)) ok = issue_scores(j + 1, g);
        }
      }
      if (!ok) status |= SPECTRA_STATUS_WAIT_TIMEOUT;
    }
  } else {
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
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int e = 0; e < kTile; e++) mx4[e & 3] = fmaxf(mx4[e & 3], s[e]);
      const float mx_s = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;   // scale > 0
      // the tile's last tokens may lie past the reconstructed ones: whatever the page holds there must not reach the
      // product as a non-finite value (their probabilities are zero), so those rows of the V tile are cleared; each
      // group does it before it reports its P (both write the same zeros; the slot is not refilled before both
      // groups' products have been issued)
      if (tok0 + kTile > kv_len) {
        const int sv = (2 * j + 1) % 3;
        if (!wait_w(&S.full[sv], (uint32_t)(((2 * j + 1) / 3) & 1))) { ok = false; break; }
        if (tok0 + r >= kv_len) {
#pragma unroll
          for (int c = 0; c < kD / 8; c++) *reinterpret_cast<uint4*>(&S.kv[sv][c * 2048 + r * 16]) = make_uint4(0, 0, 0, 0);
        }
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
      // probabilities relative to the reference (masked scores are -inf: zero), as bf16 into the K-major P operand
      float l4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int e8 = 0; e8 < kTile / 8; e8++) {
        uint32_t w[4];
#pragma unroll
        for (int e2 = 0; e2 < 4; e2++) {
          const int e = 8 * e8 + 2 * e2;
          const float p0 = pf_exp2(fmaf(s[e], p.scale_log2, -m_use)), p1 = pf_exp2(fmaf(s[e + 1], p.scale_log2, -m_use));
          l4[e2] += p0 + p1;
          const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
          w[e2] = *reinterpret_cast<const uint32_t*>(&h2);
        }
        *reinterpret_cast<uint4*>(&S.p[g][e8 * 2048 + r * 16]) = make_uint4(w[0], w[1], w[2], w[3]);
      }
      l_sum += (l4[0] + l4[1]) + (l4[2] + l4[3]);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // P (and cleared V rows): generic stores -> tensor-core reads
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
