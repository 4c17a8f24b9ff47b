// Many-query (prefill) causal attention over the reconstructed cache: Mode A of Sec. 3.3 (reconstruct, then attend)
// for a chunk of new queries.  The reconstructed keys and values sit in pools of bf16 pages of 128 tokens
// (spectra_decode_paged writes them); query i of a sequence is at position pos0 + i and attends tokens 0 .. pos0 + i.
//
// One CTA takes 128 consecutive queries of one query head and walks the key/value tiles up to its diagonal.  Both
// products run on the 5th-generation tensor cores with fp32 accumulators in tensor memory:
//   S = Q K^T       A = Q   [128 queries x 128 channels], K-major;  B = K tile [128 tokens x 128 channels], K-major
//   O += P V        A = P   [128 queries x 128 tokens],   K-major;  B = V tile [128 tokens x 128 channels], MN-major
// A page [token][channel] brought in by TMA as sixteen [128 tokens x 16 bytes] columns of core matrices is both
// layouts at once (K-major with the tokens as rows, MN-major with the tokens as the contraction index).
//
// Six warps:
//   warps 0..3  softmax: thread r owns query row r (= its tensor-memory lane): reads its 128 scores, keeps a running
//               reference m and sum l, writes the probabilities as bf16 into the P operand, rescales its row of O when
//               the reference moves (only when it grows by more than 2^8: until then the old one is kept, which is exact
//               as long as numerator and denominator use the same one), and at the end divides and stores;
//   warp 4      (one lane) producer: TMA copies of the K and V tiles, two of each in flight;
//   warp 5      (one lane) issues the MMAs: S of tile j + 1 goes out before P V of tile j, so the tensor cores work on
//               the next scores while the softmax of the current tile runs (two score buffers in tensor memory).
// Barriers (all waits bounded; a timeout sets SPECTRA_STATUS_WAIT_TIMEOUT and the waiter leaves its loop):
//   k_full[s], v_full[s]   the tile's copies have landed in ring slot s
//   k_free[s], v_free[s]   the MMAs that read slot s are complete
//   s_full[b]              the scores in buffer b are complete
//   p_full                 the four softmax warps have written P (and are done with the score buffer and with O)
//   pv_done                P V of the tile is complete: O is consistent, P may be overwritten
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

constexpr int kPfThreads = 192;
constexpr uint32_t kPfTileBytes = kTile * kD * 2;
// bf16 A and B, fp32 D, both operands K-major (scores) / B MN-major (kUmIdesc: P V)
constexpr uint32_t kPfIdescKK = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

struct PrefillSmem {
  alignas(128) uint8_t q[kPfTileBytes];
  alignas(128) uint8_t k[2][kPfTileBytes];
  alignas(128) uint8_t v[2][kPfTileBytes];
  alignas(128) uint8_t p[kPfTileBytes];
  alignas(8) uint64_t k_full[2], v_full[2], k_free[2], v_free[2], s_full[2], p_full, pv_done;
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
  const int i0 = qb * kTile;                               // first query of the block
  const int rows = min(kTile, p.n_new - i0);               // queries of the block that exist
  const int kv_len = pos0 + p.n_new;                       // reconstructed tokens of the sequence
  const int n_tiles = (pos0 + i0 + rows - 1) / kTile + 1;  // tiles up to the last row's own position

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; s++) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(um_smem_u32(&S.k_full[s])) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(um_smem_u32(&S.v_full[s])) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(um_smem_u32(&S.k_free[s])) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(um_smem_u32(&S.v_free[s])) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(um_smem_u32(&S.s_full[s])) : "memory");
    }
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 4;" ::"r"(um_smem_u32(&S.p_full)) : "memory");
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(um_smem_u32(&S.pv_done)) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {                                         // warp 0 owns the tensor-memory allocation (512 columns)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(um_smem_u32(&S.tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // Q: thread r of the softmax warps copies its row into the K-major operand (rows past the chunk's end are zero)
  if (warp < 4) {
    const int r = threadIdx.x;
    const uint4* src = reinterpret_cast<const uint4*>(p.q + (int64_t)b * p.q_stride_seq + (int64_t)(i0 + r) * p.q_stride_token +
                                                      (int64_t)h * p.q_stride_head);
#pragma unroll
    for (int c = 0; c < kD / 8; c++)
      *reinterpret_cast<uint4*>(&S.q[c * 2048 + r * 16]) = r < rows ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // Q: generic stores -> tensor-core reads
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tb = S.tmem_base;                         // columns 0..127, 128..255: scores; 256..383: O
  int status = 0;

  if (warp == 4) {
    // ------------------------------------------------------------------------------------------------ producer
    if (lane == 0) {
      bool ok = true;
#pragma unroll 1
      for (int j = 0; j < n_tiles && ok; j++) {
        const int s = j & 1;
        const int page = p.table ? p.table[(int64_t)unit * p.table_stride + j] : (int)(unit * p.table_stride + j);
        if (j >= 2) ok = um_wait(um_smem_u32(&S.k_free[s]), (uint32_t)(((j >> 1) - 1) & 1));
        if (!ok) break;
        {
          const uint32_t bar = um_smem_u32(&S.k_full[s]), dst = um_smem_u32(S.k[s]);
          asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(kPfTileBytes) : "memory");
#pragma unroll 1
          for (int c = 0; c < kD / 8; c++)
            asm volatile(
                "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
                    dst + 2048u * c),
                "l"(&kmap), "r"(8 * c), "r"(0), "r"(page), "r"(bar)
                : "memory");
        }
        if (j >= 2) ok = um_wait(um_smem_u32(&S.v_free[s]), (uint32_t)(((j >> 1) - 1) & 1));
        if (!ok) break;
        {
          const uint32_t bar = um_smem_u32(&S.v_full[s]), dst = um_smem_u32(S.v[s]);
          asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(kPfTileBytes) : "memory");
#pragma unroll 1
          for (int c = 0; c < kD / 8; c++)
            asm volatile(
                "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
                    dst + 2048u * c),
                "l"(&vmap), "r"(8 * c), "r"(0), "r"(page), "r"(bar)
                : "memory");
        }
      }
      if (!ok) status |= SPECTRA_STATUS_WAIT_TIMEOUT;
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------------------------------------------ MMA issue
    if (lane == 0) {
      const uint32_t qaddr = um_smem_u32(S.q), paddr = um_smem_u32(S.p);
      auto issue_scores = [&](int j) -> bool {
        const int s = j & 1;
        if (!um_wait(um_smem_u32(&S.k_full[s]), (uint32_t)((j >> 1) & 1))) return false;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t kaddr = um_smem_u32(S.k[s]);
#pragma unroll 1
        for (int ks = 0; ks < kD / 16; ks++)
          um_mma_ss(tb + 128u * s, um_desc(qaddr + 4096 * ks, 2048, 128), um_desc(kaddr + 4096 * ks, 2048, 128), kPfIdescKK,
                    ks != 0);
        um_commit(um_smem_u32(&S.s_full[s]));
        um_commit(um_smem_u32(&S.k_free[s]));
        return true;
      };
      bool ok = issue_scores(0);
#pragma unroll 1
      for (int j = 0; j < n_tiles && ok; j++) {
        // the score buffer of tile j + 1 was last read by the softmax of tile j - 1, which p_full(j - 1) has reported
        if (j + 1 < n_tiles) ok = issue_scores(j + 1);
        if (!ok) break;
        ok = um_wait(um_smem_u32(&S.p_full), (uint32_t)(j & 1)) && um_wait(um_smem_u32(&S.v_full[j & 1]), (uint32_t)((j >> 1) & 1));
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t vaddr = um_smem_u32(S.v[j & 1]);
#pragma unroll 1
        for (int ks = 0; ks < kTile / 16; ks++)
          um_mma_ss(tb + 256u, um_desc(paddr + 4096 * ks, 2048, 128), um_desc(vaddr + 256 * ks, 128, 2048), kUmIdesc,
                    (j | ks) != 0);
        um_commit(um_smem_u32(&S.pv_done));
        um_commit(um_smem_u32(&S.v_free[j & 1]));
      }
      if (!ok) status |= SPECTRA_STATUS_WAIT_TIMEOUT;
    }
  } else {
    // ------------------------------------------------------------------------------------------------ softmax
    const int r = threadIdx.x;                              // query row = tensor-memory lane
    const uint32_t lane_base = tb + ((uint32_t)(warp * 32) << 16);
    const int pos_row = pos0 + i0 + min(r, rows - 1);       // rows past the end repeat the last one (never stored)
    float m_use = -INFINITY, l_sum = 0.f;
    bool ok = true;
    // the outcome of a wait is made uniform over the warp: the tensor-memory accesses below are warp-wide
    auto wait_w = [&](const uint64_t* bar, uint32_t parity) { return __all_sync(0xffffffffu, um_wait(um_smem_u32(bar), parity)) != 0; };
#pragma unroll 1
    for (int j = 0; j < n_tiles && ok; j++) {
      const int sb = j & 1;
      const int tok0 = j * kTile;
      if (!wait_w(&S.s_full[sb], (uint32_t)((j >> 1) & 1))) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const bool masked = tok0 + kTile - 1 > pos0 + i0;     // some row of the block cannot see all of this tile
      const int visible = pos_row - tok0 + 1;               // tokens of this tile the row may see (can be <= 0)
      // pass 1: the row's largest visible score
      float mx = -INFINITY;
#pragma unroll 1
      for (int c = 0; c < 4; c++) {
        float s[32];
        um_ld16(lane_base + 128u * sb + 32 * c, s);
        um_ld16(lane_base + 128u * sb + 32 * c + 16, s + 16);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (masked) {
#pragma unroll
          for (int e = 0; e < 32; e++) mx = fmaxf(mx, 32 * c + e < visible ? s[e] : -INFINITY);
        } else {
#pragma unroll
          for (int e = 0; e < 32; e++) mx = fmaxf(mx, s[e]);
        }
      }
      const float mx_s = mx * p.scale_log2;                 // scale > 0
      // the tile's last tokens may lie past the reconstructed ones: whatever the page holds there must not reach the
      // product as a non-finite value (their probabilities are zero), so those rows of the V tile are cleared
      if (tok0 + kTile > kv_len) {
        if (!wait_w(&S.v_full[sb], (uint32_t)((j >> 1) & 1))) { ok = false; break; }
        if (tok0 + r >= kv_len) {
#pragma unroll
          for (int c = 0; c < kD / 8; c++) *reinterpret_cast<uint4*>(&S.v[sb][c * 2048 + r * 16]) = make_uint4(0, 0, 0, 0);
        }
      }
      if (j > 0) {
        if (!wait_w(&S.pv_done, (uint32_t)((j - 1) & 1))) { ok = false; break; }
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
            um_ld16(lane_base + 256u + 32 * c, o);
            um_ld16(lane_base + 256u + 32 * c + 16, o + 16);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
            for (int e = 0; e < 32; e++) o[e] *= alpha;
            um_st16(lane_base + 256u + 32 * c, o);
            um_st16(lane_base + 256u + 32 * c + 16, o + 16);
          }
          asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        }
        if (grow) { l_sum *= alpha; m_use = mx_s; }
      }
      // pass 2: probabilities relative to the reference, as bf16 into the K-major P operand, and their sum
#pragma unroll 1
      for (int c = 0; c < 4; c++) {
        float s[32];
        um_ld16(lane_base + 128u * sb + 32 * c, s);
        um_ld16(lane_base + 128u * sb + 32 * c + 16, s + 16);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int e8 = 0; e8 < 4; e8++) {
          uint32_t w[4];
#pragma unroll
          for (int e2 = 0; e2 < 4; e2++) {
            const int e = 8 * e8 + 2 * e2;
            float p0 = pf_exp2(fmaf(s[e], p.scale_log2, -m_use)), p1 = pf_exp2(fmaf(s[e + 1], p.scale_log2, -m_use));
            if (masked) {
              p0 = 32 * c + e < visible ? p0 : 0.f;
              p1 = 32 * c + e + 1 < visible ? p1 : 0.f;
            }
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
            const float2 back = __bfloat1622float2(h2);     // the sum takes what the product will see
            l_sum += back.x + back.y;
            w[e2] = *reinterpret_cast<const uint32_t*>(&h2);
          }
          *reinterpret_cast<uint4*>(&S.p[(4 * c + e8) * 2048 + r * 16]) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // P (and cleared V rows): generic stores -> tensor-core reads
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(um_smem_u32(&S.p_full)) : "memory");
    }
    // ---- the row's output: O / l, and lse = ln 2 * (m + log2 l)
    if (ok) ok = wait_w(&S.pv_done, (uint32_t)((n_tiles - 1) & 1));
    if (ok) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const float inv = 1.f / l_sum;
      __nv_bfloat16* dst = p.out + (int64_t)b * p.o_stride_seq + (int64_t)(i0 + r) * p.o_stride_token + (int64_t)h * p.o_stride_head;
#pragma unroll 1
      for (int c = 0; c < 4; c++) {
        float o[32];
        um_ld16(lane_base + 256u + 32 * c, o);
        um_ld16(lane_base + 256u + 32 * c + 16, o + 16);
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
      if (p.lse && r < rows) p.lse[((int64_t)b * p.n_new + i0 + r) * heads + h] = 0.6931471805599453f * (m_use + log2f(l_sum));
    } else {
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
