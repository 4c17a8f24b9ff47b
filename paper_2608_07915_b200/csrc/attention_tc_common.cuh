// Fused coded-cache decode attention on the tensor cores (mma.sync), scale_group 64; a unit of this path is a
// (sequence, kv-head, pass) triple, a pass being up to 4 query heads of the GQA group.
//
// Three kernels per call:
//   prep    (one CTA per unit)  folds W_dec,K and the softmax scale into the query (q'), turns it into
//           tensor-core B fragments per 16-strip chunk of the K tile, and lays out the per-unit descriptor;
//           one extra CTA builds the tile prefix sums and each warp's starting unit.  In a fused decode step the
//           same launch also carries one CTA per unit-side that appends the new token.
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
//   combine (one CTA per unit and head)  merges the records (log-sum-exp), folds strips back into channels, adds
//           the rotated mean and lifts the result once with W_dec,V.
//
// Codes enter the MMA as fp16 subnormals: a field masked in place inside its 16-bit half is code * 2^(p - 24)
// (p = its bit position), which the tensor core multiplies exactly; the power of two is folded into the B operand.
#pragma once
#include "attention_generic.cuh"
#include "encode_append.cuh"

namespace spectra {

constexpr int kFastGqa = 4;
constexpr int kKcMax = 40;       // upper bound of B-table entries of a K tile: 384 strips in 8 (class, group) runs, each
                                 // run rounded up to whole chunks of 16 strips and a group-1 run starting on an even strip
constexpr int kFastWarps = 4;    // warps per CTA of the main kernel
constexpr int kFastCtasPerSm = 4; // CTAs of the main kernel per SM its register budget is set for
constexpr int kRecHead = 4;      // floats of a record's per-head header: m, l, plo0, plo1
constexpr float kLog2e = 1.4426950408889634f;

struct alignas(16) UnitDesc {
  int32_t tbk, tbv;             // tile bytes (16 for a unit whose layout was refused: its copies stay harmless)
  int32_t kmeta[2], vmeta[2];   // byte offset of lo16[128] of scale group g (R16 256 bytes later), -1 if inactive
  uint32_t krun[2][4];          // K runs [scale group][class]: (byte offset of the first pair) / 16 | chunks << 16 |
                                // slot of a strip stored alone in the last chunk << 24 | (there is one) << 27
  uint32_t vcls[4];             // per V class: strips | strips of scale group 0 << 8 | (byte offset / 16) << 16
  uint32_t vfirst[4];           // index of the first V strip of each class
  int32_t n_vstrips, pad0;
  int64_t src_k, src_v;         // byte offset of the unit's first K / V tile from the cache base (0 if refused)
  float kscale[4];              // 2^-e_h
  float qlo[4][2];              // sum of q' over the active channels of a scale group
  float qconst[4];              // q' . m'_K (natural-log units)
  uint8_t vchan[kMaxStrips];    // channel of V strip k
  float vcoef[kMaxStrips];      // 2^24 * 2^shift / (2^width - 1): turns the strip's accumulator into its share of yhat
  uint4 kB[kKcMax][2][32];      // [chunk in walk order][MMAs {0,1} or {2,3}][lane] -> (b0, b1) of the two MMAs
};

struct FastArgs {
  UnitDesc* desc; int32_t* tile_prefix; int4* warp_start; float* records;
  int total_warps; int rec_stride; int vs_max;
  int n_units;       // units of the tensor path: (sequence, kv-head, pass); a pass takes up to 4 query heads of the group
  int npass;
  int depth; int slot_k, slot_v;
  int max_vblocks;   // V blocks of 16 strips whose accumulators fit the main kernel's tensor memory
};

// What the main kernel relies on for one unit, checked on the device against the widths the kernels actually read
// (the host sized the shared-memory slots and picked the kernel variant from its own copy of the widths): tiles fit
// their slots, the V blocks fit the tensor-memory columns of their accumulators, the B table fits, and both tile streams start on a
// 16-byte boundary (bulk copies).
__host__ __device__ inline bool fast_layout_ok(int tile_bytes_k, int tile_bytes_v, const int (&vblocks)[4],
                                               int k_entries, unsigned long long addr_k, unsigned long long addr_v,
                                               int slot_k, int slot_v, int max_vblocks) {
  bool ok = tile_bytes_k <= slot_k && tile_bytes_v <= slot_v && k_entries <= kKcMax;
  ok = ok && vblocks[0] + vblocks[1] + vblocks[2] + vblocks[3] <= max_vblocks;
  return ok && (addr_k & 15ull) == 0 && (addr_v & 15ull) == 0;
}

// ------------------------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// L2 policy for data that is read once (the coded tiles): first in line for eviction, so that the stream does not
// push out what the other kernels of the step re-read (parameters, descriptors, partial records).
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar), "l"(policy)
      : "memory");
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

// ------------------------------------------------------------------------------------------------ prep kernel
// These CTAs run once per call, on a cold instruction cache and with every global read paying a full memory latency.
// So: one group of reads issued together (W_dec,K by a bulk copy into shared memory; query, widths, rotated mean by plain loads
// issued together), rolled loops, all 512 threads in every phase.
struct PrepSmem {
  StripTable tk, tv;
  alignas(16) float qraw[kFastGqa][kD];
  alignas(16) float qrot[kFastGqa][kD];
  float mrot[kD];
  float kcoef[kMaxStrips];        // 2^shift / (2^width - 1) of K strip k
  __half bhi[kFastGqa][kMaxStrips];
  __half blo[kFastGqa][kMaxStrips];
  float red[4][kFastGqa][4];      // [quantity: max, q0, q1, qc][head][warp of the head's 128 threads]
  int scan[128];
  int ng0[2][4];                  // strips of scale group 0 per class: [K, V][class]
  alignas(8) unsigned long long wbar;
};
constexpr int kPrepDynSmem = kD * kD * 4 + (int)sizeof(PrepSmem);   // W_dec,K (or W_enc of an append CTA) first

__device__ inline uint32_t pack_cls(const StripTable& T, int c, int n_g0) {
  const int first = T.class_first[c], n = T.class_first[c + 1] - first;
  return (uint32_t)n | ((uint32_t)n_g0 << 8) | ((uint32_t)(T.class_off[c] / 16) << 16);
}

// Strips of class c whose channel lies in scale group 0 (channels < 64), counted by one warp.
__device__ inline int count_group0(const StripTable& T, int c, int lane) {
  int cnt = 0;
  for (int k = T.class_first[c] + lane; k < T.class_first[c + 1]; k += 32) cnt += T.chan[k] < 64;
#pragma unroll
  for (int s = 16; s; s >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, s);
  return cnt;
}

constexpr int kPrepThreads = 512;

// The work of CTA `bid` of the prep grid (f.n_units unit CTAs, then one CTA for the prefix sums).
__device__ inline void attention_prep_body(const AttnArgs& p, const FastArgs& f, int bid) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* s_w = reinterpret_cast<float*>(smem_raw);
  PrepSmem& S = *reinterpret_cast<PrepSmem*>(smem_raw + kD * kD * 4);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int kWarps = kPrepThreads / 32;
  if (bid == f.n_units) {
    // ---- tile prefix sums over units and each worker warp's first unit.  One round of global reads (the lengths);
    // counts, scan and the searches stay in shared memory when the call has at most 4096 units.
    const int n_units = f.n_units;
    __shared__ int sprefix[4097];          // units of one call; larger calls search the global copy
    const bool in_smem = n_units <= 4096;
    const int per = (n_units + 127) / 128;
    bool over = false;                     // a sequence longer than the buffers hold: reported, attended as empty
    if (in_smem) {
      for (int i = tid; i < n_units; i += kPrepThreads) {
        const int n = p.seq_len[(i / f.npass) / p.n_kv];
        over |= n > p.max_seq_len;
        sprefix[i + 1] = n > p.max_seq_len ? 0 : (n + kTile - 1) / kTile;
      }
      if (tid == 0) sprefix[0] = 0;
      __syncthreads();
      if (tid < 128) {
        int local = 0;
        for (int i = tid * per; i < min((tid + 1) * per, n_units); i++) local += sprefix[i + 1];
        S.scan[tid] = local;
      }
      __syncthreads();
      if (tid == 0) {
        int run = 0;
        for (int i = 0; i < 128; i++) { const int v = S.scan[i]; S.scan[i] = run; run += v; }
      }
      __syncthreads();
      if (tid < 128) {
        int run = S.scan[tid];
        for (int i = tid * per; i < min((tid + 1) * per, n_units); i++) { run += sprefix[i + 1]; sprefix[i + 1] = run; }
      }
      __syncthreads();
      for (int i = tid; i <= n_units; i += kPrepThreads) f.tile_prefix[i] = sprefix[i];
    } else {
      for (int b = tid; b < p.batch; b += kPrepThreads) over |= p.seq_len[b] > p.max_seq_len;
      int local = 0;
      if (tid < 128) {
        for (int i = tid * per; i < min((tid + 1) * per, n_units); i++) local += (attended_tokens(p, (i / f.npass) / p.n_kv) + kTile - 1) / kTile;
        S.scan[tid] = local;
      }
      __syncthreads();
      if (tid == 0) {
        int run = 0;
        for (int i = 0; i < 128; i++) { const int v = S.scan[i]; S.scan[i] = run; run += v; }
        f.tile_prefix[n_units] = run;
      }
      __syncthreads();
      if (tid < 128) {
        int run = S.scan[tid];
        for (int i = tid * per; i < min((tid + 1) * per, n_units); i++) {
          f.tile_prefix[i] = run;
          run += (attended_tokens(p, (i / f.npass) / p.n_kv) + kTile - 1) / kTile;
        }
      }
      __syncthreads();
      __threadfence_block();
    }
    if (over && p.status) atomicOr(p.status, SPECTRA_STATUS_CAPACITY);
    const int* pre = in_smem ? sprefix : f.tile_prefix;
    const long long total = pre[n_units];
    // each worker warp's share of the flattened tile space: first unit with a tile of the share, first tile inside
    // that unit, tiles of that unit, tiles of the share
    // floor(gw * total / W) without 64-bit divisions: total = q W + r, so it is gw q + floor(gw r / W); gw and r are
    // below 2^16 whenever W is (the grids of this library are), else the plain form is used
    const unsigned Wn = (unsigned)f.total_warps;
    const unsigned tq = (unsigned)(total / Wn), tr = (unsigned)(total % Wn);
    const bool small = Wn < 65536u;
    for (int gw = tid; gw < f.total_warps; gw += kPrepThreads) {
      long long g0, g1;
      if (small) {
        g0 = (long long)((unsigned)gw * tq) + ((unsigned)gw * tr) / Wn;
        g1 = (long long)((unsigned)(gw + 1) * tq) + ((unsigned)(gw + 1) * tr) / Wn;
      } else {
        g0 = (long long)gw * total / f.total_warps; g1 = (long long)(gw + 1) * total / f.total_warps;
      }
      int lo = 0, hi = n_units;             // first unit whose end is beyond g0
      while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (pre[mid + 1] > g0) hi = mid; else lo = mid + 1;
      }
      const int u0 = min(lo, n_units - 1);
      f.warp_start[gw] = make_int4(lo, (int)(g0 - pre[u0]), pre[u0 + 1] - pre[u0], (int)(g1 - g0));
    }
    return;
  }
  const int vu = bid;
  const int u = vu / f.npass, h0 = kFastGqa * (vu - u * f.npass);   // cache unit, first query head of this pass
  const int b = u / p.n_kv, hk = u - b * p.n_kv;
  const int ps = (int)(u % p.n_param_sets);
  const int G = min(kFastGqa, p.gqa - h0);                          // query heads of this pass
  // ---- all reads, issued together
  const int64_t off_k = p.off_k[u], off_v = p.off_v[u];             // used at the very end: fetched with the first group
  const uint32_t wbar = smem_u32(&S.wbar);
  if (tid == 0) {
    mbar_init(wbar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    mbar_expect_tx(wbar, kD * kD * 4);
    bulk_load(smem_u32(s_w), p.w_dec_k + (int64_t)ps * kD * kD, kD * kD * 4, wbar);
  }
  {
    const int h = tid >> 7, i = tid & (kD - 1);                     // 512 threads = 4 heads x 128 channels
    S.qraw[h][i] = h < G ? load_as_float(p.q, p.q_dtype, ((int64_t)b * p.n_q + hk * p.gqa + h0 + h) * kD + i) : 0.f;
    if (tid < kD) S.mrot[tid] = p.mean_rot_k ? p.mean_rot_k[(int64_t)ps * kD + tid] : 0.f;
  }
  build_strip_tables(S.tk, p.widths_k + (int64_t)ps * kD, S.tv, p.widths_v + (int64_t)ps * kD, 64);
  const StripTable& TK = S.tk;
  const StripTable& TV = S.tv;
  UnitDesc& D = f.desc[vu];
  const int nk = TK.n_strips;
  // ---- what depends on the widths only: strip coefficients, group-0 counts, the V side of the descriptor
  for (int k = tid; k < nk; k += kPrepThreads)
    S.kcoef[k] = (float)(1 << TK.shift[k]) / (float)((1 << TK.width[TK.chan[k]]) - 1);
  if (warp >= 8) {
    const int side = (warp - 8) >> 2, c = (warp - 8) & 3;
    const int cnt = count_group0(side ? TV : TK, c, lane);
    if (lane == 0) S.ng0[side][c] = cnt;
  }
  for (int k = tid; k < TV.n_strips; k += kPrepThreads) {
    const int c = TV.chan[k];
    D.vchan[k] = (uint8_t)c;
    D.vcoef[k] = 16777216.f * (float)(1 << TV.shift[k]) / (float)((1 << TV.width[c]) - 1);
  }
  // ---- q' = W_dec,K q (times the softmax scale, in the log2 domain).  A warp takes rows warp, warp + 16, .., two at
  // a time: each lane multiplies its four columns of the rows with the four heads, and a transposing butterfly leaves
  // every (row, head) sum in one lane after 9 shuffles instead of 40.
  const bool landed = mbar_wait(wbar, 0);
  if (!landed && tid == 0 && p.status) atomicOr(p.status, SPECTRA_STATUS_WAIT_TIMEOUT);
  {
    float4 qv[kFastGqa];
#pragma unroll
    for (int h = 0; h < kFastGqa; h++) qv[h] = *reinterpret_cast<const float4*>(&S.qraw[h][lane * 4]);
    const bool up16 = (lane & 16) != 0, up8 = (lane & 8) != 0, up4 = (lane & 4) != 0;
    const float out_scale = landed ? p.scale * kLog2e : 0.f;
#pragma unroll 1
    for (int row = warp; row < kD; row += 2 * kWarps) {
      const float4 wa = *reinterpret_cast<const float4*>(s_w + row * kD + lane * 4);
      const float4 wb = *reinterpret_cast<const float4*>(s_w + (row + kWarps) * kD + lane * 4);
      float pa[kFastGqa], pb[kFastGqa];
#pragma unroll
      for (int h = 0; h < kFastGqa; h++) {
        pa[h] = wa.x * qv[h].x + wa.y * qv[h].y + wa.z * qv[h].z + wa.w * qv[h].w;
        pb[h] = wb.x * qv[h].x + wb.y * qv[h].y + wb.z * qv[h].z + wb.w * qv[h].w;
      }
      // step 16 keeps heads {2 up16, 2 up16 + 1} of both rows, step 8 one head, step 4 one row
      const float a0 = (up16 ? pa[2] : pa[0]) + __shfl_xor_sync(0xffffffffu, up16 ? pa[0] : pa[2], 16);
      const float a1 = (up16 ? pa[3] : pa[1]) + __shfl_xor_sync(0xffffffffu, up16 ? pa[1] : pa[3], 16);
      const float b0 = (up16 ? pb[2] : pb[0]) + __shfl_xor_sync(0xffffffffu, up16 ? pb[0] : pb[2], 16);
      const float b1 = (up16 ? pb[3] : pb[1]) + __shfl_xor_sync(0xffffffffu, up16 ? pb[1] : pb[3], 16);
      const float ah = (up8 ? a1 : a0) + __shfl_xor_sync(0xffffffffu, up8 ? a0 : a1, 8);
      const float bh = (up8 ? b1 : b0) + __shfl_xor_sync(0xffffffffu, up8 ? b0 : b1, 8);
      float k = (up4 ? bh : ah) + __shfl_xor_sync(0xffffffffu, up4 ? ah : bh, 4);
      k += __shfl_xor_sync(0xffffffffu, k, 2);
      k += __shfl_xor_sync(0xffffffffu, k, 1);
      if ((lane & 3) == 0) S.qrot[2 * (int)up16 + (int)up8][row + (up4 ? kWarps : 0)] = k * out_scale;
    }
  }
  __syncthreads();
  // ---- per-head reductions, thread = (head, channel): largest |q' coef| over the strips (for the power-of-two
  // normalisation of the fp16 hi/lo split), sums of q' per scale group, q' . m'_K
  const int hh = tid >> 7, jj = tid & (kD - 1), wq = (tid >> 5) & 3;
  {
    float mx = 0.f;
    for (int k = jj; k < nk; k += kD) mx = fmaxf(mx, fabsf(S.qrot[hh][TK.chan[k]] * S.kcoef[k]));
    const float v = S.qrot[hh][jj];
    float q0 = (TK.width[jj] && jj < 64) ? v : 0.f, q1 = (TK.width[jj] && jj >= 64) ? v : 0.f, qc = v * S.mrot[jj];
#pragma unroll
    for (int s = 16; s; s >>= 1) {
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, s));
      q0 += __shfl_xor_sync(0xffffffffu, q0, s); q1 += __shfl_xor_sync(0xffffffffu, q1, s);
      qc += __shfl_xor_sync(0xffffffffu, qc, s);
    }
    if (lane == 0) { S.red[0][hh][wq] = mx; S.red[1][hh][wq] = q0; S.red[2][hh][wq] = q1; S.red[3][hh][wq] = qc; }
  }
  __syncthreads();
  {
    const float mx = fmaxf(fmaxf(S.red[0][hh][0], S.red[0][hh][1]), fmaxf(S.red[0][hh][2], S.red[0][hh][3]));
    int e = 0;
    if (mx > 0.f && mx <= 3.4028234e38f) e = 10 - ((int)((__float_as_uint(mx) >> 23) & 0xffu) - 126);   // mx = m 2^ex, m in [0.5, 1)
    e = max(-100, min(100, e));
    const float pow2e = __uint_as_float((uint32_t)(e + 127) << 23);
    if (jj == 0) {
      D.kscale[hh] = __uint_as_float((uint32_t)(24 - e + 127) << 23);
      D.qlo[hh][0] = (S.red[1][hh][0] + S.red[1][hh][1]) + (S.red[1][hh][2] + S.red[1][hh][3]);
      D.qlo[hh][1] = (S.red[2][hh][0] + S.red[2][hh][1]) + (S.red[2][hh][2] + S.red[2][hh][3]);
      D.qconst[hh] = ((S.red[3][hh][0] + S.red[3][hh][1]) + (S.red[3][hh][2] + S.red[3][hh][3])) / kLog2e;
    }
    for (int k = jj; k < nk; k += kD) {
      const float v = S.qrot[hh][TK.chan[k]] * S.kcoef[k] * pow2e;
      const __half hi = __float2half_rn(v);
      S.bhi[hh][k] = hi;
      S.blo[hh][k] = __float2half_rn(v - __half2float(hi));
    }
  }
  __syncthreads();
  // ---- B fragments.  The main kernel walks the K tile one scale group at a time and, inside a group, class by
  // class: run (g, c) covers the group's strips of class c in chunks of 16 strips (8 stored pairs).  The strips of
  // scale group 0 come first in a class, so its run starts at pair 0; the run of group 1 starts at the pair that
  // holds the class's first group-1 strip.  An entry's rows outside the run's group, or past the end of the class,
  // are zero.  Column n = head (n >> 1), hi (n & 1 == 0) or lo half of the fp16 split.  Variant u carries the factor
  // 2^-p_eff(u) of the unpacking.  Entries are stored in walk order.
  int ent_base[9], run_start[8];
  ent_base[0] = 0;
#pragma unroll
  for (int r = 0; r < 8; r++) {
    const int g = r >> 2, c = r & 3;
    const int n = TK.class_first[c + 1] - TK.class_first[c], n_g0 = S.ng0[0][c];
    const int sp = g ? (n_g0 >> 1) : 0;                                   // first pair of the run
    const int pairs = g ? (n > n_g0 ? ((n + 1) >> 1) - sp : 0) : ((n_g0 + 1) >> 1);
    run_start[r] = 2 * sp;
    ent_base[r + 1] = ent_base[r] + ((pairs + 7) >> 3);
  }
  const int n_entries = min(ent_base[8], kKcMax);
#pragma unroll 1
  for (int idx = tid; idx < n_entries * 4 * 32; idx += kPrepThreads) {
    const int en = idx >> 7, u4 = (idx >> 5) & 3, ln = idx & 31;
    int r = 0;
#pragma unroll
    for (int k = 1; k < 8; k++) r += en >= ent_base[k];
    int eb = 0, start = 0;
#pragma unroll
    for (int k = 0; k < 8; k++) if (k == r) { eb = ent_base[k]; start = run_start[k]; }
    const int g = r >> 2, c = r & 3;
    const int first = TK.class_first[c], n = TK.class_first[c + 1] - first, n_g0 = S.ng0[0][c];
    const int lo_s = g ? n_g0 : 0, hi_s = g ? n : n_g0;                   // strips of the class that belong to the run
    start += 16 * (en - eb);
    const int gid = ln >> 2, tg = ln & 3, h = gid >> 1, part = gid & 1;
    const int pe = c == 0 ? 0 : (c == 1 ? 4 * (u4 & 1) : (c == 2 ? 2 * u4 : u4));
    const __half scale = __ushort_as_half((unsigned short)((15 - pe) << 10));
    uint32_t rr[2];
#pragma unroll
    for (int half = 0; half < 2; half++) {
      uint32_t v = 0;
#pragma unroll
      for (int e = 0; e < 2; e++) {
        const int strip = start + 2 * tg + 8 * half + e;
        uint16_t bits = 0;
        if (strip >= lo_s && strip < hi_s && h < G)
          bits = __half_as_ushort(__hmul(part ? S.blo[h][first + strip] : S.bhi[h][first + strip], scale));
        v |= (uint32_t)bits << (16 * e);
      }
      rr[half] = v;
    }
    reinterpret_cast<uint2*>(&D.kB[en][u4 >> 1][ln])[u4 & 1] = make_uint2(rr[0], rr[1]);
  }
  if (tid < 8) {
    const int g = tid >> 2, c = tid & 3, w = 8 >> c;
    const int n = TK.class_first[c + 1] - TK.class_first[c], n_g0 = S.ng0[0][c];
    const int sp = g ? (n_g0 >> 1) : 0;
    const int pairs = g ? (n > n_g0 ? ((n + 1) >> 1) - sp : 0) : ((n_g0 + 1) >> 1);
    const int nch = (pairs + 7) >> 3;
    // a class with an odd number of strips stores its last strip alone; it belongs to the class's last run
    const bool lone = (n & 1) && pairs > 0 && (g ? true : n == n_g0);
    const int slot = lone ? (((n - 1) >> 1) - sp) & 7 : 0;
    D.krun[g][c] = (uint32_t)((TK.class_off[c] + 32 * w * sp) / 16) | ((uint32_t)nch << 16) | ((uint32_t)slot << 24) |
                   ((uint32_t)(lone ? 1 : 0) << 27);
  }
  if (tid >= 32 && tid < 36) {
    const int c = tid - 32;
    D.vcls[c] = pack_cls(TV, c, S.ng0[1][c]);
    D.vfirst[c] = TV.class_first[c];
  }
  // ---- the unit's layout against what the host assumed; a refused unit gets harmless copies and no work
  int vblocks[4];
#pragma unroll
  for (int c = 0; c < 4; c++) vblocks[c] = (TV.class_first[c + 1] - TV.class_first[c] + 15) >> 4;
  const unsigned long long addr_k = (unsigned long long)(p.cache_k + off_k), addr_v = (unsigned long long)(p.cache_v + off_v);
  const bool ok = fast_layout_ok(TK.tile_bytes, TV.tile_bytes, vblocks, ent_base[8], addr_k, addr_v, f.slot_k, f.slot_v, f.max_vblocks);
  if (tid == 64) {
    D.tbk = ok ? TK.tile_bytes : 16; D.tbv = ok ? TV.tile_bytes : 16;
    D.kmeta[0] = ok ? TK.meta_off[0] : -1; D.kmeta[1] = ok ? TK.meta_off[1] : -1;
    D.vmeta[0] = ok ? TV.meta_off[0] : -1; D.vmeta[1] = ok ? TV.meta_off[1] : -1;
    D.n_vstrips = ok ? TV.n_strips : 0; D.pad0 = 0;
    D.src_k = ok ? off_k : 0; D.src_v = ok ? off_v : 0;
    if (!ok && p.status) atomicOr(p.status, SPECTRA_STATUS_BAD_LAYOUT);
  }
  if (!ok) {
    __syncthreads();
    if (tid < 8) D.krun[tid >> 2][tid & 3] = 0;
    if (tid >= 32 && tid < 36) D.vcls[tid - 32] = 0;
  }
}

__global__ void __launch_bounds__(kPrepThreads) attention_prep_kernel(AttnArgs p, FastArgs f) {
  // the main kernel may be scheduled now: its set-up runs beside this grid, and it waits (griddepcontrol.wait) for this
  // grid's completion before it reads anything written here
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  attention_prep_body(p, f, blockIdx.x);
}

// First launch of a fused decode step: the prep grid, then one CTA per unit-side that appends the new token
// (the K side first).  The main kernel that follows reads what both parts wrote.
__global__ void __launch_bounds__(kPrepThreads, 2) decode_step_front_kernel(AttnArgs p, FastArgs f, AppendArgs ak,
                                                                         AppendArgs av, int n_cache_units) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // as in attention_prep_kernel
  const int n_prep = f.n_units + 1;
  if ((int)blockIdx.x < n_prep) { attention_prep_body(p, f, blockIdx.x); return; }
  const int i = blockIdx.x - n_prep;
  const AppendArgs& a = i < n_cache_units ? ak : av;
  const int u = i < n_cache_units ? i : i - n_cache_units;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  encode_append_body(a, u, smem_raw);
}

}  // namespace spectra
