// Fused coded-cache decode attention on the 5th-generation tensor cores (tcgen05, operands in tensor memory),
// for GQA groups of up to 4 query heads and scale_group 64.
//
// Three kernels per call:
//   prep    (one CTA per unit)  folds W_dec,K and the softmax scale into the query (q'), builds the unit's plan:
//           how a thread turns the 32-bit words of a K token string into operand registers (masks per word), the
//           matching B operand of q' (fp16 hi/lo split, pre-scaled per k-slot), the row of every V strip; one extra
//           CTA builds the tile prefix sums and each worker's first unit.
//   main    persistent, one CTA per SM = one worker over an equal contiguous range of the flattened (unit, tile)
//           space.  Warp roles: a producer streams K and V tiles into a shared-memory ring with 1-D bulk copies;
//           four "token" warps (thread = token) unpack K token strings into the A operand of the score MMA in tensor
//           memory, read the scores back, run the online softmax and write the probabilities (times the V group
//           ranges) as the B operand of the value MMA; six "strip" warps (thread = V strip) unpack V strips into
//           the A operand of the value MMA; five issuer warps feed tcgen05.mma.  Accumulators of the rotated value
//           space stay in tensor memory for the whole pass over a unit.
//   combine (one CTA per unit and head)  merges the workers' partial records (log-sum-exp), folds strips back into
//           channels, adds the rotated mean and lifts the result once with W_dec,V.
//
// Unpacking costs one logic operation per operand register (two codes): a code masked in place is the fp16
// subnormal code * 2^(p-24) (p = its bit position inside the 16-bit half), which the tensor core multiplies
// exactly; the position-dependent power of two is folded into the B operand.  A field is usable in place when it
// lies inside bits [0, 10) of its half; the others are reached through one shift of the word by 6.
#pragma once
#include "attention_generic.cuh"

namespace spectra {

constexpr int kFastGqa = 4;
constexpr int kRecHead = 4;        // floats of a record's per-head header: m, l, plo0, plo1
constexpr float kLog2e = 1.4426950408889634f;

constexpr int kKWordsMax = 16;     // 32-bit words of a K token string (remainder word included) on this path
constexpr int kKColsMax = 112;     // tensor-memory columns of the score MMA's A operand
constexpr int kKStepsMax = kKColsMax / 8;
constexpr int kVRowsMax = 192;     // V strips (accumulator rows): six strip warps
constexpr int kVGroupsMax = 3;     // (row block of 128, class) pairs
constexpr int kVSetsMax = 5;       // accumulator column sets: (issuer, group) pairs
constexpr int kVIssuers = 3;
constexpr int kNcols = 16;         // MMA N: head (4) x scale group (2) x {hi, lo}

// Slots of a word shape: (unshifted, shifted) extraction slots; a word uses the smallest shape that holds it.
__host__ __device__ constexpr int shape_u(int s) { return s == 0 ? 1 : s == 1 ? 2 : s == 2 ? 5 : 10; }
__host__ __device__ constexpr int shape_s(int s) { return s == 0 ? 1 : s == 1 ? 2 : s == 2 ? 3 : 6; }
__host__ __device__ constexpr int shape_slots(int s) { return 2 << s; }   // 2, 4, 8, 16

// ---- plans, as plain functions of the class boundaries (shared by the host eligibility check and the prep kernel)
// cfirst[c] = index of the first strip of class c (w = 8 >> c), cfirst[4] = number of strips.

// One field of a K word: strip, width, position inside its 16-bit half.
struct KField { int strip, w, p; };

// Fields of half `hf` of word i of a token string of B bits; returns their number (at most 16).
__host__ __device__ inline int k_half_fields(const int* cfirst, int B, int i, int hf, KField* out) {
  const int lo = 32 * i + 16 * hf;
  const int hi = lo + 16 < B ? lo + 16 : B;
  int n = 0, cb = 0;
  for (int c = 0; c < 4; c++) {
    const int w = 8 >> c;
    const int ce = cb + (cfirst[c + 1] - cfirst[c]) * w;
    const int o0 = lo > cb ? lo : cb, o1 = hi < ce ? hi : ce;
    for (int o = o0; o < o1; o += w) { out[n].strip = cfirst[c] + (o - cb) / w; out[n].w = w; out[n].p = o - lo; n++; }
    cb = ce;
  }
  return n;
}

// Shape of word i: counts the unshifted (p + w <= 10) and shifted fields of both halves.
__host__ __device__ inline int k_word_shape(const int* cfirst, int B, int i) {
  KField f[16];
  int nu = 0, ns = 0;
  for (int hf = 0; hf < 2; hf++) {
    const int n = k_half_fields(cfirst, B, i, hf, f);
    int u = 0;
    for (int e = 0; e < n; e++) u += f[e].p + f[e].w <= 10;
    nu = u > nu ? u : nu;
    ns = n - u > ns ? n - u : ns;
  }
  for (int s = 0; s < 3; s++)
    if (nu <= shape_u(s) && ns <= shape_s(s)) return s;
  return 3;
}

// Rows of the V strips: class by class; a class that would straddle a 128-row block and fits in one starts at the
// next block, unless that needs more than kVRowsMax rows (then rows = strips).  Returns the number of rows used.
__host__ __device__ inline int v_row_plan(const int* cfirst, int* row_first /*[4]*/) {
  int row = 0;
  for (int c = 0; c < 4; c++) {
    const int n = cfirst[c + 1] - cfirst[c];
    if (n > 0 && n <= 128 && (row & 127) + n > 128) row = (row + 127) & ~127;
    row_first[c] = row;
    row += n;
  }
  if (row > kVRowsMax) {
    for (int c = 0; c < 4; c++) row_first[c] = cfirst[c];
    row = cfirst[4];
  }
  return row;
}

// (row block, class) groups in class order; returns their number (may exceed kVGroupsMax: caller checks).
__host__ __device__ inline int v_groups(const int* cfirst, const int* row_first, int* grp /*[8]: rb | class << 8*/) {
  int n = 0;
  for (int c = 0; c < 4; c++) {
    const int cnt = cfirst[c + 1] - cfirst[c];
    if (!cnt) continue;
    for (int rb = row_first[c] >> 7; rb <= (row_first[c] + cnt - 1) >> 7; rb++) grp[n++] = rb | (c << 8);
  }
  return n;
}

// Value-MMA jobs are (group, k-step) pairs in group order, 8 per group, cut into kVIssuers contiguous slices; an
// accumulator column set belongs to one (issuer, group) pair.  Fills set_group[] / set_issuer[], returns the count.
__host__ __device__ inline int v_sets(int n_groups, int* set_group, int* set_issuer) {
  const int J = 8 * n_groups;
  int n = 0;
  for (int j = 0; j < kVIssuers; j++) {
    const int a = j * J / kVIssuers, b = (j + 1) * J / kVIssuers;
    for (int g = 0; g < n_groups; g++)
      if (a < 8 * g + 8 && b > 8 * g && a < b) { set_group[n] = g; set_issuer[n] = j; n++; }
  }
  return n;
}

// Per-unit context of the main kernel (built by prep in global memory, copied whole into shared memory).
struct alignas(128) UnitCtx {
  alignas(128) uint8_t kb[kKStepsMax * 512];  // B operand of the score MMA: per k-step a 16 (N) x 16 (K) fp16 tile
  uint32_t kmask[kKWordsMax][16];             // extraction masks per word: unshifted slots, then shifted slots
  uint32_t vrow[256];        // per row: (byte offset of the strip / 16) | class << 12 | strip << 16 | scale group << 30 | 1 << 31
  uint8_t kshape[kKWordsMax];
  uint8_t kcol[kKWordsMax];  // first operand column of the word
  int32_t tbk, tbv;
  int32_t kmeta[2], vmeta[2];
  int32_t k_full, k_rem, k_words, k_cols, k_steps;
  int32_t n_vstrips, n_vrows, n_vgroups;
  int32_t vgroup[4];         // row block | class << 8
  float kscale[4];           // 2^(24 - e_h)
  float qlo[4][2];           // sum of q' over the active channels of a scale group
  int32_t pad[2];
};
static_assert(sizeof(UnitCtx) % 128 == 0, "bulk copy size");

// What the combine kernel needs of a unit.
struct alignas(16) UnitDesc {
  int32_t n_vstrips, pad0[3];
  float qconst[4];              // q' . m'_K (natural-log units)
  uint8_t vchan[kMaxStrips];    // channel of V strip k
  float vcoef[kMaxStrips];      // 2^24 * 2^shift / (2^width - 1): turns the strip's accumulator into its share of yhat
};

struct FastArgs {
  UnitCtx* ctx; UnitDesc* desc; int32_t* tile_prefix; int32_t* worker_unit; float* records;
  int total_warps;   // number of workers (CTAs of the main kernel)
  int rec_stride; int vs_max; int n_units;
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
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void named_barrier(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ uint32_t redux_max_u32(uint32_t v) {
  uint32_t r;
  asm volatile("redux.sync.max.u32 %0, %1, 0xffffffff;" : "=r"(r) : "r"(v));
  return r;
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
__device__ __forceinline__ uint4 lds128(uint32_t a) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ void sts128(uint32_t a, uint4 v) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// ---- tensor memory and tcgen05
__device__ __forceinline__ void tmem_alloc(uint32_t result_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(result_smem), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t base, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D (tensor memory) (+)= A (tensor memory) x B (shared memory descriptor), M = 128, K = 16, fp16 in, fp32 out.
__device__ __forceinline__ void tc_mma(uint32_t d, uint32_t a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p; }" ::"r"(d),
               "r"(a), "l"(bdesc), "r"(idesc), "r"(accumulate)
               : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_st2(uint32_t a, uint32_t r0, uint32_t r1) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x2.b32 [%0], {%1,%2};" ::"r"(a), "r"(r0), "r"(r1) : "memory");
}
__device__ __forceinline__ void tc_st4(uint32_t a, const uint32_t* r) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(r[0]), "r"(r[1]), "r"(r[2]),
               "r"(r[3])
               : "memory");
}
__device__ __forceinline__ void tc_st8(uint32_t a, const uint32_t* r) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(a), "r"(r[0]), "r"(r[1]),
               "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t a, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(a),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t a, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(a)
      : "memory");
}
// Shared-memory operand descriptor, no swizzle: start address, leading and stride byte offsets (16-byte units).
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((saddr >> 4) & 0x3FFF) | ((uint64_t)((lbo >> 4) & 0x3FFF) << 16) |
         ((uint64_t)((sbo >> 4) & 0x3FFF) << 32) | ((uint64_t)1 << 46);
}
// Instruction descriptor: fp16 A and B, fp32 D, M = 128, N = kNcols; bit 16 set = B is MN-major.
constexpr uint32_t kIdescKMajor = (1u << 4) | ((uint32_t)(kNcols >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescMnMajor = kIdescKMajor | (1u << 16);

// ------------------------------------------------------------------------------------------------ prep kernel
struct PrepSmem {
  StripTable tk, tv;
  alignas(16) float qraw[kFastGqa][kD];
  alignas(16) float qrot[kFastGqa][kD];
  int escale[kFastGqa];
  int scan[128];
  int16_t slot_strip[kKWordsMax][16][2];   // strip of (word, slot, half), -1 if none
  uint8_t slot_peff[kKWordsMax][16][2];    // effective bit position of the field inside its half
  int kcol[kKWordsMax + 1];
};

constexpr int kPrepThreads = 512;

__global__ void __launch_bounds__(kPrepThreads) attention_prep_kernel(AttnArgs p, FastArgs f) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  PrepSmem& S = *reinterpret_cast<PrepSmem*>(smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int kWarps = kPrepThreads / 32;
  if ((int)blockIdx.x == f.n_units) {
    // ---- tile prefix sums over units and each worker's first unit
    const int n_units = f.n_units;
    const int per = (n_units + 127) / 128;
    int local = 0;
    if (tid < 128) {
      for (int i = tid * per; i < min((tid + 1) * per, n_units); i++) local += (p.seq_len[i / p.n_kv] + kTile - 1) / kTile;
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
        run += (p.seq_len[i / p.n_kv] + kTile - 1) / kTile;
      }
    }
    __syncthreads();
    __threadfence_block();
    __shared__ int sprefix[4097];          // units of one call; larger calls search the global copy
    const bool in_smem = n_units <= 4096;
    if (in_smem)
      for (int i = tid; i <= n_units; i += kPrepThreads) sprefix[i] = f.tile_prefix[i];
    __syncthreads();
    const int* pre = in_smem ? sprefix : f.tile_prefix;
    const long long total = pre[n_units];
    for (int gw = tid; gw < f.total_warps; gw += kPrepThreads) {
      const long long g0 = (long long)gw * total / f.total_warps;
      int lo = 0, hi = n_units;             // first unit whose end is beyond g0
      while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (pre[mid + 1] > g0) hi = mid; else lo = mid + 1;
      }
      f.worker_unit[gw] = lo;
    }
    return;
  }
  const int u = blockIdx.x;
  const int b = u / p.n_kv, hk = u - b * p.n_kv;
  const int ps = (int)(u % p.n_param_sets);
  const int G = p.gqa;
  build_strip_tables(S.tk, p.widths_k + (int64_t)ps * kD, S.tv, p.widths_v + (int64_t)ps * kD, 64);
  const StripTable& TK = S.tk;
  const StripTable& TV = S.tv;
  UnitCtx& C = f.ctx[u];
  UnitDesc& D = f.desc[u];
  for (int idx = tid; idx < kFastGqa * kD; idx += kPrepThreads) {
    const int h = idx / kD, i = idx - h * kD;
    S.qraw[h][i] = h < G ? load_as_float(p.q, p.q_dtype, ((int64_t)b * p.n_q + hk * G + h) * kD + i) : 0.f;
  }
  // zero the B operand and the mask table while the query is staged
  for (int i = tid; i < (int)sizeof(C.kb) / 16; i += kPrepThreads) reinterpret_cast<uint4*>(C.kb)[i] = make_uint4(0, 0, 0, 0);
  for (int i = tid; i < kKWordsMax * 16; i += kPrepThreads) (&C.kmask[0][0])[i] = 0u;
  for (int i = tid; i < kKWordsMax * 16 * 2; i += kPrepThreads) (&S.slot_strip[0][0][0])[i] = -1;
  __syncthreads();
  const float* wk = p.w_dec_k + (int64_t)ps * kD * kD;
  for (int j = warp; j < kD; j += kWarps) {
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
  // ---- K plan: one thread per word (warp 15 .. so that it overlaps the query fold of the other warps' tail)
  const int B = string_bits(TK), F = B >> 5, r = B & 31;
  const int n_words = F + (r ? 1 : 0);
  if (tid < n_words && tid < kKWordsMax) {
    const int i = tid;
    const int shape = k_word_shape(TK.class_first, B, i);
    C.kshape[i] = (uint8_t)shape;
    S.kcol[i + 1] = shape_slots(shape);
    KField fl[16];
    for (int hf = 0; hf < 2; hf++) {
      const int n = k_half_fields(TK.class_first, B, i, hf, fl);
      int nu = 0, ns = 0;
      for (int e = 0; e < n; e++) {
        const bool unshifted = fl[e].p + fl[e].w <= 10;
        const int slot = unshifted ? nu++ : shape_u(shape) + ns++;
        const int pe = unshifted ? fl[e].p : fl[e].p - 6;
        S.slot_strip[i][slot][hf] = (int16_t)fl[e].strip;
        S.slot_peff[i][slot][hf] = (uint8_t)pe;
        C.kmask[i][slot] |= (((1u << fl[e].w) - 1u) << pe) << (16 * hf);   // each (word, slot) is written by this thread only
      }
    }
  }
  __syncthreads();
  if (tid == 0) {
    int col = 0;
    for (int i = 0; i < n_words && i < kKWordsMax; i++) { const int n = S.kcol[i + 1]; S.kcol[i] = col; C.kcol[i] = (uint8_t)col; col += n; }
    C.k_full = F; C.k_rem = r; C.k_words = n_words; C.k_cols = col; C.k_steps = (col + 7) / 8;
    C.tbk = TK.tile_bytes; C.tbv = TV.tile_bytes;
    C.kmeta[0] = TK.meta_off[0]; C.kmeta[1] = TK.meta_off[1];
    C.vmeta[0] = TV.meta_off[0]; C.vmeta[1] = TV.meta_off[1];
    C.n_vstrips = TV.n_strips; D.n_vstrips = TV.n_strips;
    int row_first[4], grp[8];
    C.n_vrows = v_row_plan(TV.class_first, row_first);
    const int ng = v_groups(TV.class_first, row_first, grp);
    C.n_vgroups = ng;
    for (int g = 0; g < 4; g++) C.vgroup[g] = g < ng ? grp[g] : 0;
    S.scan[0] = row_first[0]; S.scan[1] = row_first[1]; S.scan[2] = row_first[2]; S.scan[3] = row_first[3];
  }
  // per-head power-of-two normalisation so that the fp16 hi/lo split of the B operand is well conditioned
  const int nk = TK.n_strips;
  if (warp < kFastGqa) {
    const int h = warp;  // one warp per head
    float mx = 0.f;
    for (int k = lane; k < nk; k += 32) {
      const int c = TK.chan[k];
      mx = fmaxf(mx, fabsf(S.qrot[h][c] * (float)(1 << TK.shift[k]) / (float)((1 << TK.width[c]) - 1)));
    }
#pragma unroll
    for (int s = 16; s; s >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, s));
    int e = 0;
    if (mx > 0.f && isfinite(mx)) { int ex; frexpf(mx, &ex); e = 14 - ex; }
    e = max(-100, min(100, e));
    if (lane == 0) { S.escale[h] = e; C.kscale[h] = ldexpf(1.f, 24 - e); }
    float q0 = 0.f, q1 = 0.f, qc = 0.f;
    for (int j = lane; j < kD; j += 32) {
      const float v = S.qrot[h][j];
      if (TK.width[j]) { if (j < 64) q0 += v; else q1 += v; }
      if (p.mean_rot_k) qc += v * p.mean_rot_k[(int64_t)ps * kD + j];
    }
#pragma unroll
    for (int s = 16; s; s >>= 1) {
      q0 += __shfl_xor_sync(0xffffffffu, q0, s); q1 += __shfl_xor_sync(0xffffffffu, q1, s);
      qc += __shfl_xor_sync(0xffffffffu, qc, s);
    }
    if (lane == 0) { C.qlo[h][0] = q0; C.qlo[h][1] = q1; D.qconst[h] = qc / kLog2e; }
  }
  __syncthreads();
  // ---- B operand of the score MMA.  k-slot (column, half) holds one field; its row carries, for head h and the
  // field's scale group g, q'_h[chan] 2^shift / (2^b - 1) 2^(e_h - p_eff) as an fp16 hi/lo pair in columns
  // n = 4 h + 2 g + {0, 1}; the other group's columns stay zero.  Per k-step (8 columns = 16 k) the tile is 16 x 16,
  // K-major, no swizzle: core (n >> 3, k >> 3) at ((n >> 3) * 2 + (k >> 3)) * 128, row n & 7 at 16 B, k & 7 at 2 B.
  for (int idx = tid; idx < kKWordsMax * 16 * 2 * kFastGqa; idx += kPrepThreads) {
    const int h = idx & 3, hf = (idx >> 2) & 1, slot = (idx >> 3) & 15, i = idx >> 7;
    const int k = i < n_words ? S.slot_strip[i][slot][hf] : -1;
    if (k < 0 || h >= G) continue;
    const int c = TK.chan[k];
    const float v = ldexpf(S.qrot[h][c] * (float)(1 << TK.shift[k]) / (float)((1 << TK.width[c]) - 1),
                           S.escale[h] - (int)S.slot_peff[i][slot][hf]);
    const __half hi = __float2half_rn(v);
    const __half lo = __float2half_rn(v - __half2float(hi));
    const int col = S.kcol[i] + slot;
    const int kk = 2 * (col & 7) + hf, n0 = 4 * h + 2 * (c >> 6);
    uint8_t* tile = C.kb + (col >> 3) * 512;
    *reinterpret_cast<__half*>(tile + ((n0 >> 3) * 2 + (kk >> 3)) * 128 + (n0 & 7) * 16 + (kk & 7) * 2) = hi;
    *reinterpret_cast<__half*>(tile + (((n0 + 1) >> 3) * 2 + (kk >> 3)) * 128 + ((n0 + 1) & 7) * 16 + (kk & 7) * 2) = lo;
  }
  // ---- V rows and what the combine kernel needs
  for (int i = tid; i < 256; i += kPrepThreads) C.vrow[i] = 0u;
  __syncthreads();
  for (int k = tid; k < TV.n_strips; k += kPrepThreads) {
    const int cls = strip_class(TV, k);
    const int c = TV.chan[k];
    const int row = S.scan[cls] + (k - TV.class_first[cls]);
    const int off = TV.class_off[cls] + 16 * (8 >> cls) * (k - TV.class_first[cls]);
    if (row < 256) C.vrow[row] = (uint32_t)(off >> 4) | ((uint32_t)cls << 12) | ((uint32_t)k << 16) | ((uint32_t)(c >> 6) << 30) | 0x80000000u;
    D.vchan[k] = (uint8_t)c;
    D.vcoef[k] = 16777216.f * (float)(1 << TV.shift[k]) / (float)((1 << TV.width[c]) - 1);
  }
}

}  // namespace spectra
