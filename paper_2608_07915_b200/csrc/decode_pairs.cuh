// Fast reconstruction path of spectra_decode: the regrouping of decode_runs.cuh
//     xhat_t = sum_g R_g(t) [ sum_{strips k of group g} field_tk W''_k ] + sum_g lo_g(t) u_g + c
// with the bracket as one tcgen05 product per scale group.  The A operand [128 tokens x K] holds the packed fields
// themselves as fp16 numbers (a field shifted to bit 0 and masked is the subnormal field * 2^-24, which the tensor
// core multiplies exactly): a worker thread takes one token and one pair of strips (K side: the 32-bit word of the
// tile already holds both halves) and turns it into a 32-bit store of the K-major operand with one load, one shift
// and one mask.  No code is assembled, dequantised or split into parts.  B = W'' scaled by a power of two and split
// into two fp16 parts (hi + lo: 22 bits; a single fp16 part left errors of 1e-3 of a vector's largest entry), rows in
// the order of the (group, class) runs, zero where a row belongs to another group or lies past its class.
// Per tile: 2 n_ksteps MMAs of 128 x 128 x 16 into one accumulator tile per group; the epilogue (thread = token and 64
// channels) reads both, scales by the token's group ranges and adds the offset terms in fp32.
//
// Persistent CTAs over (unit, tile) slots; two buffers (packed tile, operand, accumulators, metadata) alternate between
// consecutive tiles.  Warps 0..7 build operands, tile after tile; warp 16 (one lane) copies the packed tiles in and
// issues the MMAs; warps 8..15 run the epilogues: no role waits for another longer than the slowest of them needs
// per tile.  Barriers per buffer (bounded waits): raw_full, a_full (operand and metadata written), acc_full (MMAs
// complete: accumulators ready, operand free), acc_free (epilogue done: accumulators and metadata free).  Units this kernel cannot
// hold (more than two scale groups, more than twelve k-steps of 16 strips, tiles above its slot, a misaligned source)
// are skipped: decode_tc_kernel, launched behind it, takes exactly those.
#pragma once
#include "decode_runs.cuh"
#include "decode_umma.cuh"

namespace spectra {

constexpr int kDpWorkers = 512;
constexpr int kDpThreads = kDpWorkers + 32;
constexpr int kDpK = kDpMaxKsteps * 16;               // strip positions of the operands
// fp16 A and B, fp32 D, A K-major, B MN-major, N = 128, M = 128
constexpr uint32_t kDpIdesc = (1u << 4) | (1u << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

// An item of a builder warp's list (a unit's tiles all have the same items, so the list is made once per unit; see
// dp_item): x = byte offset of the class in the tile | class << 14 | (unit stored alone + 1) << 16,
// y = first unit | last unit of the run << 8 | first operand position << 16.
// A unit this kernel takes has at most twelve k-steps, i.e. 48 items (values side), handed out round robin over at most
// eight runs: a warp gets at most 48 / 8 + 8 = 14 of them.
constexpr int kDpMaxItems = 24;

struct DecodePairSmem {
  StripTable tab;
  alignas(128) uint8_t w[2][kDpK * kD * 2];            // W'' = hi + lo (two fp16 parts): element (k, n) at (n / 8) * 16 K + (k / 8) * 128 + (k % 8) * 16 + (n % 8) * 2
  struct Half {
    alignas(128) uint8_t a[kTile * kDpK * 2];          // fields: element (t, k) at (k / 8) * 2048 + t * 16 + (k % 8) * 2
    alignas(128) uint8_t raw[kDecRawMax];              // the packed tile
  } half[2];
  alignas(16) float u[2][kD];
  alignas(16) float cvec[kD];
  uint16_t meta[4][4][kTile];                          // lo16 and R16 of both groups of the last four tiles, kept for the epilogue
  DmRun run[kMaxGroups][4];
  uint2 items[8][kDpMaxItems];                         // the builder warps' items (see dp_item)
  int n_items[8];
  float row_coef[kDpK];                                // per operand row: 2^shift / L of its strip
  int16_t row_chan[kDpK];                              // its channel; -1: a zero row (another group's strip, or past its class)
  int kg[kMaxGroups + 1], wexp;
  float red[17];
  alignas(8) uint64_t raw_full[2], a_full[2], acc_full[2], acc_free[2];
  uint32_t tmem_base;
};
static_assert(sizeof(DecodePairSmem) + 128 <= 227 * 1024, "the reconstruction kernel's shared memory must fit one SM");

// One (group, class) run of a tile into the A operand, by the eight builder warps.  A warp takes four units at a time
// (K side: pairs of strips, V side: strips), a lane one unit (lane % 4) and the token lane / 4 of every group of eight
// tokens: 16 steps, each one load of the 32-bit word that holds the token's field(s), a shift, a mask and a store.
// Word offsets and shifts are a per-lane constant plus a compile-time part, so a step is those four instructions and
// a warp's store covers 8 tokens x 16 bytes: 128 contiguous bytes of the K-major operand, no bank conflicts.
// Units past the end of the run (the padding of its last k-step) repeat the last unit: they meet zero rows of W'',
// and the operand never holds anything but fields.
template <int W, bool V>
__device__ __forceinline__ void dp_item(int base, int u0, int last, int kpos0, int lone, const uint8_t* __restrict__ src,
                                        uint8_t* __restrict__ a, int lane) {
  constexpr uint32_t FM = ((1u << W) - 1u) * (V ? 1u : 0x00010001u);
  const int q = lane >> 2, pr = lane & 3;
  const uint8_t* cb = src + base + 4 * ((q * W) >> 4);
  const int shq = (q * W) & 15;
  constexpr int US = V ? 16 * W : 32 * W;                    // bytes of a unit's stretch
  const int unit = min(u0 + pr, last);
  const uint8_t* cp = cb + US * unit;
  // operand position of the unit: K side 2 strips per unit
  const int kpos = kpos0 + (V ? 1 : 2) * pr;
  uint8_t* dst = a + (kpos >> 3) * 2048 + (kpos & 7) * 2 + q * 16;
  uint32_t v[16];
  if (!V && __any_sync(0xffffffffu, unit == lone)) {
    // a strip stored alone sits among these four units: its words are half-words, the partner's half is zero
    const bool mine = unit == lone;
    const uint8_t* lp = src + base + US * unit + 2 * ((q * W) >> 4);
#pragma unroll
    for (int G = 0; G < 16; G++)
      v[G] = mine ? (uint32_t)*reinterpret_cast<const uint16_t*>(lp + 2 * ((8 * G * W) >> 4))
                  : *reinterpret_cast<const uint32_t*>(cp + 4 * ((8 * G * W) >> 4));
  } else if (V) {
#pragma unroll
    for (int G = 0; G < 16; G++)
      v[G] = *reinterpret_cast<const uint32_t*>(cp + 4 * ((G >> 2) * W + (((8 * (G & 1)) * W) >> 4)));
  } else {
    // K side: the four units of a step sit a multiple of 64 bytes apart, so their words of one token group share
    // banks.  Lane pr therefore walks the sixteen token groups in blocks of four in the order blk ^ pr: at every
    // step the four units read different banks, and the stores (row = token) stay conflict-free in any order.
    const uint8_t* cpb[4];
    uint8_t* dstb[4];
#pragma unroll
    for (int blk = 0; blk < 4; blk++) {
      const int gb = 4 * (blk ^ pr);
      cpb[blk] = cp + 4 * ((8 * gb * W) >> 4);
      dstb[blk] = dst + gb * 128;
    }
#pragma unroll
    for (int G = 0; G < 16; G++) v[G] = *reinterpret_cast<const uint32_t*>(cpb[G >> 2] + 4 * ((8 * (G & 3) * W) >> 4));
#pragma unroll
    for (int G = 0; G < 16; G++) {
      const int sh = (8 * (G & 3) * W) & 15;
      *reinterpret_cast<uint32_t*>(dstb[G >> 2] + (G & 3) * 128) = (v[G] >> (sh + shq)) & FM;
    }
    return;
  }
#pragma unroll
  for (int G = 0; G < 16; G++) {
    if (V) {
      const int sh = 16 * ((G >> 1) & 1) + (((8 * (G & 1)) * W) & 15);
      *reinterpret_cast<uint16_t*>(dst + G * 128) = (uint16_t)((v[G] >> (sh + shq)) & FM);
    } else {
      const int sh = (8 * G * W) & 15;
      *reinterpret_cast<uint32_t*>(dst + G * 128) = (v[G] >> (sh + shq)) & FM;
    }
  }
}
// Bounded wait that sleeps between polls: the waiting warps share their schedulers with the working ones.
__device__ __forceinline__ bool dp_wait(uint32_t bar, uint32_t parity) {
  uint32_t done = 0;
  for (int it = 0; it < (1 << 22) && !done; ++it) {
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3; selp.u32 %0, 1, 0, p; }"
                 : "=r"(done) : "r"(bar), "r"(parity), "r"(1000u) : "memory");
    if (!done) __nanosleep(200);
  }
  return done != 0;
}

// Channels n0 .. n0 + 15 of one token: R0 D0 + R1 D1 + lo0 u0 + lo1 u1 + c (D from tensor memory; the accumulator of
// a group without strips is cleared once per unit), two channels per instruction (packed fp32 pairs).
__device__ __forceinline__ uint64_t dp_pack2(float a, float b) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(a), "f"(b));
  return d;
}
__device__ __forceinline__ uint64_t dp_fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ void dp_zero16(uint32_t a) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
}
__device__ __forceinline__ void dp_chunk(const DecodePairSmem& S, uint32_t acc0, uint32_t acc1, float r0, float r1, float lo0,
                                         float lo1, int n0, float (&y)[16]) {
  float d0[16], d1[16];
  um_ld16(acc0 + n0, d0);
  um_ld16(acc1 + n0, d1);
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
  const uint64_t R0 = dp_pack2(r0, r0), R1 = dp_pack2(r1, r1), L0 = dp_pack2(lo0, lo0), L1 = dp_pack2(lo1, lo1);
#pragma unroll
  for (int q = 0; q < 4; q++) {
    const ulonglong2 c4 = *reinterpret_cast<const ulonglong2*>(&S.cvec[n0 + 4 * q]);
    const ulonglong2 u0 = *reinterpret_cast<const ulonglong2*>(&S.u[0][n0 + 4 * q]);
    const ulonglong2 u1 = *reinterpret_cast<const ulonglong2*>(&S.u[1][n0 + 4 * q]);
    uint64_t va = dp_fma2(L0, u0.x, dp_fma2(L1, u1.x, c4.x)), vb = dp_fma2(L0, u0.y, dp_fma2(L1, u1.y, c4.y));
    va = dp_fma2(R0, dp_pack2(d0[4 * q], d0[4 * q + 1]), va); vb = dp_fma2(R0, dp_pack2(d0[4 * q + 2], d0[4 * q + 3]), vb);
    va = dp_fma2(R1, dp_pack2(d1[4 * q], d1[4 * q + 1]), va); vb = dp_fma2(R1, dp_pack2(d1[4 * q + 2], d1[4 * q + 3]), vb);
    asm("mov.b64 {%0, %1}, %2;" : "=f"(y[4 * q]), "=f"(y[4 * q + 1]) : "l"(va));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(y[4 * q + 2]), "=f"(y[4 * q + 3]) : "l"(vb));
  }
}
__device__ __forceinline__ void dp_store16(const DecodeArgs& p, int64_t o, const float (&y)[16]) {
  const uintptr_t addr = reinterpret_cast<uintptr_t>(p.out) + (uintptr_t)o * (p.out_dtype == SPECTRA_BF16 ? 2 : 4);
  if (p.out_dtype == SPECTRA_BF16 && (addr & 31) == 0) {
    // one 32-byte store: the token's 16 channels fill a whole sector
    uint32_t h[8];
#pragma unroll
    for (int k = 0; k < 8; k++) {
      const __nv_bfloat162 v = __floats2bfloat162_rn(y[2 * k], y[2 * k + 1]);
      h[k] = *reinterpret_cast<const uint32_t*>(&v);
    }
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(addr), "r"(h[0]), "r"(h[1]), "r"(h[2]),
                 "r"(h[3]), "r"(h[4]), "r"(h[5]), "r"(h[6]), "r"(h[7])
                 : "memory");
  } else if (p.out_dtype == SPECTRA_BF16 && (addr & 15) == 0) {
    uint4* dst = reinterpret_cast<uint4*>(addr);
#pragma unroll
    for (int c = 0; c < 2; c++) {
      __nv_bfloat162 h[4];
#pragma unroll
      for (int k = 0; k < 4; k++) h[k] = __floats2bfloat162_rn(y[8 * c + 2 * k], y[8 * c + 2 * k + 1]);
      dst[c] = *reinterpret_cast<const uint4*>(h);
    }
  } else if (p.out_dtype == SPECTRA_F32 && (addr & 31) == 0) {
#pragma unroll
    for (int c = 0; c < 2; c++)
      asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(addr + 32 * c), "f"(y[8 * c]),
                   "f"(y[8 * c + 1]), "f"(y[8 * c + 2]), "f"(y[8 * c + 3]), "f"(y[8 * c + 4]), "f"(y[8 * c + 5]),
                   "f"(y[8 * c + 6]), "f"(y[8 * c + 7])
                   : "memory");
  } else if (p.out_dtype == SPECTRA_F32 && (addr & 15) == 0) {
    float4* dst = reinterpret_cast<float4*>(addr);
#pragma unroll
    for (int c = 0; c < 4; c++) dst[c] = make_float4(y[4 * c], y[4 * c + 1], y[4 * c + 2], y[4 * c + 3]);
  } else {
#pragma unroll
    for (int c = 0; c < 16; c++) store_from_float(p.out, p.out_dtype, o + c, y[c]);
  }
}

__global__ void __launch_bounds__(kDpThreads, 1) decode_pair_kernel(DecodeArgs p, int n_slots_unit, int n_slots) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned char* smem_al = smem_raw + ((128u - (um_smem_u32(smem_raw) & 127u)) & 127u);
  DecodePairSmem& S = *reinterpret_cast<DecodePairSmem*>(smem_al);
  const bool producer = threadIdx.x >= kDpWorkers;
  const int hf = (threadIdx.x >> 8) & 1;                 // which half of the workers
  const int tid = threadIdx.x & 255, lane = tid & 31, warp = tid >> 5;
  const bool side_v = p.side == SPECTRA_SIDE_V;
  if (threadIdx.x == 0) {
    for (int h = 0; h < 2; h++) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(um_smem_u32(&S.raw_full[h])) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 8;" ::"r"(um_smem_u32(&S.a_full[h])) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(um_smem_u32(&S.acc_full[h])) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 8;" ::"r"(um_smem_u32(&S.acc_free[h])) : "memory");
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < 32) {                                // warp 0 owns the tensor-memory allocation (all 512 columns)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(um_smem_u32(&S.tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  const int slot_end = (int)((long long)(blockIdx.x + 1) * n_slots / gridDim.x);
  int base0 = 0, base1 = 0;                              // tiles each buffer has taken so far: the barrier phases follow them
  int tiles_done = 0;                                    // tiles of the earlier runs (metadata slots rotate over all of them)
  int status = 0;
  const StripTable& T = S.tab;

  for (int slot = (int)((long long)blockIdx.x * n_slots / gridDim.x); slot < slot_end;) {
    // ---- the next run: tile slots [ga, gb) of unit u
    const int u = slot / n_slots_unit, ga = slot - u * n_slots_unit;
    const int gb = min(n_slots_unit, ga + (slot_end - slot));
    slot += gb - ga;
    const int ps = (int)(u % p.n_param_sets);
    const int n = p.n_tokens[u];
    const int n_tiles = min(gb, (n + kTile - 1) / kTile) - ga;
    if (n_tiles <= 0) continue;
    __syncthreads();                                     // the previous run is over
    build_strip_table(S.tab, p.widths + (int64_t)ps * kD, p.scale_group);
    const float* wsrc = p.w_dec + (int64_t)ps * kD * kD;
    const int gs = p.scale_group;
    const uint8_t* unit_ptr = p.cache + p.unit_offset[u];
    dm_build_runs(S.run, S.kg, T, side_v, gs);
    const int n_ksteps = S.kg[kMaxGroups];
    if (!dm_pairs_eligible(T, n_ksteps, unit_ptr)) continue;      // decode_tc_kernel takes this unit
    const int tile_bytes = T.tile_bytes;
    // ---- the builder warps' item lists: four units (half a k-step on the K side, a quarter on the V side) per item,
    // handed out round robin across the runs so that every warp gets the same number of them, give or take one
    if (threadIdx.x < 8) {
      const int w = threadIdx.x, per = side_v ? 16 : 8;
      int done = 0, cnt = 0;
      for (int g = 0; g < 2; g++)
        for (int c = 0; c < 4; c++) {
          const DmRun r = S.run[g][c];
          if (r.n == 0) continue;
          const int nit = (r.n + per - 1) / per * (per / 4);
          for (int item = (w - done) & 7; item < nit; item += 8)
            if (cnt < kDpMaxItems) {
              S.items[w][cnt] = make_uint2((uint32_t)r.base | (uint32_t)c << 14 | (uint32_t)(r.lone + 1) << 16,
                                           (uint32_t)(r.first + 4 * item) | (uint32_t)(r.first + r.n - 1) << 8 |
                                               (uint32_t)(16 * r.kstep0 + (side_v ? 1 : 2) * 4 * item) << 16);
              cnt++;
            }
          done += nit;
        }
      S.n_items[w] = cnt;
    }
    // ---- the operand rows: row (k-step, slot) -> channel and 2^shift / L of its strip, or a zero row (another
    // group's strip, or past the end of its class).  Done once per row, not once per entry of W''.
    for (int k = threadIdx.x; k < n_ksteps * 16; k += kDpThreads) {
      const int ks = k >> 4, row = k & 15;
      int g = 0, c = 0;
      for (int gg = 0; gg < kMaxGroups; gg++)
        for (int cc = 0; cc < 4; cc++)
          if (ks >= S.run[gg][cc].kstep0 && S.run[gg][cc].n > 0) { g = gg; c = cc; }
      const DmRun r = S.run[g][c];
      const int kk = ks - r.kstep0;
      const int first = T.class_first[c], cnt = T.class_first[c + 1] - first;
      const int s_in = side_v ? r.first + 16 * kk + row : 2 * (r.first + 8 * kk + (row >> 1)) + (row & 1);
      int ch = -1;
      float coef = 0.f;
      if (s_in < cnt) {
        const int kx = first + s_in, chx = T.chan[kx];
        if (chx >= g * gs && chx < (g + 1) * gs) {
          ch = chx;
          coef = (float)(1 << T.shift[kx]) / (float)((1 << T.width[chx]) - 1);
        }
      }
      S.row_chan[k] = (int16_t)ch; S.row_coef[k] = coef;
    }
    // ---- largest |W_dec|: the power of two that brings W'' into fp16's range
    {
      float m = 0.f;
      for (int idx = threadIdx.x; idx < kD * kD; idx += kDpThreads) m = fmaxf(m, fabsf(wsrc[idx]));
#pragma unroll
      for (int s = 16; s; s >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, s));
      if ((threadIdx.x & 31) == 0) S.red[threadIdx.x >> 5] = m;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      float m = 0.f;
      for (int i = 0; i < kDpThreads / 32; i++) m = fmaxf(m, S.red[i]);
      int e = 0;
      frexpf(m, &e);                                     // m < 2^e (m = 0: e = 0)
      S.wexp = e;
    }
    __syncthreads();
    const int wexp = S.wexp;
    {
      const float wscale = exp2f((float)(15 - wexp));
      for (int idx = threadIdx.x; idx < n_ksteps * 16 * kD; idx += kDpThreads) {
        const int nn = idx & (kD - 1), k = idx >> 7;       // operand row k = 16 k-step + slot
        const int rch = S.row_chan[k];                   // (written before the two barriers above)
        const float v = rch < 0 ? 0.f : wsrc[rch * kD + nn] * S.row_coef[k] * wscale;
        const int wo = (nn >> 3) * (16 * kDpK) + (k >> 3) * 128 + (k & 7) * 16 + (nn & 7) * 2;
        const __half hi = __float2half_rn(v);
        *reinterpret_cast<__half*>(&S.w[0][wo]) = hi;
        *reinterpret_cast<__half*>(&S.w[1][wo]) = __float2half_rn(v - __half2float(hi));
      }
      for (int idx = threadIdx.x; idx < 3 * kD; idx += kDpThreads) {     // u_0, u_1, c
        const int nn = idx & (kD - 1), g = idx >> 7;
        float acc = 0.f;
        if (g < 2) {
          if (g < T.n_groups)
            for (int j = g * gs; j < (g + 1) * gs; j++) acc += T.width[j] ? wsrc[j * kD + nn] : 0.f;
          S.u[g][nn] = acc;
        } else {
          for (int j = 0; j < kD; j++) acc = fmaf(p.mean_rot[(int64_t)ps * kD + j], wsrc[j * kD + nn], acc);
          S.cvec[nn] = acc;
        }
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");    // W'': generic stores -> tensor-core reads
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tb = S.tmem_base;
    const float rfac = exp2f((float)(24 - 15 + wexp));   // undoes 2^-24 of the fields and the scale of W''
    const int kg1 = S.kg[1], kg2 = S.kg[2];              // k-steps [0, kg1) group 0, [kg1, kg2) group 1

    if (producer) {
      if (threadIdx.x == kDpWorkers) {
        auto load_raw = [&](int tt) {                    // tile ga + tt into the packed-tile buffer of half tt & 1
          const int h = tt & 1;
          const uint32_t bar = um_smem_u32(&S.raw_full[h]);
          asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(tile_bytes) : "memory");
          asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                           um_smem_u32(S.half[h].raw)),
                       "l"(unit_ptr + p.map.page(u, ga + tt) * tile_bytes), "r"(tile_bytes), "r"(bar)
                       : "memory");
        };
        load_raw(0);
        if (n_tiles > 1) load_raw(1);
        bool ok = true;
        const uint32_t w0 = um_smem_u32(S.w[0]), w1 = um_smem_u32(S.w[1]);
#pragma unroll 1
        for (int tt = 0; tt < n_tiles && ok; tt++) {
          const int h = tt & 1, i = (h ? base1 : base0) + (tt >> 1);
          ok = um_wait(um_smem_u32(&S.a_full[h]), (uint32_t)(i & 1));
          if (!ok) break;
          if (tt + 2 < n_tiles) load_raw(tt + 2);        // the builders are done with this buffer's packed tile
          if (i >= 1) ok = um_wait(um_smem_u32(&S.acc_free[h]), (uint32_t)((i - 1) & 1));   // its accumulators are drained
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a0 = um_smem_u32(S.half[h].a);
          // descriptors once; per k-step only the address fields move (the issuing thread's own instructions bound the
          // rate at which MMAs go out)
          const uint64_t ad0 = um_desc(a0, 2048, 128), bh0 = um_desc(w0, 128, 16 * kDpK), bl0 = um_desc(w1, 128, 16 * kDpK);
#pragma unroll
          for (int g = 0; g < 2; g++) {
            const int lo = g ? kg1 : 0, hi = g ? kg2 : kg1;
            const uint32_t d = tb + 128u * (2 * h + g);
            // the fields against the high parts of W'', then against the low parts, into the same accumulator
            if (lo < hi) um_mma_ss(d, ad0 + (uint64_t)(256 * lo), bh0 + (uint64_t)(16 * lo), kDpIdesc, 0);
#pragma unroll 2
            for (int ks = lo + 1; ks < hi; ks++) um_mma_ss(d, ad0 + (uint64_t)(256 * ks), bh0 + (uint64_t)(16 * ks), kDpIdesc, 1);
#pragma unroll 2
            for (int ks = lo; ks < hi; ks++) um_mma_ss(d, ad0 + (uint64_t)(256 * ks), bl0 + (uint64_t)(16 * ks), kDpIdesc, 1);
          }
          asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(um_smem_u32(&S.acc_full[h])) : "memory");
        }
        if (!ok) status |= SPECTRA_STATUS_WAIT_TIMEOUT;
      }
    } else if (hf == 0) {
      // ------------------------------------------------------------------ builders (warps 0..7): every tile's A operand
      bool ok = true;
#pragma unroll 1
      for (int tt = 0; tt < n_tiles && ok; tt++) {
        const int bf = tt & 1, i = (bf ? base1 : base0) + (tt >> 1);
        DecodePairSmem::Half& Hs = S.half[bf];
        ok = dp_wait(um_smem_u32(&S.raw_full[bf]), (uint32_t)(i & 1));
        // the buffer's previous operand has been read by its MMAs.  (Those MMAs were issued after the epilogue of the
        // tile four back had drained their accumulators, so the metadata slot of that tile is free as well.)
        if (ok && i >= 1) ok = dp_wait(um_smem_u32(&S.acc_full[bf]), (uint32_t)((i - 1) & 1));
        if (!ok) { status |= SPECTRA_STATUS_WAIT_TIMEOUT; break; }
        const uint8_t* src = Hs.raw;
        const int my_items = S.n_items[warp];
#pragma unroll 1
        for (int it = 0; it < my_items; it++) {
          const uint2 e = S.items[warp][it];
          const int base = (int)(e.x & 0x3fffu), c = (int)(e.x >> 14) & 3, lone = (int)(e.x >> 16) - 1;
          const int u0 = (int)(e.y & 0xffu), last = (int)(e.y >> 8) & 0xff, kpos0 = (int)(e.y >> 16);
          if (side_v) {
            if (c == 0) dp_item<8, true>(base, u0, last, kpos0, lone, src, Hs.a, lane);
            else if (c == 1) dp_item<4, true>(base, u0, last, kpos0, lone, src, Hs.a, lane);
            else if (c == 2) dp_item<2, true>(base, u0, last, kpos0, lone, src, Hs.a, lane);
            else dp_item<1, true>(base, u0, last, kpos0, lone, src, Hs.a, lane);
          } else {
            if (c == 0) dp_item<8, false>(base, u0, last, kpos0, lone, src, Hs.a, lane);
            else if (c == 1) dp_item<4, false>(base, u0, last, kpos0, lone, src, Hs.a, lane);
            else if (c == 2) dp_item<2, false>(base, u0, last, kpos0, lone, src, Hs.a, lane);
            else dp_item<1, false>(base, u0, last, kpos0, lone, src, Hs.a, lane);
          }
        }
        // the tokens' group offsets and ranges, kept for the epilogue (the packed tile is handed back now)
        {
          const int g = tid >> 7, tk = tid & (kTile - 1);
          uint16_t lo = 0, rg = 0;
          if (g < T.n_groups && T.meta_off[g] >= 0) {
            const uint16_t* m = reinterpret_cast<const uint16_t*>(src + T.meta_off[g]) + tk;
            lo = m[0]; rg = m[kTile];
          }
          const int ms = (tiles_done + tt) & 3;
          S.meta[ms][2 * g][tk] = lo; S.meta[ms][2 * g + 1][tk] = rg;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");          // operand: generic stores -> tensor-core reads
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(um_smem_u32(&S.a_full[bf])) : "memory");
      }
    } else {
      // ------------------------------------------------------------------ epilogue (warps 8..15): thread = token and 64 channels
      bool ok = true;
      const int t_ep = tid & (kTile - 1), ch0 = 64 * (tid >> 7);
      // a group without strips gets no MMA: its accumulators (both buffers, this thread's lane and 64 columns) are
      // cleared once, so that the epilogue can read them unconditionally
#pragma unroll 1
      for (int g = 0; g < 2; g++) {
        if (g ? kg2 > kg1 : kg1 > 0) continue;
        for (int bf = 0; bf < 2; bf++)
          for (int c4 = 0; c4 < 4; c4++) dp_zero16(tb + 128u * (2 * bf + g) + ((uint32_t)((warp & 3) * 32) << 16) + ch0 + 16 * c4);
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        asm volatile("bar.sync 1, 256;" ::: "memory");      // the eight epilogue warps (a partner thread reads these columns too)
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      }
#pragma unroll 1
      for (int tt = 0; tt < n_tiles && ok; tt++) {
        const int bf = tt & 1, i = (bf ? base1 : base0) + (tt >> 1);
        const int tile = ga + tt, tile_pos = tile * kTile;
        const int n_here = min(n - tile_pos, kTile);
        // The MMAs of this tile were issued after its operand and metadata were complete (a_full), so their completion
        // says that the metadata are in place too.  a_full itself is not waited for here: the builders may already
        // have completed it once more (for the tile after next, which only needs this tile's MMAs) before this
        // warp looks, and a phase parity cannot tell that from "not yet".
        ok = dp_wait(um_smem_u32(&S.acc_full[bf]), (uint32_t)(i & 1));
        if (!ok) { status |= SPECTRA_STATUS_WAIT_TIMEOUT; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int ms = (tiles_done + tt) & 3;
        const float lo0 = __half2float(__ushort_as_half(S.meta[ms][0][t_ep])), r0 = __half2float(__ushort_as_half(S.meta[ms][1][t_ep])) * rfac;
        const float lo1 = __half2float(__ushort_as_half(S.meta[ms][2][t_ep])), r1 = __half2float(__ushort_as_half(S.meta[ms][3][t_ep])) * rfac;
        const bool live = t_ep < n_here;
        const uint32_t acc0 = tb + 128u * (2 * bf) + ((uint32_t)((warp & 3) * 32) << 16);
        const uint32_t acc1 = acc0 + 128u;
        const int64_t obase = p.out_index(u, tile, t_ep);
        if (p.rope_cos) {
          // Sec. 3.3: the position rotation is applied to the reconstructed key.  Channels i and i + 64 are a pair: this
          // thread takes the pairs 32 (ch0 / 64) .. + 31, 16 at a time, both halves
          const int i0 = ch0 >> 1;
          const int64_t pos = (int64_t)(p.rope_pos0 ? p.rope_pos0[u] : 0) + tile_pos + t_ep;
#pragma unroll 1
          for (int part = 0; part < 2; part++) {
            float ylo[16], yhi[16];
            dp_chunk(S, acc0, acc1, r0, r1, lo0, lo1, i0 + 16 * part, ylo);
            dp_chunk(S, acc0, acc1, r0, r1, lo0, lo1, 64 + i0 + 16 * part, yhi);
            if (live) {
              const float4* cs = reinterpret_cast<const float4*>(p.rope_cos + pos * (kD / 2) + i0 + 16 * part);
              const float4* sn = reinterpret_cast<const float4*>(p.rope_sin + pos * (kD / 2) + i0 + 16 * part);
#pragma unroll
              for (int c = 0; c < 4; c++) {
                const float4 cv = cs[c], sv = sn[c];
                const float cc[4] = {cv.x, cv.y, cv.z, cv.w}, ss[4] = {sv.x, sv.y, sv.z, sv.w};
#pragma unroll
                for (int k = 0; k < 4; k++) {
                  const float a = ylo[4 * c + k], b = yhi[4 * c + k];
                  ylo[4 * c + k] = a * cc[k] - b * ss[k];
                  yhi[4 * c + k] = b * cc[k] + a * ss[k];
                }
              }
              dp_store16(p, obase + i0 + 16 * part, ylo);
              dp_store16(p, obase + 64 + i0 + 16 * part, yhi);
            }
          }
        } else
        {
#pragma unroll 2
          for (int part = 0; part < 4; part++) {
            float y[16];
            dp_chunk(S, acc0, acc1, r0, r1, lo0, lo1, ch0 + 16 * part, y);
            if (live) dp_store16(p, obase + ch0 + 16 * part, y);
          }
        }
        // the accumulators and the metadata of this buffer may be overwritten
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(um_smem_u32(&S.acc_free[bf])) : "memory");
      }
    }
    // ---- end of the run: a timeout anywhere ends the CTA's work (the barrier phases are no longer known)
    base0 += (n_tiles + 1) >> 1; base1 += n_tiles >> 1; tiles_done += n_tiles;
    if (__syncthreads_or(status & SPECTRA_STATUS_WAIT_TIMEOUT)) break;
  }
  // ---- the warp that allocated the tensor memory frees it
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (threadIdx.x < 32) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(S.tmem_base), "r"(512u) : "memory");
  if (status && p.status) atomicOr(p.status, status);
}

}  // namespace spectra
