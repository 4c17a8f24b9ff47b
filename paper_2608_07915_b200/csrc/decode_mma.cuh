// Reconstruction path of spectra_decode with the unpacking done by the tensor cores' operand path.
//
// xhat_t = (yhat_t + m') W_dec with yhat_tj = lo_g(t) + code_tj R_g(t) / L_j (Sec. 3.2, Sec. 3.3 Mode A) is regrouped as
//     xhat_t = sum_g R_g(t) [ sum_{strips k of group g} field_tk W''_k ]  +  sum_g lo_g(t) u_g  +  c,
//     W''_k = 2^shift(k) W_dec[chan(k), :] / L_chan(k),   u_g = sum_{stored j in g} W_dec[j, :],   c = m' W_dec,
// where a strip is one sub-field (8, 4, 2 or 1 bits) of a channel's code.  The bracket is a product of small integers
// with a matrix that is fixed per unit-side: it runs as mma.sync.m16n8k16 with A = the packed fields themselves (a
// field shifted down to bit 0 of its half-word and masked is the fp16 subnormal field * 2^-24, which the tensor core
// multiplies exactly; on the K side a 32-bit word of the tile already holds the two strips of a pair for one token,
// so one shift and one mask make an A register) and B = W'' as fp16 scaled by a power of two into fp16's range.  No
// code is ever written out, dequantised or converted: per A register about three instructions instead of about
// sixty per token and channel in the tcgen05 kernel that builds its operand element by element.
//
// One CTA of eight warps per SM walks a contiguous range of (unit, tile) slots; per unit it builds the strip table,
// the (group, class) runs, the B table in MMA fragment order, u_g and c.  The two halves of the CTA take alternate
// tiles; a warp owns 32 tokens of a tile (two m16 row blocks, so that a B fragment read from shared memory serves two
// MMAs: the B table is what every warp re-reads, and shared-memory bandwidth is the first limit) and all 128 output
// channels in two passes of 64 (channels i and i + 64 in the same pass, so that the rotary pairing of the epilogue
// stays inside a thread).  Packed tiles
// arrive by bulk copies into a ring of three slots, refilled by the half that has just finished with a slot.
// Rows of B that belong to another scale group or lie past the end of a class are zero, and the unit index of such a
// row is clamped for the load, so nothing is read outside the tile.  All waits are bounded.
#pragma once
#include "decode_umma.cuh"

namespace spectra {

constexpr int kDmThreads = 256;
constexpr int kDmHalf = kDmThreads / 2;     // threads of a half: four warps, 32 tokens each
constexpr int kDmMaxKsteps = 40;          // 16 strips each; every width profile and scale group fits (see the host check)
constexpr int kDmRawSlot = 18944;         // the largest tile: 128 strips of 8 bits + four groups of metadata = 18432 bytes
constexpr int kDmSlots = 3;

struct DmRun { int base, first, n, kstep0, lone; };   // class region offset, first unit, units, first k-step, lone pair or -1

struct DecodeMmaSmem {
  StripTable tab;
  alignas(16) uint2 B[kDmMaxKsteps][16][32];          // [k-step][n block][lane] = {b0, b1} of the m16n8k16 B fragment
  alignas(128) uint8_t raw[kDmSlots][kDmRawSlot];
  alignas(16) float u[kMaxGroups][kD];                // u_g
  alignas(16) float cvec[kD];                         // c
  DmRun run[kMaxGroups][4];
  int kg[kMaxGroups + 1], wexp;
  float red[16];
  alignas(8) uint64_t full[kDmSlots];
};
static_assert(sizeof(DecodeMmaSmem) + 128 <= 227 * 1024, "the reconstruction kernel's shared memory must fit one SM");

__device__ __forceinline__ void dm_mma(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// The (group, class) runs of a unit-side's tile and their k-steps of 16 strips, by all threads of the CTA (ends with a
// barrier).  Strips of class c whose channel lies in group g are the in-class indices [sa, sb); a K-side unit is a pair
// of strips, a V-side unit one strip.  kg[g] = first k-step of group g, kg[n_groups..] = the total.
__device__ inline void dm_build_runs(DmRun (*run)[4], int* kg, const StripTable& T, bool side_v, int gs) {
  const int tid = threadIdx.x;
  if (tid < 16) {
    const int g = tid >> 2, c = tid & 3;
    DmRun r{0, 0, 0, 0, -1};
    if (g < T.n_groups) {
      const int first = T.class_first[c], cnt = T.class_first[c + 1] - first;
      int sa = 0, sb = 0;
      for (int k = 0; k < cnt; k++) {
        const int ch = T.chan[first + k];
        sa += ch < g * gs;
        sb += ch < (g + 1) * gs;
      }
      r.base = T.class_off[c];
      if (sb > sa) {
        if (side_v) { r.first = sa; r.n = sb - sa; }
        else {
          r.first = sa >> 1; r.n = ((sb - 1) >> 1) - r.first + 1;
          if ((cnt & 1) && sb == cnt) r.lone = cnt >> 1;          // the class's odd last strip, stored alone
        }
      }
    }
    run[g][c] = r;
  }
  __syncthreads();
  if (tid == 0) {
    int ks = 0;
    const int per = side_v ? 16 : 8;
    for (int g = 0; g < kMaxGroups; g++) {
      kg[g] = ks;
      for (int c = 0; c < 4; c++) {
        run[g][c].kstep0 = ks;
        ks += (run[g][c].n + per - 1) / per;
      }
    }
    kg[kMaxGroups] = ks;
  }
  __syncthreads();
}

// Entry (row of k-step ks, output channel nn) of W'' before the fp16 scale: 2^shift W_dec[chan] / L, zero for a row
// outside its run's group or past the end of its class.
__device__ inline float dm_b_value(const DmRun (*run)[4], const StripTable& T, const float* __restrict__ wsrc, bool side_v,
                                   int gs, int ks, int row, int nn) {
  int g = 0, c = 0;
#pragma unroll
  for (int gg = 0; gg < kMaxGroups; gg++)
#pragma unroll
    for (int cc = 0; cc < 4; cc++)
      if (ks >= run[gg][cc].kstep0 && run[gg][cc].n > 0) { g = gg; c = cc; }
  const DmRun r = run[g][c];
  const int kk = ks - r.kstep0;
  const int first = T.class_first[c], cnt = T.class_first[c + 1] - first;
  const int s_in = side_v ? r.first + 16 * kk + row : 2 * (r.first + 8 * kk + (row >> 1)) + (row & 1);
  if (s_in >= cnt) return 0.f;
  const int k = first + s_in, ch = T.chan[k];
  if (ch < g * gs || ch >= (g + 1) * gs) return 0.f;
  const float L = (float)((1 << T.width[ch]) - 1);
  return wsrc[ch * kD + nn] * (float)(1 << T.shift[k]) / L;
}

// Units the tcgen05 kernel of decode_pairs.cuh takes (the rest is this file's): at most two scale groups, at most
// twelve k-steps, a tile that fits that kernel's slot, a source the bulk copy accepts.
constexpr int kDpMaxKsteps = 12;
__device__ __forceinline__ bool dm_pairs_eligible(const StripTable& T, int n_ksteps, const void* unit_ptr) {
  return T.n_groups <= 2 && n_ksteps <= kDpMaxKsteps && T.tile_bytes <= kDecRawMax && (reinterpret_cast<uintptr_t>(unit_ptr) & 15) == 0;
}

// skip_pairs != 0: units that decode_pair_kernel takes are left to it
__global__ void __launch_bounds__(kDmThreads, 1) decode_mma_kernel(DecodeArgs p, int n_slots_unit, int n_slots, int skip_pairs) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned char* smem_al = smem_raw + ((128u - (um_smem_u32(smem_raw) & 127u)) & 127u);
  DecodeMmaSmem& S = *reinterpret_cast<DecodeMmaSmem*>(smem_al);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int hf = warp >> 2, wq = warp & 3;               // half of the CTA, 32-token block of the tile
  const int gid = lane >> 2, tig = lane & 3;
  const bool side_v = p.side == SPECTRA_SIDE_V;
  const StripTable& T = S.tab;
  if (tid == 0) {
    for (int s = 0; s < kDmSlots; s++) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(um_smem_u32(&S.full[s])) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  int loads_done = 0;                                    // bulk copies issued so far by this CTA (slot = count % 3)
  int status = 0;
  const int slot_end = (int)((long long)(blockIdx.x + 1) * n_slots / gridDim.x);

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
    const int gs = p.scale_group, n_groups = T.n_groups;
    const int tile_bytes = T.tile_bytes;
    const uint8_t* unit_ptr = p.cache + p.unit_offset[u];
    dm_build_runs(S.run, S.kg, T, side_v, gs);
    const int n_ksteps = S.kg[kMaxGroups];
    if (skip_pairs && dm_pairs_eligible(T, n_ksteps, unit_ptr)) continue;   // the other kernel's unit
    if (n_ksteps > kDmMaxKsteps) {                       // cannot happen with 128 channels; never index past the table
      status |= SPECTRA_STATUS_BAD_LAYOUT;
      continue;
    }
    // bulk copies need a 16-byte aligned source; a unit that is not is copied by the half's threads, two bytes at a time
    const bool bulk = (reinterpret_cast<uintptr_t>(unit_ptr) & 15) == 0;
    // the first copies go out while the tables are built
    const int load_base = loads_done;                    // tile tt of this run is copy number load_base + tt
    auto issue_load = [&](int tt) {                      // by one thread
      const int s = (load_base + tt) % kDmSlots;
      const uint32_t bar = um_smem_u32(&S.full[s]);
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(tile_bytes) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                       um_smem_u32(S.raw[s])),
                   "l"(unit_ptr + p.map.page(u, ga + tt) * tile_bytes), "r"(tile_bytes), "r"(bar)
                   : "memory");
    };
    if (tid == 0 && bulk) {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // earlier generic reads of the slots are done
      for (int tt = 0; tt < min(n_tiles, kDmSlots); tt++) issue_load(tt);
    }
    // ---- largest |W_dec| (the scale that brings W'' into fp16's range)
    {
      float m = 0.f;
      for (int idx = tid; idx < kD * kD; idx += kDmThreads) m = fmaxf(m, fabsf(wsrc[idx]));
#pragma unroll
      for (int s = 16; s; s >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, s));
      if (lane == 0) S.red[warp] = m;
    }
    __syncthreads();
    if (tid == 0) {
      float m = 0.f;
      for (int i = 0; i < kDmThreads / 32; i++) m = fmaxf(m, S.red[i]);
      int e = 0;
      frexpf(m, &e);                                     // m < 2^e (m = 0: e = 0)
      S.wexp = e;
    }
    __syncthreads();
    const int wexp = S.wexp;
    // ---- B table: W'' = 2^shift W_dec[chan] / L * 2^(15 - wexp), zero rows outside a run's group and class
    {
      const float wscale = exp2f((float)(15 - wexp));
      for (int idx = tid; idx < n_ksteps * 16 * kD; idx += kDmThreads) {
        const int nn = idx & (kD - 1), row = (idx >> 7) & 15, ks = idx >> 11;
        const float v = dm_b_value(S.run, T, wsrc, side_v, gs, ks, row, nn) * wscale;
        const int nb = nn >> 3, ln = (nn & 7) * 4 + ((row & 7) >> 1);
        reinterpret_cast<__half*>(&S.B[ks][nb][ln])[2 * (row >> 3) + (row & 1)] = __float2half_rn(v);
      }
      // u_g and c
      for (int idx = tid; idx < (kMaxGroups + 1) * kD; idx += kDmThreads) {
        const int nn = idx & (kD - 1), g = idx >> 7;
        float acc = 0.f;
        if (g < kMaxGroups) {
          if (g < n_groups)
            for (int j = g * gs; j < (g + 1) * gs; j++) acc += T.width[j] ? wsrc[j * kD + nn] : 0.f;
          S.u[g][nn] = acc;
        } else {
          for (int j = 0; j < kD; j++) acc = fmaf(p.mean_rot[(int64_t)ps * kD + j], wsrc[j * kD + nn], acc);
          S.cvec[nn] = acc;
        }
      }
    }
    __syncthreads();
    const float rfac = exp2f((float)(24 - 15 + wexp));   // undoes 2^-24 of the fields and the scale of W''

    // ---- tiles of the run: this half takes tt = hf, hf + 2, ..
    bool ok = true;
#pragma unroll 1
    for (int tt = hf; tt < n_tiles && ok; tt += 2) {
      const int cn = load_base + tt, s = cn % kDmSlots;
      const int tile = ga + tt, tile_pos = tile * kTile;
      const int n_here = min(n - tile_pos, kTile);
      if (!bulk) {
        const uint16_t* g16 = reinterpret_cast<const uint16_t*>(unit_ptr + p.map.page(u, tile) * tile_bytes);
        uint16_t* s16 = reinterpret_cast<uint16_t*>(S.raw[s]);
        for (int i = tid & (kDmHalf - 1); i < tile_bytes / 2; i += kDmHalf) s16[i] = g16[i];
        asm volatile("bar.sync %0, %1;" ::"r"(1 + hf), "n"(kDmHalf) : "memory");
      } else {   // wait (outcome uniform over the half)
        const uint32_t mine = um_wait(um_smem_u32(&S.full[s]), (uint32_t)((cn / kDmSlots) & 1)) ? 1u : 0u;
        uint32_t all;
        asm volatile("{ .reg .pred p, q; setp.ne.u32 p, %1, 0; bar.red.and.pred q, %2, %3, p; selp.u32 %0, 1, 0, q; }"
                     : "=r"(all) : "r"(mine), "r"(1 + hf), "n"(kDmHalf) : "memory");
        if (!all) { status |= SPECTRA_STATUS_WAIT_TIMEOUT; ok = false; break; }
      }
      const uint8_t* src = S.raw[s];
      // this thread's four token rows: row block rb (16 tokens), rows gid and gid + 8 of it
      const int t0 = 32 * wq + gid;                      // rows t0, t0 + 8, t0 + 16, t0 + 24
#pragma unroll 1
      for (int pass = 0; pass < 2; pass++) {
        // n blocks of this pass: channels [32 pass, 32 pass + 32) and the same + 64
        float out[2][8][4];
#pragma unroll
        for (int rb = 0; rb < 2; rb++)
#pragma unroll
          for (int j = 0; j < 8; j++)
#pragma unroll
            for (int e = 0; e < 4; e++) out[rb][j][e] = 0.f;
#pragma unroll 1
        for (int g = 0; g < n_groups; g++) {
          if (T.meta_off[g] < 0) continue;
          float acc[2][8][4];
#pragma unroll
          for (int rb = 0; rb < 2; rb++)
#pragma unroll
            for (int j = 0; j < 8; j++)
#pragma unroll
              for (int e = 0; e < 4; e++) acc[rb][j][e] = 0.f;
#pragma unroll 1
          for (int c = 0; c < 4; c++) {
            const DmRun r = S.run[g][c];
            if (r.n == 0) continue;
            const int w = 8 >> c, lw = 3 - c;
            const int nk = side_v ? (r.n + 15) >> 4 : (r.n + 7) >> 3;
            const uint32_t fmask = ((1u << w) - 1u) * (side_v ? 1u : 0x00010001u);
            // K side: word of (pair, token) = base + 32 w pair + 4 ((t w) >> 4), field at bit (t w) & 15 of both halves
            // V side: word of (strip, token) = base + 16 w strip + 4 (a w + ((i w) >> 4)), a = t >> 5, i = t & 15,
            //         field at bit 16 ((t >> 4) & 1) + ((i w) & 15)
            int tb[4], sh[4];                              // byte offset inside the unit's stretch and shift, per row
#pragma unroll
            for (int q = 0; q < 4; q++) {
              const int t = t0 + 8 * q;
              if (side_v) {
                const int i = t & 15;
                tb[q] = 4 * (((t >> 5) << lw) + ((i << lw) >> 4));
                sh[q] = 16 * ((t >> 4) & 1) + ((i << lw) & 15);
              } else {
                tb[q] = 4 * ((t << lw) >> 4);
                sh[q] = (t << lw) & 15;
              }
            }
            const int last = r.first + r.n - 1;
            const uint8_t* cbase = src + r.base;
            const int ustride = side_v ? 16 * w : 32 * w;  // bytes per unit (strip or pair)
            const uint2* bp = &S.B[r.kstep0][4 * pass][lane];
#pragma unroll 1
            for (int kk = 0; kk < nk; kk++, bp += 16 * 32) {
              uint32_t a[2][4];                            // [row block][a0..a3]
              if (side_v) {
                const int s0 = min(r.first + 16 * kk + 2 * tig, last), s1 = min(s0 + 1, last);
                const int s2 = min(r.first + 16 * kk + 2 * tig + 8, last), s3 = min(s2 + 1, last);
                const uint8_t *q0 = cbase + ustride * s0, *q1 = cbase + ustride * s1, *q2 = cbase + ustride * s2, *q3 = cbase + ustride * s3;
#pragma unroll
                for (int q = 0; q < 4; q++) {
                  const uint32_t f0 = (*reinterpret_cast<const uint32_t*>(q0 + tb[q]) >> sh[q]) & fmask;
                  const uint32_t f1 = (*reinterpret_cast<const uint32_t*>(q1 + tb[q]) >> sh[q]) & fmask;
                  const uint32_t f2 = (*reinterpret_cast<const uint32_t*>(q2 + tb[q]) >> sh[q]) & fmask;
                  const uint32_t f3 = (*reinterpret_cast<const uint32_t*>(q3 + tb[q]) >> sh[q]) & fmask;
                  a[q >> 1][q & 1] = f0 | (f1 << 16);
                  a[q >> 1][2 + (q & 1)] = f2 | (f3 << 16);
                }
              } else {
                const int p0 = min(r.first + 8 * kk + tig, last), p1 = min(r.first + 8 * kk + tig + 4, last);
                const uint8_t *c0 = cbase + ustride * p0, *c1 = cbase + ustride * p1;
                if (kk == nk - 1 && r.lone >= 0) {         // the run ends with a strip stored alone (half-words in order)
#pragma unroll
                  for (int q = 0; q < 4; q++) {
                    const uint32_t v0 = p0 == r.lone ? (uint32_t)*reinterpret_cast<const uint16_t*>(c0 + (tb[q] >> 1))
                                                     : *reinterpret_cast<const uint32_t*>(c0 + tb[q]);
                    const uint32_t v1 = p1 == r.lone ? (uint32_t)*reinterpret_cast<const uint16_t*>(c1 + (tb[q] >> 1))
                                                     : *reinterpret_cast<const uint32_t*>(c1 + tb[q]);
                    a[q >> 1][q & 1] = (v0 >> sh[q]) & fmask;
                    a[q >> 1][2 + (q & 1)] = (v1 >> sh[q]) & fmask;
                  }
                } else {
#pragma unroll
                  for (int q = 0; q < 4; q++) {
                    a[q >> 1][q & 1] = (*reinterpret_cast<const uint32_t*>(c0 + tb[q]) >> sh[q]) & fmask;
                    a[q >> 1][2 + (q & 1)] = (*reinterpret_cast<const uint32_t*>(c1 + tb[q]) >> sh[q]) & fmask;
                  }
                }
              }
#pragma unroll
              for (int j = 0; j < 8; j++) {
                const uint2 bb = bp[((j & 3) + 8 * (j >> 2)) * 32];
                dm_mma(acc[0][j], a[0][0], a[0][1], a[0][2], a[0][3], bb.x, bb.y);
                dm_mma(acc[1][j], a[1][0], a[1][1], a[1][2], a[1][3], bb.x, bb.y);
              }
            }
          }
          // the group's share, scaled by each row's range
          const uint16_t* mr = reinterpret_cast<const uint16_t*>(src + T.meta_off[g]) + kTile;
#pragma unroll
          for (int rb = 0; rb < 2; rb++) {
            const float r0 = __half2float(__ushort_as_half(mr[t0 + 16 * rb])) * rfac;
            const float r1 = __half2float(__ushort_as_half(mr[t0 + 16 * rb + 8])) * rfac;
#pragma unroll
            for (int j = 0; j < 8; j++) {
              out[rb][j][0] = fmaf(r0, acc[rb][j][0], out[rb][j][0]); out[rb][j][1] = fmaf(r0, acc[rb][j][1], out[rb][j][1]);
              out[rb][j][2] = fmaf(r1, acc[rb][j][2], out[rb][j][2]); out[rb][j][3] = fmaf(r1, acc[rb][j][3], out[rb][j][3]);
            }
          }
        }
        // ---- + sum_g lo_g u_g + c, then (keys with positions) the rotary pairing, then the stores
#pragma unroll 1
        for (int g = 0; g < n_groups; g++) {
          if (T.meta_off[g] < 0) continue;
          const uint16_t* ml = reinterpret_cast<const uint16_t*>(src + T.meta_off[g]);
          float lo[4];
#pragma unroll
          for (int q = 0; q < 4; q++) lo[q] = __half2float(__ushort_as_half(ml[t0 + 8 * q]));
#pragma unroll
          for (int j = 0; j < 8; j++) {
            const int nn = 32 * pass + 8 * (j & 3) + 64 * (j >> 2) + 2 * tig;
            const float2 ug = *reinterpret_cast<const float2*>(&S.u[g][nn]);
#pragma unroll
            for (int rb = 0; rb < 2; rb++) {
              out[rb][j][0] = fmaf(lo[2 * rb], ug.x, out[rb][j][0]); out[rb][j][1] = fmaf(lo[2 * rb], ug.y, out[rb][j][1]);
              out[rb][j][2] = fmaf(lo[2 * rb + 1], ug.x, out[rb][j][2]); out[rb][j][3] = fmaf(lo[2 * rb + 1], ug.y, out[rb][j][3]);
            }
          }
        }
#pragma unroll
        for (int j = 0; j < 8; j++) {
          const int nn = 32 * pass + 8 * (j & 3) + 64 * (j >> 2) + 2 * tig;
          const float2 cc = *reinterpret_cast<const float2*>(&S.cvec[nn]);
#pragma unroll
          for (int rb = 0; rb < 2; rb++) { out[rb][j][0] += cc.x; out[rb][j][1] += cc.y; out[rb][j][2] += cc.x; out[rb][j][3] += cc.y; }
        }
#pragma unroll
        for (int q = 0; q < 4; q++) {
          const int t = t0 + 8 * q, rb = q >> 1, e0 = 2 * (q & 1);
          if (t >= n_here) continue;
          if (p.rope_cos) {
            const int64_t pos = (p.rope_pos0 ? p.rope_pos0[u] : 0) + tile_pos + t;
#pragma unroll
            for (int j = 0; j < 4; j++) {
              const int i = 32 * pass + 8 * j + 2 * tig;                // pair index: channels i and i + 64
              const float2 cs = *reinterpret_cast<const float2*>(p.rope_cos + pos * (kD / 2) + i);
              const float2 sn = *reinterpret_cast<const float2*>(p.rope_sin + pos * (kD / 2) + i);
              const float x0 = out[rb][j][e0], x1 = out[rb][j][e0 + 1], y0 = out[rb][j + 4][e0], y1 = out[rb][j + 4][e0 + 1];
              out[rb][j][e0] = x0 * cs.x - y0 * sn.x; out[rb][j][e0 + 1] = x1 * cs.y - y1 * sn.y;
              out[rb][j + 4][e0] = y0 * cs.x + x0 * sn.x; out[rb][j + 4][e0 + 1] = y1 * cs.y + x1 * sn.y;
            }
          }
          const int64_t o = p.out_index(u, tile, t);
#pragma unroll
          for (int j = 0; j < 8; j++) {
            const int nn = 32 * pass + 8 * (j & 3) + 64 * (j >> 2) + 2 * tig;
            if (p.out_dtype == SPECTRA_BF16)
              *reinterpret_cast<__nv_bfloat162*>(reinterpret_cast<__nv_bfloat16*>(p.out) + o + nn) = __floats2bfloat162_rn(out[rb][j][e0], out[rb][j][e0 + 1]);
            else
              *reinterpret_cast<float2*>(reinterpret_cast<float*>(p.out) + o + nn) = make_float2(out[rb][j][e0], out[rb][j][e0 + 1]);
          }
        }
      }
      // ---- the half is done with the slot: refill it with the tile three further on
      asm volatile("bar.sync %0, %1;" ::"r"(1 + hf), "n"(kDmHalf) : "memory");
      if (bulk && (tid & (kDmHalf - 1)) == 0 && tt + kDmSlots < n_tiles) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        issue_load(tt + kDmSlots);
      }
    }
    if (bulk) loads_done += n_tiles;
    // ---- end of the run: a timeout anywhere ends the CTA's work (the barrier phases are no longer known)
    if (__syncthreads_or(status & SPECTRA_STATUS_WAIT_TIMEOUT)) break;
  }
  if (status && p.status) atomicOr(p.status, status);
}

}  // namespace spectra
