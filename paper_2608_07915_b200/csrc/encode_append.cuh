// Append path of spectra_encode for a handful of new tokens per unit-side (the decode step appends one).
// One CTA of 128 threads per unit-side, thread j = rotated channel j.  No staging of whole tiles: the thread
// rotates its channel, the CTA reduces the per-group minimum and maximum, every thread quantises its own code and
// writes its sub-fields into the tail tile with 16-bit read-modify-writes.  Different strips never share a
// half-word, and the CTA owns the unit-side, so no atomics are needed.
#pragma once
#include "common.cuh"

namespace spectra {

constexpr int kAppendMaxTokens = 16;

struct AppendArgs {
  const void* x; int x_dtype; int flags; int side; int scale_group;
  int64_t n_param_sets; const int32_t* pos0; int32_t n_new; int64_t stride_unit, stride_token;
  const float* w_enc; const float* mean_rot; const uint8_t* widths;
  uint8_t* cache; const int64_t* unit_offset; int32_t* status;
  const int32_t* seq_len; int n_kv;      // with pos0 == NULL: the token goes to position seq_len[u / n_kv] - 1
  int32_t capacity;                      // tokens a unit-side's buffer holds (0: not checked)
  TileMap map;
};

// Bounded wait for phase 0 of an mbarrier (each poll blocks for a bounded hardware interval).
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar) {
  for (int it = 0; it < (1 << 20); ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar)
        : "memory");
    if (ok) return true;
  }
  return false;
}

constexpr int kAppendDynSmem = kD * kD * 4 + 16;   // W_enc and the barrier of its copy

// The work of one CTA (its first 128 threads; the others leave at once) for unit-side u, thread j = rotated
// channel j.  `smem` is kAppendDynSmem bytes of 16-byte aligned shared memory.  The CTA runs on a cold instruction
// cache and every global read costs a full memory latency, so everything it reads is requested up front: W_enc by
// one bulk copy into shared memory (plain loads when the matrix is not 16-byte aligned), the width, the position,
// the new tokens, the rotated mean and the unit's offset together; the half-words that the new fields are merged
// into are read while the copy is in flight.
__device__ inline void encode_append_body(const AppendArgs& p, int u, unsigned char* smem) {
  __shared__ float xs[kAppendMaxTokens][kD];
  __shared__ float red_lo[4], red_hi[4];
  __shared__ int cls_cnt[4][4];          // [class][warp]: strips of the class owned by the warp's channels
  __shared__ int grp_act[kMaxGroups];
  if (threadIdx.x >= 128) return;
  float* s_w = reinterpret_cast<float*>(smem);
  const uint32_t wbar = (uint32_t)__cvta_generic_to_shared(smem + kD * kD * 4);
  const int ps = (int)(u % p.n_param_sets);
  const int j = threadIdx.x, lane = j & 31, warp = j >> 5;
  const int gs = p.scale_group, n_groups = kD / gs;
  const bool rotated = (p.flags & SPECTRA_ROTATED_INPUT) != 0;
  auto cta_sync = [] { asm volatile("bar.sync 1, 128;" ::: "memory"); };   // the 128 workers only
  const float* w = p.w_enc + (int64_t)ps * kD * kD;
  const bool bulk = !rotated && (reinterpret_cast<uintptr_t>(w) & 15) == 0;
  if (bulk && j == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(wbar) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(wbar), "r"(kD * kD * 4) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     (uint32_t)__cvta_generic_to_shared(s_w)),
                 "l"(w), "r"(kD * kD * 4), "r"(wbar)
                 : "memory");
  }
  const int b = p.widths[(int64_t)ps * kD + j];
  int pos_first = p.pos0 ? p.pos0[u] : p.seq_len[u / p.n_kv] - 1;
  int n_new = p.n_new;
  if (p.capacity > 0 && pos_first + n_new > p.capacity) {   // tokens past the capacity are not written; reported once
    if (j == 0 && p.status) atomicOr(p.status, SPECTRA_STATUS_CAPACITY);
    n_new = max(0, p.capacity - pos_first);
    if (n_new == 0) pos_first = -1;
  }
  const float mr = rotated ? 0.f : p.mean_rot[(int64_t)ps * kD + j];
  uint8_t* base = p.cache + p.unit_offset[u];
  for (int idx = j; idx < p.n_new * kD; idx += 128) {
    const int t = idx / kD, i = idx - t * kD;
    xs[t][i] = load_as_float(p.x, p.x_dtype, (int64_t)u * p.stride_unit + (int64_t)t * p.stride_token + i);
  }
  if (!rotated && !bulk)
    for (int i = 0; i < kD; i++) s_w[i * kD + j] = w[i * kD + j];
  if (j < kMaxGroups) grp_act[j] = 0;
  cta_sync();
  if (pos_first < 0) {                       // fused step on an empty sequence: nothing to append (CTA-uniform)
    if (bulk) mbar_wait_bounded(wbar);       // the copy must land before the shared memory is released
    return;
  }

  // ---- where this channel's strips live: rank inside each class, class offsets, tile size
  int cls_n[4], cls_off[4], my_rank[4];
  int meta_off = -1, tile_bytes = 0;
  {
    int rank_in_warp[4];
#pragma unroll
    for (int c = 0; c < 4; c++) {
      const unsigned m = __ballot_sync(0xffffffffu, (b & (8 >> c)) != 0);
      rank_in_warp[c] = __popc(m & ((1u << lane) - 1u));
      if (lane == 0) cls_cnt[c][warp] = __popc(m);
    }
    if (b) grp_act[j / gs] = 1;
    cta_sync();
    int off = 0;
#pragma unroll
    for (int c = 0; c < 4; c++) {
      int before = 0, n = 0;
#pragma unroll
      for (int wi = 0; wi < 4; wi++) { if (wi < warp) before += cls_cnt[c][wi]; n += cls_cnt[c][wi]; }
      cls_n[c] = n; cls_off[c] = off; my_rank[c] = before + rank_in_warp[c];
      off += 16 * (8 >> c) * n;
    }
    const int payload = off;
    int n_act = 0;
    for (int g = 0; g < n_groups; g++) {
      if (g == j / gs && grp_act[g]) meta_off = payload + 512 * n_act;
      n_act += grp_act[g];
    }
    tile_bytes = payload + 512 * n_act;
  }
  // Half-word and bit of this channel's field of class c for tile slot `slot`.
  auto locate = [&](int c, int slot, int& bo, int& bit) {
    const int wd = 8 >> c, k = my_rank[c], n = cls_n[c];
    if (p.side == SPECTRA_SIDE_V) {
      const int a = slot >> 5, h = (slot >> 4) & 1, i = slot & 15;
      bo = cls_off[c] + 16 * wd * k + 4 * (a * wd + ((i * wd) >> 4)) + 2 * h;
      bit = (i * wd) & 15;
    } else {
      const int hw = (slot * wd) >> 4;
      bit = (slot * wd) & 15;
      if ((k | 1) < n) bo = cls_off[c] + 32 * wd * (k >> 1) + 4 * hw + 2 * (k & 1);
      else bo = cls_off[c] + 16 * wd * k + 2 * hw;
    }
  };
  int status = 0;
  bool w_ready = rotated || !bulk;

  for (int t = 0; t < n_new; t++) {
    const int pos = pos_first + t;
    const int slot = pos & (kTile - 1);
    uint8_t* tile = base + p.map.page(u, pos / kTile) * tile_bytes;
    // the half-words the new fields go into (a tile's first token finds them cleared)
    unsigned old[4] = {0u, 0u, 0u, 0u};
    if (slot != 0) {
#pragma unroll
      for (int c = 0; c < 4; c++)
        if (b & (8 >> c)) {
          int bo, bit;
          locate(c, slot, bo, bit);
          old[c] = *reinterpret_cast<const uint16_t*>(tile + bo);
        }
    }
    if (!w_ready) {
      if (!mbar_wait_bounded(wbar)) status |= SPECTRA_STATUS_WAIT_TIMEOUT;
      w_ready = true;
    }
    // rotate + centre: y_j = sum_i x_i W_enc[i][j] - m'_j (fp32 FMA chain in ascending i)
    float y;
    if (rotated) y = xs[t][j];
    else {
      float a0 = 0.f;
#pragma unroll 8
      for (int i = 0; i < kD; i++) a0 = fmaf(xs[t][i], s_w[i * kD + j], a0);
      y = __fsub_rn(a0, mr);
    }
    if (b && !isfinite(y)) status |= SPECTRA_STATUS_NONFINITE;
    // per-group minimum and maximum over the channels with a non-zero width
    float lo = b ? y : INFINITY, hi = b ? y : -INFINITY;
    const int span = gs < 32 ? gs : 32;                      // lanes of a warp that share a group
    for (int s = span >> 1; s; s >>= 1) {
      lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, s));
      hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, s));
    }
    cta_sync();
    if (lane == 0) { red_lo[warp] = lo; red_hi[warp] = hi; }
    cta_sync();
    if (gs > 32) {
      const int w0 = (j / gs) * (gs / 32);
      lo = red_lo[w0]; hi = red_hi[w0];
      for (int k = 1; k < gs / 32; k++) { lo = fminf(lo, red_lo[w0 + k]); hi = fmaxf(hi, red_hi[w0 + k]); }
    }
    // NaN inputs: fminf/fmaxf drop NaNs, the status bit above reports them
    uint16_t code = 0;
    __half lo16 = __ushort_as_half(0), r16 = __ushort_as_half(0);
    if (meta_off >= 0) {
      float lo_c = lo;
      if (lo_c < -65504.f) { lo_c = -65504.f; status |= SPECTRA_STATUS_F16_RANGE; }
      if (lo_c > 65504.f) { lo_c = 65504.f; status |= SPECTRA_STATUS_F16_RANGE; }
      lo16 = __float2half_rd(lo_c);
      const float lo_f = __half2float(lo16);
      float R = __fsub_rn(hi, lo_f);
      if (!(R <= 65504.f)) { R = 65504.f; status |= SPECTRA_STATUS_F16_RANGE; }
      if (R < 0.f) R = 0.f;
      r16 = __float2half_ru(R);
      const float R_f = __half2float(r16);
      if (b && R_f != 0.f) {
        const float L = (float)((1 << b) - 1);
        float r = rintf(__fmul_rn(__fsub_rn(y, lo_f), __fdiv_rn(L, R_f)));
        if (!(r >= 0.f)) r = 0.f;
        if (r > L) r = L;
        code = (uint16_t)r;
      }
    }
    // ---- write into the tail tile
    if (slot == 0) {                                          // first token of a tile: clear the tile
      for (int i = j; i < tile_bytes / 16; i += 128) reinterpret_cast<uint4*>(tile)[i] = make_uint4(0, 0, 0, 0);
      cta_sync();
    }
#pragma unroll
    for (int c = 0; c < 4; c++) {
      const int wd = 8 >> c;
      if (b & wd) {
        const unsigned field = ((unsigned)code >> (b & (wd - 1))) & ((1u << wd) - 1u);
        int bo, bit;
        locate(c, slot, bo, bit);
        const unsigned below = (1u << bit) - 1u;              // earlier tokens of the half-word are kept
        *reinterpret_cast<uint16_t*>(tile + bo) = (uint16_t)((old[c] & below) | (field << bit));
      }
    }
    if (meta_off >= 0 && (j % gs) == 0) {                     // one writer per scale group
      uint16_t* m = reinterpret_cast<uint16_t*>(tile + meta_off) + slot;
      m[0] = __half_as_ushort(lo16);
      m[kTile] = __half_as_ushort(r16);
    }
    cta_sync();
  }
  if (status && p.status) atomicOr(p.status, status);
}

}  // namespace spectra
