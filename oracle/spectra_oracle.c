/*
 * SPECTRA KV-cache codec -- CPU oracle (TEST INFRASTRUCTURE, not a product path).
 *
 * A plain, slow, scalar restatement of what the codec computes, written from the
 * paper's method section and appendices.  It exists so that the CUDA library can be
 * checked element by element.  It shares no code with the CUDA path.  Only the test
 * suite, the smoke check and the benchmark's CPU-baseline leg may load it.
 *
 * What is here (one unit = one (layer, sequence, kv-head); one side = keys or values):
 *   - rotate + centre           y = x W_enc - m'            (method Sec. 3.1: the latent
 *                                c = h W_down, with measured coordinate means removed)
 *   - per-token group min/max quantiser at per-channel widths (Sec. 3.2: groups share
 *     a per-token fp16 scale and zero-point; zero-bit channels store nothing)
 *   - the packed tile format (this library's own; the paper fixes only what is stored)
 *   - dequantise + inverse rotate (Mode A reconstruction, Sec. 3.3)
 *   - attention over the coded cache, Mode A (reconstruct, then textbook softmax
 *     attention) and Mode B (latent-space attention, appendix "Latent-space attention
 *     and memory": q' = q W_up^T folded once, scores q' c^T, output lifted once)
 *   - the same two with the rotary position embedding applied to the reconstructed keys (Sec. 3.3)
 *
 * Floating point: the quantiser is IEEE fp32, round-to-nearest-even, one rounding per
 * written operation, no fused multiply-add (compile with -ffp-contract=off).  Rotations,
 * softmax and attention sums are fp64.
 *
 * Packed tile format v1 (128 tokens of one unit-side):
 *   width b in 0..8 is split into its binary digits, "sub-fields" of 8, 4, 2 or 1 bits
 *   (7 -> 4,2,1; 6 -> 4,2; 5 -> 4,1; 3 -> 2,1); the sub-field of size w holds code bits
 *   [s, s+w) with s = b & (w-1).  A "strip" is one sub-field of one channel for all 128
 *   tokens: 128*w bits = 16*w bytes, seen as 8*w little-endian 16-bit half-words; inside
 *   a half-word the field of the i-th token it holds sits at bits [i*w, i*w+w).
 *   Strips are stored by class w = 8, 4, 2, 1, and inside a class by ascending channel.
 *   The half-word order differs by side:
 *     K side: token t is in half-word n = t*w/16 of its strip.  Consecutive strips of a
 *             class are paired; a pair occupies 32*w bytes, 32-bit word n = (half-word n
 *             of the first strip) | (half-word n of the second strip) << 16.  An odd last
 *             strip of a class is stored alone, half-words in order (16*w bytes).
 *     V side: token t = 32*a + 16*h + i (a in 0..3, h in 0..1, i in 0..15) is in 32-bit
 *             word q = a*w + i*w/16 of its strip, in the low (h = 0) or high (h = 1)
 *             half-word, at bits [(i*w)%16, +w).
 *   After the strips, for every scale group that has a non-zero-width channel, in
 *   ascending order: lo16[128] then R16[128] (little-endian fp16, token order).
 *   tile bytes = 16 * sum_j b_j + 512 * (number of active scale groups).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define SPO_TILE 128
#define SPO_MAX_D 512
#define SPO_SIDE_K 0
#define SPO_SIDE_V 1

#define SPO_STATUS_NONFINITE 1
#define SPO_STATUS_F16_RANGE 2

/* ---------------------------------------------------------------- fp16 helpers */

static float spo_half_to_float(uint16_t h) {
  uint32_t sign = (uint32_t)(h >> 15) & 1u;
  int32_t e = (h >> 10) & 0x1f;
  uint32_t m = h & 0x3ffu;
  double v;
  if (e == 0) v = ldexp((double)m, -24);
  else if (e == 31) v = m ? NAN : INFINITY;
  else v = ldexp((double)(m | 0x400u), e - 25);
  return (float)(sign ? -v : v);
}

/* Largest fp16 value <= x (dir < 0) or smallest fp16 value >= x (dir > 0), for finite x
 * with |x| <= 65504.  Written as a search over the ordered fp16 number line, so that
 * the rounding direction is obvious by inspection. */
static uint16_t spo_float_to_half_dir(float x, int dir) {
  /* Map fp16 bit patterns to an ordered integer key: key k in [-31743, 31743],
   * value(k) = sign(k) * half(|k|); half(31743) = 65504 (0x7bff). */
  int lo = -0x7bff, hi = 0x7bff;
  /* binary search for the largest key with value(key) <= x */
  while (lo < hi) {
    int mid = lo + (hi - lo + 1) / 2;
    uint16_t bits = (uint16_t)(mid < 0 ? (0x8000 | (-mid)) : mid);
    if (spo_half_to_float(bits) <= x) lo = mid; else hi = mid - 1;
  }
  int k = lo;                                    /* value(k) <= x < value(k+1) */
  uint16_t bits = (uint16_t)(k < 0 ? (0x8000 | (-k)) : k);
  if (dir > 0 && spo_half_to_float(bits) < x) {
    k += 1;
    bits = (uint16_t)(k < 0 ? (0x8000 | (-k)) : k);
  }
  return bits;
}

uint16_t spo_f2h_down(float x) { return spo_float_to_half_dir(x, -1); }
uint16_t spo_f2h_up(float x) { return spo_float_to_half_dir(x, +1); }
float spo_h2f(uint16_t h) { return spo_half_to_float(h); }

/* ---------------------------------------------------------------- format */

/* Sub-fields of a width, most significant first.  Returns their number. */
int spo_subfields(int b, int* w_out, int* shift_out) {
  int n = 0;
  for (int w = 8; w >= 1; w >>= 1) {
    if (b & w) { w_out[n] = w; shift_out[n] = b & (w - 1); n++; }
  }
  return n;
}

typedef struct {
  int chan, w, shift;
  int mode;        /* 0: alone, natural order; 1: K pair, low half; 2: K pair, high half; 3: V order */
  int64_t base;    /* byte offset in the tile of the strip (mode 0, 3) or of its pair (1, 2) */
} spo_strip;

/* Enumerate the strips of a tile.  Returns their number; *payload_bytes gets the size of the strip region. */
static int spo_strips(const uint8_t* widths, int d, int side, spo_strip* out, int64_t* payload_bytes) {
  int n = 0;
  int64_t off = 0;
  for (int w = 8; w >= 1; w >>= 1) {
    int first = n;
    for (int j = 0; j < d; j++) {
      if (widths[j] & w) {
        out[n].chan = j; out[n].w = w; out[n].shift = widths[j] & (w - 1);
        n++;
      }
    }
    int cnt = n - first;
    for (int i = 0; i < cnt; i++) {
      spo_strip* s = &out[first + i];
      if (side == SPO_SIDE_V) {
        s->mode = 3; s->base = off + (int64_t)16 * w * i;
      } else if ((i | 1) < cnt) {               /* has a partner */
        s->mode = 1 + (i & 1); s->base = off + (int64_t)32 * w * (i / 2);
      } else {                                   /* odd last strip */
        s->mode = 0; s->base = off + (int64_t)16 * w * i;
      }
    }
    off += (int64_t)16 * w * cnt;
  }
  *payload_bytes = off;
  return n;
}

/* Where the field of token t of a strip lives: byte offset of its half-word, bit offset inside it. */
static void spo_locate(const spo_strip* s, int t, int64_t* byte_off, int* bit_off) {
  int w = s->w;
  if (s->mode == 3) {
    int a = t / 32, h = (t % 32) / 16, i = t % 16;
    int q = a * w + (i * w) / 16;
    *byte_off = s->base + 4 * (int64_t)q + 2 * h;
    *bit_off = (i * w) % 16;
  } else {
    int n = (t * w) / 16;
    *bit_off = (t * w) % 16;
    if (s->mode == 0) *byte_off = s->base + 2 * (int64_t)n;
    else *byte_off = s->base + 4 * (int64_t)n + 2 * (s->mode - 1);
  }
}

static int spo_active_groups(const uint8_t* widths, int d, int gs, int* active /* [d/gs] */) {
  int n = 0;
  for (int g = 0; g < d / gs; g++) {
    active[g] = 0;
    for (int j = g * gs; j < (g + 1) * gs; j++) if (widths[j]) active[g] = 1;
    n += active[g];
  }
  return n;
}

int64_t spo_tile_bytes(const uint8_t* widths, int d, int gs) {
  int active[SPO_MAX_D];
  int64_t bits = 0;
  for (int j = 0; j < d; j++) bits += widths[j];
  return 16 * bits + 512 * (int64_t)spo_active_groups(widths, d, gs, active);
}

/* Byte offset of the metadata arrays of scale group g (lo16 at the offset, R16 256 bytes later); -1 if inactive. */
static int64_t spo_meta_offset(const uint8_t* widths, int d, int gs, int g) {
  int active[SPO_MAX_D];
  spo_active_groups(widths, d, gs, active);
  if (!active[g]) return -1;
  int64_t bits = 0;
  for (int j = 0; j < d; j++) bits += widths[j];
  int before = 0;
  for (int k = 0; k < g; k++) before += active[k];
  return 16 * bits + 512 * (int64_t)before;
}

/* Export of the strip table for tests: arrays of length >= 3*d. Returns the strip count. */
int spo_strip_table(const uint8_t* widths, int d, int side, int32_t* chan, int32_t* w, int32_t* shift,
                    int32_t* mode, int64_t* base) {
  spo_strip st[3 * SPO_MAX_D];
  int64_t payload;
  int n = spo_strips(widths, d, side, st, &payload);
  for (int i = 0; i < n; i++) {
    chan[i] = st[i].chan; w[i] = st[i].w; shift[i] = st[i].shift; mode[i] = st[i].mode; base[i] = st[i].base;
  }
  return n;
}

/* ---------------------------------------------------------------- quantiser (fp32, fixed order) */

/* One token.  y[d] rotated, centred coordinates.  codes[d] (0 for zero-width channels),
 * lo16/R16 [d/gs] (0 for inactive groups).  Returns status bits. */
int spo_quantise_token(const float* y, const uint8_t* widths, int d, int gs, uint16_t* codes, uint16_t* lo16,
                       uint16_t* R16) {
  int status = 0;
  for (int g = 0; g < d / gs; g++) {
    int any = 0;
    float lo = 0.f, hi = 0.f;
    for (int j = g * gs; j < (g + 1) * gs; j++) {
      codes[j] = 0;
      if (!widths[j]) continue;
      if (!isfinite(y[j])) status |= SPO_STATUS_NONFINITE;
      if (!any) { lo = hi = y[j]; any = 1; }
      else { if (y[j] < lo) lo = y[j]; if (y[j] > hi) hi = y[j]; }
    }
    lo16[g] = 0; R16[g] = 0;
    if (!any) continue;
    float lo_c = lo;
    if (lo_c < -65504.f) { lo_c = -65504.f; status |= SPO_STATUS_F16_RANGE; }
    if (lo_c > 65504.f) { lo_c = 65504.f; status |= SPO_STATUS_F16_RANGE; }
    lo16[g] = spo_float_to_half_dir(lo_c, -1);
    float lo_f = spo_half_to_float(lo16[g]);
    float R = hi - lo_f;
    if (!(R <= 65504.f)) { R = 65504.f; status |= SPO_STATUS_F16_RANGE; }
    if (R < 0.f) R = 0.f;                        /* only reachable after saturation */
    R16[g] = spo_float_to_half_dir(R, +1);
    float R_f = spo_half_to_float(R16[g]);
    for (int j = g * gs; j < (g + 1) * gs; j++) {
      if (!widths[j]) continue;
      float L = (float)((1 << widths[j]) - 1);
      if (R_f == 0.f) { codes[j] = 0; continue; }
      float inv = L / R_f;
      float diff = y[j] - lo_f;
      float u = diff * inv;
      float r = rintf(u);                        /* ties to even */
      if (!(r >= 0.f)) r = 0.f;
      if (r > L) r = L;
      codes[j] = (uint16_t)r;
    }
  }
  return status;
}

void spo_dequantise_token(const uint16_t* codes, const uint16_t* lo16, const uint16_t* R16, const uint8_t* widths,
                          int d, int gs, float* yhat) {
  for (int j = 0; j < d; j++) {
    if (!widths[j]) { yhat[j] = 0.f; continue; }
    int g = j / gs;
    float lo_f = spo_half_to_float(lo16[g]);
    float R_f = spo_half_to_float(R16[g]);
    if (R_f == 0.f) { yhat[j] = lo_f; continue; }
    float L = (float)((1 << widths[j]) - 1);
    float step = R_f / L;
    float prod = (float)codes[j] * step;
    yhat[j] = prod + lo_f;
  }
}

/* ---------------------------------------------------------------- pack / unpack one token */

static void spo_put16(uint8_t* p, uint16_t v) { p[0] = (uint8_t)(v & 0xff); p[1] = (uint8_t)(v >> 8); }
static uint16_t spo_get16(const uint8_t* p) { return (uint16_t)(p[0] | (p[1] << 8)); }

/* Write token slot t (0..127) of a tile.  Overwrites exactly that token's bits and metadata. */
void spo_pack_token(uint8_t* tile, const uint8_t* widths, int d, int gs, int side, int t, const uint16_t* codes,
                    const uint16_t* lo16, const uint16_t* R16) {
  spo_strip st[3 * SPO_MAX_D];
  int64_t payload;
  int n = spo_strips(widths, d, side, st, &payload);
  for (int k = 0; k < n; k++) {
    int64_t bo; int bit;
    spo_locate(&st[k], t, &bo, &bit);
    uint16_t field = (uint16_t)((codes[st[k].chan] >> st[k].shift) & ((1u << st[k].w) - 1u));
    uint16_t hw = spo_get16(tile + bo);
    uint16_t mask = (uint16_t)(((1u << st[k].w) - 1u) << bit);
    hw = (uint16_t)((hw & ~mask) | (uint16_t)(field << bit));
    spo_put16(tile + bo, hw);
  }
  for (int g = 0; g < d / gs; g++) {
    int64_t mo = spo_meta_offset(widths, d, gs, g);
    if (mo < 0) continue;
    spo_put16(tile + mo + 2 * t, lo16[g]);
    spo_put16(tile + mo + 256 + 2 * t, R16[g]);
  }
}

void spo_unpack_token(const uint8_t* tile, const uint8_t* widths, int d, int gs, int side, int t, uint16_t* codes,
                      uint16_t* lo16, uint16_t* R16) {
  spo_strip st[3 * SPO_MAX_D];
  int64_t payload;
  int n = spo_strips(widths, d, side, st, &payload);
  for (int j = 0; j < d; j++) codes[j] = 0;
  for (int k = 0; k < n; k++) {
    int64_t bo; int bit;
    spo_locate(&st[k], t, &bo, &bit);
    uint16_t hw = spo_get16(tile + bo);
    uint16_t field = (uint16_t)((hw >> bit) & ((1u << st[k].w) - 1u));
    codes[st[k].chan] |= (uint16_t)(field << st[k].shift);
  }
  for (int g = 0; g < d / gs; g++) {
    int64_t mo = spo_meta_offset(widths, d, gs, g);
    if (mo < 0) { lo16[g] = 0; R16[g] = 0; continue; }
    lo16[g] = spo_get16(tile + mo + 2 * t);
    R16[g] = spo_get16(tile + mo + 256 + 2 * t);
  }
}

/* Tokens [0, n) of one unit-side, one spo_unpack_token per token: codes [n, d], lo16 and R16 [n, d / gs]. */
void spo_unpack_unit(const uint8_t* cache, int64_t tile_stride, int64_t n, const uint8_t* widths, int d, int gs,
                     int side, uint16_t* codes, uint16_t* lo16, uint16_t* R16) {
  const int ng = d / gs;
  for (int64_t t = 0; t < n; t++)
    spo_unpack_token(cache + (t / SPO_TILE) * tile_stride, widths, d, gs, side, (int)(t % SPO_TILE), codes + t * d,
                     lo16 + t * ng, R16 + t * ng);
}

/* ---------------------------------------------------------------- rotate / encode / decode */

/* y_j = sum_i x_i W_enc[i][j] - m'_j, accumulated in fp64 in index order, rounded once to fp32. */
void spo_rotate_token(const float* x, const float* w_enc, const float* mean_rot, int d, float* y) {
  for (int j = 0; j < d; j++) {
    double acc = 0.0;
    for (int i = 0; i < d; i++) acc += (double)x[i] * (double)w_enc[(int64_t)i * d + j];
    y[j] = (float)(acc - (double)mean_rot[j]);
  }
}

/* Append n_new tokens at positions pos0.. of one unit-side.  x is [n_new, d] (raw vectors, or rotated
 * centred coordinates when rotated_input != 0).  cache points at the unit-side's first tile; tiles are
 * tile_stride bytes apart.  codes_out (optional) receives [n_new, d] codes.  Returns status bits. */
int spo_encode_unit(const float* x, int rotated_input, const float* w_enc, const float* mean_rot,
                    const uint8_t* widths, int d, int gs, int side, int64_t pos0, int64_t n_new, uint8_t* cache,
                    int64_t tile_stride, uint16_t* codes_out) {
  int status = 0;
  float y[SPO_MAX_D];
  uint16_t codes[SPO_MAX_D], lo16[SPO_MAX_D], R16[SPO_MAX_D];
  for (int64_t i = 0; i < n_new; i++) {
    const float* xi = x + i * d;
    if (rotated_input) memcpy(y, xi, sizeof(float) * (size_t)d);
    else spo_rotate_token(xi, w_enc, mean_rot, d, y);
    status |= spo_quantise_token(y, widths, d, gs, codes, lo16, R16);
    int64_t pos = pos0 + i;
    spo_pack_token(cache + (pos / SPO_TILE) * tile_stride, widths, d, gs, side, (int)(pos % SPO_TILE), codes, lo16,
                   R16);
    if (codes_out) memcpy(codes_out + i * d, codes, sizeof(uint16_t) * (size_t)d);
  }
  return status;
}

/* Reconstruct tokens [0, n) of one unit-side: yhat [n, d] fp32 (optional) and
 * xhat = (yhat + m') W_dec in fp64 [n, d] (optional). */
void spo_decode_unit(const uint8_t* cache, int64_t tile_stride, int64_t n, const float* w_dec, const float* mean_rot,
                     const uint8_t* widths, int d, int gs, int side, float* yhat_out, double* xhat_out) {
  uint16_t codes[SPO_MAX_D], lo16[SPO_MAX_D], R16[SPO_MAX_D];
  float yhat[SPO_MAX_D];
  for (int64_t t = 0; t < n; t++) {
    spo_unpack_token(cache + (t / SPO_TILE) * tile_stride, widths, d, gs, side, (int)(t % SPO_TILE), codes, lo16, R16);
    spo_dequantise_token(codes, lo16, R16, widths, d, gs, yhat);
    if (yhat_out) memcpy(yhat_out + t * d, yhat, sizeof(float) * (size_t)d);
    if (xhat_out) {
      for (int i = 0; i < d; i++) {
        double acc = 0.0;
        for (int j = 0; j < d; j++)
          acc += ((double)yhat[j] + (double)mean_rot[j]) * (double)w_dec[(int64_t)j * d + i];
        xhat_out[t * d + i] = acc;
      }
    }
  }
}

/* ---------------------------------------------------------------- attention, one unit, G query heads */

/* Mode A: reconstruct K-hat, V-hat, then out_h = softmax(scale * q_h K-hat^T) V-hat over tokens [0, n).
 * q [G, d] fp64; out [G, d] fp64; lse [G] = log sum_t exp(scale * q_h . k-hat_t). */
void spo_attention_mode_a(const double* q, int G, const uint8_t* cache_k, int64_t stride_k, const uint8_t* cache_v,
                          int64_t stride_v, int64_t n, const float* w_dec_k, const float* mean_rot_k,
                          const uint8_t* widths_k, const float* w_dec_v, const float* mean_rot_v,
                          const uint8_t* widths_v, int d, int gs, double scale, double* out, double* lse) {
  double* khat = (double*)malloc(sizeof(double) * (size_t)n * d);
  double* vhat = (double*)malloc(sizeof(double) * (size_t)n * d);
  double* s = (double*)malloc(sizeof(double) * (size_t)n);
  spo_decode_unit(cache_k, stride_k, n, w_dec_k, mean_rot_k, widths_k, d, gs, SPO_SIDE_K, NULL, khat);
  spo_decode_unit(cache_v, stride_v, n, w_dec_v, mean_rot_v, widths_v, d, gs, SPO_SIDE_V, NULL, vhat);
  for (int h = 0; h < G; h++) {
    double mx = -INFINITY;
    for (int64_t t = 0; t < n; t++) {
      double acc = 0.0;
      for (int i = 0; i < d; i++) acc += q[h * d + i] * khat[t * d + i];
      s[t] = acc * scale;
      if (s[t] > mx) mx = s[t];
    }
    double l = 0.0;
    for (int64_t t = 0; t < n; t++) { s[t] = exp(s[t] - mx); l += s[t]; }
    for (int i = 0; i < d; i++) {
      double acc = 0.0;
      for (int64_t t = 0; t < n; t++) acc += s[t] * vhat[t * d + i];
      out[h * d + i] = acc / l;
    }
    if (lse) lse[h] = mx + log(l);
  }
  free(khat); free(vhat); free(s);
}

/* Mode B: q'_h = scale * W_dec,K q_h (the up-projection folded into the query once); scores
 * q'_h . (yhat_t + m'_K); o'_h = sum_t p_t yhat^V_t in the rotated value space; one lift
 * out_h = (o'_h / l + m'_V) W_dec,V.  No K-hat or V-hat vector is formed. */
void spo_attention_mode_b(const double* q, int G, const uint8_t* cache_k, int64_t stride_k, const uint8_t* cache_v,
                          int64_t stride_v, int64_t n, const float* w_dec_k, const float* mean_rot_k,
                          const uint8_t* widths_k, const float* w_dec_v, const float* mean_rot_v,
                          const uint8_t* widths_v, int d, int gs, double scale, double* out, double* lse) {
  float* yk = (float*)malloc(sizeof(float) * (size_t)n * d);
  float* yv = (float*)malloc(sizeof(float) * (size_t)n * d);
  double* s = (double*)malloc(sizeof(double) * (size_t)n);
  spo_decode_unit(cache_k, stride_k, n, w_dec_k, mean_rot_k, widths_k, d, gs, SPO_SIDE_K, yk, NULL);
  spo_decode_unit(cache_v, stride_v, n, w_dec_v, mean_rot_v, widths_v, d, gs, SPO_SIDE_V, yv, NULL);
  for (int h = 0; h < G; h++) {
    double qp[SPO_MAX_D], op[SPO_MAX_D];
    double cst = 0.0;
    for (int j = 0; j < d; j++) {
      double acc = 0.0;
      for (int i = 0; i < d; i++) acc += (double)w_dec_k[(int64_t)j * d + i] * q[h * d + i];
      qp[j] = acc * scale;
      cst += qp[j] * (double)mean_rot_k[j];
    }
    double mx = -INFINITY;
    for (int64_t t = 0; t < n; t++) {
      double acc = 0.0;
      for (int j = 0; j < d; j++) acc += qp[j] * (double)yk[t * d + j];
      s[t] = acc + cst;
      if (s[t] > mx) mx = s[t];
    }
    double l = 0.0;
    for (int64_t t = 0; t < n; t++) { s[t] = exp(s[t] - mx); l += s[t]; }
    for (int j = 0; j < d; j++) {
      double acc = 0.0;
      for (int64_t t = 0; t < n; t++) acc += s[t] * (double)yv[t * d + j];
      op[j] = acc / l + (double)mean_rot_v[j];
    }
    for (int i = 0; i < d; i++) {
      double acc = 0.0;
      for (int j = 0; j < d; j++) acc += op[j] * (double)w_dec_v[(int64_t)j * d + i];
      out[h * d + i] = acc;
    }
    if (lse) lse[h] = mx + log(l);
  }
  free(yk); free(yv); free(s);
}

/* ---------------------------------------------------------------- rotary position embedding (RoPE)
 * The paper's latent is taken before the position rotation: Mode A rebuilds K-hat and applies RoPE to it, per token
 * position, before the scores (Sec. 3.3, "Streaming decode").  Convention: the two halves of a vector are paired,
 * (x_i, x_{i + d/2}) is rotated by the angle pos * theta^(-2 i / d), i < d/2 (the "rotate-half" form).  The query
 * handed to the attention functions below is already rotated at its own position. */
void spo_rope_row(double* x, int d, double pos, double theta) {
  const int h = d / 2;
  for (int i = 0; i < h; i++) {
    const double ang = pos * pow(theta, -2.0 * (double)i / (double)d);
    const double c = cos(ang), sn = sin(ang);
    const double a = x[i], b = x[i + h];
    x[i] = a * c - b * sn;
    x[i + h] = b * c + a * sn;
  }
}

/* Reconstruct the keys of one unit and rotate token t at position pos0 + t: xhat [n, d] fp64. */
void spo_decode_unit_rope(const uint8_t* cache, int64_t tile_stride, int64_t n, const float* w_dec,
                          const float* mean_rot, const uint8_t* widths, int d, int gs, int side, double pos0,
                          double theta, double* xhat_out) {
  spo_decode_unit(cache, tile_stride, n, w_dec, mean_rot, widths, d, gs, side, NULL, xhat_out);
  for (int64_t t = 0; t < n; t++) spo_rope_row(xhat_out + t * d, d, pos0 + (double)t, theta);
}

/* Mode A with RoPE: K-hat reconstructed, rotated per position, then textbook softmax attention with V-hat. */
void spo_attention_rope_mode_a(const double* q, int G, const uint8_t* cache_k, int64_t stride_k,
                               const uint8_t* cache_v, int64_t stride_v, int64_t n, const float* w_dec_k,
                               const float* mean_rot_k, const uint8_t* widths_k, const float* w_dec_v,
                               const float* mean_rot_v, const uint8_t* widths_v, int d, int gs, double scale,
                               double pos0, double theta, double* out, double* lse) {
  double* khat = (double*)malloc(sizeof(double) * (size_t)n * d);
  double* vhat = (double*)malloc(sizeof(double) * (size_t)n * d);
  double* s = (double*)malloc(sizeof(double) * (size_t)n);
  spo_decode_unit_rope(cache_k, stride_k, n, w_dec_k, mean_rot_k, widths_k, d, gs, SPO_SIDE_K, pos0, theta, khat);
  spo_decode_unit(cache_v, stride_v, n, w_dec_v, mean_rot_v, widths_v, d, gs, SPO_SIDE_V, NULL, vhat);
  for (int h = 0; h < G; h++) {
    double mx = -INFINITY;
    for (int64_t t = 0; t < n; t++) {
      double acc = 0.0;
      for (int i = 0; i < d; i++) acc += q[h * d + i] * khat[t * d + i];
      s[t] = acc * scale;
      if (s[t] > mx) mx = s[t];
    }
    double l = 0.0;
    for (int64_t t = 0; t < n; t++) { s[t] = exp(s[t] - mx); l += s[t]; }
    for (int i = 0; i < d; i++) {
      double acc = 0.0;
      for (int64_t t = 0; t < n; t++) acc += s[t] * vhat[t * d + i];
      out[h * d + i] = acc / l;
    }
    if (lse) lse[h] = mx + log(l);
  }
  free(khat); free(vhat); free(s);
}

/* Mode B with RoPE: no K-hat is formed.  The rotation is orthogonal, so q . R(p) k-hat = (R(-p) q) . k-hat: per
 * token the query is rotated back by the token's position and folded through W_dec,K, q'_t = scale W_dec,K R(-p_t) q;
 * the score is q'_t . (yhat_t + m'_K).  The value side is that of spo_attention_mode_b. */
void spo_attention_rope_mode_b(const double* q, int G, const uint8_t* cache_k, int64_t stride_k,
                               const uint8_t* cache_v, int64_t stride_v, int64_t n, const float* w_dec_k,
                               const float* mean_rot_k, const uint8_t* widths_k, const float* w_dec_v,
                               const float* mean_rot_v, const uint8_t* widths_v, int d, int gs, double scale,
                               double pos0, double theta, double* out, double* lse) {
  float* yk = (float*)malloc(sizeof(float) * (size_t)n * d);
  float* yv = (float*)malloc(sizeof(float) * (size_t)n * d);
  double* s = (double*)malloc(sizeof(double) * (size_t)n);
  spo_decode_unit(cache_k, stride_k, n, w_dec_k, mean_rot_k, widths_k, d, gs, SPO_SIDE_K, yk, NULL);
  spo_decode_unit(cache_v, stride_v, n, w_dec_v, mean_rot_v, widths_v, d, gs, SPO_SIDE_V, yv, NULL);
  for (int h = 0; h < G; h++) {
    double qr[SPO_MAX_D], qp[SPO_MAX_D], op[SPO_MAX_D];
    double mx = -INFINITY;
    for (int64_t t = 0; t < n; t++) {
      for (int i = 0; i < d; i++) qr[i] = q[h * d + i];
      spo_rope_row(qr, d, -(pos0 + (double)t), theta);
      double acc_s = 0.0;
      for (int j = 0; j < d; j++) {
        double acc = 0.0;
        for (int i = 0; i < d; i++) acc += (double)w_dec_k[(int64_t)j * d + i] * qr[i];
        qp[j] = acc * scale;
        acc_s += qp[j] * ((double)yk[t * d + j] + (double)mean_rot_k[j]);
      }
      s[t] = acc_s;
      if (s[t] > mx) mx = s[t];
    }
    double l = 0.0;
    for (int64_t t = 0; t < n; t++) { s[t] = exp(s[t] - mx); l += s[t]; }
    for (int j = 0; j < d; j++) {
      double acc = 0.0;
      for (int64_t t = 0; t < n; t++) acc += s[t] * (double)yv[t * d + j];
      op[j] = acc / l + (double)mean_rot_v[j];
    }
    for (int i = 0; i < d; i++) {
      double acc = 0.0;
      for (int j = 0; j < d; j++) acc += op[j] * (double)w_dec_v[(int64_t)j * d + i];
      out[h * d + i] = acc;
    }
    if (lse) lse[h] = mx + log(l);
  }
  free(yk); free(yv); free(s);
}

/* ---------------------------------------------------------------- batches of independent units */

/* Units are independent; the loop over them is the only parallel loop (OpenMP, if enabled). */
int spo_encode_units(const float* x, int64_t x_unit_stride, int rotated_input, const float* w_enc,
                     const float* mean_rot, const uint8_t* widths, int d, int gs, int side, int64_t n_units,
                     int64_t pos0, int64_t n_new, uint8_t* cache, const int64_t* unit_offset,
                     const int64_t* tile_stride) {
  int status = 0;
#pragma omp parallel for schedule(dynamic) reduction(| : status)
  for (int64_t u = 0; u < n_units; u++) {
    status |= spo_encode_unit(x + u * x_unit_stride, rotated_input, w_enc + u * (int64_t)d * d, mean_rot + u * d,
                              widths + u * d, d, gs, side, pos0, n_new, cache + unit_offset[u], tile_stride[u], NULL);
  }
  return status;
}

/* q [n_units, G, d] fp64, out [n_units, G, d] fp64, lse [n_units, G]; mode 0 = A, 1 = B. */
void spo_attention_units(int mode, const double* q, int G, int64_t n_units, const int64_t* n_tokens,
                         const uint8_t* cache_k, const int64_t* off_k, const int64_t* stride_k,
                         const uint8_t* cache_v, const int64_t* off_v, const int64_t* stride_v, const float* w_dec_k,
                         const float* mean_rot_k, const uint8_t* widths_k, const float* w_dec_v,
                         const float* mean_rot_v, const uint8_t* widths_v, int d, int gs, double scale, double* out,
                         double* lse) {
#pragma omp parallel for schedule(dynamic)
  for (int64_t u = 0; u < n_units; u++) {
    const int64_t dd = (int64_t)d * d;
    if (mode == 0)
      spo_attention_mode_a(q + u * G * d, G, cache_k + off_k[u], stride_k[u], cache_v + off_v[u], stride_v[u],
                           n_tokens[u], w_dec_k + u * dd, mean_rot_k + u * d, widths_k + u * d, w_dec_v + u * dd,
                           mean_rot_v + u * d, widths_v + u * d, d, gs, scale, out + u * G * d, lse + u * G);
    else
      spo_attention_mode_b(q + u * G * d, G, cache_k + off_k[u], stride_k[u], cache_v + off_v[u], stride_v[u],
                           n_tokens[u], w_dec_k + u * dd, mean_rot_k + u * d, widths_k + u * d, w_dec_v + u * dd,
                           mean_rot_v + u * d, widths_v + u * d, d, gs, scale, out + u * G * d, lse + u * G);
  }
}

#ifdef _OPENMP
#include <omp.h>
int spo_num_threads(void) { return omp_get_max_threads(); }
void spo_set_num_threads(int n) { omp_set_num_threads(n); }
#else
int spo_num_threads(void) { return 1; }
void spo_set_num_threads(int n) { (void)n; }
#endif
