// spectra_encode and spectra_decode: rotate + per-token group quantiser + bit packing, and its inverse.
// One CTA of 128 threads owns one (unit-side, tile); no other CTA touches that tile, so the
// read-modify-write of a partly filled tail tile needs no atomics.
#include "common.cuh"
#include "encode_append.cuh"
#include "encode_umma.cuh"
#include "decode_umma.cuh"
#include "decode_pairs.cuh"
#include "tensor_map.cuh"

namespace spectra {

constexpr int kLdA = kD + 4;   // row stride of the fp32 operand tile (16-byte aligned rows)
constexpr int kLdY = kD + 1;   // row stride of the result tile (conflict-free per-token reads)
constexpr int kLdC = kD + 4;   // row stride of the byte code tile

struct CodecSmem {
  StripTable tab;
  alignas(16) float a[kTile * kLdA];       // operand rows (tokens) for the 128x128 product
  alignas(16) float y[kTile * kLdY];       // product rows
  alignas(16) uint8_t codes[kTile * kLdC];
  float bias[kD];
};

// out[t][j] = sum_i a[t][i] * W[i][j] for tokens t in [t_lo, t_hi), fp32 FMA chain in ascending i.
// Thread j owns output column j; W (global, row-major) is read through L1 with coalesced rows.
__device__ inline void tile_product(const float* __restrict__ a, const float* __restrict__ w, float* __restrict__ y,
                                    int t_lo, int t_hi) {
  const int j = threadIdx.x;
  for (int t0 = (t_lo / 8) * 8; t0 < t_hi; t0 += 8) {
    float acc[8];
#pragma unroll
    for (int r = 0; r < 8; r++) acc[r] = 0.f;
    for (int i = 0; i < kD; i += 4) {
      const float w0 = __ldg(w + (i + 0) * kD + j), w1 = __ldg(w + (i + 1) * kD + j);
      const float w2 = __ldg(w + (i + 2) * kD + j), w3 = __ldg(w + (i + 3) * kD + j);
#pragma unroll
      for (int r = 0; r < 8; r++) {
        const float4 x = *reinterpret_cast<const float4*>(a + (t0 + r) * kLdA + i);
        acc[r] = fmaf(x.x, w0, acc[r]);
        acc[r] = fmaf(x.y, w1, acc[r]);
        acc[r] = fmaf(x.z, w2, acc[r]);
        acc[r] = fmaf(x.w, w3, acc[r]);
      }
    }
#pragma unroll
    for (int r = 0; r < 8; r++) y[(t0 + r) * kLdY + j] = acc[r];
  }
}

__global__ void __launch_bounds__(128) encode_append_kernel(AppendArgs p) {
  extern __shared__ __align__(16) unsigned char append_smem[];
  encode_append_body(p, blockIdx.x, append_smem);
}

struct EncodeArgs {
  const void* x; int x_dtype; int flags; int side; int scale_group;
  int64_t n_param_sets; const int32_t* pos0; int32_t n_new; int32_t capacity; int64_t stride_unit, stride_token;
  const float* w_enc; const float* mean_rot; const uint8_t* widths;
  uint8_t* cache; const int64_t* unit_offset; int32_t* status; TileMap map;
};

__global__ void __launch_bounds__(128, 1) encode_kernel(EncodeArgs p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  CodecSmem& S = *reinterpret_cast<CodecSmem*>(smem_raw);
  const int u = blockIdx.y;
  const int ps = (int)(u % p.n_param_sets);
  const int tid = threadIdx.x;
  const int pos_first = p.pos0[u];
  int pos_end = pos_first + p.n_new;
  if (p.capacity > 0 && pos_end > p.capacity) {          // tokens past the capacity are not written; reported once
    pos_end = max(p.capacity, pos_first);
    if (blockIdx.x == 0 && tid == 0 && p.status) atomicOr(p.status, SPECTRA_STATUS_CAPACITY);
  }
  const int tile = pos_first / kTile + blockIdx.x;
  const int tile_pos = tile * kTile;
  if (tile_pos >= pos_end) return;
  const int slot_lo = max(pos_first - tile_pos, 0);            // first slot written by this call
  const int slot_hi = min(pos_end - tile_pos, kTile);          // one past the last slot written

  build_strip_table(S.tab, p.widths + (int64_t)ps * kD, p.scale_group);
  const StripTable& T = S.tab;

  // stage the new tokens of this tile (rows outside [slot_lo, slot_hi) are zero)
  const int64_t xbase = (int64_t)u * p.stride_unit + (int64_t)(tile_pos - pos_first) * p.stride_token;
  const bool rotated = (p.flags & SPECTRA_ROTATED_INPUT) != 0;
  for (int idx = tid; idx < kTile * kD; idx += blockDim.x) {
    const int t = idx / kD, i = idx - t * kD;
    float v = 0.f;
    if (t >= slot_lo && t < slot_hi) v = load_as_float(p.x, p.x_dtype, xbase + (int64_t)t * p.stride_token + i);
    if (rotated) S.y[t * kLdY + i] = v; else S.a[t * kLdA + i] = v;
  }
  __syncthreads();
  if (!rotated) {
    tile_product(S.a, p.w_enc + (int64_t)ps * kD * kD, S.y, slot_lo, slot_hi);
    __syncthreads();
    const float mr = p.mean_rot[(int64_t)ps * kD + tid];
    for (int t = slot_lo; t < slot_hi; t++) S.y[t * kLdY + tid] = __fsub_rn(S.y[t * kLdY + tid], mr);
    __syncthreads();
  }

  // quantise: thread t owns token slot t
  const int t = tid;
  const bool mine = t >= slot_lo && t < slot_hi;
  int status = 0;
  __half lo16[kMaxGroups], r16[kMaxGroups];
  for (int g = 0; g < T.n_groups; g++) {
    lo16[g] = __ushort_as_half(0); r16[g] = __ushort_as_half(0);
    if (T.meta_off[g] < 0 || !mine) continue;
    float lo = 0.f, hi = 0.f; bool any = false;
    const int j0 = g * p.scale_group, j1 = j0 + p.scale_group;
    for (int j = j0; j < j1; j++) {
      if (!T.width[j]) continue;
      const float v = S.y[t * kLdY + j];
      if (!isfinite(v)) status |= SPECTRA_STATUS_NONFINITE;
      if (!any) { lo = hi = v; any = true; } else { if (v < lo) lo = v; if (v > hi) hi = v; }
    }
    float lo_c = lo;
    if (lo_c < -65504.f) { lo_c = -65504.f; status |= SPECTRA_STATUS_F16_RANGE; }
    if (lo_c > 65504.f) { lo_c = 65504.f; status |= SPECTRA_STATUS_F16_RANGE; }
    lo16[g] = __float2half_rd(lo_c);
    const float lo_f = __half2float(lo16[g]);
    float R = __fsub_rn(hi, lo_f);
    if (!(R <= 65504.f)) { R = 65504.f; status |= SPECTRA_STATUS_F16_RANGE; }
    if (R < 0.f) R = 0.f;
    r16[g] = __float2half_ru(R);
    const float R_f = __half2float(r16[g]);
    for (int j = j0; j < j1; j++) {
      const int b = T.width[j];
      if (!b) continue;
      const float L = (float)((1 << b) - 1);
      float r = 0.f;
      if (R_f != 0.f) {
        const float inv = __fdiv_rn(L, R_f);
        const float diff = __fsub_rn(S.y[t * kLdY + j], lo_f);
        r = rintf(__fmul_rn(diff, inv));
        if (!(r >= 0.f)) r = 0.f;
        if (r > L) r = L;
      }
      S.codes[t * kLdC + j] = (uint8_t)r;
    }
  }
  if (status && p.status) atomicOr(p.status, status);
  __syncthreads();

  // pack: one half-word of the payload at a time, in storage order
  uint8_t* tile_ptr = p.cache + p.unit_offset[u] + p.map.page(u, tile) * T.tile_bytes;
  const int payload = T.class_off[4];
  if (slot_lo == 0 && slot_hi == kTile) pack_full_tile(T, p.side, S.codes, kLdC, tile_ptr, tid, blockDim.x);
  else
  for (int off = 2 * tid; off < payload; off += 2 * blockDim.x) {
    int w, first;
    const int k = halfword_owner(T, p.side, off, w, first);
    const int chan = T.chan[k], shift = T.shift[k];
    const int per = 16 / w;
    const unsigned fmask = (1u << w) - 1u;
    unsigned hw = 0, keep = 0;
    for (int e = 0; e < per; e++) {
      const int tok = first + e;
      if (tok < slot_lo) keep |= fmask << (e * w);
      else if (tok < slot_hi) hw |= (((unsigned)S.codes[tok * kLdC + chan] >> shift) & fmask) << (e * w);
    }
    uint16_t* dst = reinterpret_cast<uint16_t*>(tile_ptr + off);
    if (keep) hw |= (unsigned)(*dst) & keep;
    *dst = (uint16_t)hw;
  }
  for (int g = 0; g < T.n_groups; g++) {
    if (T.meta_off[g] < 0 || t < slot_lo) continue;
    uint16_t* lo_dst = reinterpret_cast<uint16_t*>(tile_ptr + T.meta_off[g]) + t;
    lo_dst[0] = __half_as_ushort(lo16[g]);
    lo_dst[kTile] = __half_as_ushort(r16[g]);
  }
}

__global__ void __launch_bounds__(128, 1) decode_kernel(DecodeArgs p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  CodecSmem& S = *reinterpret_cast<CodecSmem*>(smem_raw);
  const int u = blockIdx.y;
  const int ps = (int)(u % p.n_param_sets);
  const int tid = threadIdx.x;
  const int n = p.n_tokens[u];
  const int tile = blockIdx.x;
  const int tile_pos = tile * kTile;
  if (tile_pos >= n) return;
  const int n_here = min(n - tile_pos, kTile);

  build_strip_table(S.tab, p.widths + (int64_t)ps * kD, p.scale_group);
  const StripTable& T = S.tab;
  const uint8_t* tile_ptr = p.cache + p.unit_offset[u] + p.map.page(u, tile) * T.tile_bytes;
  S.bias[tid] = p.mean_rot[(int64_t)ps * kD + tid];

  // unpack: thread t gathers the fields of token slot t
  const int t = tid;
  for (int j = 0; j < kD; j += 4) *reinterpret_cast<uint32_t*>(&S.codes[t * kLdC + j]) = 0u;
  for (int k = 0; k < T.n_strips; k++) {
    int bo, bit;
    locate_field(T, p.side, k, t, bo, bit);
    const int w = 8 >> strip_class(T, k);
    const unsigned hw = *reinterpret_cast<const uint16_t*>(tile_ptr + bo);
    const unsigned field = (hw >> bit) & ((1u << w) - 1u);
    S.codes[t * kLdC + T.chan[k]] |= (uint8_t)(field << T.shift[k]);
  }
  __syncthreads();
  // dequantise
  const int64_t obase = (int64_t)u * p.stride_unit + (int64_t)(tile_pos + t) * p.stride_token;
  for (int g = 0; g < T.n_groups; g++) {
    float lo_f = 0.f, R_f = 0.f;
    if (T.meta_off[g] >= 0) {
      const uint16_t* m = reinterpret_cast<const uint16_t*>(tile_ptr + T.meta_off[g]) + t;
      lo_f = __half2float(__ushort_as_half(m[0]));
      R_f = __half2float(__ushort_as_half(m[kTile]));
    }
    for (int j = g * p.scale_group; j < (g + 1) * p.scale_group; j++) {
      const int b = T.width[j];
      float v = 0.f;
      if (b) {
        v = lo_f;
        if (R_f != 0.f) {
          const float step = __fdiv_rn(R_f, (float)((1 << b) - 1));
          v = __fadd_rn(__fmul_rn((float)S.codes[t * kLdC + j], step), lo_f);
        }
      }
      if (p.yhat_out && t < n_here) p.yhat_out[obase + j] = v;
      S.a[t * kLdA + j] = t < n_here ? v + S.bias[j] : 0.f;
    }
  }
  __syncthreads();
  if (!p.out) return;
  tile_product(S.a, p.w_dec + (int64_t)ps * kD * kD, S.y, 0, n_here);
  __syncthreads();
  for (int idx = tid; idx < n_here * kD; idx += blockDim.x) {
    const int tt = idx / kD, i = idx - tt * kD;
    store_from_float(p.out, p.out_dtype, p.out_index(u, tile, tt) + i, S.y[tt * kLdY + i]);
  }
}

}  // namespace spectra

using namespace spectra;

extern "C" int spectra_encode(const spectra_config* cfg, int side, const void* x, int x_dtype, int flags,
                              int64_t n_units, int64_t n_param_sets, const int32_t* pos0, int32_t n_new,
                              int64_t stride_unit, int64_t stride_token, const float* w_enc, const float* mean_rot,
                              const uint8_t* widths, uint8_t* cache, const int64_t* unit_offset,
                              int32_t capacity_tokens, const int32_t* tile_table, int64_t table_stride,
                              int32_t* status_word, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if ((side != SPECTRA_SIDE_K && side != SPECTRA_SIDE_V) || n_units < 0 || n_new < 0 || n_param_sets < 1 ||
      capacity_tokens < 0 || table_stride < 0)
    return SPECTRA_INVALID_ARG;
  const TileMap map{tile_table, table_stride};
  if (x_dtype != SPECTRA_F32 && x_dtype != SPECTRA_BF16) return SPECTRA_INVALID_ARG;
  if (flags & ~SPECTRA_ROTATED_INPUT) return SPECTRA_INVALID_ARG;
  if ((flags & SPECTRA_ROTATED_INPUT) && x_dtype != SPECTRA_F32) return SPECTRA_INVALID_ARG;
  if (n_units == 0 || n_new == 0) return SPECTRA_OK;
  if (!x || !pos0 || !widths || !cache || !unit_offset) return SPECTRA_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(cache) & 15) return SPECTRA_INVALID_ARG;      // tiles are cleared and packed with 16- and 4-byte stores
  if (!(flags & SPECTRA_ROTATED_INPUT) && (!w_enc || !mean_rot)) return SPECTRA_INVALID_ARG;
  if (n_units > 65535) return SPECTRA_UNSUPPORTED;
  if (n_new <= kAppendMaxTokens) {   // decode-step appends: one light CTA per unit-side
    AppendArgs ap{x, x_dtype, flags, side, cfg->scale_group, n_param_sets, pos0, n_new, stride_unit, stride_token,
                  w_enc, mean_rot, widths, cache, unit_offset, status_word, nullptr, 1, capacity_tokens, map};
    if (cudaFuncSetAttribute(encode_append_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kAppendDynSmem) !=
        cudaSuccess)
      return SPECTRA_CUDA_ERROR;
    encode_append_kernel<<<(unsigned)n_units, 128, kAppendDynSmem, (cudaStream_t)stream>>>(ap);
    return launch_status();
  }
  if (x_dtype == SPECTRA_BF16 && !(flags & SPECTRA_ROTATED_INPUT) && cfg->scale_group == 64 &&
      stride_token % 8 == 0 && stride_unit % 8 == 0 && (reinterpret_cast<uintptr_t>(x) & 15) == 0) {
    // bf16 bulk encode: rotation on the tensor cores
    EncodeTcArgs ta{reinterpret_cast<const __nv_bfloat16*>(x), side, n_param_sets, pos0, n_new, capacity_tokens, stride_unit,
                    stride_token, w_enc, mean_rot, widths, cache, unit_offset, status_word, map};
    // rotation on the 5th-generation tensor cores (accumulator tiles in tensor memory); the token tiles arrive by
    // TMA: a 3-D map over x [unit][token][channel] whose box is 8 channels x 128 tokens
    CUtensorMap xmap;
    if (make_token_map(&xmap, x, n_new, n_units, stride_token, stride_unit, true)) {
      const size_t um_smem = sizeof(EncodeUmmaSmem) + 1024;
      if (cudaFuncSetAttribute(encode_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)um_smem) !=
          cudaSuccess)
        return SPECTRA_CUDA_ERROR;
      const unsigned tiles = (unsigned)((n_new + 2 * kTile - 2) / kTile);
      const int n_groups = (int)tiles;                   // tile slots per unit
      const long long n_items = (long long)n_groups * n_units;
      const int sms = sm_count();
      if (sms <= 0 || n_items > 0x7fffffffLL) return SPECTRA_CUDA_ERROR;
      const unsigned grid = (unsigned)(n_items < sms ? n_items : sms);
      encode_umma_kernel<<<grid, kUmThreads, um_smem, (cudaStream_t)stream>>>(ta, xmap, n_groups, (int)n_items);
      return launch_status();
    }
  }
  EncodeArgs a{x, x_dtype, flags, side, cfg->scale_group, n_param_sets, pos0, n_new, capacity_tokens, stride_unit, stride_token,
               w_enc, mean_rot, widths, cache, unit_offset, status_word, map};
  if (cudaFuncSetAttribute(encode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(CodecSmem)) !=
      cudaSuccess)
    return SPECTRA_CUDA_ERROR;
  dim3 grid((unsigned)((n_new + 2 * kTile - 2) / kTile), (unsigned)n_units);
  encode_kernel<<<grid, 128, sizeof(CodecSmem), (cudaStream_t)stream>>>(a);
  return launch_status();
}

namespace {
int decode_impl(const spectra_config* cfg, int side, const uint8_t* cache, const int64_t* unit_offset, int64_t n_units,
                int64_t n_param_sets, const int32_t* n_tokens, int32_t max_tokens, const float* w_dec,
                const float* mean_rot, const uint8_t* widths, void* out, int out_dtype, float* yhat_out,
                int64_t stride_unit, int64_t stride_token, const int32_t* tile_table, int64_t table_stride,
                const int32_t* rope_pos0, const float* rope_cos, const float* rope_sin, const int32_t* out_table,
                int64_t out_table_stride, int32_t* status_word, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if ((side != SPECTRA_SIDE_K && side != SPECTRA_SIDE_V) || n_units < 0 || max_tokens < 0 || n_param_sets < 1 ||
      table_stride < 0)
    return SPECTRA_INVALID_ARG;
  if (out_dtype != SPECTRA_F32 && out_dtype != SPECTRA_BF16) return SPECTRA_INVALID_ARG;
  if (n_units == 0 || max_tokens == 0) return SPECTRA_OK;
  if (!cache || !unit_offset || !n_tokens || !widths || !mean_rot) return SPECTRA_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(cache) & 1) return SPECTRA_INVALID_ARG;       // the packed fields are read as half-words
  if (!out && !yhat_out) return SPECTRA_INVALID_ARG;
  if (out && !w_dec) return SPECTRA_INVALID_ARG;
  if (n_units > 65535) return SPECTRA_UNSUPPORTED;
  DecodeArgs a{cache, unit_offset, side, cfg->scale_group, n_param_sets, n_tokens, w_dec, mean_rot, widths, out,
               out_dtype, yhat_out, stride_unit, stride_token, status_word, TileMap{tile_table, table_stride},
               rope_cos, rope_sin, rope_pos0, TileMap{out_table, out_table_stride}};
  if (out && !yhat_out) {
    // reconstruction with the packed fields themselves as the tensor-core operand: decode_pair_kernel takes the units it
    // can hold (up to two scale groups and 192 strip positions, tiles up to 10 KB, aligned sources), decode_tc_kernel
    // behind it exactly the others
    const int tiles = (int)((max_tokens + kTile - 1) / kTile);
    const long long n_slots = (long long)tiles * n_units;
    const int sms = sm_count();
    if (sms <= 0 || n_slots > 0x7fffffffLL) return SPECTRA_CUDA_ERROR;
    const unsigned grid = (unsigned)(n_slots < sms ? n_slots : sms);
    const size_t smem_p = sizeof(DecodePairSmem) + 128, smem_t = sizeof(DecodeTcSmem) + 128;
    if (cudaFuncSetAttribute(decode_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_p) != cudaSuccess ||
        cudaFuncSetAttribute(decode_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_t) != cudaSuccess)
      return SPECTRA_CUDA_ERROR;
    decode_pair_kernel<<<grid, kDpThreads, smem_p, (cudaStream_t)stream>>>(a, tiles, (int)n_slots);
    if (launch_status()) return SPECTRA_CUDA_ERROR;
    decode_tc_kernel<<<grid, kDecThreads, smem_t, (cudaStream_t)stream>>>(a, tiles, (int)n_slots, 1);
    return launch_status();
  }
  if (out) {   // reconstruction: inverse rotation on the tensor cores (tcgen05), persistent grid
    const size_t dec_smem = sizeof(DecodeTcSmem) + 128;
    if (cudaFuncSetAttribute(decode_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dec_smem) !=
        cudaSuccess)
      return SPECTRA_CUDA_ERROR;
    const int tiles = (int)((max_tokens + kTile - 1) / kTile);
    const long long n_slots = (long long)tiles * n_units;
    const int sms = sm_count();
    if (sms <= 0 || n_slots > 0x7fffffffLL) return SPECTRA_CUDA_ERROR;
    const unsigned grid_tc = (unsigned)(n_slots < sms ? n_slots : sms);
    decode_tc_kernel<<<grid_tc, kDecThreads, dec_smem, (cudaStream_t)stream>>>(a, tiles, (int)n_slots, 0);
    return launch_status();
  }
  if (cudaFuncSetAttribute(decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(CodecSmem)) !=
      cudaSuccess)
    return SPECTRA_CUDA_ERROR;
  dim3 grid((unsigned)((max_tokens + kTile - 1) / kTile), (unsigned)n_units);
  decode_kernel<<<grid, 128, sizeof(CodecSmem), (cudaStream_t)stream>>>(a);
  return launch_status();
}
}  // namespace

extern "C" int spectra_decode(const spectra_config* cfg, int side, const uint8_t* cache, const int64_t* unit_offset,
                              int64_t n_units, int64_t n_param_sets, const int32_t* n_tokens, int32_t max_tokens,
                              const float* w_dec, const float* mean_rot, const uint8_t* widths, void* out,
                              int out_dtype, float* yhat_out, int64_t stride_unit, int64_t stride_token,
                              const int32_t* tile_table, int64_t table_stride, int32_t* status_word, void* stream) {
  return decode_impl(cfg, side, cache, unit_offset, n_units, n_param_sets, n_tokens, max_tokens, w_dec, mean_rot, widths,
                     out, out_dtype, yhat_out, stride_unit, stride_token, tile_table, table_stride, nullptr, nullptr,
                     nullptr, nullptr, 0, status_word, stream);
}

extern "C" int spectra_decode_rope(const spectra_config* cfg, const uint8_t* cache, const int64_t* unit_offset,
                                   int64_t n_units, int64_t n_param_sets, const int32_t* n_tokens, int32_t max_tokens,
                                   const float* w_dec, const float* mean_rot, const uint8_t* widths, void* out,
                                   int out_dtype, int64_t stride_unit, int64_t stride_token, const int32_t* tile_table,
                                   int64_t table_stride, const int32_t* position0, const float* rope_cos,
                                   const float* rope_sin, int32_t* status_word, void* stream) {
  if (!out || !rope_cos || !rope_sin) return SPECTRA_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(rope_cos) | reinterpret_cast<uintptr_t>(rope_sin)) & 15) return SPECTRA_INVALID_ARG;
  return decode_impl(cfg, SPECTRA_SIDE_K, cache, unit_offset, n_units, n_param_sets, n_tokens, max_tokens, w_dec,
                     mean_rot, widths, out, out_dtype, nullptr, stride_unit, stride_token, tile_table, table_stride,
                     position0, rope_cos, rope_sin, nullptr, 0, status_word, stream);
}

extern "C" int spectra_decode_paged(const spectra_config* cfg, int side, const uint8_t* cache, const int64_t* unit_offset,
                                    int64_t n_units, int64_t n_param_sets, const int32_t* n_tokens, int32_t max_tokens,
                                    const float* w_dec, const float* mean_rot, const uint8_t* widths, void* out_pool,
                                    int out_dtype, int64_t stride_page, int64_t stride_token, const int32_t* tile_table,
                                    int64_t table_stride, const int32_t* out_table, int64_t out_table_stride,
                                    const int32_t* position0, const float* rope_cos, const float* rope_sin,
                                    int32_t* status_word, void* stream) {
  if (!out_pool || !out_table || out_table_stride < (max_tokens + kTile - 1) / kTile) return SPECTRA_INVALID_ARG;
  if ((rope_cos == nullptr) != (rope_sin == nullptr)) return SPECTRA_INVALID_ARG;
  if (rope_cos && side != SPECTRA_SIDE_K) return SPECTRA_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(rope_cos) | reinterpret_cast<uintptr_t>(rope_sin)) & 15) return SPECTRA_INVALID_ARG;
  return decode_impl(cfg, side, cache, unit_offset, n_units, n_param_sets, n_tokens, max_tokens, w_dec, mean_rot, widths,
                     out_pool, out_dtype, nullptr, stride_page, stride_token, tile_table, table_stride, position0,
                     rope_cos, rope_sin, out_table, out_table_stride, status_word, stream);
}

extern "C" int spectra_selftest_quotients(int64_t* mismatches, void* stream) {
  if (!mismatches) return SPECTRA_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemsetAsync(mismatches, 0, sizeof(int64_t), st) != cudaSuccess) return SPECTRA_CUDA_ERROR;
  selftest_quotients_kernel<<<0x7c00 / 256, 256, 0, st>>>(reinterpret_cast<unsigned long long*>(mismatches));
  return launch_status();
}
