// spectra_decode_attention entry point and host-side helpers of the library.
#include "attention_generic.cuh"

using namespace spectra;

namespace {

int generic_splits(int n_units, int max_seq_len) {
  const int n_tiles = (max_seq_len + kTile - 1) / kTile;
  int splits = (4 * 148 + n_units - 1) / n_units;
  if (splits > n_tiles) splits = n_tiles;
  if (splits < 1) splits = 1;
  if (splits > 1024) splits = 1024;
  return splits;
}

}  // namespace

extern "C" size_t spectra_attention_workspace_bytes(const spectra_config* cfg, int32_t batch, int32_t n_kv_heads,
                                                    int32_t n_q_heads, int32_t max_seq_len) {
  if (check_config(cfg) || batch < 0 || n_kv_heads < 1 || n_q_heads < n_kv_heads || max_seq_len < 0) return 0;
  const int64_t n_units = (int64_t)batch * n_kv_heads;
  if (n_units == 0) return 16;
  const int splits = generic_splits((int)n_units, max_seq_len);
  return (size_t)n_units * splits * (n_q_heads / n_kv_heads) * kPartialStride * sizeof(float) + 16;
}

extern "C" int spectra_decode_attention(const spectra_config* cfg, const void* q, int q_dtype, int32_t batch,
                                        int32_t n_kv_heads, int32_t n_q_heads, const int32_t* seq_len,
                                        int32_t max_seq_len, const uint8_t* cache_k, const int64_t* unit_offset_k,
                                        const uint8_t* cache_v, const int64_t* unit_offset_v, int64_t n_param_sets,
                                        const float* w_dec_k, const float* mean_rot_k, const uint8_t* widths_k,
                                        const float* w_dec_v, const float* mean_rot_v, const uint8_t* widths_v,
                                        float softmax_scale, void* out, int out_dtype, float* lse, void* workspace,
                                        size_t workspace_bytes, int32_t* status_word, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if (batch < 0 || n_kv_heads < 1 || n_q_heads < 1 || n_q_heads % n_kv_heads || max_seq_len < 0 || n_param_sets < 1)
    return SPECTRA_INVALID_ARG;
  if ((q_dtype != SPECTRA_F32 && q_dtype != SPECTRA_BF16) || (out_dtype != SPECTRA_F32 && out_dtype != SPECTRA_BF16))
    return SPECTRA_INVALID_ARG;
  const int gqa = n_q_heads / n_kv_heads;
  if (gqa > kMaxGqa) return SPECTRA_UNSUPPORTED;
  if (batch == 0) return SPECTRA_OK;
  if (!q || !seq_len || !cache_k || !cache_v || !unit_offset_k || !unit_offset_v || !w_dec_k || !w_dec_v ||
      !mean_rot_v || !widths_k || !widths_v || !out || !workspace)
    return SPECTRA_INVALID_ARG;
  if (lse && !mean_rot_k) return SPECTRA_INVALID_ARG;
  const int64_t n_units = (int64_t)batch * n_kv_heads;
  if (n_units > 65535) return SPECTRA_UNSUPPORTED;
  if (workspace_bytes < spectra_attention_workspace_bytes(cfg, batch, n_kv_heads, n_q_heads, max_seq_len))
    return SPECTRA_WORKSPACE_TOO_SMALL;
  AttnArgs a{};
  a.q = q; a.q_dtype = q_dtype; a.batch = batch; a.n_kv = n_kv_heads; a.n_q = n_q_heads; a.gqa = gqa;
  a.seq_len = seq_len; a.scale_group = cfg->scale_group;
  a.cache_k = cache_k; a.off_k = unit_offset_k; a.cache_v = cache_v; a.off_v = unit_offset_v;
  a.n_param_sets = n_param_sets;
  a.w_dec_k = w_dec_k; a.mean_rot_k = mean_rot_k; a.widths_k = widths_k;
  a.w_dec_v = w_dec_v; a.mean_rot_v = mean_rot_v; a.widths_v = widths_v;
  a.scale = softmax_scale != 0.f ? softmax_scale : 1.0f / sqrtf((float)kD);
  a.out = out; a.out_dtype = out_dtype; a.lse = lse;
  a.partials = reinterpret_cast<float*>(workspace);
  a.n_splits = generic_splits((int)n_units, max_seq_len);
  a.status = status_word;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaFuncSetAttribute(attention_generic_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)sizeof(GenericSmem)) != cudaSuccess)
    return SPECTRA_CUDA_ERROR;
  dim3 grid((unsigned)a.n_splits, (unsigned)n_units);
  attention_generic_kernel<<<grid, 128, sizeof(GenericSmem), st>>>(a);
  if (launch_status()) return SPECTRA_CUDA_ERROR;
  attention_combine_kernel<<<(unsigned)n_units, 128, 0, st>>>(a);
  return launch_status();
}

extern "C" size_t spectra_tile_bytes(const spectra_config* cfg, const uint8_t* widths_host) {
  if (check_config(cfg) || !widths_host) return 0;
  size_t bits = 0;
  int n_act = 0;
  for (int g = 0; g < kD / cfg->scale_group; g++) {
    bool any = false;
    for (int j = g * cfg->scale_group; j < (g + 1) * cfg->scale_group; j++) {
      if (widths_host[j] > 8) return 0;
      bits += widths_host[j];
      any |= widths_host[j] != 0;
    }
    n_act += any;
  }
  return 16 * bits + 512 * (size_t)n_act;
}

extern "C" void spectra_config_default(spectra_config* cfg) {
  if (!cfg) return;
  cfg->head_dim = kD; cfg->tile_tokens = kTile; cfg->scale_group = 64; cfg->width_group = 1; cfg->b_max = 8;
  cfg->gain_mode = SPECTRA_GAIN_SQRT; cfg->layout_version = 1;
}

extern "C" const char* spectra_status_string(int code) {
  switch (code) {
    case SPECTRA_OK: return "SPECTRA_OK";
    case SPECTRA_INVALID_ARG: return "SPECTRA_INVALID_ARG";
    case SPECTRA_UNSUPPORTED: return "SPECTRA_UNSUPPORTED";
    case SPECTRA_WORKSPACE_TOO_SMALL: return "SPECTRA_WORKSPACE_TOO_SMALL";
    case SPECTRA_CAPACITY: return "SPECTRA_CAPACITY";
    case SPECTRA_CUDA_ERROR: return "SPECTRA_CUDA_ERROR";
    default: return "SPECTRA_UNKNOWN";
  }
}
