// spectra_decode_attention entry point and host-side helpers of the library.
#include "attention_tc_main.cuh"
#include "attention_tc_combine.cuh"

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

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Token positions of a fused step on the generic path: unit u appends at seq_len[u / n_kv] - 1.
__global__ void step_positions_kernel(const int32_t* seq_len, int n_kv, int n_units, int32_t* pos) {
  const int u = blockIdx.x * blockDim.x + threadIdx.x;
  if (u < n_units) pos[u] = seq_len[u / n_kv] - 1;
}

// Workspace carve-up of the tensor-core path.
struct FastLayout {
  size_t desc_off, prefix_off, warp_off, rec_off, total;
  int total_warps, rec_stride;
};

FastLayout fast_layout(int64_t n_units, int total_warps, int vs_max) {
  FastLayout L{};
  L.total_warps = total_warps;
  L.rec_stride = kFastGqa * (kRecHead + vs_max);
  size_t off = 0;
  L.desc_off = off; off = align_up(off + sizeof(UnitDesc) * (size_t)n_units, 256);
  L.prefix_off = off; off = align_up(off + sizeof(int32_t) * (size_t)(n_units + 1), 256);
  L.warp_off = off; off = align_up(off + sizeof(int4) * (size_t)total_warps, 256);
  L.rec_off = off; off = align_up(off + sizeof(float) * (size_t)L.rec_stride * (size_t)(total_warps + n_units), 256);
  L.total = off;
  return L;
}

// What the host learns from the widths: tile sizes, V strip and block counts.
struct WidthFacts { int max_tile_k = 0, max_tile_v = 0, max_vstrips = 0, max_vblocks = 0; int vb[4] = {0, 0, 0, 0}; bool ok = true; };

WidthFacts width_facts(const uint8_t* wk, const uint8_t* wv, int64_t n_sets) {
  WidthFacts F;
  for (int64_t s = 0; s < n_sets; s++) {
    for (int side = 0; side < 2; side++) {
      const uint8_t* w = (side ? wv : wk) + s * kD;
      int bits = 0, cnt[4] = {0, 0, 0, 0}, act[2] = {0, 0};
      for (int j = 0; j < kD; j++) {
        if (w[j] > 8) { F.ok = false; return F; }
        bits += w[j];
        act[j / 64] |= w[j] != 0;
        for (int c = 0; c < 4; c++) cnt[c] += (w[j] & (8 >> c)) != 0;
      }
      const int tb = 16 * bits + 512 * (act[0] + act[1]);
      if (side == 0) F.max_tile_k = tb > F.max_tile_k ? tb : F.max_tile_k;
      else {
        F.max_tile_v = tb > F.max_tile_v ? tb : F.max_tile_v;
        const int strips = cnt[0] + cnt[1] + cnt[2] + cnt[3];
        const int blocks = (cnt[0] + 15) / 16 + (cnt[1] + 15) / 16 + (cnt[2] + 15) / 16 + (cnt[3] + 15) / 16;
        F.max_vstrips = strips > F.max_vstrips ? strips : F.max_vstrips;
        F.max_vblocks = blocks > F.max_vblocks ? blocks : F.max_vblocks;
        for (int c = 0; c < 4; c++) F.vb[c] = (cnt[c] + 15) / 16 > F.vb[c] ? (cnt[c] + 15) / 16 : F.vb[c];
      }
    }
  }
  return F;
}

template <bool PAGED>
int launch_fast_main_as(const AttnArgs& a, const FastArgs& f, int grid, size_t smem, cudaStream_t st) {
  if (cudaFuncSetAttribute(attention_mma_kernel<PAGED>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
      cudaSuccess)
    return SPECTRA_CUDA_ERROR;
  // programmatic dependent launch: the kernel's set-up (barriers, tensor-memory allocation) overlaps the preceding
  // prep / front kernel; it waits for that kernel's completion before it reads the descriptors
  cudaLaunchConfig_t lc{};
  lc.gridDim = dim3((unsigned)grid); lc.blockDim = dim3(kFastWarps * 32);
  lc.dynamicSmemBytes = smem; lc.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at; lc.numAttrs = 1;
  if (cudaLaunchKernelEx(&lc, attention_mma_kernel<PAGED>, a, f) != cudaSuccess) return SPECTRA_CUDA_ERROR;
  return launch_status();
}
int launch_fast_main(const AttnArgs& a, const FastArgs& f, int grid, size_t smem, cudaStream_t st) {
  return a.map_k.table ? launch_fast_main_as<true>(a, f, grid, smem, st) : launch_fast_main_as<false>(a, f, grid, smem, st);
}

constexpr int kMaxVBlocks = kAccColumns / 4;   // V blocks of 16 strips a warp's share of tensor memory holds

// Launch shape of the tensor-core path for a set of widths: shared-memory slot sizes, CTAs per SM, ring depth and
// whether the V accumulators fit their tensor-memory columns (fits false or depth < 1: the CUDA-core kernel runs).
struct FastPlan { int slot_k, slot_v, ctas_per_sm, depth; bool fits; };

FastPlan plan_fast(const WidthFacts& F) {
  FastPlan P{};
  P.slot_k = (int)align_up((size_t)(F.max_tile_k > 16 ? F.max_tile_k : 16), 128);
  P.slot_v = (int)align_up((size_t)(F.max_tile_v > 16 ? F.max_tile_v : 16), 128);
  const size_t pair = (size_t)P.slot_k + P.slot_v;
  const size_t budget = 200 * 1024;
  P.ctas_per_sm = kFastCtasPerSm;
  while (P.ctas_per_sm > 1 &&
         (size_t)P.ctas_per_sm * (kFastWarps * pair + 2048 + kFastWarps * (64 + kWarpStateBytes)) > budget)
    P.ctas_per_sm--;
  P.depth = (int)(budget / ((size_t)P.ctas_per_sm * kFastWarps * pair));
  if (P.depth > 4) P.depth = 4;
  P.fits = F.max_vblocks <= kMaxVBlocks;
  return P;
}

}  // namespace

extern "C" size_t spectra_attention_workspace_bytes(const spectra_config* cfg, int32_t batch, int32_t n_kv_heads,
                                                    int32_t n_q_heads, int32_t max_seq_len) {
  if (check_config(cfg) || batch < 0 || n_kv_heads < 1 || n_q_heads < n_kv_heads || max_seq_len < 0) return 0;
  const int64_t n_units = (int64_t)batch * n_kv_heads;
  if (n_units == 0) return 16;
  const int splits = generic_splits((int)n_units, max_seq_len);
  const size_t generic = (size_t)n_units * splits * (n_q_heads / n_kv_heads) * kPartialStride * sizeof(float) + 16;
  int sms = sm_count();
  if (sms <= 0) sms = 160;
  const int npass = (n_q_heads / n_kv_heads + kFastGqa - 1) / kFastGqa;
  const size_t fast = fast_layout(n_units * npass, sms * kFastCtasPerSm * kFastWarps, kMaxStrips).total;
  return generic > fast ? generic : fast;
}

namespace {

// New key and value vectors of a fused decode step (NULL new_k: plain attention call).
struct StepAppend {
  const void* new_k; const void* new_v; int x_dtype;
  const float* w_enc_k; const float* w_enc_v; uint8_t* cache_k; uint8_t* cache_v;
};

int attention_impl(const spectra_config* cfg, const void* q, int q_dtype, int32_t batch, int32_t n_kv_heads,
                   int32_t n_q_heads, const int32_t* seq_len, int32_t max_seq_len, const uint8_t* cache_k,
                   const int64_t* unit_offset_k, const uint8_t* cache_v, const int64_t* unit_offset_v,
                   int64_t n_param_sets, const float* w_dec_k, const float* mean_rot_k, const uint8_t* widths_k,
                   const float* w_dec_v, const float* mean_rot_v, const uint8_t* widths_v,
                   const uint8_t* widths_k_host, const uint8_t* widths_v_host, float softmax_scale, void* out,
                   int out_dtype, float* lse, void* workspace, size_t workspace_bytes, int32_t* status_word,
                   void* stream, const StepAppend* app, const int32_t* tile_table_k, const int32_t* tile_table_v,
                   int64_t table_stride) {
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
  if ((widths_k_host == nullptr) != (widths_v_host == nullptr)) return SPECTRA_INVALID_ARG;
  if ((tile_table_k == nullptr) != (tile_table_v == nullptr) || table_stride < 0) return SPECTRA_INVALID_ARG;
  // the kernels read the parameter matrices, the caches and the workspace with 16-byte accesses and bulk copies
  if ((((uintptr_t)w_dec_k | (uintptr_t)w_dec_v | (uintptr_t)cache_k | (uintptr_t)cache_v | (uintptr_t)workspace) & 15) != 0)
    return SPECTRA_INVALID_ARG;
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
  a.max_seq_len = max_seq_len;
  a.map_k = TileMap{tile_table_k, table_stride}; a.map_v = TileMap{tile_table_v, table_stride};
  cudaStream_t st = (cudaStream_t)stream;

  // ---- tensor-core path: scale group 64, host copy of the widths available; a GQA group of more than 4 query
  // heads is taken in passes of 4 (each pass is a unit of its own that reads the same tiles)
  const int npass = (gqa + kFastGqa - 1) / kFastGqa;
  const int64_t n_vunits = n_units * npass;
  if (widths_k_host && cfg->scale_group == 64 && n_vunits <= 65534) {
    const WidthFacts F = width_facts(widths_k_host, widths_v_host, n_param_sets);
    if (!F.ok) return SPECTRA_INVALID_ARG;
    const int sms = sm_count();
    if (sms <= 0) return SPECTRA_CUDA_ERROR;
    const FastPlan P = plan_fast(F);
    const int slot_k = P.slot_k, slot_v = P.slot_v, ctas_per_sm = P.ctas_per_sm, depth = P.depth;
    const size_t pair = (size_t)slot_k + slot_v;
    if (depth >= 1 && P.fits) {
      const int vs_max = (F.max_vstrips + 3) & ~3;     // records are fetched with bulk copies: 16-byte multiples
      FastLayout L = fast_layout(n_vunits, sms * ctas_per_sm * kFastWarps, vs_max);
      if (L.total > workspace_bytes) return SPECTRA_WORKSPACE_TOO_SMALL;
      char* ws = reinterpret_cast<char*>(workspace);
      FastArgs f{};
      f.desc = reinterpret_cast<UnitDesc*>(ws + L.desc_off);
      f.tile_prefix = reinterpret_cast<int32_t*>(ws + L.prefix_off);
      f.warp_start = reinterpret_cast<int4*>(ws + L.warp_off);
      f.records = reinterpret_cast<float*>(ws + L.rec_off);
      f.total_warps = L.total_warps; f.rec_stride = L.rec_stride; f.vs_max = vs_max;
      f.n_units = (int)n_vunits; f.npass = npass; f.depth = depth; f.slot_k = slot_k; f.slot_v = slot_v;
      f.max_vblocks = kMaxVBlocks;
      if (cudaFuncSetAttribute(decode_step_front_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPrepDynSmem) !=
              cudaSuccess ||
          cudaFuncSetAttribute(attention_prep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPrepDynSmem) !=
              cudaSuccess)
        return SPECTRA_CUDA_ERROR;
      if (app) {
        AppendArgs ak{app->new_k, app->x_dtype, 0, SPECTRA_SIDE_K, cfg->scale_group, n_param_sets, nullptr, 1, kD, kD,
                      app->w_enc_k, mean_rot_k, widths_k, app->cache_k, unit_offset_k, status_word, seq_len, n_kv_heads,
                      max_seq_len, a.map_k};
        AppendArgs av{app->new_v, app->x_dtype, 0, SPECTRA_SIDE_V, cfg->scale_group, n_param_sets, nullptr, 1, kD, kD,
                      app->w_enc_v, mean_rot_v, widths_v, app->cache_v, unit_offset_v, status_word, seq_len, n_kv_heads,
                      max_seq_len, a.map_v};
        decode_step_front_kernel<<<(unsigned)(n_vunits + 1 + 2 * n_units), kPrepThreads, kPrepDynSmem, st>>>(
            a, f, ak, av, (int)n_units);
      } else {
        attention_prep_kernel<<<(unsigned)n_vunits + 1, kPrepThreads, kPrepDynSmem, st>>>(a, f);
      }
      if (launch_status()) return SPECTRA_CUDA_ERROR;
      // the last chunk of a K run and the last block of a V class read up to 15 strips past the end of their class
      // (zero rows of B, unused accumulator rows): the pad keeps those reads inside the CTA's shared memory
      const size_t smem = (size_t)kFastWarps * depth * pair + kFastWarps * 64 + kFastWarps * kWarpStateBytes + 2048;
      const int grid = sms * ctas_per_sm;
      rc = launch_fast_main(a, f, grid, smem, st);
      if (rc) return rc;
      if (cudaFuncSetAttribute(attention_mma_combine_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               kCombineDynSmem) != cudaSuccess)
        return SPECTRA_CUDA_ERROR;
      {
        // the combine kernel may start while the main kernel drains: its first group of reads does not depend on the
        // main kernel, and it waits (griddepcontrol.wait) before it touches the partial records
        cudaLaunchConfig_t lc{};
        lc.gridDim = dim3((unsigned)(n_vunits * kFastGqa)); lc.blockDim = dim3(128);
        lc.dynamicSmemBytes = kCombineDynSmem; lc.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = at; lc.numAttrs = 1;
        if (cudaLaunchKernelEx(&lc, attention_mma_combine_kernel, a, f) != cudaSuccess) return SPECTRA_CUDA_ERROR;
      }
      return launch_status();
    }
  }

  // ---- generic path (a fused step appends through the ordinary encode launches first)
  if (app) {
    // positions: lengths minus one, written into the head of the workspace (the partials come after the appends)
    int32_t* pos = reinterpret_cast<int32_t*>(workspace);
    step_positions_kernel<<<(unsigned)((n_units + 255) / 256), 256, 0, st>>>(seq_len, n_kv_heads, (int)n_units, pos);
    rc = spectra_encode(cfg, SPECTRA_SIDE_K, app->new_k, app->x_dtype, 0, n_units, n_param_sets, pos, 1, kD, kD,
                        app->w_enc_k, mean_rot_k, widths_k, app->cache_k, unit_offset_k, max_seq_len, tile_table_k, table_stride,
                        status_word, stream);
    if (rc) return rc;
    rc = spectra_encode(cfg, SPECTRA_SIDE_V, app->new_v, app->x_dtype, 0, n_units, n_param_sets, pos, 1, kD, kD,
                        app->w_enc_v, mean_rot_v, widths_v, app->cache_v, unit_offset_v, max_seq_len, tile_table_v, table_stride,
                        status_word, stream);
    if (rc) return rc;
  }
  if (cudaFuncSetAttribute(attention_generic_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)sizeof(GenericSmem)) != cudaSuccess)
    return SPECTRA_CUDA_ERROR;
  dim3 grid((unsigned)a.n_splits, (unsigned)n_units);
  attention_generic_kernel<<<grid, 128, sizeof(GenericSmem), st>>>(a);
  if (launch_status()) return SPECTRA_CUDA_ERROR;
  attention_combine_kernel<<<(unsigned)n_units, 128, 0, st>>>(a);
  return launch_status();
}

}  // namespace

extern "C" int spectra_decode_attention(const spectra_config* cfg, const void* q, int q_dtype, int32_t batch,
                                        int32_t n_kv_heads, int32_t n_q_heads, const int32_t* seq_len,
                                        int32_t max_seq_len, const uint8_t* cache_k, const int64_t* unit_offset_k,
                                        const uint8_t* cache_v, const int64_t* unit_offset_v, int64_t n_param_sets,
                                        const float* w_dec_k, const float* mean_rot_k, const uint8_t* widths_k,
                                        const float* w_dec_v, const float* mean_rot_v, const uint8_t* widths_v,
                                        const uint8_t* widths_k_host, const uint8_t* widths_v_host,
                                        float softmax_scale, void* out, int out_dtype, float* lse, void* workspace,
                                        size_t workspace_bytes, const int32_t* tile_table_k,
                                        const int32_t* tile_table_v, int64_t table_stride, int32_t* status_word,
                                        void* stream) {
  return attention_impl(cfg, q, q_dtype, batch, n_kv_heads, n_q_heads, seq_len, max_seq_len, cache_k, unit_offset_k,
                        cache_v, unit_offset_v, n_param_sets, w_dec_k, mean_rot_k, widths_k, w_dec_v, mean_rot_v,
                        widths_v, widths_k_host, widths_v_host, softmax_scale, out, out_dtype, lse, workspace,
                        workspace_bytes, status_word, stream, nullptr, tile_table_k, tile_table_v, table_stride);
}

extern "C" int spectra_decode_step(const spectra_config* cfg, const void* q, int q_dtype, const void* new_k,
                                   const void* new_v, int x_dtype, int32_t batch, int32_t n_kv_heads,
                                   int32_t n_q_heads, const int32_t* seq_len, int32_t max_seq_len, uint8_t* cache_k,
                                   const int64_t* unit_offset_k, uint8_t* cache_v, const int64_t* unit_offset_v,
                                   int64_t n_param_sets, const float* w_enc_k, const float* w_dec_k,
                                   const float* mean_rot_k, const uint8_t* widths_k, const float* w_enc_v,
                                   const float* w_dec_v, const float* mean_rot_v, const uint8_t* widths_v,
                                   const uint8_t* widths_k_host, const uint8_t* widths_v_host, float softmax_scale,
                                   void* out, int out_dtype, float* lse, void* workspace, size_t workspace_bytes,
                                   const int32_t* tile_table_k, const int32_t* tile_table_v, int64_t table_stride,
                                   int32_t* status_word, void* stream) {
  if (!new_k || !new_v || !w_enc_k || !w_enc_v || !mean_rot_k || !mean_rot_v) return SPECTRA_INVALID_ARG;
  if (x_dtype != SPECTRA_F32 && x_dtype != SPECTRA_BF16) return SPECTRA_INVALID_ARG;
  const StepAppend app{new_k, new_v, x_dtype, w_enc_k, w_enc_v, cache_k, cache_v};
  return attention_impl(cfg, q, q_dtype, batch, n_kv_heads, n_q_heads, seq_len, max_seq_len, cache_k, unit_offset_k,
                        cache_v, unit_offset_v, n_param_sets, w_dec_k, mean_rot_k, widths_k, w_dec_v, mean_rot_v,
                        widths_v, widths_k_host, widths_v_host, softmax_scale, out, out_dtype, lse, workspace,
                        workspace_bytes, status_word, stream, &app, tile_table_k, tile_table_v, table_stride);
}

extern "C" int spectra_attention_path(const spectra_config* cfg, int32_t n_kv_heads, int32_t n_q_heads,
                                      int64_t n_param_sets, const uint8_t* widths_k_host,
                                      const uint8_t* widths_v_host) {
  if (check_config(cfg) || n_kv_heads < 1 || n_q_heads < 1 || n_q_heads % n_kv_heads || n_param_sets < 1) return -1;
  if (n_q_heads / n_kv_heads > kMaxGqa) return -1;
  if (!widths_k_host || !widths_v_host || cfg->scale_group != 64) return SPECTRA_PATH_CUDA_CORE;
  const WidthFacts F = width_facts(widths_k_host, widths_v_host, n_param_sets);
  if (!F.ok) return -1;
  const FastPlan P = plan_fast(F);
  return P.depth >= 1 && P.fits ? SPECTRA_PATH_TENSOR_CORE : SPECTRA_PATH_CUDA_CORE;
}

extern "C" size_t spectra_cache_bytes(const spectra_config* cfg, const uint8_t* widths_host, int64_t capacity_tokens) {
  const size_t tb = spectra_tile_bytes(cfg, widths_host);
  if (tb == 0 || capacity_tokens < 0) return 0;
  return tb * (size_t)((capacity_tokens + kTile - 1) / kTile);
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
