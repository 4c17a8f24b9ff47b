// spectra_prefill_attention: many-query causal attention over the reconstructed (bf16, paged) cache.
#include <cuda_runtime.h>
#include "../../include/spectra.h"
#include "common.cuh"
#include "prefill_umma.cuh"
#include "tensor_map.cuh"

using namespace spectra;

extern "C" int spectra_prefill_attention(const void* q, const void* k_pool, const void* v_pool, int64_t n_pages,
                                         int64_t stride_page, int64_t stride_token, const int32_t* page_table,
                                         int64_t table_stride, int64_t n_seqs, int32_t n_kv_heads, int32_t n_q_heads,
                                         const int32_t* pos0, int32_t n_new, int64_t q_stride_seq,
                                         int64_t q_stride_token, int64_t q_stride_head, float scale, void* out,
                                         int64_t out_stride_seq, int64_t out_stride_token, int64_t out_stride_head,
                                         float* lse, int32_t* status_word, void* stream) {
  if (n_seqs < 0 || n_new < 0 || n_kv_heads < 1 || n_q_heads < n_kv_heads || n_q_heads % n_kv_heads || n_pages < 0 ||
      table_stride < 0 || !(scale > 0.f))
    return SPECTRA_INVALID_ARG;
  if (n_seqs == 0 || n_new == 0) return SPECTRA_OK;
  if (!q || !k_pool || !v_pool || !pos0 || !out || n_pages < 1) return SPECTRA_INVALID_ARG;
  if (!page_table && table_stride < 1) return SPECTRA_INVALID_ARG;
  // rows are moved as 16-byte pieces, the pools are read through tensor maps
  const uintptr_t ptrs = reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out) |
                         reinterpret_cast<uintptr_t>(k_pool) | reinterpret_cast<uintptr_t>(v_pool);
  if (ptrs & 15) return SPECTRA_INVALID_ARG;
  if ((q_stride_seq | q_stride_token | q_stride_head | out_stride_seq | out_stride_token | out_stride_head | stride_page |
       stride_token) & 7)
    return SPECTRA_INVALID_ARG;
  if (stride_token < kD || stride_page < stride_token) return SPECTRA_INVALID_ARG;
  const int n_qblocks = (n_new + kPfRows - 1) / kPfRows;
  const long long grid = (long long)n_qblocks * n_q_heads * n_seqs;
  if (grid > 0x7fffffffLL) return SPECTRA_UNSUPPORTED;
  CUtensorMap kmap, vmap;
  if (!make_token_map(&kmap, k_pool, kTile, n_pages, stride_token, stride_page, kPfSwizzle) ||
      !make_token_map(&vmap, v_pool, kTile, n_pages, stride_token, stride_page, kPfSwizzle))
    return SPECTRA_CUDA_ERROR;
  PrefillArgs a{reinterpret_cast<const __nv_bfloat16*>(q), reinterpret_cast<__nv_bfloat16*>(out), lse,
                q_stride_seq, q_stride_token, q_stride_head, out_stride_seq, out_stride_token, out_stride_head,
                pos0, n_new, (int)n_seqs, n_kv_heads, n_q_heads / n_kv_heads, scale * 1.4426950408889634f,
                page_table, table_stride, status_word, n_qblocks};
  const size_t smem = sizeof(PrefillSmem) + 1024;
  if (cudaFuncSetAttribute(prefill_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return SPECTRA_CUDA_ERROR;
  prefill_attention_kernel<<<(unsigned)grid, kPfThreads, smem, (cudaStream_t)stream>>>(a, kmap, vmap);
  return launch_status();
}
