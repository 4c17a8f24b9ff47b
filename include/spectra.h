/*
 * libspectra -- SPECTRA KV-cache codec, data-parallel hot path, for NVIDIA B200 (sm_100a).
 *
 * C ABI.  Every pointer marked "device" is caller-owned device memory (any allocator);
 * pointers marked "host" are ordinary host memory.  The library allocates nothing and carries
 * no results from one call to the next (all it remembers is, per device, the address of the fixed
 * scratch array of spectra_fit_basis_static).  All work is enqueued on `stream` (a cudaStream_t passed as void*,
 * NULL = the legacy default stream) and the calls return without synchronising.  Arguments
 * are validated on the host before anything is launched; a non-zero return value means that
 * nothing was enqueued.  Data-dependent anomalies (non-finite input, metadata beyond the
 * fp16 range, a token position beyond the stated capacity, a unit whose layout does not match
 * the host's copy of the widths) are OR-ed into a caller-supplied device status word, never trapped.
 *
 * Vocabulary (paper notation).  A unit is one (sequence, kv-head) of one layer; a side is its
 * keys (K) or values (V).  d = head_dim = 128.  Per unit-side the codec holds a decorrelating
 * transform fitted from the cache's own second moment (Sec. 3.1, Eq. 3-4):
 *     W_enc [d, d] (rotate + gain), W_dec [d, d] (its inverse), m' [d] (rotated mean),
 * and integer per-channel bit widths b_j in [0, b_max] from reverse water-filling (Sec. 3.2,
 * Eq. 5).  A token x (row vector) is stored as codes of y = x W_enc - m'.
 *
 * Parameter sets.  Transforms and widths usually depend on (layer, kv-head) only and are
 * shared by the sequences of a batch: calls take `n_param_sets`, and unit u uses parameter
 * set (u % n_param_sets).  With units ordered [sequence][kv-head] and n_param_sets = number
 * of kv-heads this is "one set per head".
 *
 * Quantiser (Sec. 3.2: per-token min/max per group, one fp16 zero-point and scale per token
 * per group, zero-bit channels dropped).  For each token and each scale group G of
 * `scale_group` adjacent channels, over the channels with b_j > 0 only, in IEEE fp32,
 * round-to-nearest-even, one rounding per operation, nothing fused:
 *     lo = min y_j, hi = max y_j
 *     lo16 = fp16 round-down(clamp(lo, +-65504));  lo_f = float(lo16)
 *     R16  = fp16 round-up(min(hi - lo_f, 65504)); R_f  = float(R16)
 *     L_j = 2^b_j - 1;  code_j = 0 if R_f == 0 else clamp(rint((y_j - lo_f) * (L_j / R_f)), 0, L_j)
 *     reconstruction: yhat_j = lo_f if R_f == 0 else (float(code_j) * (R_f / L_j)) + lo_f;  b_j == 0: yhat_j = 0
 *
 * Packed tile format v1 (128 consecutive tokens of one unit-side; tiles of a unit-side are
 * contiguous, tile t of unit u starts at cache + unit_offset[u] + t * spectra_tile_bytes()):
 *   - A width b is split into its binary digits, sub-fields of 8, 4, 2 or 1 bits
 *     (7 -> 4,2,1; 6 -> 4,2; 5 -> 4,1; 3 -> 2,1); the sub-field of size w holds code bits
 *     [s, s+w), s = b & (w-1).
 *   - A strip is one sub-field of one channel for the 128 tokens: 16*w bytes, seen as 8*w
 *     little-endian 16-bit half-words; the i-th token of a half-word sits at bits [i*w, i*w+w).
 *   - Strips are stored by class w = 8, 4, 2, 1 and, inside a class, by ascending channel.
 *   - K side: token t is in half-word n = t*w/16.  Consecutive strips of a class are paired;
 *     a pair takes 32*w bytes and its 32-bit word n is (half-word n of the first strip) |
 *     (half-word n of the second) << 16.  An odd last strip is stored alone, half-words in order.
 *   - V side: token t = 32a + 16h + i (a < 4, h < 2, i < 16) is in 32-bit word q = a*w + i*w/16
 *     of its strip, low (h = 0) or high (h = 1) half-word, at bits [(i*w) % 16, +w).
 *   - Then, for each scale group with a non-zero-width channel, ascending: lo16[128], R16[128]
 *     (little-endian fp16, token order).
 *   - tile bytes = 16 * sum_j b_j + 512 * (number of active scale groups); always a multiple of 16.
 *   Paged caches.  Every call that addresses tiles takes an optional tile table (device int32) and its row stride:
 *   with a table, unit_offset[u] is the base of a pool of tile-sized pages (spectra_tile_bytes each; units that share
 *   a parameter set may share a pool) and tile t of unit u is page tile_table[u * table_stride + t] of that pool.
 *   NULL means contiguous tiles as above.  The streaming cache of Sec. 3.3 then grows one page at a time.
 *   The K-side pairing puts two channels of one token 16 bits apart in a word, the V-side order
 *   puts two tokens of one channel 16 bits apart: what the tensor-core operand registers of the
 *   score and of the value contraction need, respectively.
 */
#ifndef SPECTRA_H_
#define SPECTRA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* return codes */
#define SPECTRA_OK 0
#define SPECTRA_INVALID_ARG 1
#define SPECTRA_UNSUPPORTED 2
#define SPECTRA_WORKSPACE_TOO_SMALL 3
#define SPECTRA_CAPACITY 4
#define SPECTRA_CUDA_ERROR 5

/* element types of caller tensors */
#define SPECTRA_F32 0
#define SPECTRA_BF16 1

#define SPECTRA_SIDE_K 0
#define SPECTRA_SIDE_V 1

/* spectra_encode flags */
#define SPECTRA_ROTATED_INPUT 1 /* x already holds y = x W_enc - m' in fp32; the rotation is skipped */

/* bits of the device status word */
#define SPECTRA_STATUS_NONFINITE 1 /* a non-finite coordinate reached the quantiser */
#define SPECTRA_STATUS_F16_RANGE 2 /* a group minimum or range was saturated to the fp16 range */
#define SPECTRA_STATUS_WAIT_TIMEOUT 4 /* a bounded wait on an on-chip copy gave up; the results are invalid */
#define SPECTRA_STATUS_CAPACITY 8 /* a token position beyond the stated capacity: that token was not written (append) or
                                     the sequence was attended as empty (attention) */
#define SPECTRA_STATUS_BAD_LAYOUT 16 /* the tensor-core attention path found a unit whose device-side widths or offsets
                                        do not match what the host copy of the widths promised (tile larger than its
                                        shared-memory slot, more strips than the kernel variant holds, tile stream not
                                        16-byte aligned): the unit's tiles were not read and its output is invalid */

/* return values of spectra_attention_path */
#define SPECTRA_PATH_CUDA_CORE 0
#define SPECTRA_PATH_TENSOR_CORE 1

#define SPECTRA_GAIN_ROTATE 0 /* gamma = 1: a pure rotation */
#define SPECTRA_GAIN_SQRT 1   /* gamma_j = lambda_j^(-1/4): the paper's square-root split (Eq. 3) */
#define SPECTRA_GAIN_WHITEN 2 /* gamma_j = var_j^(-1/2): the pure-whitening split of the paper's footnote */

typedef struct spectra_config {
  int32_t head_dim;       /* 128 (other values: SPECTRA_UNSUPPORTED) */
  int32_t tile_tokens;    /* 128 */
  int32_t scale_group;    /* channels sharing one (lo16, R16) per token: 32, 64 (paper default) or 128 */
  int32_t width_group;    /* adjacent channels sharing one width in spectra_alloc_bits: power of two, 1..scale_group */
  int32_t b_max;          /* largest width, 1..8 */
  int32_t gain_mode;      /* SPECTRA_GAIN_* (used by spectra_fit_basis only) */
  int32_t layout_version; /* 1 */
} spectra_config;

/* ------------------------------------------------------------------------------------------------
 * spectra_fit_basis -- Sec. 3.1, Eq. 3-4 and the appendix "G-Weighted SVD", restated on cache vectors:
 * the right singular basis of the whitened weight is the eigenbasis of the uncentred second moment of
 * the produced keys, so per unit-side
 *     C = X^T X / N, mu = mean(X)            (fp32 partial sums over at most 256 tokens, fp64 across them)
 *     C = U diag(lambda) U^T, lambda descending, each eigenvector's largest component positive (fp64 Jacobi)
 *     m = mu U, var_j = max(lambda_j - m_j^2, 0), gains gamma per cfg->gain_mode (floor 1e-12 lambda_1)
 *     W_enc = U diag(gamma), W_dec = diag(1/gamma) U^T, m' = m * gamma,
 *     var_alloc = var * gamma^2 (ROTATE, SQRT) or var (WHITEN)
 * x: device, element type x_dtype; unit u, token t, channel i at x[u*stride_unit + t*stride_token + i]
 *    (strides in elements).  n_tokens >= 1.
 * Outputs (device, fp32): w_enc, w_dec, basis_u [n_units, d, d] row-major; mean_rot, var_alloc, eigval
 *    [n_units, d].  basis_u and eigval may be NULL.
 * workspace: device, at least spectra_fit_workspace_bytes(cfg, n_units) bytes, 16-byte aligned.
 * bf16 input with a 16-byte aligned x and strides that are multiples of 8 elements forms X^T X on the tensor cores,
 * one CTA per unit-side with the partial sums added in token order: two calls on the same input give the same bits.
 * Other inputs use a CUDA-core kernel whose fp64 atomic additions leave the last bits run-dependent.  Should a
 * bounded wait of the tensor-core kernel give up, that unit's outputs are NaN.
 */
int spectra_fit_basis(const spectra_config* cfg, const void* x, int x_dtype, int64_t n_units, int64_t n_tokens,
                      int64_t stride_unit, int64_t stride_token, float* w_enc, float* w_dec, float* mean_rot,
                      float* var_alloc, float* eigval, float* basis_u, void* workspace, size_t workspace_bytes,
                      void* stream);
size_t spectra_fit_workspace_bytes(const spectra_config* cfg, int64_t n_units);

/* ------------------------------------------------------------------------------------------------
 * spectra_fit_basis_static -- the paper has no counterpart; this is a packaging variant of spectra_fit_basis for
 * callers that may not allocate device memory at the point where they calibrate: a serving plug-in that lives
 * inside a host process with a fixed, pre-carved memory arena, or a component started after the process has
 * frozen its allocator (allocation there would synchronise the device or is simply forbidden).  It takes the
 * same inputs and writes the same outputs, but needs no workspace argument: the scratch (second-moment sums and
 * means, fp64) lives in a fixed array inside the library image, sized for at most
 * SPECTRA_FIT_STATIC_MAX_UNITS unit-sides per call (about 132 KB each, 1.1 MB in all, held by every device that
 * loads the library until the process exits).
 *   - n_units > SPECTRA_FIT_STATIC_MAX_UNITS returns SPECTRA_CAPACITY and enqueues nothing; fit larger sets in
 *     slices of that many unit-sides.
 *   - The first call on a device looks up the device address of the array (with that device current); make that
 *     first call outside any stream capture.  Later calls on the same device reuse the address.
 *   - The call allocates nothing and calls no allocating routine.  All calls on a device share the one array,
 *     which still holds the previous call's contents when a call starts; the call clears what it accumulates
 *     into.  Two calls whose GPU work overlaps (different streams, no ordering between them) would race on the
 *     array: order them.
 */
#define SPECTRA_FIT_STATIC_MAX_UNITS 8
int spectra_fit_basis_static(const spectra_config* cfg, const void* x, int x_dtype, int64_t n_units,
                             int64_t n_tokens, int64_t stride_unit, int64_t stride_token, float* w_enc,
                             float* w_dec, float* mean_rot, float* var_alloc, float* eigval, float* basis_u,
                             void* stream);

/* ------------------------------------------------------------------------------------------------
 * spectra_alloc_bits -- Sec. 3.2, Eq. 5 and the appendix "Reverse water-filling derivation": integer
 * widths minimising sum_j v_j 4^(-b_j) subject to sum_j b_j <= Btot = floor(16 d / ratio), 0 <= b_j <= b_max,
 * with cfg->width_group adjacent channels sharing one width taken from the group's mean variance.
 * Realised as greedy marginal return (one bit at a time to the group with the largest v_G 4^(-b_G),
 * ties to the lowest index), which is the exact integer optimum of that objective.
 * var_alloc: device fp32 [n_units, d].  widths: device uint8 [n_units, d].  ratio > 0.
 */
int spectra_alloc_bits(const spectra_config* cfg, const float* var_alloc, int64_t n_units, double ratio,
                       uint8_t* widths, void* stream);

/* ------------------------------------------------------------------------------------------------
 * spectra_alloc_bits_pooled -- the same rule with the budget pooled over pool_units consecutive units (Sec. 3.2 and
 * the appendix's bit-profile figure: the paper's latent spans all KV heads of a layer, so a head with little energy
 * gives its bits to the others; with cfg->width_group = 64 this is the paper's structure, one width per group of 64
 * energy-ordered coordinates).  Every run of pool_units units gets pool_units * Btot bits over its pool_units * d
 * channels; ties go to the lowest unit, then channel.  n_units must be a multiple of pool_units; at most 2048 width
 * groups per pool (SPECTRA_UNSUPPORTED beyond).
 * spectra_split_ratio -- the key/value budget split of Sec. 3.1 (last paragraph) and the appendix on hyperparameters:
 * of the bits a nominal ratio gives keys and values together, the keys get the fraction kappa (0 < kappa < 1) and the
 * values the rest: ratio_k = ratio / (2 kappa), ratio_v = ratio / (2 (1 - kappa)); kappa = 0.5 leaves both at ratio.
 * Host only.
 */
int spectra_alloc_bits_pooled(const spectra_config* cfg, const float* var_alloc, int64_t n_units, int64_t pool_units,
                              double ratio, uint8_t* widths, void* stream);
int spectra_split_ratio(double ratio, double kappa, double* ratio_k, double* ratio_v);

/* ------------------------------------------------------------------------------------------------
 * spectra_encode -- Sec. 3.2-3.3 (Mode A streaming: each token is down-projected, quantised per token at
 * the group widths and appended).  Appends n_new tokens to each of n_units unit-sides: unit u gets tokens
 * x[u*stride_unit + i*stride_token + 0..d) for i < n_new at cache positions pos0[u] + i.
 * Token slots of a touched tile that lie before pos0[u] are preserved, slots after the last appended token
 * are written as zero, so a tile needs no initialisation when its slot 0 is appended first.
 * x: device; x_dtype SPECTRA_F32 or SPECTRA_BF16; with SPECTRA_ROTATED_INPUT x must be SPECTRA_F32.
 * pos0: device int32 [n_units].  w_enc: device fp32 [n_param_sets, d, d]; mean_rot [n_param_sets, d];
 * widths: device uint8 [n_param_sets, d].  cache: device; unit_offset: device int64 [n_units], byte offset
 * of the unit-side's first tile, multiple of 16.  status_word: device int32, OR-ed with SPECTRA_STATUS_* bits,
 * may be NULL.
 * capacity_tokens: tokens every unit-side's buffer holds (spectra_cache_bytes); a token whose position is at or
 * beyond it is not written and SPECTRA_STATUS_CAPACITY is set in the status word.  0 switches the check off: the
 * caller then guarantees that every touched tile lies inside its buffer.  cache must be 16-byte aligned
 * (SPECTRA_INVALID_ARG otherwise).
 * Speed, not results, depends on alignment: bf16 input with a 16-byte aligned x and strides that are multiples of 8
 * elements (and scale_group 64, more than 16 tokens) takes the tensor-core path; anything else a CUDA-core kernel.
 */
int spectra_encode(const spectra_config* cfg, int side, const void* x, int x_dtype, int flags, int64_t n_units,
                   int64_t n_param_sets, const int32_t* pos0, int32_t n_new, int64_t stride_unit,
                   int64_t stride_token, const float* w_enc, const float* mean_rot, const uint8_t* widths,
                   uint8_t* cache, const int64_t* unit_offset, int32_t capacity_tokens, const int32_t* tile_table,
                   int64_t table_stride, int32_t* status_word, void* stream);

/* ------------------------------------------------------------------------------------------------
 * spectra_decode -- Sec. 3.3 (Mode A reconstruction): xhat = (yhat + m') W_dec for tokens [0, n_tokens[u])
 * of every unit-side; fp32 accumulation.  out: device, out_dtype SPECTRA_F32 or SPECTRA_BF16, element
 * (u, t, i) at out[u*stride_unit + t*stride_token + i].  n_tokens: device int32 [n_units];
 * max_tokens (host value) bounds it.  yhat_out (device fp32, same strides, may be NULL) receives the
 * dequantised rotated coordinates.  cache must be 2-byte aligned (SPECTRA_INVALID_ARG otherwise).
 * Speed, not the contract, depends on the call's shape.  With yhat_out NULL the sum is regrouped per scale group,
 * xhat = sum_g R_g (fields x W_dec rows / L) + sum_g lo_g u_g + m' W_dec, and the packed sub-fields themselves are the
 * tensor-core operand (exact as fp16 numbers; the W_dec rows enter as two fp16 parts: same accuracy as the
 * element-wise path, about 1e-5 of a vector's largest entry): one tcgen05 kernel takes the units with at most two
 * scale groups, at most 192 strip positions, tiles up to 10 KB and a 16-byte aligned cache + unit_offset[u]; the
 * element-wise kernel, launched behind it, takes the other units.  With yhat_out the codes are dequantised one by one
 * in the oracle's operation order (yhat bit-exact) and rotated with
 * tcgen05.  status_word: device int32 or NULL; a bounded wait that gives up sets SPECTRA_STATUS_WAIT_TIMEOUT there
 * (the reconstruction is then invalid).
 */
int spectra_decode(const spectra_config* cfg, int side, const uint8_t* cache, const int64_t* unit_offset,
                   int64_t n_units, int64_t n_param_sets, const int32_t* n_tokens, int32_t max_tokens,
                   const float* w_dec, const float* mean_rot, const uint8_t* widths, void* out, int out_dtype,
                   float* yhat_out, int64_t stride_unit, int64_t stride_token, const int32_t* tile_table,
                   int64_t table_stride, int32_t* status_word, void* stream);

/* ------------------------------------------------------------------------------------------------
 * spectra_decode_rope -- Sec. 3.3: the latent is taken before the rotary position embedding, and the position
 * rotation is applied to the key after its reconstruction.  spectra_decode for keys (tensor-core kernel) with that
 * rotation in its epilogue: channels i and i + d/2 of token t of unit u are rotated by the angle of position
 * position0[u] + t.  rope_cos, rope_sin: device fp32 [n_positions, d / 2], cos and sin of position * frequency_i
 * (the tables a model keeps anyway), 16-byte aligned, n_positions > the largest position touched.  position0: device
 * int32 [n_units] or NULL (all zero).  Other arguments as in spectra_decode (out must not be NULL).  The fused
 * latent-space attention does not take positions: q . R(p) k-hat = (R(-p) q) . k-hat makes the folded query depend on
 * the token, so a latent-space score needs the full d x d lift per token; callers with rotary models reconstruct
 * (this call) and attend, as the paper's Mode A does.
 */
int spectra_decode_rope(const spectra_config* cfg, const uint8_t* cache, const int64_t* unit_offset, int64_t n_units,
                        int64_t n_param_sets, const int32_t* n_tokens, int32_t max_tokens, const float* w_dec,
                        const float* mean_rot, const uint8_t* widths, void* out, int out_dtype, int64_t stride_unit,
                        int64_t stride_token, const int32_t* tile_table, int64_t table_stride,
                        const int32_t* position0, const float* rope_cos, const float* rope_sin, int32_t* status_word,
                        void* stream);

/* ------------------------------------------------------------------------------------------------
 * spectra_decode_paged -- Sec. 3.3 (Mode A): reconstruction into a pool of pages of 128 tokens, the form a paged
 * attention kernel reads.  out_pool: device, out_dtype SPECTRA_F32 or SPECTRA_BF16; token slot s (0..127) of tile t of
 * unit u goes to out_pool[out_table[u * out_table_stride + t] * stride_page + s * stride_token + i], i = 0..d-1.
 * out_table: device int32 [n_units, out_table_stride], out_table_stride >= ceil(max_tokens / 128) (SPECTRA_INVALID_ARG
 * otherwise); the caller guarantees that every page index lies inside the pool.  It may be the same table as
 * tile_table (the pages of the coded cache; NULL: contiguous).  Only tokens below n_tokens[u] are written.  rope_cos,
 * rope_sin, position0: as in spectra_decode_rope, both tables NULL for no position rotation (keys only:
 * SPECTRA_INVALID_ARG with side V).  Other arguments as in spectra_decode.
 */
int spectra_decode_paged(const spectra_config* cfg, int side, const uint8_t* cache, const int64_t* unit_offset,
                         int64_t n_units, int64_t n_param_sets, const int32_t* n_tokens, int32_t max_tokens,
                         const float* w_dec, const float* mean_rot, const uint8_t* widths, void* out_pool, int out_dtype,
                         int64_t stride_page, int64_t stride_token, const int32_t* tile_table, int64_t table_stride,
                         const int32_t* out_table, int64_t out_table_stride, const int32_t* position0,
                         const float* rope_cos, const float* rope_sin, int32_t* status_word, void* stream);

/* ------------------------------------------------------------------------------------------------
 * spectra_prefill_attention -- Sec. 3.3 (Mode A, reconstruct then attend) for a chunk of new queries: causal
 * softmax attention of n_new queries per sequence over the reconstructed cache.  Query i of sequence b sits at
 * position pos0[b] + i and attends tokens 0 .. pos0[b] + i; the pools must hold the reconstruction of all
 * pos0[b] + n_new tokens (spectra_encode the chunk, then spectra_decode_paged both sides).  head_dim 128, bf16.
 *   q, out    device bf16, element (b, i, h, c) at [b * stride_seq + i * stride_token + h * stride_head + c],
 *             h = 0 .. n_q_heads - 1 (query head h uses KV head h / (n_q_heads / n_kv_heads)); 16-byte aligned,
 *             strides multiples of 8 elements
 *   k_pool, v_pool   device bf16 pools of n_pages pages [128 tokens][d]: token slot s of page g at
 *             [g * stride_page + s * stride_token]; 16-byte aligned, strides multiples of 8 elements
 *   page_table       device int32 [n_seqs * n_kv_heads, table_stride]: page of tile t of unit (b, kv head); NULL: the
 *             page is unit * table_stride + t (table_stride = pages per unit, >= 1)
 *   pos0      device int32 [n_seqs]; n_new: host value, the same for every sequence
 *   scale     softmax scale (> 0), usually 1 / sqrt(d)
 *   lse       device fp32 [n_seqs, n_new, n_q_heads] or NULL: natural logarithm of the sum of exp(scale q.k)
 * Products run on the tensor cores with bf16 operands (probabilities are rounded to bf16 before P V, the row sum
 * is taken in fp32 before that rounding) and fp32 accumulation.  Slots of the last page past the sequence's end may hold anything.
 * status_word: SPECTRA_STATUS_WAIT_TIMEOUT if a bounded wait gave up (the output is then invalid).
 * Returns SPECTRA_INVALID_ARG for NULL or misaligned arguments, SPECTRA_UNSUPPORTED if the grid would not fit.
 */
int spectra_prefill_attention(const void* q, const void* k_pool, const void* v_pool, int64_t n_pages,
                              int64_t stride_page, int64_t stride_token, const int32_t* page_table,
                              int64_t table_stride, int64_t n_seqs, int32_t n_kv_heads, int32_t n_q_heads,
                              const int32_t* pos0, int32_t n_new, int64_t q_stride_seq, int64_t q_stride_token,
                              int64_t q_stride_head, float scale, void* out, int64_t out_stride_seq,
                              int64_t out_stride_token, int64_t out_stride_head, float* lse, int32_t* status_word,
                              void* stream);

/* ------------------------------------------------------------------------------------------------
 * spectra_decode_attention -- appendix "Latent-space attention and memory" (Mode B): one decode query per
 * (sequence, query head) attends to the whole coded cache of its kv-head without reconstructing it:
 *     q' = softmax_scale * W_dec,K q      (the up-projection folded into the query, once per call)
 *     s_t = q' . yhat^K_t                 (codes unpacked and dequantised in registers; the constant
 *                                          q' . m'_K is dropped from the softmax and restored in lse)
 *     o' = sum_t softmax(s)_t yhat^V_t    (online softmax, rotated value space, sequence split across CTAs)
 *     out = (o' + m'_V) W_dec,V           (one lift per query head)
 * Units are ordered u = sequence * n_kv_heads + kv_head; query head hq belongs to kv-head hq / (n_q_heads /
 * n_kv_heads).  q: device [batch, n_q_heads, d], q_dtype.  seq_len: device int32 [batch] (tokens attended; 0 gives
 * a zero output row and lse = -inf).  max_seq_len (host value) is the capacity of every sequence's buffers in tokens:
 * a sequence whose seq_len exceeds it sets SPECTRA_STATUS_CAPACITY and is treated as empty, nothing past the end of a
 * buffer is read.  cache_k/v with unit_offset_k/v: as in
 * spectra_encode.  Parameter arrays as in spectra_encode/decode ([n_param_sets, ...]); mean_rot_k is read
 * only when lse != NULL and may be NULL otherwise.  widths_k_host / widths_v_host: HOST copies of the two width
 * arrays ([n_param_sets, d], the same values the caller already needs for spectra_tile_bytes); read during the
 * call only.  They let the host size shared-memory rings and pick the kernel variant without a device
 * round-trip.  With both NULL, or scale_group != 64, or width profiles outside the built variants, a slower
 * CUDA-core kernel runs (spectra_attention_path tells which).  The tensor-core path checks every unit on the device
 * against the widths the kernels read: a unit that does not match the host copy (see SPECTRA_STATUS_BAD_LAYOUT) is
 * skipped, never copied from.  w_dec_k, w_dec_v, cache_k, cache_v and workspace must be 16-byte aligned
 * (SPECTRA_INVALID_ARG otherwise: the kernels use 16-byte accesses and bulk copies).  A GQA group of 5 to 8 query
 * heads is taken in two passes over the tiles.  On the tensor-core path the partial sums of a sequence are merged in a fixed order (results are
 * bit-reproducible from run to run); the CUDA-core kernel accumulates with shared-memory atomics (they are not).
 * softmax_scale 0 means 1/sqrt(d).
 * out: device [batch, n_q_heads, d], out_dtype.  lse: device fp32 [batch, n_q_heads] or NULL.
 * workspace: device, >= spectra_attention_workspace_bytes(...), 16-byte aligned; scratch only, nothing is
 * carried between calls.  status_word: device int32 or NULL.
 */
int spectra_decode_attention(const spectra_config* cfg, const void* q, int q_dtype, int32_t batch,
                             int32_t n_kv_heads, int32_t n_q_heads, const int32_t* seq_len, int32_t max_seq_len,
                             const uint8_t* cache_k, const int64_t* unit_offset_k, const uint8_t* cache_v,
                             const int64_t* unit_offset_v, int64_t n_param_sets, const float* w_dec_k,
                             const float* mean_rot_k, const uint8_t* widths_k, const float* w_dec_v,
                             const float* mean_rot_v, const uint8_t* widths_v, const uint8_t* widths_k_host,
                             const uint8_t* widths_v_host, float softmax_scale, void* out, int out_dtype,
                             float* lse, void* workspace, size_t workspace_bytes, const int32_t* tile_table_k,
                             const int32_t* tile_table_v, int64_t table_stride, int32_t* status_word, void* stream);
size_t spectra_attention_workspace_bytes(const spectra_config* cfg, int32_t batch, int32_t n_kv_heads,
                                         int32_t n_q_heads, int32_t max_seq_len);

/* ------------------------------------------------------------------------------------------------
 * spectra_decode_step -- one decode step of one layer: Sec. 3.3 (each new token's key and value are
 * down-projected, quantised and appended to the coded cache) followed by the latent-space attention of
 * spectra_decode_attention over the grown cache, with the append folded into the attention's first launch.
 * Same results, bit for bit in the cache, as spectra_encode(K), spectra_encode(V) (one new token per unit at
 * position seq_len[sequence] - 1) followed by spectra_decode_attention.
 * new_k, new_v: device [batch * n_kv_heads, d] (one vector per unit, unit order as above), x_dtype SPECTRA_F32
 * or SPECTRA_BF16.  seq_len: device int32 [batch], the lengths INCLUDING the appended token (a sequence with
 * length 0 gets no append and a zero output row).
 * w_enc_k/v, mean_rot_k/v as in spectra_encode; every other argument as in spectra_decode_attention
 * (mean_rot_k is required here).  cache_k / cache_v are written (the appended token) and read.  A sequence with
 * seq_len > max_seq_len gets no append (SPECTRA_STATUS_CAPACITY) and is attended as empty.
 */
int spectra_decode_step(const spectra_config* cfg, const void* q, int q_dtype, const void* new_k, const void* new_v,
                        int x_dtype, int32_t batch, int32_t n_kv_heads, int32_t n_q_heads, const int32_t* seq_len,
                        int32_t max_seq_len, uint8_t* cache_k, const int64_t* unit_offset_k, uint8_t* cache_v,
                        const int64_t* unit_offset_v, int64_t n_param_sets, const float* w_enc_k,
                        const float* w_dec_k, const float* mean_rot_k, const uint8_t* widths_k, const float* w_enc_v,
                        const float* w_dec_v, const float* mean_rot_v, const uint8_t* widths_v,
                        const uint8_t* widths_k_host, const uint8_t* widths_v_host, float softmax_scale, void* out,
                        int out_dtype, float* lse, void* workspace, size_t workspace_bytes,
                        const int32_t* tile_table_k, const int32_t* tile_table_v, int64_t table_stride,
                        int32_t* status_word, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Helpers (host only, no device work).
 * spectra_tile_bytes: size of one packed tile for the given widths (host uint8 [d]); 0 on bad arguments.
 * spectra_cache_bytes: bytes of one unit-side's buffer for capacity_tokens tokens (whole tiles); 0 on bad arguments.
 * spectra_attention_path: which kernels spectra_decode_attention / spectra_decode_step will run for these host
 *   widths ([n_param_sets, d] each, may be NULL): SPECTRA_PATH_TENSOR_CORE or SPECTRA_PATH_CUDA_CORE; -1 on bad
 *   arguments.
 * spectra_config_default: fills cfg with head_dim 128, tile 128, scale_group 64, width_group 1, b_max 8,
 *   SPECTRA_GAIN_SQRT, layout 1.
 * spectra_total_bits: Btot = floor(16 d / ratio) clamped to b_max * d.
 * spectra_status_string: name of a return code.
 *
 * spectra_selftest_quotients (device work): the bulk bf16 encoder takes the quotients (2^b - 1) / R16, b = 1..8, of
 *   the quantiser (Sec. 3.2: code = round((y - lo) (2^b - 1) / R)) from one shared reciprocal and fused
 *   multiply-add corrections instead of eight divisions.  This call runs that computation for every positive finite
 *   fp16 value of R16 and every b on the device and writes to mismatches[0] (device pointer, one int64) how many of
 *   the 8 x 31 743 quotients differ in any bit from the IEEE single-precision division; 0 is the only acceptable
 *   answer.  Enqueued on `stream`; returns SPECTRA_INVALID_ARG for a NULL pointer, SPECTRA_CUDA_ERROR if the launch
 *   failed.
 */
size_t spectra_tile_bytes(const spectra_config* cfg, const uint8_t* widths_host);
size_t spectra_cache_bytes(const spectra_config* cfg, const uint8_t* widths_host, int64_t capacity_tokens);
int spectra_attention_path(const spectra_config* cfg, int32_t n_kv_heads, int32_t n_q_heads, int64_t n_param_sets,
                           const uint8_t* widths_k_host, const uint8_t* widths_v_host);
void spectra_config_default(spectra_config* cfg);
int32_t spectra_total_bits(const spectra_config* cfg, double ratio);
const char* spectra_status_string(int code);
int spectra_selftest_quotients(int64_t* mismatches, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SPECTRA_H_ */
