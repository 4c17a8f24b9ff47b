// Reconstruction path of spectra_decode (xhat = (yhat + m') W_dec) with the inverse rotation on the 5th-generation
// tensor cores (tcgen05).  Both operands enter as two-way bf16 splits (a = a1 + a2, W = W1 + W2) and the three
// products a1 W1 + a1 W2 + a2 W1 are accumulated in fp32 in tensor memory: relative error about 2^-16, far inside the
// 2e-3 bound of the reconstruction.  Operand layouts in shared memory as in encode_umma.cuh (a: K-major, W: MN-major
// core matrices).
//
// The grid is persistent: the (unit, tile) slots of the call are cut into one contiguous range per CTA; a CTA takes
// the consecutive tiles of one unit as one run and builds the tables and the two parts of W_dec once per run.
// Seventeen warps:
//   warp 16 (one lane) is the producer: it brings the packed tiles in with one bulk copy each (two tiles ahead) and
//     issues the 24 MMAs of a tile when its operand is complete;
//   warps 0..15 are two halves of 8 warps that take alternate tiles, each with an operand buffer, a packed-tile
//     buffer and an accumulator tile (128 tensor-memory columns) of its own, so one half's MMAs run under the other
//     half's scalar work.  A worker thread owns one token and 64 consecutive channels: it pulls the channel's
//     sub-fields straight out of the packed tile (no intermediate code array), dequantises in the oracle's operation
//     order, adds the rotated mean, splits into two bf16 parts and stores 16-byte pieces of the K-major operand;
//     after the MMAs it reads its token's 64 output channels from tensor memory and stores them.
// The quotient R / L of the dequantiser is the correctly rounded one, computed without a division: with y = RN(1 / L),
// q0 = RN(R y), r = R - q0 L (exact in an FMA), q = RN(q0 + r y) equals RN(R / L) for every fp16 R and every
// L = 2^b - 1, b = 1..8 (checked exhaustively on the host).
// Barriers per half (all waits bounded; a timeout sets SPECTRA_STATUS_WAIT_TIMEOUT and ends the CTA's work):
//   raw_full   the packed tile has landed            (workers wait)
//   a_full     the eight warps have written the operand, and are done with the packed tile   (producer waits)
//   acc_full   the MMAs are complete                 (workers wait)
#pragma once
#include "encode_umma.cuh"
#include "decode_runs.cuh"

namespace spectra {

constexpr int kDecWorkers = 512;
constexpr int kDecThreads = kDecWorkers + 32;

struct DecodeArgs {
  const uint8_t* cache; const int64_t* unit_offset; int side; int scale_group; int64_t n_param_sets;
  const int32_t* n_tokens; const float* w_dec; const float* mean_rot; const uint8_t* widths;
  void* out; int out_dtype; float* yhat_out; int64_t stride_unit, stride_token;
  int32_t* status; TileMap map;
  // rotary position embedding of the reconstructed vectors (NULL tables: none): cos and sin of position * frequency,
  // [positions, d / 2] fp32, and the position of each unit's token 0 (NULL: 0)
  const float* rope_cos; const float* rope_sin; const int32_t* rope_pos0;
  // paged output (table != NULL): token slot t of tile `tile` of unit u goes to page omap.page(u, tile) of a pool whose
  // pages are stride_unit elements apart; otherwise unit u's tokens are stride_token apart from u * stride_unit on
  TileMap omap;
  __device__ __forceinline__ int64_t out_index(int64_t u, int tile, int t) const {
    return omap.table ? omap.page(u, tile) * stride_unit + (int64_t)t * stride_token
                      : u * stride_unit + ((int64_t)tile * kTile + t) * stride_token;
  }
};

struct DecodeTcSmem {
  StripTable tab;
  alignas(128) uint8_t w[2][kD * kD * 2];          // the two bf16 parts of W_dec, MN-major core layout
  struct Half {
    alignas(128) uint8_t a[2][kTile * kD * 2];     // the two bf16 parts of yhat + m', K-major core layout
    alignas(128) uint8_t raw[kDecRawMax];          // the packed tile
  } half[2];
  alignas(16) float4 chq[kD];                      // per channel {L, RN(1 / L), stored ? 1 : 0, m'}, L = 2^width - 1
  uint32_t field1[kD];                             // the channel's first (widest) sub-field: see field_desc()
  uint16_t sbase[4][kD];                           // per class: byte offset of the channel's strip; bit 15: stored alone
  uint8_t more[kD];                                // classes of the channel's further sub-fields (bit c), usually 0
  DmRun run[kMaxGroups][4];                        // only to tell which units the packed-field kernel takes
  int kg[kMaxGroups + 1];
  alignas(8) uint64_t raw_full[2], a_full[2], acc_full[2];
  uint32_t tmem_base;
};
static_assert(sizeof(DecodeTcSmem) + 128 <= 227 * 1024, "the reconstruction kernel's shared memory must fit one SM");

// skip_pairs != 0: units that decode_pair_kernel (decode_pairs.cuh) takes are left to it
__global__ void __launch_bounds__(kDecThreads, 1) decode_tc_kernel(DecodeArgs p, int n_slots_unit, int n_slots, int skip_pairs) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned char* smem_al = smem_raw + ((128u - (um_smem_u32(smem_raw) & 127u)) & 127u);
  DecodeTcSmem& S = *reinterpret_cast<DecodeTcSmem*>(smem_al);
  const bool producer = threadIdx.x >= kDecWorkers;
  const int hf = (threadIdx.x >> 8) & 1;                 // which half of the workers
  const int tid = threadIdx.x & 255, lane = tid & 31, warp = tid >> 5;
  const int t = tid & (kTile - 1);                       // this thread's token slot (= its tensor-memory lane)
  const int ch0 = 64 * (tid >> 7);                       // its 64 channels
  if (threadIdx.x == 0) {
    for (int h = 0; h < 2; h++) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(um_smem_u32(&S.raw_full[h])) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 8;" ::"r"(um_smem_u32(&S.a_full[h])) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(um_smem_u32(&S.acc_full[h])) : "memory");
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < 32) {                                // warp 0 owns the tensor-memory allocation (256 columns)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(um_smem_u32(&S.tmem_base)), "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  const int slot_end = (int)((long long)(blockIdx.x + 1) * n_slots / gridDim.x);
  int base0 = 0, base1 = 0;                              // tiles each half has taken so far: the barrier phases follow them
  int status = 0;
  const StripTable& T = S.tab;
  // this thread's token inside a strip of class c (field width w = 8 >> c): byte offset of its half-word relative to
  // the strip (paired strips of the K side and all strips of the V side; a strip stored alone uses half of it) and the
  // field's bit inside the half-word
  int tokoff[4], bitpos[4];
  unsigned long long tokpack = 0;                        // both, 16 bits per class: offset (8 bits) | bit << 8
#pragma unroll
  for (int c = 0; c < 4; c++) {
    const int w = 8 >> c;
    if (p.side == SPECTRA_SIDE_V) {
      const int a = t >> 5, h = (t >> 4) & 1, i = t & 15;
      tokoff[c] = 4 * (a * w + ((i * w) >> 4)) + 2 * h;
      bitpos[c] = (i * w) & 15;
    } else {
      tokoff[c] = 4 * ((t * w) >> 4);
      bitpos[c] = (t * w) & 15;
    }
    tokpack |= (unsigned long long)(tokoff[c] | (bitpos[c] << 8)) << (16 * c);
  }

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
    if (skip_pairs) {
      dm_build_runs(S.run, S.kg, S.tab, p.side == SPECTRA_SIDE_V, p.scale_group);
      if (dm_pairs_eligible(S.tab, S.kg[kMaxGroups], p.cache + p.unit_offset[u])) continue;
    }
    const float* wsrc = p.w_dec + (int64_t)ps * kD * kD;
    for (int idx = threadIdx.x; idx < kD * kD; idx += kDecThreads) {
      const int k = idx / kD, nn = idx - k * kD;
      const float v = wsrc[idx];
      const __nv_bfloat16 w1 = __float2bfloat16_rn(v);
      const int off = (nn >> 3) * 2048 + (k >> 3) * 128 + (k & 7) * 16 + (nn & 7) * 2;
      *reinterpret_cast<__nv_bfloat16*>(&S.w[0][off]) = w1;
      *reinterpret_cast<__nv_bfloat16*>(&S.w[1][off]) = __float2bfloat16_rn(v - __bfloat162float(w1));
    }
    for (int k = threadIdx.x; k < T.n_strips; k += kDecThreads) {
      const int c = strip_class(T, k);
      const int w = 8 >> c, i_in = k - T.class_first[c], cnt = T.class_first[c + 1] - T.class_first[c];
      int sb;
      if (p.side == SPECTRA_SIDE_V) sb = T.class_off[c] + 16 * w * i_in;
      else if ((i_in | 1) < cnt) sb = T.class_off[c] + 32 * w * (i_in >> 1) + 2 * (i_in & 1);
      else sb = (T.class_off[c] + 16 * w * i_in) | 0x8000;
      S.sbase[c][T.chan[k]] = (uint16_t)sb;
    }
    __syncthreads();
    if (threadIdx.x < kD) {
      const int j = threadIdx.x, b = T.width[j];
      const float L = (float)((1 << b) - 1);
      S.chq[j] = b ? make_float4(L, __frcp_rn(L), 1.f, p.mean_rot[(int64_t)ps * kD + j])
                   : make_float4(0.f, 0.f, 0.f, p.mean_rot[(int64_t)ps * kD + j]);
      // first sub-field: strip offset (bits 0..15, bit 15 = stored alone), class (16..17), position of the field inside
      // the code (18..20), field mask (24..31; 0: the channel stores nothing)
      uint32_t d = 0, more = 0;
      for (int c = 0; c < 4; c++) {
        const int w = 8 >> c;
        if (!(b & w)) continue;
        if (!d) d = (uint32_t)S.sbase[c][j] | ((uint32_t)c << 16) | ((uint32_t)(b & (w - 1)) << 18) | (((1u << w) - 1u) << 24);
        else more |= 1u << c;
      }
      S.field1[j] = d;
      S.more[j] = (uint8_t)more;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");    // W parts: generic stores -> tensor-core reads
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tb = S.tmem_base;
    const int tile_bytes = T.tile_bytes;
    const uint8_t* unit_ptr = p.cache + p.unit_offset[u];
    // packed tiles are staged in shared memory when they fit and the bulk copy's alignment rule holds
    const bool staged = tile_bytes <= kDecRawMax && (reinterpret_cast<uintptr_t>(unit_ptr) & 15) == 0;

    if (producer) {
      if (threadIdx.x == kDecWorkers) {
        auto load_raw = [&](int tt) {                    // tile ga + tt into the packed-tile buffer of half tt & 1
          const int h = tt & 1;
          const uint32_t bar = um_smem_u32(&S.raw_full[h]);
          asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(tile_bytes) : "memory");
          asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                           um_smem_u32(S.half[h].raw)),
                       "l"(unit_ptr + p.map.page(u, ga + tt) * tile_bytes), "r"(tile_bytes), "r"(bar)
                       : "memory");
        };
        if (staged) {
          load_raw(0);
          if (n_tiles > 1) load_raw(1);
        }
        bool ok = true;
#pragma unroll 1
        for (int tt = 0; tt < n_tiles && ok; tt++) {
          const int h = tt & 1, i = (h ? base1 : base0) + (tt >> 1);
          ok = um_wait(um_smem_u32(&S.a_full[h]), (uint32_t)(i & 1));
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          if (staged && tt + 2 < n_tiles) load_raw(tt + 2);          // the workers are done with this half's buffer
          const uint32_t dcol = tb + 128u * h;
          const uint32_t a0 = um_smem_u32(S.half[h].a[0]), a1 = um_smem_u32(S.half[h].a[1]);
          const uint32_t w0 = um_smem_u32(S.w[0]), w1 = um_smem_u32(S.w[1]);
#pragma unroll 1
          for (int pr = 0; pr < 3; pr++) {               // a1 W1, a1 W2, a2 W1
            const uint32_t aa = pr == 2 ? a1 : a0, ww = pr == 1 ? w1 : w0;
#pragma unroll 1
            for (int ks = 0; ks < kD / 16; ks++)
              um_mma_ss(dcol, um_desc(aa + 4096 * ks, 2048, 128), um_desc(ww + 256 * ks, 128, 2048), kUmIdesc,
                        (pr | ks) != 0);
          }
          asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(um_smem_u32(&S.acc_full[h])) : "memory");
        }
        if (!ok) status |= SPECTRA_STATUS_WAIT_TIMEOUT;
      }
    } else {
      DecodeTcSmem::Half& Hs = S.half[hf];
      const int gs = p.scale_group;
      bool ok = true;
      for (int tt = hf; tt < n_tiles && ok; tt += 2) {
        const int i = (hf ? base1 : base0) + (tt >> 1);
        const int tile = ga + tt;
        const int tile_pos = tile * kTile;
        const int n_here = min(n - tile_pos, kTile);
        const bool live = t < n_here;
        const uint8_t* tile_ptr = unit_ptr + p.map.page(u, tile) * tile_bytes;
        if (staged) {
          ok = um_wait(um_smem_u32(&S.raw_full[hf]), (uint32_t)(i & 1));
          if (!ok) { status |= SPECTRA_STATUS_WAIT_TIMEOUT; break; }
        }
        const uint8_t* src = staged ? Hs.raw : tile_ptr;           // generic pointer: shared or global
        // ---- this thread: token t, channels ch0 .. ch0 + 63, eight at a time (one 16-byte piece of each operand part)
        float lo_f = 0.f, R_f = 0.f;
#pragma unroll 1
        for (int kb = 0; kb < 8; kb++) {
          const int j0 = ch0 + 8 * kb;
          if ((j0 % gs) == 0 || kb == 0) {                          // a new scale group starts: its offset and range
            const int mo = T.meta_off[j0 / gs];
            lo_f = 0.f; R_f = 0.f;
            if (mo >= 0) {
              const uint16_t* m = reinterpret_cast<const uint16_t*>(src + mo) + t;
              lo_f = __half2float(__ushort_as_half(m[0]));
              R_f = __half2float(__ushort_as_half(m[kTile]));
            }
          }
          float a[8];
#pragma unroll
          for (int e = 0; e < 8; e++) {
            const int j = j0 + e;
            // the code: its first sub-field without a branch (all per-channel facts are warp-uniform), further ones
            // (widths 3, 5, 6, 7) class by class
            const uint32_t d = S.field1[j];
            const uint32_t tk = (uint32_t)(tokpack >> ((d >> 12) & 0x30u)) & 0xfffu;     // this token in that class
            const uint32_t off = (d & 0x7fffu) + ((d & 0x8000u) ? (tk & 0xffu) >> 1 : (tk & 0xffu));
            const uint32_t hw = *reinterpret_cast<const uint16_t*>(src + off);
            uint32_t code = ((hw >> (tk >> 8)) & (d >> 24)) << ((d >> 18) & 7u);
            const uint32_t more = S.more[j];
            if (more) {
              const uint32_t b = T.width[j];
#pragma unroll
              for (int c = 1; c < 4; c++) {
                const uint32_t w = 8u >> c;
                if (more & (1u << c)) {
                  const uint32_t sb = S.sbase[c][j];
                  const uint32_t o2 = (sb & 0x7fffu) + ((sb & 0x8000u) ? (uint32_t)tokoff[c] >> 1 : (uint32_t)tokoff[c]);
                  const uint32_t h2 = *reinterpret_cast<const uint16_t*>(src + o2);
                  code |= ((h2 >> bitpos[c]) & ((1u << w) - 1u)) << (b & (w - 1u));
                }
              }
            }
            // v = code * (R / L) + lo for a stored channel, 0 otherwise (R = 0 gives q = 0 and v = lo)
            const float4 cq = S.chq[j];
            const float q0 = __fmul_rn(R_f, cq.y);
            const float q = __fmaf_rn(__fmaf_rn(-q0, cq.x, R_f), cq.y, q0);           // RN(R / L), see the header
            const float cf = __uint_as_float(0x4B000000u | code) - 8388608.f;         // (float)code
            const float v = __fadd_rn(__fmul_rn(cf, q), __fmul_rn(lo_f, cq.z));
            if (p.yhat_out && live)
              p.yhat_out[(int64_t)u * p.stride_unit + (int64_t)(tile_pos + t) * p.stride_token + j] = v;
            a[e] = live ? v + cq.w : 0.f;
          }
          uint32_t hi[4], lw[4];
#pragma unroll
          for (int e = 0; e < 4; e++) {
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(a[2 * e], a[2 * e + 1]);
            const float2 hf2 = __bfloat1622float2(h2);
            const __nv_bfloat162 l2 = __floats2bfloat162_rn(a[2 * e] - hf2.x, a[2 * e + 1] - hf2.y);
            hi[e] = *reinterpret_cast<const uint32_t*>(&h2);
            lw[e] = *reinterpret_cast<const uint32_t*>(&l2);
          }
          const int off = (j0 >> 3) * 2048 + t * 16;                // K-major cores: k block j0 / 8, row t
          *reinterpret_cast<uint4*>(&Hs.a[0][off]) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
          *reinterpret_cast<uint4*>(&Hs.a[1][off]) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");          // operand: generic stores -> tensor-core reads
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(um_smem_u32(&S.a_full[hf])) : "memory");
        if (!p.out) continue;
        // ---- xhat: this token's 64 output channels from tensor memory (lane quarter = warp % 4, columns ch0 ..)
        ok = um_wait(um_smem_u32(&S.acc_full[hf]), (uint32_t)(i & 1));
        if (!ok) { status |= SPECTRA_STATUS_WAIT_TIMEOUT; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (p.rope_cos) {
          // Sec. 3.3: the position rotation is applied to the reconstructed key.  Channels i and i + 64 are a pair; any
          // thread of a token's lane can read all of its columns, so this thread takes pairs 32 (ch0 / 64) .. + 31:
          // 16 at a time, both halves, rotated by the angle of the token's position, stored as two pieces.
          const uint32_t lane_acc = tb + 128u * hf + ((uint32_t)((warp & 3) * 32) << 16);
          const int i0 = ch0 >> 1;
          const int64_t pos = (int64_t)(p.rope_pos0 ? p.rope_pos0[u] : 0) + tile_pos + t;
#pragma unroll 1
          for (int part = 0; part < 2; part++) {
            float ylo[16], yhi[16];
            um_ld16(lane_acc + i0 + 16 * part, ylo); um_ld16(lane_acc + 64 + i0 + 16 * part, yhi);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (live) {
              const float4* cs = reinterpret_cast<const float4*>(p.rope_cos + pos * (kD / 2) + i0 + 16 * part);
              const float4* sn = reinterpret_cast<const float4*>(p.rope_sin + pos * (kD / 2) + i0 + 16 * part);
#pragma unroll
              for (int c = 0; c < 4; c++) {
                const float4 cv = cs[c], sv = sn[c];
                const float cc[4] = {cv.x, cv.y, cv.z, cv.w}, ss[4] = {sv.x, sv.y, sv.z, sv.w};
#pragma unroll
                for (int e = 0; e < 4; e++) {
                  const float a = ylo[4 * c + e], b = yhi[4 * c + e];
                  ylo[4 * c + e] = a * cc[e] - b * ss[e];
                  yhi[4 * c + e] = b * cc[e] + a * ss[e];
                }
              }
#pragma unroll
              for (int half = 0; half < 2; half++) {
                const float* y = half ? yhi : ylo;
                const int64_t o = p.out_index(u, tile, t) + 64 * half + i0 + 16 * part;
                const uintptr_t addr = reinterpret_cast<uintptr_t>(p.out) + (uintptr_t)o * (p.out_dtype == SPECTRA_BF16 ? 2 : 4);
                if ((addr & 15) == 0 && p.out_dtype == SPECTRA_BF16) {
                  uint4* dst = reinterpret_cast<uint4*>(addr);
#pragma unroll
                  for (int c = 0; c < 2; c++) {
                    __nv_bfloat162 h[4];
#pragma unroll
                    for (int e = 0; e < 4; e++) h[e] = __floats2bfloat162_rn(y[8 * c + 2 * e], y[8 * c + 2 * e + 1]);
                    dst[c] = *reinterpret_cast<const uint4*>(h);
                  }
                } else if ((addr & 15) == 0) {
                  float4* dst = reinterpret_cast<float4*>(addr);
#pragma unroll
                  for (int c = 0; c < 4; c++) dst[c] = make_float4(y[4 * c], y[4 * c + 1], y[4 * c + 2], y[4 * c + 3]);
                } else {
#pragma unroll
                  for (int c = 0; c < 16; c++) store_from_float(p.out, p.out_dtype, o + c, y[c]);
                }
              }
            }
          }
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          continue;
        }
        const uint32_t acc = tb + 128u * hf + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)ch0;
#pragma unroll 1
        for (int part = 0; part < 2; part++) {
          float y[32];
          um_ld16(acc + 32 * part, y); um_ld16(acc + 32 * part + 16, y + 16);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
          if (live) {
            const int64_t o = p.out_index(u, tile, t) + ch0 + 32 * part;
            const uintptr_t addr = reinterpret_cast<uintptr_t>(p.out) + (uintptr_t)o * (p.out_dtype == SPECTRA_BF16 ? 2 : 4);
            if ((addr & 15) == 0 && p.out_dtype == SPECTRA_BF16) {
              uint4* dst = reinterpret_cast<uint4*>(addr);
#pragma unroll
              for (int c = 0; c < 4; c++) {
                __nv_bfloat162 h[4];
#pragma unroll
                for (int e = 0; e < 4; e++) h[e] = __floats2bfloat162_rn(y[8 * c + 2 * e], y[8 * c + 2 * e + 1]);
                dst[c] = *reinterpret_cast<const uint4*>(h);
              }
            } else if ((addr & 15) == 0) {
              float4* dst = reinterpret_cast<float4*>(addr);
#pragma unroll
              for (int c = 0; c < 8; c++) dst[c] = make_float4(y[4 * c], y[4 * c + 1], y[4 * c + 2], y[4 * c + 3]);
            } else {
#pragma unroll
              for (int c = 0; c < 32; c++) store_from_float(p.out, p.out_dtype, o + c, y[c]);
            }
          }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      }
    }
    // ---- end of the run: a timeout anywhere ends the CTA's work (the barrier phases are no longer known)
    base0 += (n_tiles + 1) >> 1; base1 += n_tiles >> 1;
    if (__syncthreads_or(status & SPECTRA_STATUS_WAIT_TIMEOUT)) break;
  }
  // ---- the warp that allocated the tensor memory frees it
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (threadIdx.x < 32) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(S.tmem_base), "r"(256u) : "memory");
  if (status && p.status) atomicOr(p.status, status);
}

}  // namespace spectra
