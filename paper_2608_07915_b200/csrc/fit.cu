// spectra_fit_basis (second-moment accumulation + fp64 Jacobi eigensolver + transform assembly) and
// spectra_alloc_bits (greedy integer reverse water-filling).
#include "common.cuh"
#include "moments_umma.cuh"
#include "tensor_map.cuh"

namespace spectra {

// ------------------------------------------------------------------------------------------------
// Moments: S = sum_t x_t^T x_t and s = sum_t x_t.  Each CTA takes a chunk of tokens, forms the
// chunk's products in fp32 (each thread an 8x8 block of S) and adds them to the fp64 totals.
constexpr int kMomChunk = 256;

struct FitWorkspace {   // per unit, all fp64
  double S[kD * kD];
  double s[kD];
};

__global__ void __launch_bounds__(256) moments_kernel(const void* x, int x_dtype, int64_t n_tokens,
                                                      int64_t stride_unit, int64_t stride_token, FitWorkspace* ws) {
  __shared__ float xs[32][kD + 4];
  const int u = blockIdx.y;
  const int64_t t_begin = (int64_t)blockIdx.x * kMomChunk;
  const int64_t t_end = min(t_begin + (int64_t)kMomChunk, n_tokens);
  const int tid = threadIdx.x;
  const int r0 = (tid / 16) * 8, c0 = (tid % 16) * 8;
  float acc[8][8];
#pragma unroll
  for (int a = 0; a < 8; a++)
#pragma unroll
    for (int b = 0; b < 8; b++) acc[a][b] = 0.f;
  float colsum = 0.f;  // threads 0..127: sum of channel tid
  for (int64_t t0 = t_begin; t0 < t_end; t0 += 32) {
    __syncthreads();
    for (int idx = tid; idx < 32 * kD; idx += blockDim.x) {
      const int tt = idx / kD, i = idx - tt * kD;
      xs[tt][i] = t0 + tt < t_end ? load_as_float(x, x_dtype, (int64_t)u * stride_unit + (t0 + tt) * stride_token + i)
                                  : 0.f;
    }
    __syncthreads();
    for (int tt = 0; tt < 32; tt++) {
      float xr[8], xc[8];
#pragma unroll
      for (int a = 0; a < 8; a++) { xr[a] = xs[tt][r0 + a]; xc[a] = xs[tt][c0 + a]; }
#pragma unroll
      for (int a = 0; a < 8; a++)
#pragma unroll
        for (int b = 0; b < 8; b++) acc[a][b] = fmaf(xr[a], xc[b], acc[a][b]);
      if (tid < kD) colsum += xs[tt][tid];
    }
  }
  FitWorkspace& W = ws[u];
#pragma unroll
  for (int a = 0; a < 8; a++)
#pragma unroll
    for (int b = 0; b < 8; b++) atomicAdd(&W.S[(r0 + a) * kD + c0 + b], (double)acc[a][b]);
  if (tid < kD) atomicAdd(&W.s[tid], (double)colsum);
}

// ------------------------------------------------------------------------------------------------
// Eigensolver: cyclic two-sided Jacobi in fp64, round-robin ordering (127 rounds of 64 disjoint plane rotations per
// sweep), one CTA of 512 threads per matrix.  Everything a round touches is in shared memory: the symmetric matrix
// as its packed upper triangle (66 KB) and the accumulated eigenvectors (rows, 132 KB).  A round is one barrier
// pair: 64 threads derive the rotations from the 2 x 2 diagonal blocks; then every 2 x 2 block (pair i, pair j),
// i <= j, of the matrix is transformed by one thread as J_i^T B J_j (a matrix entry belongs to exactly one block, so
// the rows-then-columns order of the textbook update needs no barrier in between), and the eigenvector rows of each
// pair are rotated by eight threads.
constexpr int kLdV = kD + 1;                       // row stride of the eigenvector array (bank spread)
constexpr int kTri = kD * (kD + 1) / 2;            // entries of the packed upper triangle
constexpr int kPairs = kD / 2;                     // rotations per round
constexpr int kBlocks = kPairs * (kPairs - 1) / 2; // off-diagonal 2 x 2 blocks per round
constexpr int kMaxSweeps = 30;

struct EigSmem {
  double A[kTri];                                  // entry (r, c), r <= c, at tri(r, c)
  double VT[kD * kLdV];                            // rows are eigenvectors
  double c[kPairs], s[kPairs];
  int pp[kPairs], qq[kPairs];
  double red[16];
  double lam[kD], lam_sorted[kD];
  int order[kD];
  double mu[kD], m[kD], gam[kD];
  unsigned short blk[kBlocks];                     // (i << 8) | j of the off-diagonal blocks, i < j
};

struct FitOut {
  float* w_enc; float* w_dec; float* mean_rot; float* var_alloc; float* eigval; float* basis_u;
  int gain_mode; int64_t n_tokens;
};

__device__ __forceinline__ int tri(int r, int c) {              // r <= c
  return r * kD - ((r * (r - 1)) >> 1) + (c - r);
}
__device__ __forceinline__ int sym(int r, int c) { return r <= c ? tri(r, c) : tri(c, r); }

__device__ inline double block_sum_512(double v, double* red) {
#pragma unroll
  for (int s = 16; s; s >>= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  double t = 0.0;
  for (int i = 0; i < 16; i++) t += red[i];
  return t;
}

__global__ void __launch_bounds__(512, 1) eigen_kernel(FitWorkspace* ws, FitOut o) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  EigSmem& E = *reinterpret_cast<EigSmem*>(smem_raw);
  const int u = blockIdx.x, tid = threadIdx.x;
  FitWorkspace& W = ws[u];
  const double inv_n = 1.0 / (double)o.n_tokens;
  for (int idx = tid; idx < kD * kD; idx += 512) {
    const int r = idx / kD, c = idx - r * kD;
    // symmetrise: the two triangles were accumulated by different threads in the same order, but keep it exact
    if (r <= c) E.A[tri(r, c)] = 0.5 * (W.S[r * kD + c] + W.S[c * kD + r]) * inv_n;
    E.VT[r * kLdV + c] = r == c ? 1.0 : 0.0;
  }
  for (int b = tid; b < kBlocks; b += 512) {                    // enumerate i < j once
    int i = 0, rem = b;
    while (rem >= kPairs - 1 - i) { rem -= kPairs - 1 - i; i++; }
    E.blk[b] = (unsigned short)((i << 8) | (i + 1 + rem));
  }
  if (tid < kD) E.mu[tid] = W.s[tid] * inv_n;
  __syncthreads();
  double fro = 0.0;
  for (int idx = tid; idx < kTri; idx += 512) { const double v = E.A[idx]; fro += v * v; }
  double diag2 = 0.0;
  if (tid < kD) { const double v = E.A[tri(tid, tid)]; diag2 = v * v; }
  fro = 2.0 * block_sum_512(fro, E.red) - block_sum_512(diag2, E.red);
  const double tol2 = 1e-28 * fro;   // (1e-14 ||C||_F)^2

  const int pair = tid >> 3, sub = tid & 7;
  for (int sweep = 0; sweep < kMaxSweeps; sweep++) {
    double all2 = 0.0, dg2 = 0.0;
    for (int idx = tid; idx < kTri; idx += 512) { const double v = E.A[idx]; all2 += v * v; }
    if (tid < kD) { const double v = E.A[tri(tid, tid)]; dg2 = v * v; }
    const double off = 2.0 * (block_sum_512(all2, E.red) - block_sum_512(dg2, E.red));
    if (off <= tol2) break;
    for (int round = 0; round < kD - 1; round++) {
      if (tid < kPairs) {
        int p, q;
        if (tid == 0) { p = kD - 1; q = round; }
        else { p = (round + tid) % (kD - 1); q = (round - tid + (kD - 1)) % (kD - 1); }
        if (p > q) { const int t = p; p = q; q = t; }
        const double app = E.A[tri(p, p)], aqq = E.A[tri(q, q)], apq = E.A[tri(p, q)];
        double c = 1.0, s = 0.0;
        if (apq != 0.0 && fabs(apq) > 1e-300) {
          const double tau = (aqq - app) / (2.0 * apq);
          const double t = (tau >= 0.0 ? 1.0 : -1.0) / (fabs(tau) + sqrt(1.0 + tau * tau));
          c = 1.0 / sqrt(1.0 + t * t);
          s = t * c;
        }
        E.c[tid] = c; E.s[tid] = s; E.pp[tid] = p; E.qq[tid] = q;
      }
      __syncthreads();
      // the matrix: A <- J^T A J, block by block.  With J^T = [[c, -s], [s, c]] on rows (p, q):
      //   rows:    x_p' = c x_p - s x_q,  x_q' = s x_p + c x_q;  columns the same with the other pair's (c, s)
      for (int b = tid; b < kBlocks + kPairs; b += 512) {
        if (b < kBlocks) {
          const int i = E.blk[b] >> 8, j = E.blk[b] & 0xff;
          const int pi = E.pp[i], qi = E.qq[i], pj = E.pp[j], qj = E.qq[j];
          const double ci = E.c[i], si = E.s[i], cj = E.c[j], sj = E.s[j];
          const int i00 = sym(pi, pj), i01 = sym(pi, qj), i10 = sym(qi, pj), i11 = sym(qi, qj);
          const double b00 = E.A[i00], b01 = E.A[i01], b10 = E.A[i10], b11 = E.A[i11];
          const double r00 = ci * b00 - si * b10, r01 = ci * b01 - si * b11;      // rows by pair i
          const double r10 = si * b00 + ci * b10, r11 = si * b01 + ci * b11;
          E.A[i00] = cj * r00 - sj * r01; E.A[i01] = sj * r00 + cj * r01;        // columns by pair j
          E.A[i10] = cj * r10 - sj * r11; E.A[i11] = sj * r10 + cj * r11;
        } else {
          const int i = b - kBlocks;
          const int p = E.pp[i], q = E.qq[i];
          const double c = E.c[i], s = E.s[i];
          const double app = E.A[tri(p, p)], aqq = E.A[tri(q, q)], apq = E.A[tri(p, q)];
          const double r00 = c * app - s * apq, r01 = c * apq - s * aqq;          // rows
          const double r10 = s * app + c * apq, r11 = s * apq + c * aqq;
          E.A[tri(p, p)] = c * r00 - s * r01;                                     // columns
          E.A[tri(q, q)] = s * r10 + c * r11;
          E.A[tri(p, q)] = s * r00 + c * r01;
        }
      }
      // the eigenvector rows: VT <- J^T VT
      {
        const int p = E.pp[pair], q = E.qq[pair];
        const double c = E.c[pair], s = E.s[pair];
        for (int k = sub; k < kD; k += 8) {
          const double vp = E.VT[p * kLdV + k], vq = E.VT[q * kLdV + k];
          E.VT[p * kLdV + k] = c * vp - s * vq;
          E.VT[q * kLdV + k] = s * vp + c * vq;
        }
      }
      __syncthreads();
    }
  }
  // ---- order eigenvalues (descending, ties by index), fix signs, assemble the transform
  if (tid < kD) E.lam[tid] = E.A[tri(tid, tid)];
  __syncthreads();
  if (tid < kD) {
    const double l = E.lam[tid];
    int rank = 0;
    for (int k = 0; k < kD; k++) rank += (E.lam[k] > l) || (E.lam[k] == l && k < tid);
    E.order[rank] = tid;
  }
  __syncthreads();
  if (tid < kD) {
    // output column j = tid comes from Jacobi row order[j]
    const int src = E.order[tid];
    const double* v = E.VT + src * kLdV;
    int kmax = 0; double amax = -1.0;
    for (int k = 0; k < kD; k++) { const double a = fabs(v[k]); if (a > amax) { amax = a; kmax = k; } }
    const double sign = v[kmax] < 0.0 ? -1.0 : 1.0;
    double m = 0.0;
    for (int k = 0; k < kD; k++) m += E.mu[k] * v[k];
    m *= sign;
    const double lam = fmax(E.lam[src], 0.0);
    E.m[tid] = m;
    E.gam[tid] = sign;            // stash the sign; replaced by the gain below
    E.lam_sorted[tid] = lam;      // eigenvalue j in descending order
  }
  __syncthreads();
  if (tid < kD) {
    const double lam = E.lam_sorted[tid];
    const double lam1 = E.lam_sorted[0];
    const double m = E.m[tid];
    const double var = fmax(lam - m * m, 0.0);
    const double floor_v = 1e-12 * lam1;
    double g = 1.0;
    if (o.gain_mode == SPECTRA_GAIN_SQRT) g = 1.0 / sqrt(sqrt(fmax(lam, floor_v)));
    else if (o.gain_mode == SPECTRA_GAIN_WHITEN) g = 1.0 / sqrt(fmax(var, floor_v));
    const double sign = E.gam[tid];
    const int64_t base = (int64_t)u * kD;
    o.mean_rot[base + tid] = (float)(m * g);
    o.var_alloc[base + tid] = (float)(o.gain_mode == SPECTRA_GAIN_WHITEN ? var : var * g * g);
    if (o.eigval) o.eigval[base + tid] = (float)lam;
    const double* v = E.VT + E.order[tid] * kLdV;
    const int64_t mb = (int64_t)u * kD * kD;
    for (int k = 0; k < kD; k++) {
      const double ukj = sign * v[k];                       // U[k][j], j = tid
      o.w_enc[mb + k * kD + tid] = (float)(ukj * g);        // W_enc = U diag(gamma)
      o.w_dec[mb + tid * kD + k] = (float)(ukj / g);        // W_dec = diag(1/gamma) U^T
      if (o.basis_u) o.basis_u[mb + k * kD + tid] = (float)ukj;
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Allocation: one warp per unit.  Lane l holds groups l, l+32, l+64, l+96 (when present).
__global__ void __launch_bounds__(128) alloc_kernel(const float* __restrict__ var_alloc, int64_t n_units, int btot,
                                                    int b_max, int wg, uint8_t* __restrict__ widths) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t u = (int64_t)blockIdx.x * 4 + warp;
  if (u >= n_units) return;
  const int ng = kD / wg;
  double v[4];
  int b[4];
#pragma unroll
  for (int r = 0; r < 4; r++) {
    const int g = lane + 32 * r;
    b[r] = 0; v[r] = -1.0;
    if (g < ng) {
      float acc = var_alloc[u * kD + g * wg];
      for (int j = 1; j < wg; j++) acc = __fadd_rn(acc, var_alloc[u * kD + g * wg + j]);
      v[r] = (double)(wg == 1 ? acc : __fdiv_rn(acc, (float)wg));
    }
  }
  int steps = btot / wg;
  if (steps > ng * b_max) steps = ng * b_max;
  for (int it = 0; it < steps; it++) {
    double best = -1.0; int best_g = 1 << 30;
#pragma unroll
    for (int r = 0; r < 4; r++) {
      const int g = lane + 32 * r;
      if (g < ng && b[r] < b_max) {
        const double val = scalbn(v[r], -2 * b[r]);
        if (val > best || (val == best && g < best_g)) { best = val; best_g = g; }
      }
    }
#pragma unroll
    for (int s = 16; s; s >>= 1) {
      const double ob = __shfl_xor_sync(0xffffffffu, best, s);
      const int og = __shfl_xor_sync(0xffffffffu, best_g, s);
      if (ob > best || (ob == best && og < best_g)) { best = ob; best_g = og; }
    }
#pragma unroll
    for (int r = 0; r < 4; r++) if (lane + 32 * r == best_g) b[r]++;
  }
#pragma unroll
  for (int r = 0; r < 4; r++) {
    const int g = lane + 32 * r;
    if (g < ng) for (int j = 0; j < wg; j++) widths[u * kD + g * wg + j] = (uint8_t)b[r];
  }
}

// Allocation with the budget pooled over `pool` consecutive units (the heads of one layer: the paper's latent spans
// all of them): one CTA per pool, the groups' variances and widths in shared memory, the same greedy rule over all
// pool * d / wg groups (index order = unit, then channel, so ties go to the lowest unit and channel).
constexpr int kPoolMaxGroups = 2048;
__global__ void __launch_bounds__(128) alloc_pooled_kernel(const float* __restrict__ var_alloc, int pool, int btot,
                                                           int b_max, int wg, uint8_t* __restrict__ widths) {
  __shared__ double v[kPoolMaxGroups];
  __shared__ uint8_t b[kPoolMaxGroups];
  __shared__ double red_v[4];
  __shared__ int red_g[4];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ng = pool * kD / wg;
  const float* src = var_alloc + (int64_t)blockIdx.x * pool * kD;
  for (int g = tid; g < ng; g += 128) {
    float acc = src[g * wg];
    for (int j = 1; j < wg; j++) acc = __fadd_rn(acc, src[g * wg + j]);
    v[g] = (double)(wg == 1 ? acc : __fdiv_rn(acc, (float)wg));
    b[g] = 0;
  }
  __syncthreads();
  long long steps = (long long)pool * btot / wg;
  if (steps > (long long)ng * b_max) steps = (long long)ng * b_max;
  for (long long it = 0; it < steps; it++) {
    double best = -1.0; int best_g = 1 << 30;
    for (int g = tid; g < ng; g += 128) {
      if (b[g] < b_max) {
        const double val = scalbn(v[g], -2 * (int)b[g]);
        if (val > best || (val == best && g < best_g)) { best = val; best_g = g; }
      }
    }
#pragma unroll
    for (int s = 16; s; s >>= 1) {
      const double ob = __shfl_xor_sync(0xffffffffu, best, s);
      const int og = __shfl_xor_sync(0xffffffffu, best_g, s);
      if (ob > best || (ob == best && og < best_g)) { best = ob; best_g = og; }
    }
    if (lane == 0) { red_v[warp] = best; red_g[warp] = best_g; }
    __syncthreads();
    if (tid == 0) {
      for (int w = 1; w < 4; w++)
        if (red_v[w] > best || (red_v[w] == best && red_g[w] < best_g)) { best = red_v[w]; best_g = red_g[w]; }
      if (best_g < ng) b[best_g]++;
    }
    __syncthreads();
  }
  uint8_t* dst = widths + (int64_t)blockIdx.x * pool * kD;
  for (int j = tid; j < pool * kD; j += 128) dst[j] = b[j / wg];
}

}  // namespace spectra

using namespace spectra;

extern "C" size_t spectra_fit_workspace_bytes(const spectra_config* cfg, int64_t n_units) {
  if (check_config(cfg) || n_units < 0) return 0;
  return sizeof(FitWorkspace) * (size_t)n_units;
}

extern "C" int spectra_fit_basis(const spectra_config* cfg, const void* x, int x_dtype, int64_t n_units,
                                 int64_t n_tokens, int64_t stride_unit, int64_t stride_token, float* w_enc,
                                 float* w_dec, float* mean_rot, float* var_alloc, float* eigval, float* basis_u,
                                 void* workspace, size_t workspace_bytes, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if (n_units < 0 || n_tokens < 1) return SPECTRA_INVALID_ARG;
  if (x_dtype != SPECTRA_F32 && x_dtype != SPECTRA_BF16) return SPECTRA_INVALID_ARG;
  if (n_units == 0) return SPECTRA_OK;
  if (!x || !w_enc || !w_dec || !mean_rot || !var_alloc || !workspace) return SPECTRA_INVALID_ARG;
  if (workspace_bytes < sizeof(FitWorkspace) * (size_t)n_units) return SPECTRA_WORKSPACE_TOO_SMALL;
  if (n_units > 65535) return SPECTRA_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  FitWorkspace* ws = reinterpret_cast<FitWorkspace*>(workspace);
  // bf16 inputs whose layout a tensor map can describe: X^T X on the tensor cores, one CTA per unit, sums in a fixed
  // order (reproducible); anything else: the CUDA-core kernel with fp64 atomics
  CUtensorMap xmap;
  const bool tensor_path = x_dtype == SPECTRA_BF16 && (reinterpret_cast<uintptr_t>(x) & 15) == 0 && stride_token % 8 == 0 &&
                           stride_unit % 8 == 0 && n_tokens < (1LL << 31) &&
                           make_token_map(&xmap, x, n_tokens, n_units, stride_token, stride_unit, true);
  if (tensor_path) {
    const size_t smem = sizeof(MomentsSmem) + 1024;
    if (cudaFuncSetAttribute(moments_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return SPECTRA_CUDA_ERROR;
    double* base = reinterpret_cast<double*>(ws);
    moments_umma_kernel<<<(unsigned)n_units, kMuThreads, smem, st>>>(xmap, n_tokens, base, base + kD * kD,
                                                                     (int64_t)(sizeof(FitWorkspace) / sizeof(double)), nullptr);
  } else {
    if (cudaMemsetAsync(ws, 0, sizeof(FitWorkspace) * (size_t)n_units, st) != cudaSuccess) return SPECTRA_CUDA_ERROR;
    dim3 grid((unsigned)((n_tokens + kMomChunk - 1) / kMomChunk), (unsigned)n_units);
    moments_kernel<<<grid, 256, 0, st>>>(x, x_dtype, n_tokens, stride_unit, stride_token, ws);
  }
  if (launch_status()) return SPECTRA_CUDA_ERROR;
  if (cudaFuncSetAttribute(eigen_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(EigSmem)) !=
      cudaSuccess)
    return SPECTRA_CUDA_ERROR;
  FitOut o{w_enc, w_dec, mean_rot, var_alloc, eigval, basis_u, cfg->gain_mode, n_tokens};
  eigen_kernel<<<(unsigned)n_units, 512, sizeof(EigSmem), st>>>(ws, o);
  return launch_status();
}

// ------------------------------------------------------------------------------------------------
// Variant without a caller workspace: the scratch is a fixed array in the library image.
static __device__ __align__(256) unsigned char g_fit_static_scratch[sizeof(FitWorkspace) * SPECTRA_FIT_STATIC_MAX_UNITS];

namespace {
constexpr int kMaxDevices = 64;
void* g_fit_static_addr[kMaxDevices];   // device address of the array, per device, looked up on first use
}  // namespace

extern "C" int spectra_fit_basis_static(const spectra_config* cfg, const void* x, int x_dtype, int64_t n_units,
                                        int64_t n_tokens, int64_t stride_unit, int64_t stride_token, float* w_enc,
                                        float* w_dec, float* mean_rot, float* var_alloc, float* eigval,
                                        float* basis_u, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if (n_units < 0) return SPECTRA_INVALID_ARG;
  if (n_units > SPECTRA_FIT_STATIC_MAX_UNITS) return SPECTRA_CAPACITY;
  if (n_units == 0) return SPECTRA_OK;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SPECTRA_CUDA_ERROR;
  if (!g_fit_static_addr[dev]) {
    // In host code the array's name is only a handle; the kernels need its address on the current device.
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_fit_static_scratch) != cudaSuccess || !ptr) return SPECTRA_CUDA_ERROR;
    g_fit_static_addr[dev] = ptr;
  }
  return spectra_fit_basis(cfg, x, x_dtype, n_units, n_tokens, stride_unit, stride_token, w_enc, w_dec, mean_rot,
                           var_alloc, eigval, basis_u, g_fit_static_addr[dev],
                           sizeof(FitWorkspace) * (size_t)n_units, stream);
}

extern "C" int32_t spectra_total_bits(const spectra_config* cfg, double ratio) {
  if (check_config(cfg) || !(ratio > 0.0)) return -1;
  double bits = 16.0 * kD / ratio + 1e-9;
  int64_t b = (int64_t)bits;
  const int64_t cap = (int64_t)cfg->b_max * kD;
  return (int32_t)(b > cap ? cap : b);
}

extern "C" int spectra_alloc_bits(const spectra_config* cfg, const float* var_alloc, int64_t n_units, double ratio,
                                  uint8_t* widths, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if (n_units < 0 || !(ratio > 0.0)) return SPECTRA_INVALID_ARG;
  if (n_units == 0) return SPECTRA_OK;
  if (!var_alloc || !widths) return SPECTRA_INVALID_ARG;
  const int btot = spectra_total_bits(cfg, ratio);
  alloc_kernel<<<(unsigned)((n_units + 3) / 4), 128, 0, (cudaStream_t)stream>>>(var_alloc, n_units, btot, cfg->b_max,
                                                                                cfg->width_group, widths);
  return launch_status();
}

extern "C" int spectra_alloc_bits_pooled(const spectra_config* cfg, const float* var_alloc, int64_t n_units,
                                         int64_t pool_units, double ratio, uint8_t* widths, void* stream) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if (n_units < 0 || pool_units < 1 || !(ratio > 0.0)) return SPECTRA_INVALID_ARG;
  if (n_units == 0) return SPECTRA_OK;
  if (n_units % pool_units) return SPECTRA_INVALID_ARG;
  if (!var_alloc || !widths) return SPECTRA_INVALID_ARG;
  if (pool_units * kD / cfg->width_group > kPoolMaxGroups) return SPECTRA_UNSUPPORTED;
  const int btot = spectra_total_bits(cfg, ratio);
  alloc_pooled_kernel<<<(unsigned)(n_units / pool_units), 128, 0, (cudaStream_t)stream>>>(
      var_alloc, (int)pool_units, btot, cfg->b_max, cfg->width_group, widths);
  return launch_status();
}

extern "C" int spectra_split_ratio(double ratio, double kappa, double* ratio_k, double* ratio_v) {
  if (!(ratio > 0.0) || !(kappa > 0.0) || !(kappa < 1.0) || !ratio_k || !ratio_v) return SPECTRA_INVALID_ARG;
  *ratio_k = ratio / (2.0 * kappa);
  *ratio_v = ratio / (2.0 * (1.0 - kappa));
  return SPECTRA_OK;
}
