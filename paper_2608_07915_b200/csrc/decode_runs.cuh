// Tables shared by the reconstruction kernels that regroup the sum per scale group,
//     xhat_t = sum_g R_g(t) [ sum_{strips k of group g} field_tk W''_k ]  +  sum_g lo_g(t) u_g  +  c,
//     W''_k = 2^shift(k) W_dec[chan(k), :] / L_chan(k),   u_g = sum_{stored j in g} W_dec[j, :],   c = m' W_dec
// (Sec. 3.2 dequantiser, Sec. 3.3 Mode A reconstruction; a strip is one sub-field of 8, 4, 2 or 1 bits of a channel's
// code): the (group, class) runs of a tile, their k-steps of 16 strip positions, the rows of W'' in that order, and the
// test that says which units the tcgen05 kernel of decode_pairs.cuh takes.
#pragma once
#include "common.cuh"

namespace spectra {

constexpr int kDecRawMax = 10240;      // packed tiles up to this size are staged in shared memory by the tcgen05 kernels

struct DmRun { int base, first, n, kstep0, lone; };   // class region offset, first unit, units, first k-step, lone pair or -1

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

// Units the tcgen05 kernel of decode_pairs.cuh takes (decode_tc_kernel takes the rest): at most two scale groups, at
// most twelve k-steps, a tile that fits that kernel's slot, a source the bulk copy accepts.
constexpr int kDpMaxKsteps = 12;
__device__ __forceinline__ bool dm_pairs_eligible(const StripTable& T, int n_ksteps, const void* unit_ptr) {
  return T.n_groups <= 2 && n_ksteps <= kDpMaxKsteps && T.tile_bytes <= kDecRawMax && (reinterpret_cast<uintptr_t>(unit_ptr) & 15) == 0;
}

}  // namespace spectra
