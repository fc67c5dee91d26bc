// Expert utilisation and the load-balancing bias update (Section 4.3): after a step,
// with p_i the fraction of the routed assignments of an (outer) layer that went to its
// expert i and p*_i the target (uniform 1/N_r unless given), b_i decreases by gamma if
// p_i > p*_i and increases by gamma if p_i < p*_i.  One warp per (outer) layer; lane i
// owns expert i.  The comparison is done in fp64 on exactly representable integer counts,
// so the decision is the same as a double-precision host evaluation.
#pragma once

#include "common.cuh"

namespace cmoe {

__global__ void __launch_bounds__(256)
bias_update_kernel(const int32_t* __restrict__ counts, int n_outer, int n_r,
                   const float* __restrict__ target /* [n_outer*n_r] or null: uniform */, float gamma,
                   float* __restrict__ b, float* __restrict__ share /* [n_outer*n_r] or null */) {
  const int lane = threadIdx.x & 31;
  const int outer = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (outer >= n_outer) return;
  const bool live = lane < n_r;
  const int c = live ? counts[outer * n_r + lane] : 0;
  int total = c;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
  if (!live || total == 0) {
    if (live && share) share[outer * n_r + lane] = 0.0f;
    return;
  }
  const double p = (double)c / (double)total;
  const double p_star = target ? (double)target[outer * n_r + lane] : 1.0 / (double)n_r;
  if (share) share[outer * n_r + lane] = (float)p;
  float bi = b[outer * n_r + lane];
  if (p > p_star) bi -= gamma;
  else if (p < p_star) bi += gamma;
  b[outer * n_r + lane] = bi;
}

}  // namespace cmoe
