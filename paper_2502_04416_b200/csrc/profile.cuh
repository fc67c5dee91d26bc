// Activation profiling (Section 4.1 "Activation Profiling"; Appendix, Complete Activation
// Analysis Pipeline, steps 2-4): per token the K_a hidden activations of largest magnitude
// (ATopK) as bits of the neurons' activation feature vectors c_i, the per-neuron activation
// counts q * mu_i, and the N_s * m neurons of highest rate.  Step 1, H itself, is the gate/up
// GEMM of a layer whose neurons all sit in the always-on expert.
#pragma once

#include "common.cuh"

namespace cmoe {

constexpr int kAtopkThreads = 256;

// Sort key of |h|: the bit pattern of a non-negative float orders like its value; NaN ranks
// last (key 0), as in a descending sort that puts NaN at the end.
__device__ __forceinline__ uint32_t magnitude_key(float h) {
  return (h != h) ? 0u : (__float_as_uint(h) & 0x7fffffffu);
}

// One block per token row: exact K_a-th largest key by a 4-pass, 8-bits-per-pass radix
// select (shared-memory histogram of the keys that still match the prefix found so far),
// then one ordered pass that takes every key above the threshold and, among keys equal to
// it, the lowest neuron indices until K_a are taken.  A taken neuron i sets bit
// (token0 + row) of its word row in act_bits and adds 1 to act_count[i]: integer OR / ADD,
// so the result does not depend on the order in which blocks run.
template <typename T>
__global__ void __launch_bounds__(kAtopkThreads)
atopk_kernel(const T* __restrict__ h, int ld, int d_h, int k_a, int token0, uint32_t* __restrict__ act_bits,
             int words_per_neuron, int32_t* __restrict__ act_count) {
  __shared__ int hist[256];
  __shared__ uint32_t sh_prefix;
  __shared__ int sh_remaining;
  __shared__ int warp_eq[kAtopkThreads / 32];
  __shared__ int sh_taken_eq;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const T* row = h + (size_t)blockIdx.x * ld;
  uint32_t prefix = 0, mask = 0;
  int remaining = k_a;                        // how many of the keys matching the prefix are still to be taken
  for (int pass = 3; pass >= 0; --pass) {
    hist[tid] = 0;
    __syncthreads();
    for (int i = tid; i < d_h; i += kAtopkThreads) {
      const uint32_t key = magnitude_key(to_float(row[i]));
      if ((key & mask) == prefix) atomicAdd(&hist[(key >> (8 * pass)) & 255u], 1);
    }
    __syncthreads();
    if (warp == 0) {                          // lane l owns bins [8l, 8l + 8); find the bin that holds the cut
      int own = 0;
#pragma unroll
      for (int b = 0; b < 8; ++b) own += hist[8 * lane + b];
      int run = own;                          // suffix sum: keys in this lane's bins and in those of higher lanes
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_down_sync(0xffffffffu, run, o);
        if (lane + o < 32) run += v;
      }
      const int above = run - own;
      if (above < remaining && remaining <= above + own) {
        int acc = above, bin = 8 * lane + 7;
        for (; bin > 8 * lane; --bin) {
          if (acc + hist[bin] >= remaining) break;
          acc += hist[bin];
        }
        sh_prefix = prefix | ((uint32_t)bin << (8 * pass));
        sh_remaining = remaining - acc;
      }
    }
    __syncthreads();
    prefix = sh_prefix;
    remaining = sh_remaining;
    mask |= 255u << (8 * pass);
    __syncthreads();
  }
  // prefix is the K_a-th largest key; `remaining` of the keys equal to it are taken, lowest index first
  const uint32_t thr = prefix;
  const int token = token0 + blockIdx.x;
  uint32_t* word_col = act_bits + (token >> 5);
  const uint32_t bit = 1u << (token & 31);
  if (tid == 0) sh_taken_eq = 0;
  __syncthreads();
  for (int base = 0; base < d_h; base += kAtopkThreads) {
    const int i = base + tid;
    const uint32_t key = i < d_h ? magnitude_key(to_float(row[i])) : 0u;
    const bool eq = i < d_h && key == thr;
    const unsigned eq_mask = __ballot_sync(0xffffffffu, eq);
    if (lane == 0) warp_eq[warp] = __popc(eq_mask);
    __syncthreads();
    int before = sh_taken_eq;                 // equal keys at lower indices
    for (int w = 0; w < warp; ++w) before += warp_eq[w];
    before += __popc(eq_mask & ((1u << lane) - 1u));
    const bool take = i < d_h && (key > thr || (eq && before < remaining));
    if (take) {
      atomicOr(word_col + (size_t)i * words_per_neuron, bit);
      atomicAdd(act_count + i, 1);
    }
    __syncthreads();
    if (tid == 0) {
      int total = 0;
      for (int w = 0; w < kAtopkThreads / 32; ++w) total += warp_eq[w];
      sh_taken_eq += total;
    }
    __syncthreads();
  }
}

// Step 4: neuron i's rank is the number of neurons with a higher count, or the same count and
// a lower index; the n_select first ranks are written in rank order.  d_h^2 comparisons, no scratch.
__global__ void __launch_bounds__(256)
select_shared_kernel(const int32_t* __restrict__ act_count, int d_h, int n_select, int32_t* __restrict__ shared_idx) {
  __shared__ int32_t tile[1024];
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  const int32_t mine = i < d_h ? act_count[i] : 0;
  int rank = 0;
  for (int j0 = 0; j0 < d_h; j0 += 1024) {
    for (int j = threadIdx.x; j < 1024; j += blockDim.x) tile[j] = j0 + j < d_h ? act_count[j0 + j] : -1;
    __syncthreads();
    const int n = min(1024, d_h - j0);
    for (int j = 0; j < n; ++j) {
      const int32_t c = tile[j];
      rank += (c > mine || (c == mine && j0 + j < i)) ? 1 : 0;
    }
    __syncthreads();
  }
  if (i < d_h && rank < n_select) shared_idx[rank] = i;
}

}  // namespace cmoe
