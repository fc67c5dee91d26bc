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

// Key width of a storage type: bf16 magnitudes are their 15 value bits, fp32 magnitudes 31.
template <typename T> struct KeyOf;
template <> struct KeyOf<bf16> {
  typedef uint16_t type;
  static constexpr int kBits = 15;
  static __device__ __forceinline__ uint16_t make(bf16 h) { return (uint16_t)(magnitude_key(to_float(h)) >> 16); }
};
template <> struct KeyOf<float> {
  typedef uint32_t type;
  static constexpr int kBits = 31;
  static __device__ __forceinline__ uint32_t make(float h) { return magnitude_key(h); }
};

// Sum of one int per thread over the block (all threads get it); `red` holds one slot per warp.
__device__ __forceinline__ int block_sum(int v, int* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();                               // the previous result has been read by everyone
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  int total = 0;
#pragma unroll
  for (int w = 0; w < kAtopkThreads / 32; ++w) total += red[w];
  return total;
}

constexpr int kAtopkCap = 1024;     // candidates ranked directly
// static shared memory of atopk_kernel: two candidate arrays, two per-warp arrays, two scalars (rounded up)
constexpr int kAtopkStaticSmem = 2 * kAtopkCap * 4 + 2 * (kAtopkThreads / 32) * 4 + 192;

// One block per token row; the row's magnitude keys are staged once in shared memory.
// Fast path (K_a small against d_h, the paper's K_a = 10): the K_a-th largest of the 256
// per-thread maxima is a lower bound of the row's K_a-th largest key (those maxima are distinct
// elements), so only the few keys at or above it can be selected; they are gathered and ranked
// by (key descending, neuron index ascending) against one another.  General path (more than
// kAtopkCap candidates): the K_a-th largest key is built bit by bit from the top (the largest
// value v with at least K_a keys >= v: one counting pass per bit), and one ordered pass takes
// every key above that threshold and, among keys equal to it, the lowest neuron indices until
// K_a are taken.  Both are exact and give the same set.  A taken neuron i sets bit
// (token0 + row) of its word row in act_bits and adds 1 to act_count[i]: integer OR / ADD, so
// the result does not depend on the order in which blocks run.  Dynamic shared memory: d_h keys.
template <typename T>
__global__ void __launch_bounds__(kAtopkThreads)
atopk_kernel(const T* __restrict__ h, int ld, int d_h, int k_a, int token0, uint32_t* __restrict__ act_bits,
             int words_per_neuron, int32_t* __restrict__ act_count) {
  typedef typename KeyOf<T>::type Key;
  extern __shared__ __align__(16) uint8_t atopk_smem[];
  Key* keys = reinterpret_cast<Key*>(atopk_smem);
  __shared__ int red[kAtopkThreads / 32];
  __shared__ int warp_eq[kAtopkThreads / 32];
  __shared__ int sh_taken_eq;
  __shared__ uint32_t cand_key[kAtopkCap];
  __shared__ int32_t cand_idx[kAtopkCap];
  __shared__ int sh_n_cand;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const T* row = h + (size_t)blockIdx.x * ld;
  const int token = token0 + blockIdx.x;
  uint32_t* word_col = act_bits + (token >> 5);
  const uint32_t bit = 1u << (token & 31);
  uint32_t my_max = 0;
  for (int i = tid; i < d_h; i += kAtopkThreads) {
    const Key k = KeyOf<T>::make(row[i]);
    keys[i] = k;
    my_max = max(my_max, (uint32_t)k);
  }
  if (tid == 0) sh_n_cand = 0;
  __syncthreads();
  uint32_t bound = 0;                          // K_a-th largest of the per-thread maxima (0: no bound)
  if (k_a <= kAtopkThreads) {
    for (int b = KeyOf<T>::kBits - 1; b >= 0; --b) {
      const uint32_t cand = bound | (1u << b);
      if (block_sum(my_max >= cand ? 1 : 0, red) >= k_a) bound = cand;
    }
  }
  int n_cand = 0;
  for (int i = tid; i < d_h; i += kAtopkThreads) n_cand += (uint32_t)keys[i] >= bound ? 1 : 0;
  n_cand = block_sum(n_cand, red);
  if (n_cand <= kAtopkCap) {
    for (int i = tid; i < d_h; i += kAtopkThreads) {
      const uint32_t k = keys[i];
      if (k >= bound) {
        const int slot = atomicAdd(&sh_n_cand, 1);       // any order: the rank below does not depend on it
        cand_key[slot] = k;
        cand_idx[slot] = i;
      }
    }
    __syncthreads();
    for (int c = tid; c < n_cand; c += kAtopkThreads) {
      const uint32_t k = cand_key[c];
      const int32_t idx = cand_idx[c];
      int rank = 0;
      for (int j = 0; j < n_cand; ++j) {
        const uint32_t kj = cand_key[j];
        rank += (kj > k || (kj == k && cand_idx[j] < idx)) ? 1 : 0;
      }
      if (rank < k_a) {
        atomicOr(word_col + (size_t)idx * words_per_neuron, bit);
        atomicAdd(act_count + idx, 1);
      }
    }
    return;
  }
  uint32_t thr = 0;
  for (int b = KeyOf<T>::kBits - 1; b >= 0; --b) {
    const uint32_t cand = thr | (1u << b);
    int n = 0;
    for (int i = tid; i < d_h; i += kAtopkThreads) n += (uint32_t)keys[i] >= cand ? 1 : 0;
    if (block_sum(n, red) >= k_a) thr = cand;
  }
  int n_above = 0;
  for (int i = tid; i < d_h; i += kAtopkThreads) n_above += (uint32_t)keys[i] > thr ? 1 : 0;
  const int remaining = k_a - block_sum(n_above, red);       // keys equal to the threshold still to take (>= 1)
  if (tid == 0) sh_taken_eq = 0;
  __syncthreads();
  for (int base = 0; base < d_h; base += kAtopkThreads) {
    const int i = base + tid;
    const uint32_t key = i < d_h ? (uint32_t)keys[i] : 0u;
    const bool eq = i < d_h && key == thr;
    const unsigned eq_mask = __ballot_sync(0xffffffffu, eq);
    const unsigned any_above = __ballot_sync(0xffffffffu, i < d_h && key > thr);
    if (__syncthreads_or((eq_mask | any_above) != 0u) == 0) continue;      // nothing to take in this stretch
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
// a lower index; the n_select first ranks are written in rank order.  d_h^2 comparisons, no
// scratch: a block ranks 32 neurons, its eight warps each compare against one eighth of the
// counts, and the eight partial ranks are added through shared memory.
__global__ void __launch_bounds__(256)
select_shared_kernel(const int32_t* __restrict__ act_count, int d_h, int n_select, int32_t* __restrict__ shared_idx) {
  __shared__ int part[8][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int i = blockIdx.x * 32 + lane;
  const int32_t mine = i < d_h ? __ldg(act_count + i) : 0;
  const int per = (d_h + 7) / 8, j_lo = warp * per, j_hi = min(d_h, j_lo + per);
  int rank = 0;
  for (int j = j_lo; j < j_hi; ++j) {
    const int32_t c = __ldg(act_count + j);              // same address across the warp: one broadcast load
    rank += (c > mine || (c == mine && j < i)) ? 1 : 0;
  }
  part[warp][lane] = rank;
  __syncthreads();
  if (warp == 0) {
    int total = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) total += part[w][lane];
    if (i < d_h && total < n_select) shared_idx[total] = i;
  }
}

}  // namespace cmoe
