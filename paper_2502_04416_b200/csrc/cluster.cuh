// Data-parallel pieces of the balanced K-means over the neurons' activation feature vectors
// (Appendix "Balanced Clustering Algorithm for Routed Experts"; Eq. rep_neuron): centroid
// update, neuron-to-centroid distances and the representative neuron of every cluster.  The
// vectors c_i are the bit rows written by the profiling stage.  A centroid is the mean of
// binary vectors, so it is kept exactly as an integer count vector n_j[k] = #members active
// for token k together with the member count s_j (chat_j = n_j / s_j), and the squared
// distance is carried as the integer
//     S_ij = s_j^2 * || c_i - n_j / s_j ||^2 = s_j^2 |c_i| - 2 s_j <c_i, n_j> + ||n_j||^2
// (c is binary, so c^2 = c).  Everything here is integer arithmetic: results are exact and
// independent of the order in which threads run.  The assignment solver is not part of this.
#pragma once

#include "common.cuh"

namespace cmoe {

constexpr int kClusterMax = 32;      // clusters per call (N_r of one layer)

// Centroid update, first half.  One block per cluster j: count the members (rows i with
// assign[i] == j); a cluster without members keeps its centroid, otherwise its size is set and
// its count vector cleared for the second half.
__global__ void __launch_bounds__(256)
cluster_reset_kernel(const int32_t* __restrict__ assign, int n, int q, int32_t* __restrict__ centroid_count,
                     int32_t* __restrict__ cluster_size) {
  __shared__ int red[8];
  __shared__ int sh_members;
  const int j = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int mine = 0;
  for (int i = tid; i < n; i += 256) mine += assign[i] == j ? 1 : 0;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
  if (lane == 0) red[warp] = mine;
  __syncthreads();
  if (tid == 0) {
    int total = 0;
    for (int w = 0; w < 8; ++w) total += red[w];
    sh_members = total;
  }
  __syncthreads();
  const int members = sh_members;
  if (members == 0) return;
  int32_t* cc = centroid_count + (size_t)j * q;
  for (int k = tid; k < q; k += 256) cc[k] = 0;
  if (tid == 0) cluster_size[j] = members;
}

// Centroid update, second half.  One warp per listed neuron with a cluster: lanes walk its
// words and add 1 to the cluster's count for every set bit (few: K_a per token over all neurons).
__global__ void __launch_bounds__(256)
cluster_accumulate_kernel(const uint32_t* __restrict__ act_bits, int words, int q,
                          const int32_t* __restrict__ neuron_idx, const int32_t* __restrict__ assign, int n,
                          int n_clusters, int32_t* __restrict__ centroid_count) {
  const int lane = threadIdx.x & 31;
  const int i = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (i >= n) return;
  const int j = assign[i];
  if (j < 0 || j >= n_clusters) return;
  const uint32_t* row = act_bits + (size_t)neuron_idx[i] * words;
  int32_t* cc = centroid_count + (size_t)j * q;
  for (int w = lane; w < words; w += 32) {
    uint32_t bits = row[w];
    while (bits) {
      const int b = __ffs(bits) - 1;
      bits &= bits - 1;
      const int k = 32 * w + b;
      if (k < q) atomicAdd(cc + k, 1);
    }
  }
}

// ||n_j||^2 of every cluster, one block each.
__global__ void __launch_bounds__(256)
centroid_norm_kernel(const int32_t* __restrict__ centroid_count, int q, long long* __restrict__ sqnorm) {
  __shared__ long long red[8];
  const int j = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int32_t* cc = centroid_count + (size_t)j * q;
  long long acc = 0;
  for (int k = tid; k < q; k += 256) { const long long v = cc[k]; acc += v * v; }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) red[warp] = acc;
  __syncthreads();
  if (tid == 0) {
    long long total = 0;
    for (int w = 0; w < 8; ++w) total += red[w];
    sqnorm[j] = total;
  }
}

// One warp per listed neuron: |c_i| and <c_i, n_j> for every cluster from the neuron's set
// bits, then lane j writes S_ij.
__global__ void __launch_bounds__(256)
cluster_distance_kernel(const uint32_t* __restrict__ act_bits, int words, int q,
                        const int32_t* __restrict__ neuron_idx, int n,
                        const int32_t* __restrict__ centroid_count, const int32_t* __restrict__ cluster_size,
                        const long long* __restrict__ sqnorm, int n_clusters, long long* __restrict__ scaled_sq_dist) {
  const int lane = threadIdx.x & 31;
  const int i = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (i >= n) return;
  const uint32_t* row = act_bits + (size_t)neuron_idx[i] * words;
  int ones = 0;
  int dot[kClusterMax];
#pragma unroll
  for (int j = 0; j < kClusterMax; ++j) dot[j] = 0;
  for (int w = lane; w < words; w += 32) {
    uint32_t bits = row[w];
    while (bits) {
      const int b = __ffs(bits) - 1;
      bits &= bits - 1;
      const int k = 32 * w + b;
      if (k < q) {
        ++ones;
#pragma unroll
        for (int j = 0; j < kClusterMax; ++j)
          if (j < n_clusters) dot[j] += __ldg(centroid_count + (size_t)j * q + k);
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ones += __shfl_xor_sync(0xffffffffu, ones, o);
  long long my_dot = 0;
#pragma unroll
  for (int j = 0; j < kClusterMax; ++j) {
    int v = dot[j];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane == j) my_dot = v;
  }
  if (lane < n_clusters) {
    const long long s = cluster_size[lane];
    scaled_sq_dist[(size_t)i * n_clusters + lane] = s * s * ones - 2 * s * my_dot + sqnorm[lane];
  }
}

// One block per cluster: the member with the smallest distance to its own centroid, equal
// distances to the lower position in the list; -1 for a cluster without members.  Within one
// cluster the scale s_j^2 is common, so S_ij orders like the distance.
__global__ void __launch_bounds__(256)
cluster_representative_kernel(const long long* __restrict__ scaled_sq_dist, const int32_t* __restrict__ neuron_idx,
                              const int32_t* __restrict__ assign, int n, int n_clusters,
                              int32_t* __restrict__ rep_neuron) {
  __shared__ long long best_d[8];
  __shared__ int best_i[8];
  const int j = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  long long bd = 0x7fffffffffffffffLL;
  int bi = 0x7fffffff;
  for (int i = tid; i < n; i += 256) {
    if (assign[i] != j) continue;
    const long long dd = scaled_sq_dist[(size_t)i * n_clusters + j];
    if (dd < bd || (dd == bd && i < bi)) { bd = dd; bi = i; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const long long d2 = __shfl_xor_sync(0xffffffffu, bd, o);
    const int i2 = __shfl_xor_sync(0xffffffffu, bi, o);
    if (d2 < bd || (d2 == bd && i2 < bi)) { bd = d2; bi = i2; }
  }
  if (lane == 0) { best_d[warp] = bd; best_i[warp] = bi; }
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < 8; ++w)
      if (best_d[w] < bd || (best_d[w] == bd && best_i[w] < bi)) { bd = best_d[w]; bi = best_i[w]; }
    rep_neuron[j] = bi == 0x7fffffff ? -1 : neuron_idx[bi];
  }
}

}  // namespace cmoe
