// Analytical router (Eq. router) and gate logic (Eq. final_gate); top-level
// router of a hierarchical layer (Section 4.4).  One warp owns two rows; the
// N_r <= 32 routed experts of a row live one per lane for the softmax and the
// warp-shuffle top-k.
#pragma once

#include "common.cuh"

namespace cmoe {

// Index of the outer expert whose row range [off[g], off[g+1]) holds row r.
__device__ __forceinline__ int find_outer(const int32_t* __restrict__ off, int n_outer, int r) {
  int g = 0;
  for (int i = 1; i < n_outer; ++i) g += (__ldg(off + i) <= r) ? 1 : 0;
  return g;
}

// Warp-wide arg-max over (key, index): the larger key wins, equal keys go to the
// lower index.  Lanes that do not take part pass index >= 64.
__device__ __forceinline__ void warp_argmax(float& key, int& idx) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float k2 = __shfl_xor_sync(0xffffffffu, key, o);
    const int i2 = __shfl_xor_sync(0xffffffffu, idx, o);
    if (k2 > key || (k2 == key && i2 < idx)) { key = k2; idx = i2; }
  }
}

// Gate logic for one row held across a warp: lane j < n_r carries the gate and up
// pre-activations (a, v) of routed expert j's representative neuron.
__device__ __forceinline__ void gate_row(int lane, int n_r, int n_k, float a, float v,
                                         const float* __restrict__ u, const float* __restrict__ b,
                                         int group_base, float* __restrict__ scores_row,
                                         float* __restrict__ keys_row, int32_t* __restrict__ idx_row,
                                         float* __restrict__ gates_row) {
  const bool live = lane < n_r;
  const float s = live ? silu_accurate(a) * v : -INFINITY;            // Eq. router
  const float s_max = warp_max(s);
  const float e = live ? expf(s - s_max) : 0.0f;
  const float s_prime = e / warp_sum(e);                               // Softmax over all N_r
  const float key = live ? s_prime + __ldg(b + lane) : -INFINITY;
  if (live) { scores_row[lane] = s; keys_row[lane] = key; }
  const float gate = live ? 1.0f + s_prime * __ldg(u + lane) : 0.0f;   // 1 + s'_i u_i
  const float rank_key = (key != key) ? -INFINITY : key;               // NaN ranks last
  bool taken = !live;
  for (int i = 0; i < n_k; ++i) {
    float best = taken ? -INFINITY : rank_key;
    int who = taken ? 64 + lane : lane;
    warp_argmax(best, who);
    const float g = __shfl_sync(0xffffffffu, gate, who & 31);
    if (lane == who) taken = true;
    if (lane == 0) { idx_row[i] = group_base + who; gates_row[i] = g; }
  }
}

// The same gate logic with W lanes per row (W = 8, 16 or 32 >= n_r): a warp handles 32 / W rows at
// once.  `sub` is the lane's position in its W-lane group; every lane of the warp must call it (the
// shuffles name the full warp), `live_row` = false for groups that hold no row.  The arithmetic and
// its order per row are those of gate_row with the idle lanes removed, so the results are the same bits.
template <int W>
__device__ __forceinline__ void gate_row_sub(int sub, bool live_row, int n_r, int n_k, float a, float v,
                                             const float* __restrict__ u, const float* __restrict__ b,
                                             int group_base, float* __restrict__ scores_row,
                                             float* __restrict__ keys_row, int32_t* __restrict__ idx_row,
                                             float* __restrict__ gates_row) {
  const bool live = live_row && sub < n_r;
  const float s = live ? silu_accurate(a) * v : -INFINITY;
  float s_max = s;
#pragma unroll
  for (int o = W / 2; o > 0; o >>= 1) s_max = fmaxf(s_max, __shfl_xor_sync(0xffffffffu, s_max, o));
  const float e = live ? expf(s - s_max) : 0.0f;
  float e_sum = e;
#pragma unroll
  for (int o = W / 2; o > 0; o >>= 1) e_sum += __shfl_xor_sync(0xffffffffu, e_sum, o);
  const float s_prime = e / e_sum;
  const float key = live ? s_prime + __ldg(b + sub) : -INFINITY;
  if (live) { scores_row[sub] = s; keys_row[sub] = key; }
  const float gate = live ? 1.0f + s_prime * __ldg(u + sub) : 0.0f;
  const float rank_key = (key != key) ? -INFINITY : key;
  const int lane = threadIdx.x & 31, group0 = lane - sub;
  bool taken = !live;
  for (int i = 0; i < n_k; ++i) {
    float best = taken ? -INFINITY : rank_key;
    int who = taken ? 64 + sub : sub;
#pragma unroll
    for (int o = W / 2; o > 0; o >>= 1) {
      const float k2 = __shfl_xor_sync(0xffffffffu, best, o);
      const int i2 = __shfl_xor_sync(0xffffffffu, who, o);
      if (k2 > best || (k2 == best && i2 < who)) { best = k2; who = i2; }
    }
    const float g = __shfl_sync(0xffffffffu, gate, group0 + (who & (W - 1)));
    if (sub == who) taken = true;
    if (live_row && sub == 0) { idx_row[i] = group_base + who; gates_row[i] = g; }
  }
}

template <typename T, int NACC>
__global__ void __launch_bounds__(256)
router_kernel(const T* __restrict__ xo, int n_rows, int d, int n_r, int n_rp, int n_k,
              const T* __restrict__ w_rep, const float* __restrict__ u, const float* __restrict__ b,
              const int32_t* __restrict__ outer_off, int n_outer,
              float* __restrict__ scores, float* __restrict__ keys,
              int32_t* __restrict__ topk_idx, float* __restrict__ topk_gate) {
  const int lane = threadIdx.x & 31;
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int r0 = warp * 2;
  if (r0 >= n_rows) return;
  const bool has1 = r0 + 1 < n_rows;
  const int r1 = has1 ? r0 + 1 : r0;
  const int g0 = outer_off ? find_outer(outer_off, n_outer, r0) : 0;
  const int g1 = outer_off ? find_outer(outer_off, n_outer, r1) : 0;
  const int n2 = 2 * n_rp;      // W^R block: n_rp gate rows (zero-padded), then n_rp up rows
  const T* x0 = xo + (size_t)r0 * d;
  const T* x1 = xo + (size_t)r1 * d;
  const T* w0 = w_rep + (size_t)g0 * n2 * d;
  const T* w1 = w_rep + (size_t)g1 * n2 * d;
  const bool same = g0 == g1;

  float acc0[NACC], acc1[NACC];
#pragma unroll
  for (int j = 0; j < NACC; ++j) { acc0[j] = 0.0f; acc1[j] = 0.0f; }

  for (int k = lane * 8; k < d; k += 256) {
    float xa[8], xb[8];
    load8(x0 + k, xa);
    load8(x1 + k, xb);
#pragma unroll
    for (int j = 0; j < NACC; ++j) {
      if (j < n2) {
        float wa[8];
        load8(w0 + (size_t)j * d + k, wa);
        float t0 = acc0[j];
#pragma unroll
        for (int q = 0; q < 8; ++q) t0 = fmaf(wa[q], xa[q], t0);
        acc0[j] = t0;
        if (!same) load8(w1 + (size_t)j * d + k, wa);
        float t1 = acc1[j];
#pragma unroll
        for (int q = 0; q < 8; ++q) t1 = fmaf(wa[q], xb[q], t1);
        acc1[j] = t1;
      }
    }
  }

  float a0 = 0.f, v0 = 0.f, a1 = 0.f, v1 = 0.f;
#pragma unroll
  for (int j = 0; j < NACC; ++j) {
    if (j < n2) {
      const float t0 = warp_sum(acc0[j]);
      const float t1 = warp_sum(acc1[j]);
      if (lane == j) { a0 = t0; a1 = t1; }
      if (lane == j - n_rp) { v0 = t0; v1 = t1; }
    }
  }
  gate_row(lane, n_r, n_k, a0, v0, u + g0 * n_r, b + g0 * n_r, g0 * n_r,
           scores + (size_t)r0 * n_r, keys + (size_t)r0 * n_r,
           topk_idx + (size_t)r0 * n_k, topk_gate + (size_t)r0 * n_k);
  if (has1)
    gate_row(lane, n_r, n_k, a1, v1, u + g1 * n_r, b + g1 * n_r, g1 * n_r,
             scores + (size_t)r1 * n_r, keys + (size_t)r1 * n_r,
             topk_idx + (size_t)r1 * n_k, topk_gate + (size_t)r1 * n_k);
}

// Top-level router of an existing MoE layer: logits = W_r x, the outer_k largest
// logits (ties: lower index), weights = softmax over the selected logits.
template <typename T>
__global__ void __launch_bounds__(256)
outer_router_kernel(const T* __restrict__ x, int n_tokens, int d, int n_outer, int outer_k,
                    const T* __restrict__ w_router, float* __restrict__ logits,
                    int32_t* __restrict__ outer_idx, float* __restrict__ outer_w) {
  const int lane = threadIdx.x & 31;
  const int t = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (t >= n_tokens) return;
  float acc[kMaxOuter];
#pragma unroll
  for (int j = 0; j < kMaxOuter; ++j) acc[j] = 0.0f;
  const T* xr = x + (size_t)t * d;
  for (int k = lane * 8; k < d; k += 256) {
    float xa[8];
    load8(xr + k, xa);
#pragma unroll
    for (int j = 0; j < kMaxOuter; ++j) {
      if (j < n_outer) {
        float wa[8];
        load8(w_router + (size_t)j * d + k, wa);
        float s = acc[j];
#pragma unroll
        for (int q = 0; q < 8; ++q) s = fmaf(wa[q], xa[q], s);
        acc[j] = s;
      }
    }
  }
  float logit = -INFINITY;
#pragma unroll
  for (int j = 0; j < kMaxOuter; ++j) {
    if (j < n_outer) {
      const float s = warp_sum(acc[j]);
      if (lane == j) logit = s;
    }
  }
  const bool live = lane < n_outer;
  if (live) logits[(size_t)t * n_outer + lane] = logit;
  const float rank_key = (logit != logit) ? -INFINITY : logit;
  bool taken = !live;
  float sel_logit = -INFINITY;   // lane i < outer_k keeps the i-th selected logit
  int sel_who = 0;
  for (int i = 0; i < outer_k; ++i) {
    float best = taken ? -INFINITY : rank_key;
    int who = taken ? 64 + lane : lane;
    warp_argmax(best, who);
    const float l = __shfl_sync(0xffffffffu, logit, who & 31);
    if (lane == who) taken = true;
    if (lane == i) { sel_logit = l; sel_who = who; }
  }
  const float mx = warp_max(lane < outer_k ? sel_logit : -INFINITY);
  const float e = lane < outer_k ? expf(sel_logit - mx) : 0.0f;
  const float w = e / warp_sum(e);
  if (lane < outer_k) {
    outer_idx[(size_t)t * outer_k + lane] = sel_who;
    outer_w[(size_t)t * outer_k + lane] = w;
  }
}

}  // namespace cmoe
