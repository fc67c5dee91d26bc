// Row gather into expert-contiguous order, per-forward group row ranges, and the
// gate-weighted combine back into token order (Eq. moe_output; Section 4.4 for the
// two-level form).
#pragma once

#include "common.cuh"

namespace cmoe {

// dst[r, :] = src[idx[r], :], 16 bytes per thread step.  row bytes % 16 == 0.
__global__ void __launch_bounds__(256)
gather_rows_kernel(const uint4* __restrict__ src, const int32_t* __restrict__ idx, int n_rows,
                   int row_vec /* 16-byte vectors per row */, uint4* __restrict__ dst) {
  const int r = blockIdx.x;
  if (r >= n_rows) return;
  const uint4* s = src + (size_t)__ldg(idx + r) * row_vec;
  uint4* o = dst + (size_t)r * row_vec;
  for (int v = threadIdx.x; v < row_vec; v += blockDim.x) o[v] = __ldg(s + v);
}

// Row range of every group for this forward.  Groups: n_outer shared groups (rows of
// the outer-row order), then n_outer*n_r routed groups (rows of the routed order).
__global__ void plan_groups_kernel(int n_outer, int n_r, int n_tokens,
                                   const int32_t* __restrict__ outer_off /* null: plain layer */,
                                   const int32_t* __restrict__ counts, const int32_t* __restrict__ offsets,
                                   GroupRows* __restrict__ gr) {
  const int n_groups = n_outer + n_outer * n_r;
  for (int g = threadIdx.x; g < n_groups; g += blockDim.x) {
    GroupRows r;
    if (g < n_outer) {
      r.row0 = outer_off ? outer_off[g] : 0;
      r.count = outer_off ? outer_off[g + 1] - outer_off[g] : n_tokens;
    } else {
      r.row0 = offsets[g - n_outer];
      r.count = counts[g - n_outer];
    }
    gr[g] = r;
  }
}

// out[t] = sum_slot w[t,slot] * ( Y_s[orow] + sum_j g[orow,j] * Y_r[row_of[orow,j]] ),
// orow = outer_row_of[t,slot] (plain layer: one slot, orow = t, w = 1).  Routed terms are
// added in ascending group index; fp32 accumulation, one rounding to the output type.
template <typename T>
__global__ void __launch_bounds__(256)
combine_kernel(const T* __restrict__ y_s, const T* __restrict__ y_r,
               const int32_t* __restrict__ topk_idx, const float* __restrict__ topk_gate,
               const int32_t* __restrict__ row_of, const int32_t* __restrict__ outer_row_of,
               const float* __restrict__ outer_w, int outer_k, int n_k, int d, T* __restrict__ out) {
  __shared__ int32_t s_row[kMaxTopK][kMaxTopK];
  __shared__ float s_gate[kMaxTopK][kMaxTopK];
  __shared__ int32_t s_orow[kMaxTopK];
  __shared__ float s_w[kMaxTopK];
  const int t = blockIdx.x;
  if ((int)threadIdx.x < outer_k) {
    const int slot = threadIdx.x;
    const int orow = outer_row_of ? outer_row_of[(size_t)t * outer_k + slot] : t;
    s_orow[slot] = orow;
    s_w[slot] = outer_w ? outer_w[(size_t)t * outer_k + slot] : 1.0f;
    int idx[kMaxTopK];
    for (int j = 0; j < n_k; ++j) {                    // insertion sort by group index
      const int e = topk_idx[(size_t)orow * n_k + j];
      int p = j;
      while (p > 0 && idx[p - 1] > e) {
        idx[p] = idx[p - 1];
        s_row[slot][p] = s_row[slot][p - 1];
        s_gate[slot][p] = s_gate[slot][p - 1];
        --p;
      }
      idx[p] = e;
      s_row[slot][p] = row_of[(size_t)orow * n_k + j];
      s_gate[slot][p] = topk_gate[(size_t)orow * n_k + j];
    }
  }
  __syncthreads();
  if (sizeof(T) == 2 && (d & 15) == 0) {            // bf16 rows in 32-byte pieces
    const bf16* ys = reinterpret_cast<const bf16*>(y_s);
    const bf16* yr = reinterpret_cast<const bf16*>(y_r);
    bf16* o = reinterpret_cast<bf16*>(out);
    for (int c = threadIdx.x * 16; c < d; c += blockDim.x * 16) {
      float acc[16];
#pragma unroll
      for (int q = 0; q < 16; ++q) acc[q] = 0.0f;
      for (int slot = 0; slot < outer_k; ++slot) {
        float inner[16];
#pragma unroll
        for (int q = 0; q < 16; ++q) inner[q] = 0.0f;
        if (ys) load16(ys + (size_t)s_orow[slot] * d + c, inner);
        for (int j = 0; j < n_k; ++j) {
          float v[16];
          load16(yr + (size_t)s_row[slot][j] * d + c, v);
          const float g = s_gate[slot][j];
#pragma unroll
          for (int q = 0; q < 16; ++q) inner[q] = fmaf(g, v[q], inner[q]);
        }
        const float w = s_w[slot];
#pragma unroll
        for (int q = 0; q < 16; ++q) acc[q] = fmaf(w, inner[q], acc[q]);
      }
      store16(o + (size_t)t * d + c, acc);
    }
    return;
  }
  for (int c = threadIdx.x * 8; c < d; c += blockDim.x * 8) {
    float acc[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) acc[q] = 0.0f;
    for (int slot = 0; slot < outer_k; ++slot) {
      float inner[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) inner[q] = 0.0f;
      if (y_s) load8(y_s + (size_t)s_orow[slot] * d + c, inner);
      for (int j = 0; j < n_k; ++j) {
        float v[8];
        load8(y_r + (size_t)s_row[slot][j] * d + c, v);
        const float g = s_gate[slot][j];
#pragma unroll
        for (int q = 0; q < 8; ++q) inner[q] = fmaf(g, v[q], inner[q]);
      }
      const float w = s_w[slot];
#pragma unroll
      for (int q = 0; q < 8; ++q) acc[q] = fmaf(w, inner[q], acc[q]);
    }
    store8(out + (size_t)t * d + c, acc);
  }
}

}  // namespace cmoe
