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
// added in the order of the selection (descending key), a fixed order, so results are
// reproducible run to run; fp32 accumulation, one rounding to the output type.  Every
// thread reads the token's few routing words itself (same addresses across the block, so
// they broadcast from L1) and then streams its 16 (bf16) or 8 columns of every row.
template <typename T>
__global__ void __launch_bounds__(256)
combine_kernel(const T* __restrict__ y_s, const T* __restrict__ y_r,
               const int32_t* __restrict__ topk_idx, const float* __restrict__ topk_gate,
               const int32_t* __restrict__ row_of, const int32_t* __restrict__ outer_row_of,
               const float* __restrict__ outer_w, int outer_k, int n_k, int d, T* __restrict__ out) {
  grid_dep_wait();
  grid_dep_trigger();
  (void)topk_idx;
  const int t = blockIdx.x;
  constexpr bool kWide = sizeof(T) == 2;
  constexpr int kCols = kWide ? 16 : 8;
  const bool wide_ok = (d % kCols) == 0;
  for (int c = threadIdx.x * kCols; c < d; c += blockDim.x * kCols) {
    float acc[kCols];
#pragma unroll
    for (int q = 0; q < kCols; ++q) acc[q] = 0.0f;
    for (int slot = 0; slot < outer_k; ++slot) {
      const int orow = outer_row_of ? __ldg(outer_row_of + (size_t)t * outer_k + slot) : t;
      const float w = outer_w ? __ldg(outer_w + (size_t)t * outer_k + slot) : 1.0f;
      float inner[kCols];
#pragma unroll
      for (int q = 0; q < kCols; ++q) inner[q] = 0.0f;
      if constexpr (kWide) {
        const bf16* ys = reinterpret_cast<const bf16*>(y_s);
        const bf16* yr = reinterpret_cast<const bf16*>(y_r);
        if (wide_ok) {
          if (ys) load16(ys + (size_t)orow * d + c, inner);
          for (int j = 0; j < n_k; ++j) {
            const int row = __ldg(row_of + (size_t)orow * n_k + j);
            const float g = __ldg(topk_gate + (size_t)orow * n_k + j);
            float v[16];
            load16(yr + (size_t)row * d + c, v);
#pragma unroll
            for (int q = 0; q < 16; ++q) inner[q] = fmaf(g, v[q], inner[q]);
          }
        } else {                                    // d % 16 == 8: two 8-column halves
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            if (c + h * 8 < d) {
              float v[8], part[8];
#pragma unroll
              for (int q = 0; q < 8; ++q) part[q] = 0.0f;
              if (ys) load8(ys + (size_t)orow * d + c + h * 8, part);
              for (int j = 0; j < n_k; ++j) {
                const int row = __ldg(row_of + (size_t)orow * n_k + j);
                const float g = __ldg(topk_gate + (size_t)orow * n_k + j);
                load8(yr + (size_t)row * d + c + h * 8, v);
#pragma unroll
                for (int q = 0; q < 8; ++q) part[q] = fmaf(g, v[q], part[q]);
              }
#pragma unroll
              for (int q = 0; q < 8; ++q) inner[h * 8 + q] = part[q];
            }
          }
        }
      } else {
        float v[8];
        if (y_s) { load8(y_s + (size_t)orow * d + c, v);
#pragma unroll
          for (int q = 0; q < 8; ++q) inner[q] = v[q]; }
        for (int j = 0; j < n_k; ++j) {
          const int row = __ldg(row_of + (size_t)orow * n_k + j);
          const float g = __ldg(topk_gate + (size_t)orow * n_k + j);
          load8(y_r + (size_t)row * d + c, v);
#pragma unroll
          for (int q = 0; q < 8; ++q) inner[q] = fmaf(g, v[q], inner[q]);
        }
      }
#pragma unroll
      for (int q = 0; q < kCols; ++q) acc[q] = fmaf(w, inner[q], acc[q]);
    }
    if constexpr (kWide) {
      bf16* o = reinterpret_cast<bf16*>(out) + (size_t)t * d + c;
      if (wide_ok) {
        store16(o, acc);
      } else {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (c + h * 8 < d) {
            float v[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) v[q] = acc[h * 8 + q];
            store8(o + h * 8, v);
          }
        }
      }
    } else {
      float v[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) v[q] = acc[q];
      store8(reinterpret_cast<float*>(out) + (size_t)t * d + c, v);
    }
  }
}

// The same sum for a plain (one-level) bf16 layer with d % 16 == 0 and n_k <= NK, written for
// bandwidth: a block strides over tokens with one thread per 16 columns (one pass over the
// row whatever d is), all 1 + n_k row loads of a token are issued before any arithmetic, and
// the next token's routing words are fetched while the current rows are in flight.  The
// arithmetic and its order are those of combine_kernel, so both give the same bits.
__device__ __forceinline__ void ld256_stream(const bf16* p, uint32_t (&w)[8]) {
  // volatile + memory clobber: the load must stay below griddepcontrol.wait (its source is written
  // by the preceding kernel of a chained launch)
  asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
               : "l"(p) : "memory");
}

template <int NK>
__global__ void __launch_bounds__(1024)
combine_plain_bf16_kernel(const bf16* __restrict__ y_s, const bf16* __restrict__ y_r,
                          const float* __restrict__ topk_gate, const int32_t* __restrict__ row_of,
                          int n_tok, int n_k, int d, bf16* __restrict__ out) {
  grid_dep_wait();
  grid_dep_trigger();
  const int c = threadIdx.x * 16;
  if (c >= d) return;
  int t = blockIdx.x;
  if (t >= n_tok) return;
  int rows[NK], rows_next[NK];
  float g[NK], g_next[NK];
#pragma unroll
  for (int j = 0; j < NK; ++j) {
    rows[j] = j < n_k ? __ldg(row_of + (size_t)t * n_k + j) : 0;
    g[j] = j < n_k ? __ldg(topk_gate + (size_t)t * n_k + j) : 0.0f;
  }
  while (true) {
    uint32_t ws[8], wr[NK][8];
    if (y_s) ld256_stream(y_s + (size_t)t * d + c, ws);
#pragma unroll
    for (int j = 0; j < NK; ++j)
      if (j < n_k) ld256_stream(y_r + (size_t)rows[j] * d + c, wr[j]);
    const int t_next = t + gridDim.x;
    if (t_next < n_tok) {
#pragma unroll
      for (int j = 0; j < NK; ++j) {
        rows_next[j] = j < n_k ? __ldg(row_of + (size_t)t_next * n_k + j) : 0;
        g_next[j] = j < n_k ? __ldg(topk_gate + (size_t)t_next * n_k + j) : 0.0f;
      }
    }
    float inner[16];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      inner[2 * q] = y_s ? __uint_as_float(ws[q] << 16) : 0.0f;
      inner[2 * q + 1] = y_s ? __uint_as_float(ws[q] & 0xffff0000u) : 0.0f;
    }
#pragma unroll
    for (int j = 0; j < NK; ++j) {
      if (j < n_k) {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          inner[2 * q] = fmaf(g[j], __uint_as_float(wr[j][q] << 16), inner[2 * q]);
          inner[2 * q + 1] = fmaf(g[j], __uint_as_float(wr[j][q] & 0xffff0000u), inner[2 * q + 1]);
        }
      }
    }
    store16(out + (size_t)t * d + c, inner);      // outer weight 1: fmaf(1, inner, 0) == inner
    if (t_next >= n_tok) break;
    t = t_next;
#pragma unroll
    for (int j = 0; j < NK; ++j) { rows[j] = rows_next[j]; g[j] = g_next[j]; }
  }
}

}  // namespace cmoe
