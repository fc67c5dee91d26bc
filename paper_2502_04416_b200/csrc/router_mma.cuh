// bf16 router on the warp-level tensor-core path: the router is a skinny contraction
// [rows, d] x [d, 2*N_r] (Eq. router), far too narrow for a tcgen05 tile and, on CUDA
// cores, latency-bound; mma.sync.m16n8k16 with fp32 accumulation keeps it a small,
// bandwidth-bound kernel.  A block owns ROWS = 16*MT rows; its warps split K and their
// partial sums are added in a fixed order (deterministic), then each row's N_r score
// pairs go through the same warp-shuffle softmax / top-k as the SIMT router.
//
// Operand fragments are loaded straight from global memory, 16 bytes per lane.  The k
// index inside a 32-wide chunk is permuted identically for the x and the W fragments
// (a lane's 8 consecutive elements stand for the fragment's k = 2t,2t+1,2t+8,2t+9 of
// two consecutive k16 steps), which leaves every dot product unchanged.
#pragma once

#include "common.cuh"
#include "router.cuh"

namespace cmoe {

constexpr int kRmStride = 72;    // floats per row of the partial / final tiles (64 + pad)

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// fin[r][n] = sum_k x[row0 + r][k] * w[n][k] for r < 16*MT, n < n2 (n2 <= 64), all warps of
// the block cooperating.  Rows beyond n_rows repeat the last valid row (callers skip them).
template <int WARPS, int MT>
__device__ __forceinline__ void block_dot_tile(const bf16* __restrict__ x, int n_rows, int row0, int d,
                                               const bf16* __restrict__ w, int n2,
                                               float (*part)[16 * MT][kRmStride],
                                               float (*fin)[kRmStride], const int* row_take /*null: all*/,
                                               int take_value) {
  constexpr int ROWS = 16 * MT;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int n_tiles = (n2 + 7) >> 3;
  float acc[MT][8][4];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int nt = 0; nt < 8; ++nt)
#pragma unroll
      for (int q = 0; q < 4; ++q) acc[mt][nt][q] = 0.0f;

  const bf16* xr[MT][2];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    xr[mt][0] = x + (size_t)min(row0 + mt * 16 + g, n_rows - 1) * d;
    xr[mt][1] = x + (size_t)min(row0 + mt * 16 + g + 8, n_rows - 1) * d;
  }
  const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
  for (int k0 = warp * 32; k0 < d; k0 += WARPS * 32) {
    const int k = k0 + 8 * t;
    const bool kin = k < d;
    uint4 a[MT][2];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      a[mt][0] = kin ? __ldg(reinterpret_cast<const uint4*>(xr[mt][0] + k)) : zero;
      a[mt][1] = kin ? __ldg(reinterpret_cast<const uint4*>(xr[mt][1] + k)) : zero;
    }
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      if (nt < n_tiles) {
        const int n = nt * 8 + g;
        const uint4 bw = (kin && n < n2) ? __ldg(reinterpret_cast<const uint4*>(w + (size_t)n * d + k)) : zero;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          mma_bf16_16816(acc[mt][nt], a[mt][0].x, a[mt][1].x, a[mt][0].y, a[mt][1].y, bw.x, bw.y);
          mma_bf16_16816(acc[mt][nt], a[mt][0].z, a[mt][1].z, a[mt][0].w, a[mt][1].w, bw.z, bw.w);
        }
      }
    }
  }
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      if (nt < n_tiles) {
        float* p0 = &part[warp][mt * 16 + g][nt * 8 + 2 * t];
        float* p1 = &part[warp][mt * 16 + g + 8][nt * 8 + 2 * t];
        p0[0] = acc[mt][nt][0]; p0[1] = acc[mt][nt][1];
        p1[0] = acc[mt][nt][2]; p1[1] = acc[mt][nt][3];
      }
    }
  __syncthreads();
  for (int i = threadIdx.x; i < ROWS * 64; i += WARPS * 32) {
    const int r = i >> 6, n = i & 63;
    if (n < n_tiles * 8 && (row_take == nullptr || row_take[r] == take_value)) {
      float s = 0.0f;
#pragma unroll
      for (int wq = 0; wq < WARPS; ++wq) s += part[wq][r][n];      // fixed order: deterministic
      fin[r][n] = s;
    }
  }
  __syncthreads();
}

template <int WARPS, int MT>
__global__ void __launch_bounds__(WARPS * 32)
router_mma_kernel(const bf16* __restrict__ xo, int n_rows, int d, int n_r, int n_rp, int n_k,
                  const bf16* __restrict__ w_rep, const float* __restrict__ u, const float* __restrict__ b,
                  const int32_t* __restrict__ outer_off, int n_outer,
                  float* __restrict__ scores, float* __restrict__ keys,
                  int32_t* __restrict__ topk_idx, float* __restrict__ topk_gate) {
  constexpr int ROWS = 16 * MT;
  __shared__ float part[WARPS][ROWS][kRmStride];
  __shared__ float fin[ROWS][kRmStride];
  __shared__ int row_group[ROWS];
  const int row0 = blockIdx.x * ROWS;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n2 = 2 * n_rp;      // W^R block: n_rp gate rows (zero-padded), then n_rp up rows
  if (threadIdx.x < ROWS)
    row_group[threadIdx.x] = outer_off ? find_outer(outer_off, n_outer, min(row0 + (int)threadIdx.x, n_rows - 1)) : 0;
  __syncthreads();
  const int g_lo = row_group[0], g_hi = row_group[ROWS - 1];
  for (int go = g_lo; go <= g_hi; ++go)          // one pass, except for tiles that straddle outer experts
    block_dot_tile<WARPS, MT>(xo, n_rows, row0, d, w_rep + (size_t)go * n2 * d, n2, part, fin,
                              g_lo == g_hi ? nullptr : row_group, go);
  for (int r = warp; r < ROWS; r += WARPS) {
    const int row = row0 + r;
    if (row >= n_rows) break;
    const int go = row_group[r];
    const float a = lane < n_r ? fin[r][lane] : 0.0f;
    const float v = lane < n_r ? fin[r][n_rp + lane] : 0.0f;
    gate_row(lane, n_r, n_k, a, v, u + go * n_r, b + go * n_r, go * n_r, scores + (size_t)row * n_r,
             keys + (size_t)row * n_r, topk_idx + (size_t)row * n_k, topk_gate + (size_t)row * n_k);
  }
}

// Top-level router of a hierarchical layer on the same contraction: logits = W_r x.
template <int WARPS, int MT>
__global__ void __launch_bounds__(WARPS * 32)
outer_router_mma_kernel(const bf16* __restrict__ x, int n_tokens, int d, int n_outer, int outer_k,
                        const bf16* __restrict__ w_router, float* __restrict__ logits,
                        int32_t* __restrict__ outer_idx, float* __restrict__ outer_w) {
  constexpr int ROWS = 16 * MT;
  __shared__ float part[WARPS][ROWS][kRmStride];
  __shared__ float fin[ROWS][kRmStride];
  const int row0 = blockIdx.x * ROWS;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  block_dot_tile<WARPS, MT>(x, n_tokens, row0, d, w_router, n_outer, part, fin, nullptr, 0);
  for (int r = warp; r < ROWS; r += WARPS) {
    const int tkn = row0 + r;
    if (tkn >= n_tokens) break;
    const bool live = lane < n_outer;
    const float logit = live ? fin[r][lane] : -INFINITY;
    if (live) logits[(size_t)tkn * n_outer + lane] = logit;
    const float rank_key = (logit != logit) ? -INFINITY : logit;
    bool taken = !live;
    float sel_logit = -INFINITY;
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
    const float wgt = e / warp_sum(e);
    if (lane < outer_k) {
      outer_idx[(size_t)tkn * outer_k + lane] = sel_who;
      outer_w[(size_t)tkn * outer_k + lane] = wgt;
    }
  }
}

}  // namespace cmoe
