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
#include "permute.cuh"
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
  grid_dep_wait();
  grid_dep_trigger();
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

namespace cmoe {

// ---------------------------------------------------------------------------------------
// Router for at most kRskMaxRows rows (decode): the dot products are split over K across
// the grid so that every 16-byte load of x and W^R is in flight at once instead of in a
// per-warp sequence.  Block s owns the k slice [128 s, 128 s + 128); a warp takes one
// (16-row tile, 64-wide half slice) unit; the block adds its two halves in a fixed order
// and writes the slice's partial sums to scratch [slice][row][64]; the block that takes
// the last ticket adds the slices in ascending order (deterministic) and runs the gate
// logic, then resets the ticket for the next call.  With at most kRskFuseGroups routed
// groups the same block goes on to the histogram / scan / permutation of the selections
// (and the groups' row ranges), which saves two launches per decode step.
// Larger batches run the same kernel on a two-dimensional grid: block (s, c) owns k slice s of row chunk c
// (chunk_rows = 16, so that the chunks' reductions and gate logic run on many SMs, or 64 for routers of at
// most 8 columns, whose gate logic runs four rows per warp; kRskMaxTotalRows rows at most), and each chunk
// has its own scratch and ticket.  The chunks' last
// blocks take a second ticket, and the block that takes the last of those permutes the whole batch (up to
// kPermChunk rows; beyond that the permutation is left to the permutation kernels).
constexpr int kRskMaxRows = 64;
constexpr int kRskMaxChunks = 32;
constexpr int kRskMaxTotalRows = 512;       // rows of a batch this kernel takes (scratch: a [slices][64] block per row)
constexpr int kRskSliceK = 128;
constexpr int kRskMaxSlices = 64;           // d <= 8192
constexpr int kRskThreads = 256;
constexpr int kRskFuseGroups = 64;

// SUB8: the gate logic of the last block runs four rows per warp (8 lanes each; needs n_r <= 8),
// which pays for batches of more than 16 rows; the plain form is launched otherwise.
template <bool SUB8>
__global__ void __launch_bounds__(kRskThreads)
router_splitk_kernel(const bf16* __restrict__ xo, int n_rows, int d, int n_r, int n_rp, int n_k,
                     const bf16* __restrict__ w_rep, const float* __restrict__ u, const float* __restrict__ b,
                     const int32_t* __restrict__ outer_off, int n_outer,
                     float* __restrict__ part /*[chunks][slices][chunk_rows][64]*/,
                     int32_t* __restrict__ ticket /*[kRskMaxChunks + 1], zero between launches*/, int chunk_rows,
                     float* __restrict__ scores, float* __restrict__ keys,
                     int32_t* topk_idx, float* __restrict__ topk_gate,
                     int fuse_permute, int n_groups, int32_t* __restrict__ counts, int32_t* __restrict__ offsets,
                     int32_t* __restrict__ row_token, int32_t* __restrict__ row_of, const GroupPlanOut po) {
  grid_dep_wait();
  grid_dep_trigger();
  static_assert(kRskThreads == kPermChunk, "the fused permutation is written for one 256-row chunk");
  // this block's chunk of rows: from here on rows are counted within the chunk
  const int n_rows_all = n_rows;
  const int32_t* topk_idx_all = topk_idx;
  int32_t* ticket_chunks = ticket + kRskMaxChunks;
  const int row_base = blockIdx.y * chunk_rows;
  n_rows = min(chunk_rows, n_rows - row_base);
  xo += (size_t)row_base * d;
  scores += (size_t)row_base * n_r; keys += (size_t)row_base * n_r;
  topk_idx += (size_t)row_base * n_k; topk_gate += (size_t)row_base * n_k;
  part += (size_t)blockIdx.y * gridDim.x * chunk_rows * 64;
  ticket += blockIdx.y;
  __shared__ __align__(16) float unit[8][16][kRmStride];       // [unit = half*m_tiles + m-tile][row in tile][n]
  __shared__ int row_group[kRskMaxRows];
  __shared__ int is_last;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int n2 = 2 * n_rp, n_tiles = n2 >> 3;
  const int m_tiles = (n_rows + 15) >> 4;
  const int k_base = blockIdx.x * kRskSliceK;
  for (int r = threadIdx.x; r < kRskMaxRows; r += kRskThreads)
    row_group[r] = (outer_off && r < n_rows) ? find_outer(outer_off, n_outer, row_base + r) : 0;
  __syncthreads();
  const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
  const int un = warp;                           // at most 2 * 4 units for 8 warps
  if (un < 2 * m_tiles) {
    const int mt = un % m_tiles, half = un / m_tiles;
    const int r_lo = min(mt * 16 + g, n_rows - 1), r_hi = min(mt * 16 + g + 8, n_rows - 1);
    const int k0 = k_base + half * 64 + 8 * t, k1 = k0 + 32;
    const bool in0 = k0 < d, in1 = k1 < d;
    const uint4 a0_lo = in0 ? __ldg(reinterpret_cast<const uint4*>(xo + (size_t)r_lo * d + k0)) : zero;
    const uint4 a0_hi = in0 ? __ldg(reinterpret_cast<const uint4*>(xo + (size_t)r_hi * d + k0)) : zero;
    const uint4 a1_lo = in1 ? __ldg(reinterpret_cast<const uint4*>(xo + (size_t)r_lo * d + k1)) : zero;
    const uint4 a1_hi = in1 ? __ldg(reinterpret_cast<const uint4*>(xo + (size_t)r_hi * d + k1)) : zero;
    const int g_first = row_group[mt * 16], g_last = row_group[min(mt * 16 + 15, n_rows - 1)];
    for (int go = g_first; go <= g_last; ++go) {       // one pass unless the tile straddles outer experts
      const bf16* w = w_rep + (size_t)go * n2 * d;
      uint4 b0[8], b1[8];
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        const bf16* wr = w + (size_t)(nt * 8 + g) * d;
        b0[nt] = (nt < n_tiles && in0) ? __ldg(reinterpret_cast<const uint4*>(wr + k0)) : zero;
        b1[nt] = (nt < n_tiles && in1) ? __ldg(reinterpret_cast<const uint4*>(wr + k1)) : zero;
      }
      const bool take_lo = row_group[r_lo] == go, take_hi = row_group[r_hi] == go;
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        if (nt < n_tiles) {
          float acc[4] = {0.f, 0.f, 0.f, 0.f};
          mma_bf16_16816(acc, a0_lo.x, a0_hi.x, a0_lo.y, a0_hi.y, b0[nt].x, b0[nt].y);
          mma_bf16_16816(acc, a0_lo.z, a0_hi.z, a0_lo.w, a0_hi.w, b0[nt].z, b0[nt].w);
          mma_bf16_16816(acc, a1_lo.x, a1_hi.x, a1_lo.y, a1_hi.y, b1[nt].x, b1[nt].y);
          mma_bf16_16816(acc, a1_lo.z, a1_hi.z, a1_lo.w, a1_hi.w, b1[nt].z, b1[nt].w);
          const int col = nt * 8 + 2 * t;
          if (take_lo) { unit[un][g][col] = acc[0]; unit[un][g][col + 1] = acc[1]; }
          if (take_hi) { unit[un][g + 8][col] = acc[2]; unit[un][g + 8][col + 1] = acc[3]; }
        }
      }
    }
  }
  __syncthreads();
  // slice partial = first half + second half
  float* mine = part + (size_t)blockIdx.x * chunk_rows * 64;
  for (int i = threadIdx.x; i < n_rows * n2; i += kRskThreads) {
    const int r = i / n2, n = i - r * n2;
    const int mt = r >> 4, rr = r & 15;
    mine[r * 64 + n] = unit[mt][rr][n] + unit[m_tiles + mt][rr][n];
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = (atomicAdd(ticket, 1) == (int)gridDim.x - 1);
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  // Sum the slices in ascending order (a fixed order: deterministic), all threads at once, sixteen
  // 16-byte loads in flight per thread; the totals go to shared memory (the unit tiles are free now).
  float (*total)[kRmStride] = reinterpret_cast<float (*)[kRmStride]>(&unit[0][0][0]);   // [64][72]
  const int n_slices = (int)gridDim.x;
  const int n4 = n2 >> 2;                          // n2 is a multiple of 8: whole float4 groups
  const size_t kSliceStride4 = (size_t)chunk_rows * 64 / 4;
  for (int i = threadIdx.x; i < n_rows * n4; i += kRskThreads) {
    const int r = i / n4, n = (i - r * n4) * 4;
    const float4* ps = reinterpret_cast<const float4*>(part + (size_t)r * 64 + n);
    float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
    int s = 0;
    for (; s + 16 <= n_slices; s += 16) {
      float4 t[16];
#pragma unroll
      for (int q = 0; q < 16; ++q) t[q] = __ldcg(ps + (size_t)(s + q) * kSliceStride4);
#pragma unroll
      for (int q = 0; q < 16; ++q) { sum.x += t[q].x; sum.y += t[q].y; sum.z += t[q].z; sum.w += t[q].w; }
    }
    for (; s < n_slices; ++s) {
      const float4 t = __ldcg(ps + (size_t)s * kSliceStride4);
      sum.x += t.x; sum.y += t.y; sum.z += t.z; sum.w += t.w;
    }
    *reinterpret_cast<float4*>(&total[r][n]) = sum;
  }
  __syncthreads();
  if (SUB8) {                                      // four rows per warp at a time, 8 lanes each
    const int sub = lane & 7, grp = lane >> 3;
    for (int r0 = warp * 4; r0 < n_rows; r0 += (kRskThreads / 32) * 4) {
      const int r = r0 + grp;
      const bool live_row = r < n_rows;
      const int rr = live_row ? r : 0;
      const float a = (live_row && sub < n_r) ? total[rr][sub] : 0.0f;
      const float v = (live_row && sub < n_r) ? total[rr][n_rp + sub] : 0.0f;
      const int go = row_group[rr];
      gate_row_sub<8>(sub, live_row, n_r, n_k, a, v, u + go * n_r, b + go * n_r, go * n_r, scores + (size_t)rr * n_r,
                      keys + (size_t)rr * n_r, topk_idx + (size_t)rr * n_k, topk_gate + (size_t)rr * n_k);
    }
  } else {
    for (int r = warp; r < n_rows; r += kRskThreads / 32) {
      const float a = lane < n_r ? total[r][lane] : 0.0f;
      const float v = lane < n_r ? total[r][n_rp + lane] : 0.0f;
      const int go = row_group[r];
      gate_row(lane, n_r, n_k, a, v, u + go * n_r, b + go * n_r, go * n_r, scores + (size_t)r * n_r,
               keys + (size_t)r * n_r, topk_idx + (size_t)r * n_k, topk_gate + (size_t)r * n_k);
    }
  }
  if (threadIdx.x == 0) *ticket = 0;
  if (!fuse_permute) return;
  if (gridDim.y > 1) {                             // the last chunk to finish permutes the batch
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(ticket_chunks, 1) == (int)gridDim.y - 1);
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    if (threadIdx.x == 0) *ticket_chunks = 0;
    n_rows = n_rows_all;
    topk_idx = const_cast<int32_t*>(topk_idx_all);
  }
  // ---- histogram / scan / stable permutation of the selections just written (at most kPermChunk rows)
  __syncthreads();
  int32_t* sm = reinterpret_cast<int32_t*>(&unit[0][0][0]);     // the partial sums are no longer needed
  int32_t* hist = sm;                              // [n_groups]
  int32_t* offs = hist + n_groups;                 // [n_groups + 1]
  int32_t* sums = offs + n_groups + 1;             // [kPermChunk]
  int32_t* warp_cnt = sums + kPermChunk;           // [8][n_groups]
  int32_t* sel = warp_cnt + 8 * n_groups;          // [n_rows * n_k] copy of the selections
  for (int i = threadIdx.x; i < n_rows * n_k; i += kRskThreads) sel[i] = __ldcg(topk_idx + i);
  __syncthreads();
  const int row = threadIdx.x;
  chunk_histogram(sel, n_rows, n_k, n_groups, row, hist);
  block_scan_groups(hist, offs, n_groups, sums);
  for (int gq = threadIdx.x; gq < n_groups; gq += kRskThreads) { counts[gq] = hist[gq]; offsets[gq] = offs[gq]; }
  if (threadIdx.x == 0) offsets[n_groups] = offs[n_groups];
  write_group_rows(po, n_groups, hist, offs);
  chunk_scatter(sel, n_rows, n_k, n_groups, row, offs, warp_cnt, row_token, row_of);
}

}  // namespace cmoe
