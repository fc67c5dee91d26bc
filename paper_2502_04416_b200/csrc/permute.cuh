// Token histogram, exclusive scan and stable permutation into expert-contiguous
// order.  Integer only and deterministic: the result is the list of selected
// (row, group) pairs sorted by (group, row).
//
// Rows are cut into chunks of kPermChunk; a chunk's per-group counts go to a
// scratch matrix [n_chunks][n_groups], one block scans it group by group, and
// every chunk then places its pairs at (group offset + pairs of earlier chunks +
// rank inside the chunk).  With a single chunk everything runs in one block.
#pragma once

#include "common.cuh"

namespace cmoe {

constexpr int kPermChunk = 256;      // rows per block, one thread per row
constexpr int kPermMaxGroups = 1024;

__device__ __forceinline__ void chunk_histogram(const int32_t* __restrict__ topk_idx, int n_rows,
                                                int n_k, int n_groups, int row, int32_t* hist) {
  for (int g = threadIdx.x; g < n_groups; g += blockDim.x) hist[g] = 0;
  __syncthreads();
  if (row < n_rows)
    for (int j = 0; j < n_k; ++j) {
      const int e = topk_idx[(size_t)row * n_k + j];
      if ((unsigned)e < (unsigned)n_groups) atomicAdd(&hist[e], 1);   // out-of-range entries are ignored
    }
  __syncthreads();
}

// Exclusive scan of counts[0..n_groups) into offsets[0..n_groups]; sums[] holds
// blockDim.x ints of shared memory.
__device__ __forceinline__ void block_scan_groups(const int32_t* counts, int32_t* offsets,
                                                  int n_groups, int32_t* sums) {
  const int per = (n_groups + blockDim.x - 1) / blockDim.x;
  const int lo = min((int)threadIdx.x * per, n_groups);
  const int hi = min(lo + per, n_groups);
  int s = 0;
  for (int g = lo; g < hi; ++g) s += counts[g];
  sums[threadIdx.x] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    int run = 0;
    for (int i = 0; i < (int)blockDim.x; ++i) { const int v = sums[i]; sums[i] = run; run += v; }
    offsets[n_groups] = run;
  }
  __syncthreads();
  int run = sums[threadIdx.x];
  for (int g = lo; g < hi; ++g) { offsets[g] = run; run += counts[g]; }
  __syncthreads();
}

// Places the pairs of one chunk.  base[g] = first free row of group g for this chunk.
__device__ __forceinline__ void chunk_scatter(const int32_t* __restrict__ topk_idx, int n_rows,
                                              int n_k, int n_groups, int row, const int32_t* base,
                                              int32_t* warp_cnt /*[8][n_groups]*/,
                                              int32_t* __restrict__ row_token,
                                              int32_t* __restrict__ row_of) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned lt = (1u << lane) - 1u;
  int sel[kMaxTopK], rank[kMaxTopK];
#pragma unroll
  for (int j = 0; j < kMaxTopK; ++j) {
    sel[j] = (row < n_rows && j < n_k) ? topk_idx[(size_t)row * n_k + j] : -1;
    if ((unsigned)sel[j] >= (unsigned)n_groups) sel[j] = -1;
    rank[j] = 0;
  }
  for (int g = 0; g < n_groups; ++g) {
    bool has = false;
#pragma unroll
    for (int j = 0; j < kMaxTopK; ++j) has |= (sel[j] == g);
    const unsigned vote = __ballot_sync(0xffffffffu, has);
#pragma unroll
    for (int j = 0; j < kMaxTopK; ++j)
      if (sel[j] == g) rank[j] = __popc(vote & lt);
    if (lane == 0) warp_cnt[warp * n_groups + g] = __popc(vote);
  }
  __syncthreads();
#pragma unroll
  for (int j = 0; j < kMaxTopK; ++j) {
    if (sel[j] >= 0) {
      int pos = base[sel[j]] + rank[j];
      for (int w = 0; w < warp; ++w) pos += warp_cnt[w * n_groups + sel[j]];
      row_token[pos] = row;
      row_of[(size_t)row * n_k + j] = pos;
    }
  }
}

// Optional by-product of the permutation inside a layer's forward: the row range of every
// expert group (n_outer shared groups over the outer rows, then the routed groups), which
// the grouped GEMMs' tile schedulers read.  gr == nullptr: not wanted.
struct GroupPlanOut {
  GroupRows* gr = nullptr;
  int n_outer = 0, n_tokens = 0;
  const int32_t* outer_off = nullptr;    // hierarchical: row ranges of the outer experts
};

__device__ __forceinline__ void write_group_rows(const GroupPlanOut& po, int n_groups, const int32_t* counts,
                                                 const int32_t* offsets) {
  if (po.gr == nullptr) return;
  for (int g = threadIdx.x; g < po.n_outer + n_groups; g += blockDim.x) {
    GroupRows r;
    if (g < po.n_outer) {
      r.row0 = po.outer_off ? po.outer_off[g] : 0;
      r.count = po.outer_off ? po.outer_off[g + 1] - po.outer_off[g] : po.n_tokens;
    } else {
      r.row0 = offsets[g - po.n_outer];
      r.count = counts[g - po.n_outer];
    }
    po.gr[g] = r;
  }
}

// n_rows <= kPermChunk: histogram, scan and scatter in one block.
__global__ void __launch_bounds__(kPermChunk)
permute_single_kernel(const int32_t* __restrict__ topk_idx, int n_rows, int n_k, int n_groups,
                      int32_t* __restrict__ counts, int32_t* __restrict__ offsets,
                      int32_t* __restrict__ row_token, int32_t* __restrict__ row_of, const GroupPlanOut po) {
  grid_dep_wait();
  grid_dep_trigger();
  extern __shared__ int32_t sm[];
  int32_t* hist = sm;                              // [n_groups]
  int32_t* offs = hist + n_groups;                 // [n_groups + 1]
  int32_t* sums = offs + n_groups + 1;             // [kPermChunk]
  int32_t* warp_cnt = sums + kPermChunk;           // [8][n_groups]
  const int row = threadIdx.x;
  chunk_histogram(topk_idx, n_rows, n_k, n_groups, row, hist);
  block_scan_groups(hist, offs, n_groups, sums);
  for (int g = threadIdx.x; g < n_groups; g += blockDim.x) { counts[g] = hist[g]; offsets[g] = offs[g]; }
  if (threadIdx.x == 0) offsets[n_groups] = offs[n_groups];
  write_group_rows(po, n_groups, hist, offs);
  chunk_scatter(topk_idx, n_rows, n_k, n_groups, row, offs, warp_cnt, row_token, row_of);
}

__global__ void __launch_bounds__(kPermChunk)
permute_count_kernel(const int32_t* __restrict__ topk_idx, int n_rows, int n_k, int n_groups,
                     int32_t* __restrict__ chunk_cnt /*[n_chunks][n_groups]*/) {
  grid_dep_wait();
  grid_dep_trigger();
  extern __shared__ int32_t sm[];
  const int row = blockIdx.x * kPermChunk + threadIdx.x;
  chunk_histogram(topk_idx, n_rows, n_k, n_groups, row, sm);
  for (int g = threadIdx.x; g < n_groups; g += blockDim.x)
    chunk_cnt[(size_t)blockIdx.x * n_groups + g] = sm[g];
}

// One block: per group, a warp turns the column of chunk counts into the chunks'
// exclusive prefixes inside the group; then the scan over groups.
__global__ void __launch_bounds__(1024)
permute_scan_kernel(int32_t* chunk_cnt, int n_chunks, int n_groups,
                    int32_t* __restrict__ counts, int32_t* __restrict__ offsets, const GroupPlanOut po) {
  grid_dep_wait();
  grid_dep_trigger();
  __shared__ int32_t sums[1024];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  for (int g = warp; g < n_groups; g += n_warps) {
    int run = 0;
    for (int c0 = 0; c0 < n_chunks; c0 += 32) {
      const int c = c0 + lane;
      const int v = c < n_chunks ? chunk_cnt[(size_t)c * n_groups + g] : 0;
      int incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
      }
      if (c < n_chunks) chunk_cnt[(size_t)c * n_groups + g] = run + incl - v;
      run += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) counts[g] = run;
  }
  __syncthreads();
  block_scan_groups(counts, offsets, n_groups, sums);
  write_group_rows(po, n_groups, counts, offsets);
}

__global__ void __launch_bounds__(kPermChunk)
permute_scatter_kernel(const int32_t* __restrict__ topk_idx, int n_rows, int n_k, int n_groups,
                       const int32_t* __restrict__ chunk_cnt, const int32_t* __restrict__ offsets,
                       int32_t* __restrict__ row_token, int32_t* __restrict__ row_of) {
  grid_dep_wait();
  grid_dep_trigger();
  extern __shared__ int32_t sm[];
  int32_t* base = sm;                      // [n_groups]
  int32_t* warp_cnt = base + n_groups;     // [8][n_groups]
  for (int g = threadIdx.x; g < n_groups; g += blockDim.x)
    base[g] = offsets[g] + chunk_cnt[(size_t)blockIdx.x * n_groups + g];
  __syncthreads();
  const int row = blockIdx.x * kPermChunk + threadIdx.x;
  chunk_scatter(topk_idx, n_rows, n_k, n_groups, row, base, warp_cnt, row_token, row_of);
}

// Scan and scatter in one launch, for count matrices small enough to be re-read by every block
// (n_chunks * n_groups <= kPermFusedCells): block c adds up, per group, the counts of the chunks
// before it and of all chunks, scans the group totals itself and places its chunk; block 0 also
// publishes counts, offsets and the groups' row ranges.  The same integers as the three-kernel
// form, one launch fewer.
constexpr int kPermFusedCells = 16384;

__global__ void __launch_bounds__(kPermChunk)
permute_scan_scatter_kernel(const int32_t* __restrict__ topk_idx, int n_rows, int n_k, int n_groups, int n_chunks,
                            const int32_t* __restrict__ chunk_cnt, int32_t* __restrict__ counts,
                            int32_t* __restrict__ offsets, int32_t* __restrict__ row_token,
                            int32_t* __restrict__ row_of, const GroupPlanOut po) {
  grid_dep_wait();
  grid_dep_trigger();
  extern __shared__ int32_t sm[];
  int32_t* total = sm;                         // [n_groups]
  int32_t* offs = total + n_groups;            // [n_groups + 1]
  int32_t* base = offs + n_groups + 1;         // [n_groups]
  int32_t* sums = base + n_groups;             // [kPermChunk]
  int32_t* warp_cnt = sums + kPermChunk;       // [8][n_groups]
  const int c = blockIdx.x;
  for (int g = threadIdx.x; g < n_groups; g += blockDim.x) {
    int before = 0, all = 0;
    for (int cc = 0; cc < n_chunks; ++cc) {
      const int v = __ldg(chunk_cnt + (size_t)cc * n_groups + g);
      before += cc < c ? v : 0;
      all += v;
    }
    total[g] = all;
    base[g] = before;
  }
  __syncthreads();
  block_scan_groups(total, offs, n_groups, sums);
  for (int g = threadIdx.x; g < n_groups; g += blockDim.x) base[g] += offs[g];
  if (c == 0) {
    for (int g = threadIdx.x; g < n_groups; g += blockDim.x) { counts[g] = total[g]; offsets[g] = offs[g]; }
    if (threadIdx.x == 0) offsets[n_groups] = offs[n_groups];
    write_group_rows(po, n_groups, total, offs);
  }
  __syncthreads();
  const int row = c * kPermChunk + threadIdx.x;
  chunk_scatter(topk_idx, n_rows, n_k, n_groups, row, base, warp_cnt, row_token, row_of);
}

inline int64_t permute_scratch_bytes(int n_rows, int n_groups) {
  const int64_t n_chunks = (n_rows + kPermChunk - 1) / kPermChunk;
  const int64_t b = n_chunks * n_groups * (int64_t)sizeof(int32_t);
  return (b + 255) / 256 * 256;
}

// Enqueues the permutation; returns the number of kernels launched.
inline int launch_token_permute(const int32_t* topk_idx, int n_rows, int n_k, int n_groups,
                                int32_t* counts, int32_t* offsets, int32_t* row_token,
                                int32_t* row_of, int32_t* scratch, cudaStream_t stream,
                                const GroupPlanOut po = GroupPlanOut(), bool dep = false) {
  if (n_rows <= kPermChunk) {
    const size_t smem = (size_t)(n_groups * 2 + 1 + kPermChunk + 8 * n_groups) * sizeof(int32_t);
    launch_kernel(dep, permute_single_kernel, dim3(1), dim3(kPermChunk), smem, stream, topk_idx, n_rows, n_k,
                  n_groups, counts, offsets, row_token, row_of, po);
    return 1;
  }
  const int n_chunks = (n_rows + kPermChunk - 1) / kPermChunk;
  launch_kernel(dep, permute_count_kernel, dim3(n_chunks), dim3(kPermChunk), n_groups * sizeof(int32_t), stream,
                topk_idx, n_rows, n_k, n_groups, scratch);
  if ((long long)n_chunks * n_groups <= kPermFusedCells && n_groups <= 1024) {
    const size_t smem = (size_t)(n_groups * 3 + 1 + kPermChunk + 8 * n_groups) * sizeof(int32_t);
    launch_kernel(dep, permute_scan_scatter_kernel, dim3(n_chunks), dim3(kPermChunk), smem, stream, topk_idx, n_rows,
                  n_k, n_groups, n_chunks, (const int32_t*)scratch, counts, offsets, row_token, row_of, po);
    return 2;
  }
  launch_kernel(dep, permute_scan_kernel, dim3(1), dim3(1024), 0, stream, scratch, n_chunks, n_groups, counts,
                offsets, po);
  launch_kernel(dep, permute_scatter_kernel, dim3(n_chunks), dim3(kPermChunk), 9 * n_groups * sizeof(int32_t), stream,
                topk_idx, n_rows, n_k, n_groups, scratch, offsets, row_token, row_of);
  return 3;
}

}  // namespace cmoe
