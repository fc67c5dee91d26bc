// Plain SIMT grouped expert GEMMs (fp32 FMA, fp32 accumulate).  They serve the
// fp32 storage type and every shape the tensor-core path does not take, and give
// a second, structurally different implementation to check the tensor path against.
//
//   GEMM-1: H[r, n] = Swish(sum_k A[r,k] Wg[n,k]) * (sum_k A[r,k] Wu[n,k])   (Eq. ori_ffn_method)
//   GEMM-2: Y[r, c] = sum_n H[r,n] Wd[c,n]
// per group g (one shared expert per outer expert, then every routed expert), on the
// group's rows [row0, row0+count) of its row space.
#pragma once

#include "common.cuh"

namespace cmoe {

constexpr int kSimtTile = 64;
constexpr int kSimtBK = 32;

template <typename T>
__device__ __forceinline__ void load_seg(const T* row_ptr, int k, int K, bool vec, float (&v)[8]) {
  if (row_ptr == nullptr) {
#pragma unroll
    for (int q = 0; q < 8; ++q) v[q] = 0.0f;
  } else if (vec && k + 8 <= K) {
    load8(row_ptr + k, v);
  } else {
#pragma unroll
    for (int q = 0; q < 8; ++q) v[q] = (k + q < K) ? to_float(row_ptr[k + q]) : 0.0f;
  }
}

// One 64x64 tile of C = A B^T (and, if DUAL, of A B2^T) into acc / acc2.
// A: M x K (lda), B/B2: N x K (ldb); (m0, n0) tile origin.  256 threads.
template <typename T, bool DUAL>
__device__ __forceinline__ void simt_tile(const T* __restrict__ A, int lda, int M, const T* __restrict__ B,
                                          const T* __restrict__ B2, int ldb, int N, int K, int m0, int n0,
                                          bool vec_a, bool vec_b, float (&acc)[4][4], float (&acc2)[4][4]) {
  __shared__ float As[kSimtBK][kSimtTile + 1];
  __shared__ float Bs[kSimtBK][kSimtTile + 1];
  __shared__ float Bs2[DUAL ? kSimtBK : 1][kSimtTile + 1];
  const int tid = threadIdx.x;
  const int lrow = tid >> 2, kseg = (tid & 3) * 8;
  const int ty = tid >> 4, tx = tid & 15;
  const T* a_row = (m0 + lrow < M) ? A + (size_t)(m0 + lrow) * lda : nullptr;
  const T* b_row = (n0 + lrow < N) ? B + (size_t)(n0 + lrow) * ldb : nullptr;
  const T* b2_row = (DUAL && n0 + lrow < N) ? B2 + (size_t)(n0 + lrow) * ldb : nullptr;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) { acc[i][j] = 0.0f; acc2[i][j] = 0.0f; }

  for (int k0 = 0; k0 < K; k0 += kSimtBK) {
    float va[8], vb[8], vb2[8];
    load_seg(a_row, k0 + kseg, K, vec_a, va);
    load_seg(b_row, k0 + kseg, K, vec_b, vb);
    if (DUAL) load_seg(b2_row, k0 + kseg, K, vec_b, vb2);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      As[kseg + q][lrow] = va[q];
      Bs[kseg + q][lrow] = vb[q];
      if (DUAL) Bs2[kseg + q][lrow] = vb2[q];
    }
    __syncthreads();
#pragma unroll 8
    for (int kk = 0; kk < kSimtBK; ++kk) {
      float a[4], b[4], b2[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        b[j] = Bs[kk][tx * 4 + j];
        b2[j] = DUAL ? Bs2[kk][tx * 4 + j] : 0.0f;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
          if (DUAL) acc2[i][j] = fmaf(a[i], b2[j], acc2[i][j]);
        }
    }
    __syncthreads();
  }
}

template <typename T>
struct SimtGemmArgs {
  const GroupStatic* gs;
  const GroupRows* gr;
  const T* a_shared;   // GEMM-1: outer rows of x [R, d];            GEMM-2: H_s [R, shared width]
  const T* a_routed;   // GEMM-1: permuted rows of x [R*N_k, d];     GEMM-2: H_r [R*N_k, m]
  const T* w_gate;     // GEMM-1: packed W_gate [rows, d];           GEMM-2: packed W_down
  const T* w_up;       // GEMM-1: packed W_up
  T* c_shared;         // GEMM-1: H_s;  GEMM-2: Y_s [R, d]
  T* c_routed;         // GEMM-1: H_r;  GEMM-2: Y_r [R*N_k, d]
  int d;
  int shared_width, routed_width;
};

// grid = (row tiles, column tiles, groups)
template <typename T>
__global__ void __launch_bounds__(256) simt_gemm1_kernel(SimtGemmArgs<T> p) {
  const GroupStatic g = p.gs[blockIdx.z];
  const GroupRows r = p.gr[blockIdx.z];
  const int m0 = blockIdx.x * kSimtTile, n0 = blockIdx.y * kSimtTile;
  if (m0 >= r.count || n0 >= g.width) return;
  const int ldc = g.is_shared ? p.shared_width : p.routed_width;
  const T* A = (g.is_shared ? p.a_shared : p.a_routed) + (size_t)r.row0 * p.d;
  const T* Bg = p.w_gate + (size_t)g.w_row0 * p.d;
  const T* Bu = p.w_up + (size_t)g.w_row0 * p.d;
  T* C = (g.is_shared ? p.c_shared : p.c_routed) + (size_t)r.row0 * ldc;
  float acc_g[4][4], acc_u[4][4];
  simt_tile<T, true>(A, p.d, r.count, Bg, Bu, p.d, g.width, p.d, m0, n0, true, true, acc_g, acc_u);
  const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = m0 + ty * 4 + i;
    if (row >= r.count) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n < g.width) C[(size_t)row * ldc + n] = from_float<T>(silu_accurate(acc_g[i][j]) * acc_u[i][j]);
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(256) simt_gemm2_kernel(SimtGemmArgs<T> p) {
  const GroupStatic g = p.gs[blockIdx.z];
  const GroupRows r = p.gr[blockIdx.z];
  const int m0 = blockIdx.x * kSimtTile, n0 = blockIdx.y * kSimtTile;
  if (m0 >= r.count || n0 >= p.d || g.width == 0) return;
  const int lda = g.is_shared ? p.shared_width : p.routed_width;
  const T* A = (g.is_shared ? p.a_shared : p.a_routed) + (size_t)r.row0 * lda;
  const T* B = p.w_gate + g.wd_offset;                     // [d, width], ld = width
  T* C = (g.is_shared ? p.c_shared : p.c_routed) + (size_t)r.row0 * p.d;
  const bool vec = (g.width % 8 == 0) && (lda % 8 == 0) && (g.wd_offset % 8 == 0);
  float acc[4][4], unused[4][4];
  simt_tile<T, false>(A, lda, r.count, B, nullptr, g.width, p.d, g.width, m0, n0, vec, vec, acc, unused);
  const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = m0 + ty * 4 + i;
    if (row >= r.count) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = n0 + tx * 4 + j;
      if (c < p.d) C[(size_t)row * p.d + c] = from_float<T>(acc[i][j]);
    }
  }
}

}  // namespace cmoe
