// Tensor-core kernels for sm_100a: tcgen05.mma with the accumulator in tensor memory
// (TMEM), operands staged in shared memory by TMA, one persistent CTA per SM,
// warp-specialised (TMA producer warp / MMA issuer / 4 epilogue warps), TMEM accumulator
// double-buffered so the epilogue of one tile overlaps the MMAs of the next.
//
//   MODE 1, gate/up GEMM: H[r, n] = Swish(x_r . Wg[n]) * (x_r . Wu[n])      (Eq. ori_ffn_method)
//       A tile  : 128 rows of x x 64 k.  Shared groups read consecutive outer rows by TMA.
//                 Routed groups gather their rows straight from x, so no permuted copy of
//                 x is ever written: four extra warps (one thread per tile row) issue
//                 16-byte cp.async copies into the 128-byte-swizzled layout the MMA expects
//                 and arrive on the stage's barrier when their copies land.  (TMA
//                 tile::gather4 does the same with one copy per 4 rows; it is correct but a
//                 full tile needs 32 copies per stage, which the TMA unit issues ~3x slower
//                 than one tiled box, so it is kept only for batches of a few rows.)
//       B tile  : bn gate rows + bn up rows of the group's neurons x 64 k (one 3-D TMA box)
//       D (TMEM): 128 lanes x 2*bn fp32 columns; epilogue fuses SiLU(gate)*up -> bf16 H
//   MODE 2, down GEMM: Y[r, c] = sum_n H[r, n] Wd[c, n]
//       A tile  : 128 rows of H x 64 k ;  B tile: 256 output channels of the group's W_down
//       block x 64 k ;  D: 128 x 256 fp32 ; epilogue rounds to bf16 Y.
//   MODE 3, router: a_j = x_r . w_gate^{R_j}, v_j = x_r . w_up^{R_j}          (Eq. router)
//       B tile  : the (outer) layer's padded representative rows, gate block then up block;
//       epilogue: one thread per row does Swish(a)*v, the softmax over all N_r scores, the
//       biased top-N_k and the gates 1 + s'u                                 (Eq. final_gate).
// All operands are K-major with the 128-byte swizzle; rows or k beyond a tensor's extent
// are zero-filled by TMA, rows beyond a group's count are computed but never stored.
//
// Every mbarrier wait is bounded (about a second of SM clock); a wait that runs out sets
// the layer's device error word, raises a CTA-wide abort flag that the other waits poll,
// and the CTA falls through to the common teardown, which frees its TMEM.
#pragma once

#include <cuda.h>

#include <cstdio>

#include "common.cuh"

namespace cmoe {

constexpr int kUmmaBM = 128;          // rows per tile (UMMA M)
constexpr int kUmmaBK = 64;           // k per stage: 64 bf16 = one 128-byte swizzle row
constexpr int kUmmaStages = 4;
constexpr int kUmmaABytes = kUmmaBM * kUmmaBK * 2;       // 16 KB
constexpr int kUmmaBBytes = 256 * kUmmaBK * 2;           // 32 KB (up to 256 B rows)
constexpr int kUmmaStageBytes = kUmmaABytes + kUmmaBBytes;
constexpr int kUmmaMaxGroups = 1088;
constexpr int kUmmaThreads = 192;     // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue
constexpr int kUmmaGatherThreads = 128;   // mode 1 only: warps 6..9, one thread per A-tile row
constexpr int kUmmaTmemCols = 512;    // two accumulator buffers of 256 columns
constexpr int kUmmaSmemBytes = 1024 /*alignment slack*/ + kUmmaStages * kUmmaStageBytes +
                               256 /*barriers*/ + (kUmmaMaxGroups + 1) * 4;
constexpr long long kUmmaWaitCycles = 2000000000LL;   // ~1 s at SM clock

enum { kErrWaitFull = 1, kErrWaitEmpty = 2, kErrWaitAccFull = 3, kErrWaitAccEmpty = 4 };

// ----------------------------------------------------------------------------- PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false if the wait ran out (error word + abort flag set) or another wait
// of this CTA already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int32_t* err_word, int code, long long limit = kUmmaWaitCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > limit) {
      *abort_flag = 1;
      atomicCAS(err_word, 0, code);
      return false;
    }
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1,
                                            int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1,
                                            int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
// Four rows r0..r3 of a 2-D tensor (box: 64 columns x 1 row) to four consecutive 128-byte rows.
__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int r0,
                                            int r1, int r2, int r3) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(r0), "r"(r1), "r"(r2), "r"(r3) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t smem_slot, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_slot), "r"(cols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// D[tmem] (+)= A[smem desc] * B[smem desc]^T, bf16 inputs, fp32 accumulate.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc]^T, E4M3 inputs (32 k values per step), fp32 accumulate.
__device__ __forceinline__ void umma_e4m3(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// mbarrier arrives once all tcgen05 operations issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 16 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major tile, 128-byte rows, 128-byte swizzle, 8-row
// groups 1024 bytes apart; `addr` is the 1024-byte-aligned tile base plus the k offset.
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3FFF);
  d |= (uint64_t)1 << 16;                 // leading-dimension offset (unused with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;       // stride between 8-row groups
  d |= (uint64_t)1 << 46;                 // descriptor version of sm_100
  d |= (uint64_t)2 << 61;                 // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t umma_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kUmmaBM >> 4) << 24);
}

// One warp waits, with a limit of `limit` SM cycles, on an mbarrier that nobody arrives on, through the
// same mbar_wait the tensor-core kernels use: the wait gives up, the error word takes the code,
// the kernel returns normally.  No copy is in flight and no tensor memory is held.
__global__ void wait_timeout_probe_kernel(int32_t* err_word, long long limit) {
  __shared__ __align__(8) unsigned long long bar_mem;
  __shared__ int abort_flag;
  const uint32_t bar = smem_u32(&bar_mem);
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  if (threadIdx.x == 0) mbar_wait(bar, 0, &abort_flag, err_word, kErrWaitFull, limit);
  __syncwarp();
}

// Instruction descriptor of kind::f8f6f4: E4M3 x E4M3 (operand format code 0) -> fp32, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t umma_idesc_e4m3(int n) {
  return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kUmmaBM >> 4) << 24);
}

// ----------------------------------------------------------------------------- kernel
struct UmmaArgs {
  const GroupStatic* gs;
  const GroupRows* gr;
  int n_groups, n_outer, n_r;
  int d;                 // model width: K of modes 1 and 3, N of mode 2
  int bn_s, bn_r;        // mode 1: neurons per tile for shared / routed groups
  bf16* out_s;           // mode 1: H_s ; mode 2: Y_s
  bf16* out_r;           // mode 1: H_r ; mode 2: Y_r
  int ld_out_s, ld_out_r;
  const int32_t* row_token;   // mode 1: outer row held by each routed row (gather source)
  int band_mt;                // row tiles per band of the tile order (see umma_decode)
  int use_gather;             // mode 1, routed A rows: 0 permuted copy by TMA, 1 TMA gather4 from x, 2 cp.async from x
  const bf16* x_rows_ptr;     // mode 1: the outer rows of x (source of the cp.async gather)
  int32_t* err;
  // mode 3 (router)
  int ksplit;                 // K slices per tile (>= 1): a tile's k range is cut so that more SMs take part
  float* rt_part;             // ksplit > 1: [unit][2 n_rp columns][128 rows] fp32 partial sums
  int32_t* rt_ticket;         // ksplit > 1: [tile][4 epilogue warps], zero between launches
  const int32_t* outer_off;   // row ranges of the outer experts, or null (one range [0, n_rows))
  int n_rows, n_rp, n_k;      // n_rp: N_r rounded up to 8 (rows per block of the padded W^R)
  const float* u;
  const float* b;
  float* scores;
  float* keys;
  int32_t* topk_idx;
  float* topk_gate;
};

struct TileCoord { int g, mt, nt, row0, count; };

template <int MODE>
__device__ __forceinline__ GroupRows umma_rows(const UmmaArgs& p, int g) {
  if (MODE == 3) {
    GroupRows r;
    r.row0 = p.outer_off ? p.outer_off[g] : 0;
    r.count = p.outer_off ? p.outer_off[g + 1] - p.outer_off[g] : p.n_rows;
    return r;
  }
  return p.gr[g];
}

template <int MODE>
__device__ __forceinline__ int umma_n_tiles(const UmmaArgs& p, int g) {
  if (MODE == 3) return 1;
  const GroupStatic gs = p.gs[g];
  if (MODE == 1) {
    const int bn = gs.is_shared ? p.bn_s : p.bn_r;
    return (gs.width + bn - 1) / bn;
  }
  return gs.width > 0 ? (p.d + 255) / 256 : 0;
}

template <int MODE>
__device__ __forceinline__ TileCoord umma_decode(const UmmaArgs& p, const int32_t* tile_start, int n_groups,
                                                 int t) {
  int lo = 0, hi = n_groups;                 // last g with tile_start[g] <= t
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (tile_start[mid] <= t) lo = mid; else hi = mid;
  }
  const int local = t - tile_start[lo];
  const GroupRows r = umma_rows<MODE>(p, lo);
  // Order inside a group: bands of p.band_mt row tiles; inside a band the row tiles run fastest (CTAs
  // working side by side share a weight tile), then the n-tiles, then the next band.  A band's rows of A
  // (about 16 MB) stay in L2 while the n-tiles pass over them; without bands a large group's rows left L2
  // between two n-tiles and were read again for each (5.6 GB of DRAM reads instead of 0.45 GB in the gate/up
  // GEMM of the 16384-token workload), while letting the n-tiles run fastest everywhere was slower for the
  // groups that do fit (every CTA then streams a different weight tile).
  const int m_tiles = (r.count + kUmmaBM - 1) / kUmmaBM;
  const int n_tiles = umma_n_tiles<MODE>(p, lo);
  const int band_mt = MODE == 3 ? m_tiles : max(p.band_mt, 1);
  const int per_band = band_mt * n_tiles;
  const int band = local / per_band, in_band = local - band * per_band;
  const int cur_mt = min(band_mt, m_tiles - band * band_mt);
  TileCoord c;
  c.g = lo; c.nt = in_band / cur_mt; c.mt = band * band_mt + in_band % cur_mt; c.row0 = r.row0; c.count = r.count;
  return c;
}

// Router epilogue for one row (Eq. router, Eq. final_gate): a[j], v[j] are the gate / up
// pre-activations of routed expert j's representative neuron, j < n_r <= 32.
__device__ __forceinline__ void router_row_epilogue(const float (&a)[32], const float (&v)[32], int n_r, int n_k,
                                                    const float* __restrict__ u, const float* __restrict__ b,
                                                    int group_base, float* __restrict__ scores_row,
                                                    float* __restrict__ keys_row, int32_t* __restrict__ idx_row,
                                                    float* __restrict__ gates_row) {
  float s[32];
  float s_max = -INFINITY;
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    s[j] = j < n_r ? silu_accurate(a[j]) * v[j] : -INFINITY;
    s_max = fmaxf(s_max, s[j]);
  }
  float sum = 0.0f;
  float e[32];
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    e[j] = j < n_r ? expf(s[j] - s_max) : 0.0f;
    sum += e[j];
  }
  float key[32];
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    if (j < n_r) {
      e[j] = e[j] / sum;                              // s'_j
      const float k = e[j] + __ldg(b + j);
      scores_row[j] = s[j];
      keys_row[j] = k;
      key[j] = (k != k) ? -INFINITY : k;              // NaN ranks last
    } else {
      key[j] = -INFINITY;
    }
  }
  uint32_t taken = 0;
  for (int i = 0; i < n_k; ++i) {
    int who = -1;
    float best = 0.0f, best_sp = 0.0f;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      if (j < n_r && !((taken >> j) & 1u) && (who < 0 || key[j] > best)) {   // ties: lower index
        who = j; best = key[j]; best_sp = e[j];
      }
    }
    taken |= 1u << who;
    idx_row[i] = group_base + who;
    gates_row[i] = 1.0f + best_sp * __ldg(u + who);
  }
}

template <int MODE>
__global__ void __launch_bounds__(MODE == 1 ? kUmmaThreads + kUmmaGatherThreads : kUmmaThreads, 1)
umma_grouped_kernel(const __grid_constant__ CUtensorMap tm_a_s, const __grid_constant__ CUtensorMap tm_a_r,
                    const __grid_constant__ CUtensorMap tm_b_s, const __grid_constant__ CUtensorMap tm_b_r,
                    const UmmaArgs p) {
  grid_dep_wait();
  grid_dep_trigger();
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);                       // generic pointer to the aligned base
  constexpr int kStages = MODE == 3 ? 8 : kUmmaStages;             // the router's B tile is at most 8 KB
  constexpr int kStageBytes = MODE == 3 ? kUmmaABytes + 8192 : kUmmaStageBytes;
  const uint32_t bars = base + kStages * kStageBytes;   // barrier block
  uint8_t* bars_gen = gen + kStages * kStageBytes;
  // barrier block: full[8] empty[8] acc_full[2] acc_empty[2] (8 B each), tmem slot, abort flag
  const uint32_t full0 = bars, empty0 = bars + 64, accf0 = bars + 128, acce0 = bars + 144;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars_gen + 160);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars_gen + 164);
  int32_t* tile_start = reinterpret_cast<int32_t*>(bars_gen + 256);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_groups = MODE == 3 ? p.n_outer : p.n_groups;

  if (threadIdx.x == 0) {
    // mode 1: besides the producer's expect_tx arrival, every gather thread arrives once per stage
    const uint32_t full_count = MODE == 1 ? 1 + kUmmaGatherThreads : 1;
    for (int s = 0; s < kStages; ++s) { mbar_init(full0 + 8 * s, full_count); mbar_init(empty0 + 8 * s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(accf0 + 8 * b, 1); mbar_init(acce0 + 8 * b, 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), kUmmaTmemCols);
    tmem_relinquish();
  }
  // tiles of every group, then their exclusive prefix
  for (int g = threadIdx.x; g < n_groups; g += blockDim.x) {
    const int m_tiles = (umma_rows<MODE>(p, g).count + kUmmaBM - 1) / kUmmaBM;
    tile_start[g + 1] = m_tiles * umma_n_tiles<MODE>(p, g);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int run = 0;
    tile_start[0] = 0;
    for (int g = 0; g < n_groups; ++g) { run += tile_start[g + 1]; tile_start[g + 1] = run; }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int total_tiles = tile_start[n_groups];
  const int ksplit = MODE == 3 ? max(p.ksplit, 1) : 1;
  const int total_units = total_tiles * ksplit;
  const int k_blocks_fixed = (p.d + kUmmaBK - 1) / kUmmaBK;      // modes 1 and 3: K = d

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (whole warp)
    uint32_t it = 0;
    bool ok = true;
    for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
      const int t = u / ksplit, kz = u - t * ksplit;
      const TileCoord c = umma_decode<MODE>(p, tile_start, n_groups, t);
      GroupStatic g;
      if (MODE != 3) g = p.gs[c.g]; else { g.is_shared = 1; g.outer = c.g; g.width = 0; g.w_row0 = 0; }
      const int row = c.row0 + c.mt * kUmmaBM;
      const bool gather = MODE == 1 && !g.is_shared && p.use_gather == 1;
      const bool by_threads = MODE == 1 && !g.is_shared && p.use_gather == 2;   // the gather warps fill A
      const CUtensorMap* ta = g.is_shared ? &tm_a_s : &tm_a_r;
      const CUtensorMap* tb = g.is_shared ? &tm_b_s : &tm_b_r;
      int k_blocks, b_bytes, b_row = 0, j = 0;
      int a_bytes = kUmmaABytes, n_issue = 0;
      int gr0 = 0, gr1 = 0, gr2 = 0, gr3 = 0;
      if (MODE == 1) {
        const int bn = g.is_shared ? p.bn_s : p.bn_r;
        k_blocks = k_blocks_fixed;
        b_bytes = 2 * bn * kUmmaBK * 2;
        b_row = g.w_row0 + c.nt * bn;
        if (gather) {                          // this lane's four rows; rows past the group repeat its last row
          n_issue = (min(kUmmaBM, c.count - c.mt * kUmmaBM) + 3) >> 2;    // copies that carry valid rows
          a_bytes = n_issue * 512;
          const int last = c.row0 + c.count - 1;
          const int r = row + 4 * lane;
          gr0 = __ldg(p.row_token + min(r, last));
          gr1 = __ldg(p.row_token + min(r + 1, last));
          gr2 = __ldg(p.row_token + min(r + 2, last));
          gr3 = __ldg(p.row_token + min(r + 3, last));
        }
      } else if (MODE == 2) {
        k_blocks = (g.width + kUmmaBK - 1) / kUmmaBK;
        b_bytes = kUmmaBBytes;
        b_row = c.nt * 256;
        j = g.is_shared ? 0 : (c.g - p.n_outer) - g.outer * p.n_r;
      } else {
        k_blocks = k_blocks_fixed;
        b_bytes = 2 * p.n_rp * kUmmaBK * 2;
      }
      const int kb_lo = kz * k_blocks / ksplit, kb_hi = (kz + 1) * k_blocks / ksplit;      // this unit's k slice
      for (int kb = kb_lo; kb < kb_hi; ++kb, ++it) {
        const uint32_t s = it % kStages, n = it / kStages;
        if (!mbar_wait(empty0 + 8 * s, (n & 1) ^ 1, abort_flag, p.err, kErrWaitEmpty)) { ok = false; break; }
        const uint32_t fb = full0 + 8 * s;
        const uint32_t sa = base + s * kStageBytes, sb = sa + kUmmaABytes;
        if (lane == 0) mbar_expect_tx(fb, (by_threads ? 0 : a_bytes) + b_bytes);
        __syncwarp();
        if (gather) {
          if (lane < n_issue) tma_gather4(sa + lane * 512, ta, fb, kb * kUmmaBK, gr0, gr1, gr2, gr3);
        } else if (lane == 0 && !by_threads) {
          tma_load_2d(sa, ta, fb, kb * kUmmaBK, row);
        }
        if (lane == 0) {
          if (MODE == 1) tma_load_3d(sb, tb, fb, kb * kUmmaBK, b_row, 0);
          else if (MODE == 3) tma_load_3d(sb, tb, fb, kb * kUmmaBK, 0, c.g);
          else if (g.is_shared) tma_load_3d(sb, tb, fb, kb * kUmmaBK, b_row, g.outer);
          else tma_load_4d(sb, tb, fb, kb * kUmmaBK, b_row, j, g.outer);
        }
      }
    }
    if (!ok) for (int i = 0; i < 200; ++i) __nanosleep(1000);   // let copies in flight land
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t it = 0, tile_n = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x, ++tile_n) {
        const int t = u / ksplit, kz = u - t * ksplit;
        const TileCoord c = umma_decode<MODE>(p, tile_start, n_groups, t);
        int k_blocks, n_mma;
        if (MODE == 1) {
          const GroupStatic g = p.gs[c.g];
          k_blocks = k_blocks_fixed; n_mma = 2 * (g.is_shared ? p.bn_s : p.bn_r);
        } else if (MODE == 2) {
          k_blocks = (p.gs[c.g].width + kUmmaBK - 1) / kUmmaBK; n_mma = 256;
        } else {
          k_blocks = k_blocks_fixed; n_mma = 2 * p.n_rp;
        }
        const uint32_t idesc = umma_idesc(n_mma);
        const uint32_t buf = tile_n & 1, use = tile_n >> 1;
        if (!mbar_wait(acce0 + 8 * buf, (use & 1) ^ 1, abort_flag, p.err, kErrWaitAccEmpty)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * 256;
        const int kb_lo = kz * k_blocks / ksplit, kb_hi = (kz + 1) * k_blocks / ksplit;
        for (int kb = kb_lo; kb < kb_hi; ++kb, ++it) {
          const uint32_t s = it % kStages, n = it / kStages;
          if (!mbar_wait(full0 + 8 * s, n & 1, abort_flag, p.err, kErrWaitFull)) { ok = false; break; }
          if (MODE == 1) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // cp.async-written rows
          tc_fence_after();
          const uint32_t sa = base + s * kStageBytes, sb = sa + kUmmaABytes;
#pragma unroll
          for (int k = 0; k < kUmmaBK / 16; ++k)
            umma_bf16(d_tmem, umma_smem_desc(sa + k * 32), umma_smem_desc(sb + k * 32), idesc,
                      (kb != kb_lo || k != 0) ? 1u : 0u);
          umma_commit(empty0 + 8 * s);         // stage reusable once these MMAs have read it
        }
        if (ok) umma_commit(accf0 + 8 * buf);  // accumulator complete
      }
    }
  } else if (MODE == 1 && warp >= 6) {
    // ------------------------------------------------------------ A-row gather (mode 1, warps 6..9)
    // For routed groups (use_gather == 2) the 128 threads copy the tile's 128 rows x 128 bytes of
    // this k block from x: eight consecutive threads cover one row (coalesced 128-byte reads), 16
    // rows per pass, 8 passes; 16-byte chunk c of row r goes to the swizzled chunk c ^ (r & 7).
    // Otherwise the threads only arrive.
    const int gt = threadIdx.x - kUmmaThreads;
    const int ch = gt & 7, r_sub = gt >> 3;
    uint32_t it = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
      const TileCoord c = umma_decode<MODE>(p, tile_start, n_groups, t);
      const GroupStatic g = p.gs[c.g];
      const bool mine = !g.is_shared && p.use_gather == 2;
      const bf16* src_row[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        src_row[i] = nullptr;
        if (mine) {                                   // rows past the group repeat its last row
          const int r = c.row0 + min(c.mt * kUmmaBM + i * 16 + r_sub, c.count - 1);
          src_row[i] = p.x_rows_ptr + (size_t)__ldg(p.row_token + r) * p.d;
        }
      }
      for (int kb = 0; kb < k_blocks_fixed; ++kb, ++it) {
        const uint32_t s = it % kStages, n = it / kStages;
        if (!mbar_wait(empty0 + 8 * s, (n & 1) ^ 1, abort_flag, p.err, kErrWaitEmpty)) { ok = false; break; }
        const uint32_t fb = full0 + 8 * s;
        if (mine) {
          const int k = kb * kUmmaBK + ch * 8;
          const uint32_t bytes = k < p.d ? 16u : 0u;                        // zero-fill past the end of the row
          const int k_src = k < p.d ? k : 0;
          const uint32_t sa = base + s * kStageBytes;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int r = i * 16 + r_sub;
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;"
                         ::"r"(sa + r * 128 + ((ch ^ (r & 7)) << 4)), "l"(src_row[i] + k_src), "r"(bytes)
                         : "memory");
          }
          asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(fb) : "memory");
        } else {
          mbar_arrive(fb);
        }
      }
    }
    if (!ok) asm volatile("cp.async.wait_all;" ::: "memory");
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int quad = warp & 3;                 // TMEM lane quadrant this warp may read
    uint32_t tile_n = 0;
    bool ok = true;
    for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x, ++tile_n) {
      const int t = u / ksplit, kz = u - t * ksplit;
      const TileCoord c = umma_decode<MODE>(p, tile_start, n_groups, t);
      const uint32_t buf = tile_n & 1, use = tile_n >> 1;
      if (!mbar_wait(accf0 + 8 * buf, use & 1, abort_flag, p.err, kErrWaitAccFull)) { ok = false; break; }
      tc_fence_after();
      const int row_in_group = c.mt * kUmmaBM + quad * 32 + lane;
      const bool row_ok = row_in_group < c.count;
      const uint32_t taddr = tmem_base + buf * 256 + ((uint32_t)(quad * 32) << 16);
      if (MODE == 1) {
        const GroupStatic g = p.gs[c.g];
        const int bn = g.is_shared ? p.bn_s : p.bn_r;
        const int ld = g.is_shared ? p.ld_out_s : p.ld_out_r;
        const int n0 = c.nt * bn;
        const int n_valid = min(bn, g.width - n0);
        bf16* dst = (g.is_shared ? p.out_s : p.out_r) + (size_t)(c.row0 + row_in_group) * ld + n0;
        const bool wide = ((ld | n0) & 15) == 0;          // 32-byte aligned row segments
        for (int c0 = 0; c0 < n_valid; c0 += 16) {
          float gt[16], up[16];
          tmem_ld16(taddr + c0, gt);
          tmem_ld16(taddr + bn + c0, up);
          tmem_ld_wait();
          if (row_ok) {
            float h16[16];
#pragma unroll
            for (int q = 0; q < 16; ++q) h16[q] = gt[q] / (1.0f + __expf(-gt[q])) * up[q];
            if (wide && c0 + 16 <= n_valid) {
              store16(dst + c0, h16);
            } else {
#pragma unroll
              for (int h = 0; h < 2; ++h) {
                if (c0 + h * 8 < n_valid) {
                  float v[8];
#pragma unroll
                  for (int q = 0; q < 8; ++q) v[q] = h16[h * 8 + q];
                  store8(dst + c0 + h * 8, v);
                }
              }
            }
          }
        }
      } else if (MODE == 2) {
        const GroupStatic g = p.gs[c.g];
        const int n0 = c.nt * 256;
        const int n_valid = min(256, p.d - n0);
        bf16* dst = (g.is_shared ? p.out_s : p.out_r) + (size_t)(c.row0 + row_in_group) * p.d + n0;
        const bool wide = (p.d & 15) == 0;
        for (int c0 = 0; c0 < n_valid; c0 += 16) {
          float acc[16];
          tmem_ld16(taddr + c0, acc);
          tmem_ld_wait();
          if (row_ok && wide && c0 + 16 <= n_valid) {
            store16(dst + c0, acc);
          } else if (row_ok) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              if (c0 + h * 8 < n_valid) {
                float v[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) v[q] = acc[h * 8 + q];
                store8(dst + c0 + h * 8, v);
              }
            }
          }
        }
      } else {
        float a[32], v[32];
        tmem_ld16(taddr, a);
        tmem_ld16(taddr + p.n_rp, v);
        if (p.n_rp > 16) {                     // warp-uniform
          tmem_ld16(taddr + 16, a + 16);
          tmem_ld16(taddr + p.n_rp + 16, v + 16);
        }
        tmem_ld_wait();
        bool finish_row = true;
        if (ksplit > 1) {
          // K slice of a split tile: park this row's partial sums ([column][row]: a warp's store is one
          // 128-byte line), take the warp's ticket for the tile; the warp that takes the last one adds
          // the slices in ascending order (a fixed order: deterministic) and goes on to the gate logic
          const int row128 = quad * 32 + lane;
          float* mine = p.rt_part + ((size_t)t * ksplit + kz) * (64 * 128) + row128;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            if (j < p.n_rp) { __stcg(mine + (size_t)j * 128, a[j]); __stcg(mine + (size_t)(32 + j) * 128, v[j]); }
          }
          __threadfence();
          __syncwarp();
          int32_t* tk = p.rt_ticket + (size_t)t * 4 + quad;
          int last = 0;
          if (lane == 0) last = atomicAdd(tk, 1) == ksplit - 1;
          last = __shfl_sync(0xffffffffu, last, 0);
          finish_row = last != 0;
          if (finish_row) {
            __threadfence();
            const float* all = p.rt_part + (size_t)t * ksplit * (64 * 128) + row128;
#pragma unroll
            for (int j = 0; j < 32; ++j) { a[j] = 0.0f; v[j] = 0.0f; }
            for (int z = 0; z < ksplit; ++z) {
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                if (j < p.n_rp) {
                  a[j] += __ldcg(all + (size_t)z * (64 * 128) + (size_t)j * 128);
                  v[j] += __ldcg(all + (size_t)z * (64 * 128) + (size_t)(32 + j) * 128);
                }
              }
            }
            if (lane == 0) *tk = 0;            // ready for the next launch
          }
        }
        if (row_ok && finish_row) {
          const size_t row = (size_t)(c.row0 + row_in_group);
          router_row_epilogue(a, v, p.n_r, p.n_k, p.u + c.g * p.n_r, p.b + c.g * p.n_r, c.g * p.n_r,
                              p.scores + row * p.n_r, p.keys + row * p.n_r, p.topk_idx + row * p.n_k,
                              p.topk_gate + row * p.n_k);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acce0 + 8 * buf);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kUmmaTmemCols);
  }
}

// ----------------------------------------------------------------------------- host
struct UmmaShape {
  int d = 0, m = 0, shared_width = 0, d_ff = 0, n_outer = 1, n_r = 0, n_rp = 0, n_k = 0;
  size_t max_outer_rows = 0, max_routed_rows = 0;
};

struct UmmaBuffers {
  const void* w_gate_up = nullptr;   // [2][n_outer*d_ff][d]
  const void* w_down = nullptr;      // packed W_down
  const void* w_rep = nullptr;       // [n_outer][2*n_rp][d] padded representative rows
  const void* x_fixed = nullptr;     // hierarchical: the layer's own outer-row copy of x
  const void* x_perm = nullptr;      // routed rows of x in expert-contiguous order
  void *h_s = nullptr, *h_r = nullptr, *y_s = nullptr, *y_r = nullptr;
  const GroupStatic* gs_dev = nullptr;
  const float *u = nullptr, *b = nullptr;
  float *scores = nullptr, *keys = nullptr, *topk_gate = nullptr;
  int32_t* topk_idx = nullptr;
  const int32_t* row_token = nullptr;
};

typedef CUresult (*PFN_encodeTiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                    CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                    CUtensorMapFloatOOBfill);

struct UmmaPlan {
  bool built = false;
  char error[256] = "";
  UmmaShape shape;
  UmmaBuffers buf;
  int bn_s = 128, bn_r = 128, n_sms = 0, n_groups = 0;
  float* rt_part = nullptr;                // router K-slice partials: n_sms units x 64 columns x 128 rows (caller's workspace)
  int32_t* rt_ticket = nullptr;            // [n_sms][4], zeroed once
  bool has_s = false, has_r = false;
  PFN_encodeTiled encode = nullptr;
  CUtensorMap x_rows, x_gather;            // x: 64 x 128 boxes for consecutive rows, 64 x 1 for gather4
  CUtensorMap x_perm;                      // permuted copy of x
  CUtensorMap b1_s, b1_r;                  // stacked gate+up rows, box heights bn_s / bn_r
  CUtensorMap a2_s, a2_r, b2_s, b2_r;      // H_s / H_r / shared W_down / routed W_down blocks
  CUtensorMap w_rep;                       // padded representative rows
};

// Neurons per gate/up tile: 128 (N = 256 MMAs, the fewest passes over the A rows) when that pads the width
// by at most 5 %, else the multiple of 8 in [96, 128] that wastes the least of the last tile.  (Measured on
// widths 864 / 1728 at 16384 tokens: 128 against 96, which pads nothing, is 12 % faster in the gate/up GEMM:
// seven instead of nine passes over the gathered rows outweigh 3.7 % of padded MMA work.)
inline int umma_pick_bn(int width) {
  if (width <= 0) return 128;
  if ((long long)((width + 127) / 128 * 128) * 100 <= (long long)width * 105) return 128;
  int best = 128, best_pad = (width + 127) / 128 * 128;
  for (int bn = 120; bn >= 96; bn -= 8) {
    const int pad = (width + bn - 1) / bn * bn;
    if (pad < best_pad) { best = bn; best_pad = pad; }
  }
  return best;
}

inline bool umma_encode(UmmaPlan* P, CUtensorMap* tm, const void* base, int rank, const cuuint64_t* dims,
                        const cuuint64_t* strides_bytes, const cuuint32_t* box, const char* what) {
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  for (int i = 0; i < rank; ++i)
    if (dims[i] == 0) { snprintf(P->error, sizeof(P->error), "tensor map %s: zero extent", what); return false; }
  const CUresult r = P->encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base),
                               dims, strides_bytes, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(P->error, sizeof(P->error), "cuTensorMapEncodeTiled(%s) failed with CUresult %d", what, (int)r);
    return false;
  }
  return true;
}

// [rows, cols] row-major bf16 matrix, box 64 columns x box_rows.
inline bool umma_encode_rows(UmmaPlan* P, CUtensorMap* tm, const void* base, size_t rows, size_t cols,
                             int box_rows, const char* what) {
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t str[1] = {cols * 2};
  const cuuint32_t box[2] = {kUmmaBK, (cuuint32_t)box_rows};
  return umma_encode(P, tm, base, 2, dims, str, box, what);
}

// Tensor maps of x for this forward: the caller's buffer for a plain layer (a host-side
// struct fill, no allocation), fixed at plan creation for a hierarchical layer.
inline bool umma_bind_x(UmmaPlan* P, const void* x_rows, int n_rows) {
  if (P->buf.x_fixed) return true;
  return umma_encode_rows(P, &P->x_rows, x_rows, (size_t)n_rows, (size_t)P->shape.d, kUmmaBM, "x") &&
         umma_encode_rows(P, &P->x_gather, x_rows, (size_t)n_rows, (size_t)P->shape.d, 1, "x (gather)");
}

// 0: plan built; 1: shape not taken by this path; -5: a driver call failed (P->error).
inline int umma_plan_create(UmmaPlan* P, const UmmaShape& s, const UmmaBuffers& buf, int n_groups) {
  P->built = false;
  P->has_s = s.shared_width > 0 && s.max_outer_rows > 0;
  P->has_r = s.n_r > 0 && s.n_k > 0 && s.max_routed_rows > 0;
  const bool has_s = P->has_s, has_r = P->has_r;
  if (!has_s && !has_r) return 1;
  if (s.d % 8 || s.m % 8 || s.shared_width % 8 || n_groups > kUmmaMaxGroups) return 1;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn ||
      q != cudaDriverEntryPointSuccess) {
    snprintf(P->error, sizeof(P->error), "cuTensorMapEncodeTiled entry point not found");
    return -5;
  }
  P->encode = reinterpret_cast<PFN_encodeTiled>(fn);
  P->shape = s;
  P->buf = buf;
  P->n_groups = n_groups;
  P->bn_s = umma_pick_bn(s.shared_width);
  P->bn_r = umma_pick_bn(s.m);
  int dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&P->n_sms, cudaDevAttrMultiProcessorCount, dev);

  const size_t d = s.d, rows_w = (size_t)s.n_outer * s.d_ff;
  bool ok = true;
  // gate/up weights stacked, [2][rows_w][d]; box = 64 k x bn rows x 2 planes
  for (int shared = 0; shared < 2 && ok; ++shared) {
    const int bn = shared ? P->bn_s : P->bn_r;
    const cuuint64_t dims[3] = {d, rows_w, 2};
    const cuuint64_t str[2] = {d * 2, rows_w * d * 2};
    const cuuint32_t box[3] = {kUmmaBK, (cuuint32_t)bn, 2};
    ok = umma_encode(P, shared ? &P->b1_s : &P->b1_r, buf.w_gate_up, 3, dims, str, box, "gate/up weights");
  }
  if (ok && has_r) ok = umma_encode_rows(P, &P->a2_r, buf.h_r, s.max_routed_rows, s.m, kUmmaBM, "H routed");
  if (ok && has_r) ok = umma_encode_rows(P, &P->x_perm, buf.x_perm, s.max_routed_rows, d, kUmmaBM, "permuted x");
  if (ok && has_s) ok = umma_encode_rows(P, &P->a2_s, buf.h_s, s.max_outer_rows, s.shared_width, kUmmaBM, "H shared");
  // W_down: shared block [d, W_s] of every outer expert; routed blocks [d, m] x N_r of every outer expert
  if (ok && has_s) {
    const cuuint64_t dims[3] = {(cuuint64_t)s.shared_width, d, (cuuint64_t)s.n_outer};
    const cuuint64_t str[2] = {(cuuint64_t)s.shared_width * 2, d * s.d_ff * 2};
    const cuuint32_t box[3] = {kUmmaBK, 256, 1};
    ok = umma_encode(P, &P->b2_s, buf.w_down, 3, dims, str, box, "shared W_down");
  }
  if (ok && has_r) {
    const cuuint64_t dims[4] = {(cuuint64_t)s.m, d, (cuuint64_t)s.n_r, (cuuint64_t)s.n_outer};
    const cuuint64_t str[3] = {(cuuint64_t)s.m * 2, d * s.m * 2, d * s.d_ff * 2};
    const cuuint32_t box[4] = {kUmmaBK, 256, 1, 1};
    ok = umma_encode(P, &P->b2_r, (const bf16*)buf.w_down + (size_t)s.shared_width * d, 4, dims, str, box,
                     "routed W_down");
  }
  if (ok && s.n_r > 0) {
    const cuuint64_t dims[3] = {d, (cuuint64_t)2 * s.n_rp, (cuuint64_t)s.n_outer};
    const cuuint64_t str[2] = {d * 2, (cuuint64_t)2 * s.n_rp * d * 2};
    const cuuint32_t box[3] = {kUmmaBK, (cuuint32_t)(2 * s.n_rp), 1};
    ok = umma_encode(P, &P->w_rep, buf.w_rep, 3, dims, str, box, "representative rows");
  }
  if (ok && buf.x_fixed)
    ok = umma_encode_rows(P, &P->x_rows, buf.x_fixed, s.max_outer_rows, d, kUmmaBM, "outer rows of x") &&
         umma_encode_rows(P, &P->x_gather, buf.x_fixed, s.max_outer_rows, d, 1, "outer rows of x (gather)");
  if (!ok) return -5;
  // placeholders for absent operand classes (never dereferenced: such groups have no tiles)
  if (!has_r) { P->a2_r = P->a2_s; P->b2_r = P->b2_s; }
  if (!has_s) { P->a2_s = P->a2_r; P->b2_s = P->b2_r; }
  if (s.n_r == 0) P->w_rep = P->b1_s;
  cudaError_t e = cudaSuccess;
  if (e == cudaSuccess) e = cudaFuncSetAttribute(umma_grouped_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kUmmaSmemBytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(umma_grouped_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kUmmaSmemBytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(umma_grouped_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, kUmmaSmemBytes);
  if (e != cudaSuccess) {
    snprintf(P->error, sizeof(P->error), "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    return -5;
  }
  P->built = true;
  return 0;
}

inline void umma_plan_destroy(UmmaPlan* P) { P->built = false; }

// Row tiles per band of the tile order: about 16 MB of A rows (k_extent bf16 elements per row), an even count.
inline int umma_band_tiles(int k_extent) {
  const long long tile_bytes = (long long)kUmmaBM * k_extent * 2;
  long long n = (16ll << 20) / (tile_bytes > 0 ? tile_bytes : 1);
  n = n < 2 ? 2 : n;
  return (int)(n & ~1ll);
}

inline UmmaArgs umma_base_args(const UmmaPlan* P, const GroupRows* gr, int32_t* err_word) {
  const UmmaShape& s = P->shape;
  UmmaArgs a{};
  a.gs = P->buf.gs_dev; a.gr = gr; a.n_groups = P->n_groups; a.n_outer = s.n_outer; a.n_r = s.n_r;
  a.d = s.d; a.bn_s = P->bn_s; a.bn_r = P->bn_r; a.err = err_word;
  a.row_token = P->buf.row_token;
  a.x_rows_ptr = nullptr;
  a.n_rp = s.n_rp; a.n_k = s.n_k; a.u = P->buf.u; a.b = P->buf.b;
  a.scores = P->buf.scores; a.keys = P->buf.keys; a.topk_idx = P->buf.topk_idx; a.topk_gate = P->buf.topk_gate;
  return a;
}

// Router on the tensor path (mode 3).  Requires umma_bind_x for this forward.  Returns launches or -1.
inline int umma_router_forward(UmmaPlan* P, int n_rows, const int32_t* outer_off, int32_t* err_word,
                               cudaStream_t st) {
  UmmaArgs a = umma_base_args(P, nullptr, err_word);
  a.outer_off = outer_off; a.n_rows = n_rows;
  const int tiles = (n_rows + kUmmaBM - 1) / kUmmaBM + P->shape.n_outer;     // upper bound of the tile count
  // with few tiles, cut each tile's K range so that up to four times as many SMs stream x
  int ksplit = 1;
  if (P->rt_part && P->rt_ticket) {
    const int kb = (P->shape.d + kUmmaBK - 1) / kUmmaBK;
    ksplit = P->n_sms / tiles;
    if (ksplit > 4) ksplit = 4;
    if (ksplit > kb / 8) ksplit = kb / 8;
    if (ksplit < 1) ksplit = 1;
  }
  a.ksplit = ksplit; a.rt_part = P->rt_part; a.rt_ticket = P->rt_ticket;
  const int units = tiles * ksplit;
  const int grid = units < P->n_sms ? units : P->n_sms;
  umma_grouped_kernel<3><<<grid, kUmmaThreads, kUmmaSmemBytes, st>>>(P->x_rows, P->x_rows, P->w_rep, P->w_rep, a);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    snprintf(P->error, sizeof(P->error), "tensor-core router launch: %s", cudaGetErrorString(e));
    return -1;
  }
  return 1;
}

// Enqueues the gate/up and the down GEMM over all groups.  gather_mode: how routed groups get
// their rows of x (0 permuted copy, 1 TMA gather4, 2 cp.async gather).  Requires umma_bind_x for this
// forward.  which: bit 0 the gate/up GEMM, bit 1 the down GEMM.  Returns the number of kernels
// launched, or -1 (P->error).
inline int umma_forward(UmmaPlan* P, const GroupRows* gr, int gather_mode, const void* x_rows, int32_t* err_word,
                        cudaStream_t st, cudaEvent_t mid, bool dep = false, int which = 3) {
  const UmmaShape& s = P->shape;
  UmmaArgs a = umma_base_args(P, gr, err_word);
  a.out_s = (bf16*)P->buf.h_s; a.out_r = (bf16*)P->buf.h_r; a.ld_out_s = s.shared_width; a.ld_out_r = s.m;
  a.use_gather = gather_mode;
  a.x_rows_ptr = (const bf16*)x_rows;
  a.band_mt = umma_band_tiles(s.d);
  if (which & 1)
    launch_kernel(dep, umma_grouped_kernel<1>, dim3(P->n_sms), dim3(kUmmaThreads + kUmmaGatherThreads), kUmmaSmemBytes,
                  st, P->x_rows, (gather_mode != 0 || !P->has_r) ? P->x_gather : P->x_perm, P->b1_s, P->b1_r, a);
  if (mid && (which & 1)) cudaEventRecord(mid, st);
  a.out_s = (bf16*)P->buf.y_s; a.out_r = (bf16*)P->buf.y_r; a.ld_out_s = s.d; a.ld_out_r = s.d;
  a.band_mt = umma_band_tiles(s.shared_width > s.m ? s.shared_width : s.m);
  if (which & 2)
    launch_kernel(dep, umma_grouped_kernel<2>, dim3(P->n_sms), dim3(kUmmaThreads), kUmmaSmemBytes, st, P->a2_s,
                  P->a2_r, P->b2_s, P->b2_r, a);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    snprintf(P->error, sizeof(P->error), "tensor-core GEMM launch: %s", cudaGetErrorString(e));
    return -1;
  }
  return (which & 1) + ((which >> 1) & 1);
}

}  // namespace cmoe
