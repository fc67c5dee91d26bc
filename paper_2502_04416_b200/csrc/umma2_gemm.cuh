// Expert GEMMs on CTA pairs (tcgen05 cta_group::2): two CTAs of a 2-CTA cluster, on
// neighbouring SMs, compute one 256 x N tile.  Each CTA stages its own 128 rows of A and
// only HALF of the B tile (the MMA reads the other half from the peer's shared memory),
// so a stage is 16 KB + 16 KB instead of 16 KB + 32 KB: six stages fit instead of four,
// and the L2 -> SM traffic for the weights halves.  The leader CTA (cluster rank 0) issues
// every MMA for the pair; accumulators sit in both CTAs' TMEM (128 lanes each).
//
//   MODE 1, gate/up: the leader stages the bn gate rows, the peer the bn up rows, so the
//           accumulator columns are [gate | up] exactly as in the single-CTA kernel.
//   MODE 2, down:    each CTA stages 128 of the tile's 256 output channels.
// The two 128-row halves are two m-tiles of the same group and n-tile; a group with an odd
// number of m-tiles leaves one half computing rows that are never stored.
// Routed groups of the gate/up GEMM gather their A rows straight from x (no permuted copy):
// four extra warps per CTA copy the CTA's 128 rows of each k block with 16-byte cp.async into the
// swizzled layout and arrive, copy-completion-bound, on a barrier of their own CTA; a relay
// thread per CTA forwards each completed block to the leader's full barrier.  (Waiting for the
// copies in the gather threads themselves, cp.async.wait_group + proxy fence per block, drained
// the copies in flight at every block and ran three times slower.)
//
// Synchronisation (all waits bounded):
//   full[s]      leader's barrier; the leader's producer arrives with the byte count of BOTH
//                CTAs' TMA copies, which complete on it; in the gate/up kernel each CTA's relay
//                thread arrives on it as well (2 more arrivals).
//   afull[s]     gate/up only, one per CTA: its 128 gather threads, then its relay waits on it.
//   empty[s]     one per CTA; the leader's tcgen05.commit is multicast to both.
//   acc_full[b]  one per CTA, multicast commit;  acc_empty[b]: leader's, 8 arrivals (the
//                four epilogue warps of each CTA, the peer's arriving remotely).
#pragma once

#include "umma_decode.cuh"
#include "umma_gemm.cuh"

namespace cmoe {

constexpr int kU2Stages = 6;
constexpr int kU2ABytes = kUmmaBM * kUmmaBK * 2;        // 16 KB: this CTA's 128 rows
constexpr int kU2BBytes = 128 * kUmmaBK * 2;            // 16 KB: this CTA's half of B
constexpr int kU2StageBytes = kU2ABytes + kU2BBytes;
constexpr int kU2SmemBytes = 1024 + kU2Stages * kU2StageBytes + 256 + (kUmmaMaxGroups + 1) * 4;
constexpr int kU2Threads1 = kUmmaThreads + kUmmaGatherThreads + 32;   // gate/up: + 4 gather warps + 1 relay warp

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of `local` (a shared::cta address) in the shared memory of cluster CTA `rank`.
__device__ __forceinline__ uint32_t mapa_shared(uint32_t local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrive on a barrier of a cluster CTA with the default (CTA-scope release) semantics: the data
// the arrival stands for was written by cp.async and fenced towards the async proxy, and is read
// only by tcgen05.mma.  (Cluster-scope acquire / release on this per-k-block path cost more than
// the MMAs of the block.)
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA loads of a CTA pair: data lands in this CTA, completion bytes go to `bar`, a
// shared::cluster address that may lie in the peer (leader) CTA.
__device__ __forceinline__ void tma2_load_2d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma2_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1,
                                             int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma2_load_4d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1,
                                             int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tmem_alloc2(uint32_t smem_slot, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_slot), "r"(cols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish2() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D (both CTAs' TMEM, 256 x N) (+)= A (each CTA's 128 rows) * B (N/2 rows from each CTA)^T.
__device__ __forceinline__ void umma2_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                           uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrive on the barrier at this shared-memory offset in BOTH CTAs of the pair once all
// tcgen05 operations issued so far by this thread have completed.
__device__ __forceinline__ void umma2_commit_both(uint32_t bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ uint32_t umma2_idesc(int n) {     // M = 256 across the pair
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}

struct Pair2Coord { int g, mp, nt, row0, count; };

template <int MODE>
__device__ __forceinline__ int umma2_pairs(const UmmaArgs& p, int g) {
  const int m_tiles = (p.gr[g].count + kUmmaBM - 1) / kUmmaBM;
  return ((m_tiles + 1) >> 1) * umma_n_tiles<MODE>(p, g);
}

template <int MODE>
__device__ __forceinline__ Pair2Coord umma2_decode(const UmmaArgs& p, const int32_t* tile_start, int t) {
  int lo = 0, hi = p.n_groups;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (tile_start[mid] <= t) lo = mid; else hi = mid;
  }
  const int local = t - tile_start[lo];
  const GroupRows r = p.gr[lo];
  // bands of row-tile pairs, row tiles fastest inside a band, then n-tiles (see umma_decode)
  const int m_pairs = ((r.count + kUmmaBM - 1) / kUmmaBM + 1) >> 1;
  const int n_tiles = umma_n_tiles<MODE>(p, lo);
  const int band_mp = max(p.band_mt >> 1, 1);
  const int per_band = band_mp * n_tiles;
  const int band = local / per_band, in_band = local - band * per_band;
  const int cur_mp = min(band_mp, m_pairs - band * band_mp);
  Pair2Coord c;
  c.g = lo; c.nt = in_band / cur_mp; c.mp = band * band_mp + in_band % cur_mp; c.row0 = r.row0; c.count = r.count;
  return c;
}

template <int MODE>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(MODE == 1 ? kU2Threads1 : kUmmaThreads, 1)
umma2_grouped_kernel(const __grid_constant__ CUtensorMap tm_a_s, const __grid_constant__ CUtensorMap tm_a_r,
                     const __grid_constant__ CUtensorMap tm_b_s, const __grid_constant__ CUtensorMap tm_b_r,
                     const UmmaArgs p) {
  grid_dep_wait();
  grid_dep_trigger();
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const uint32_t bars = base + kU2Stages * kU2StageBytes;
  uint8_t* bars_gen = gen + kU2Stages * kU2StageBytes;
  // barrier block: full[8] empty[8] acc_full[2] acc_empty[2], tmem slot, abort flag
  const uint32_t full0 = bars, empty0 = bars + 64, accf0 = bars + 128, acce0 = bars + 144, afull0 = bars + 192;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars_gen + 160);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars_gen + 164);
  int32_t* tile_start = reinterpret_cast<int32_t*>(bars_gen + 256);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    const uint32_t full_count = MODE == 1 ? 3 : 1;      // gate/up: plus one relay arrival per CTA
    for (int s = 0; s < kU2Stages; ++s) {
      mbar_init(full0 + 8 * s, full_count); mbar_init(empty0 + 8 * s, 1); mbar_init(afull0 + 8 * s, kUmmaGatherThreads);
    }
    for (int b = 0; b < 2; ++b) { mbar_init(accf0 + 8 * b, 1); mbar_init(acce0 + 8 * b, 8); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  for (int g = threadIdx.x; g < p.n_groups; g += blockDim.x) tile_start[g + 1] = umma2_pairs<MODE>(p, g);
  __syncthreads();
  if (threadIdx.x == 0) {
    int run = 0;
    tile_start[0] = 0;
    for (int g = 0; g < p.n_groups; ++g) { run += tile_start[g + 1]; tile_start[g + 1] = run; }
  }
  cluster_sync_all();                         // both CTAs' barriers exist before any remote use
  if (warp == 1) {
    tmem_alloc2(smem_u32(tmem_slot), kUmmaTmemCols);
    tmem_relinquish2();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int total_tiles = tile_start[p.n_groups];
  const int k_blocks_fixed = (p.d + kUmmaBK - 1) / kUmmaBK;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (one lane per CTA)
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int t = pair_id; t < total_tiles && ok; t += n_pairs) {
        const Pair2Coord c = umma2_decode<MODE>(p, tile_start, t);
        const GroupStatic g = p.gs[c.g];
        const int row = c.row0 + (2 * c.mp + (int)rank) * kUmmaBM;     // this CTA's m-tile
        const CUtensorMap* ta = g.is_shared ? &tm_a_s : &tm_a_r;
        const CUtensorMap* tb = g.is_shared ? &tm_b_s : &tm_b_r;
        const bool by_threads = MODE == 1 && !g.is_shared && p.use_gather == 2;   // the gather warps fill A
        int k_blocks, b_half, b_row, j = 0;
        if (MODE == 1) {
          const int bn = g.is_shared ? p.bn_s : p.bn_r;
          k_blocks = k_blocks_fixed;
          b_half = bn * kUmmaBK * 2;
          b_row = g.w_row0 + c.nt * bn;
        } else {
          k_blocks = (g.width + kUmmaBK - 1) / kUmmaBK;
          b_half = kU2BBytes;
          b_row = c.nt * 256 + (int)rank * 128;
          j = g.is_shared ? 0 : (c.g - p.n_outer) - g.outer * p.n_r;
        }
        for (int kb = 0; kb < k_blocks; ++kb, ++it) {
          const uint32_t s = it % kU2Stages, n = it / kU2Stages;
          if (!mbar_wait(empty0 + 8 * s, (n & 1) ^ 1, abort_flag, p.err, kErrWaitEmpty)) { ok = false; break; }
          const uint32_t fb_local = full0 + 8 * s;
          const uint32_t fb = mapa_shared(fb_local, 0);               // the leader's barrier
          const uint32_t sa = base + s * kU2StageBytes, sb = sa + kU2ABytes;
          if (leader) mbar_expect_tx(fb_local, 2 * ((by_threads ? 0 : kU2ABytes) + b_half));
          if (!by_threads) tma2_load_2d(sa, ta, fb, kb * kUmmaBK, row);
          if (MODE == 1) tma2_load_3d(sb, tb, fb, kb * kUmmaBK, b_row, (int)rank);   // plane 0 gate, 1 up
          else if (g.is_shared) tma2_load_3d(sb, tb, fb, kb * kUmmaBK, b_row, g.outer);
          else tma2_load_4d(sb, tb, fb, kb * kUmmaBK, b_row, j, g.outer);
        }
      }
      if (!ok) for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader CTA only)
    if (leader && lane == 0) {
      uint32_t it = 0, tile_n = 0;
      bool ok = true;
      for (int t = pair_id; t < total_tiles && ok; t += n_pairs, ++tile_n) {
        const Pair2Coord c = umma2_decode<MODE>(p, tile_start, t);
        const GroupStatic g = p.gs[c.g];
        int k_blocks, n_mma;
        if (MODE == 1) { k_blocks = k_blocks_fixed; n_mma = 2 * (g.is_shared ? p.bn_s : p.bn_r); }
        else { k_blocks = (g.width + kUmmaBK - 1) / kUmmaBK; n_mma = 256; }
        const uint32_t idesc = umma2_idesc(n_mma);
        const uint32_t buf = tile_n & 1, use = tile_n >> 1;
        if (!mbar_wait(acce0 + 8 * buf, (use & 1) ^ 1, abort_flag, p.err, kErrWaitAccEmpty)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * 256;
        for (int kb = 0; kb < k_blocks; ++kb, ++it) {
          const uint32_t s = it % kU2Stages, n = it / kU2Stages;
          if (!mbar_wait(full0 + 8 * s, n & 1, abort_flag, p.err, kErrWaitFull)) { ok = false; break; }
          if (MODE == 1) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          tc_fence_after();
          const uint32_t sa = base + s * kU2StageBytes, sb = sa + kU2ABytes;
#pragma unroll
          for (int k = 0; k < kUmmaBK / 16; ++k)
            umma2_bf16(d_tmem, umma_smem_desc(sa + k * 32), umma_smem_desc(sb + k * 32), idesc,
                       (kb | k) != 0 ? 1u : 0u);
          umma2_commit_both(empty0 + 8 * s);
        }
        if (ok) umma2_commit_both(accf0 + 8 * buf);
      }
    }
  } else if (MODE == 1 && warp == 10) {
    // ------------------------------------------------------------ relay (gate/up, warp 10, both CTAs)
    // Waits until this CTA's 128 gather threads have landed a k block (local barrier), fences
    // those generic-proxy writes towards the async proxy and arrives on the leader's full barrier.
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int t = pair_id; t < total_tiles && ok; t += n_pairs) {
        for (int kb = 0; kb < k_blocks_fixed; ++kb, ++it) {
          const uint32_t s = it % kU2Stages, n = it / kU2Stages;
          if (!mbar_wait(afull0 + 8 * s, n & 1, abort_flag, p.err, kErrWaitFull)) { ok = false; break; }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          mbar_arrive_remote(mapa_shared(full0 + 8 * s, 0));
        }
      }
    }
  } else if (MODE == 1 && warp >= 6) {
    // ------------------------------------------------------------ A-row gather (gate/up, warps 6..9, both CTAs)
    // Eight consecutive threads cover one 128-byte row segment, 16 rows per pass, 8 passes; 16-byte
    // chunk c of row r goes to the swizzled chunk c ^ (r & 7).  Each thread's arrival on the CTA's
    // local barrier is tied to the completion of its copies (cp.async.mbarrier.arrive.noinc).
    const int gt = threadIdx.x - kUmmaThreads;
    const int ch = gt & 7, r_sub = gt >> 3;
    uint32_t it = 0;
    bool ok = true;
    for (int t = pair_id; t < total_tiles && ok; t += n_pairs) {
      const Pair2Coord c = umma2_decode<MODE>(p, tile_start, t);
      const GroupStatic g = p.gs[c.g];
      const bool mine = !g.is_shared && p.use_gather == 2;
      const bf16* src_row[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        src_row[i] = nullptr;
        if (mine) {                                   // rows past the group repeat its last row
          const int r = c.row0 + min((2 * c.mp + (int)rank) * kUmmaBM + i * 16 + r_sub, c.count - 1);
          src_row[i] = p.x_rows_ptr + (size_t)__ldg(p.row_token + r) * p.d;
        }
      }
      for (int kb = 0; kb < k_blocks_fixed; ++kb, ++it) {
        const uint32_t s = it % kU2Stages, n = it / kU2Stages;
        if (!mbar_wait(empty0 + 8 * s, (n & 1) ^ 1, abort_flag, p.err, kErrWaitEmpty)) { ok = false; break; }
        const uint32_t ab = afull0 + 8 * s;
        if (mine) {
          const int k = kb * kUmmaBK + ch * 8;
          const uint32_t bytes = k < p.d ? 16u : 0u;                        // zero-fill past the end of the row
          const int k_src = k < p.d ? k : 0;
          const uint32_t sa = base + s * kU2StageBytes;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int r = i * 16 + r_sub;
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;"
                         ::"r"(sa + r * 128 + ((ch ^ (r & 7)) << 4)), "l"(src_row[i] + k_src), "r"(bytes)
                         : "memory");
          }
          asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(ab) : "memory");
        } else {
          mbar_arrive(ab);
        }
      }
    }
    if (!ok) asm volatile("cp.async.wait_all;" ::: "memory");
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5, both CTAs)
    const int quad = warp & 3;
    uint32_t tile_n = 0;
    bool ok = true;
    for (int t = pair_id; t < total_tiles && ok; t += n_pairs, ++tile_n) {
      const Pair2Coord c = umma2_decode<MODE>(p, tile_start, t);
      const GroupStatic g = p.gs[c.g];
      const uint32_t buf = tile_n & 1, use = tile_n >> 1;
      if (!mbar_wait(accf0 + 8 * buf, use & 1, abort_flag, p.err, kErrWaitAccFull)) { ok = false; break; }
      tc_fence_after();
      const int row_in_group = (2 * c.mp + (int)rank) * kUmmaBM + quad * 32 + lane;
      const bool row_ok = row_in_group < c.count;
      const uint32_t taddr = tmem_base + buf * 256 + ((uint32_t)(quad * 32) << 16);
      if (MODE == 1) {
        const int bn = g.is_shared ? p.bn_s : p.bn_r;
        const int ld = g.is_shared ? p.ld_out_s : p.ld_out_r;
        const int n0 = c.nt * bn;
        const int n_valid = min(bn, g.width - n0);
        bf16* dst = (g.is_shared ? p.out_s : p.out_r) + (size_t)(c.row0 + row_in_group) * ld + n0;
        const bool wide = ((ld | n0) & 15) == 0;
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
      } else {
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
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa_shared(acce0 + 8 * buf, 0));
    }
  }
  tc_fence_before();
  cluster_sync_all();                         // the peer is done with this CTA's smem and TMEM use
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc2(tmem_base, kUmmaTmemCols);
  }
}

// ----------------------------------------------------------------------------- host
struct Umma2Plan {
  bool built = false;
  int grid = 0;                    // 2 x the number of CTA pairs that can be resident at once
  CUtensorMap b1_s, b1_r;          // stacked gate/up rows, box 64 k x bn rows x 1 plane
};

inline bool umma2_plan_create(UmmaPlan* P, Umma2Plan* Q) {
  const UmmaShape& s = P->shape;
  const size_t d = s.d, rows_w = (size_t)s.n_outer * s.d_ff;
  bool ok = true;
  for (int shared = 0; shared < 2 && ok; ++shared) {
    const int bn = shared ? P->bn_s : P->bn_r;
    const cuuint64_t dims[3] = {d, rows_w, 2};
    const cuuint64_t str[2] = {d * 2, rows_w * d * 2};
    const cuuint32_t box[3] = {kUmmaBK, (cuuint32_t)bn, 1};
    ok = umma_encode(P, shared ? &Q->b1_s : &Q->b1_r, P->buf.w_gate_up, 3, dims, str, box,
                     "gate/up weights (CTA pair)");
  }
  if (!ok) return false;
  cudaError_t e = cudaFuncSetAttribute(umma2_grouped_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kU2SmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(umma2_grouped_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kU2SmemBytes);
  if (e != cudaSuccess) {
    snprintf(P->error, sizeof(P->error), "cudaFuncSetAttribute (CTA pair): %s", cudaGetErrorString(e));
    return false;
  }
  // persistent grid: as many pairs as the device can hold at once (GPCs with an odd SM count leave one SM out)
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(P->n_sms & ~1, 1, 1);
  cfg.blockDim = dim3(kU2Threads1, 1, 1);
  cfg.dynamicSmemBytes = kU2SmemBytes;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  int n_clusters = 0;
  e = cudaOccupancyMaxActiveClusters(&n_clusters, umma2_grouped_kernel<1>, &cfg);
  if (e != cudaSuccess || n_clusters <= 0) {
    snprintf(P->error, sizeof(P->error), "cudaOccupancyMaxActiveClusters: %s", cudaGetErrorString(e));
    return false;
  }
  Q->grid = 2 * (n_clusters < P->n_sms / 2 ? n_clusters : P->n_sms / 2);
  Q->built = true;
  return true;
}

// Gate/up and down GEMM on CTA pairs.  gather_mode 2: routed rows are gathered from x_rows inside
// the gate/up kernel; 0: they come from the permuted copy of x by TMA.
// `D` supplies the 128-channel W_down maps (shared with the decode path).  Requires
// umma_bind_x for this forward.  which: bit 0 the gate/up GEMM, bit 1 the down GEMM.  Returns launches or -1.
inline int umma2_forward(UmmaPlan* P, Umma2Plan* Q, DecodePlan* D, const GroupRows* gr, int gather_mode,
                         const void* x_rows, int32_t* err_word, cudaStream_t st, cudaEvent_t mid, bool dep = false,
                         int which = 3) {
  const UmmaShape& s = P->shape;
  UmmaArgs a = umma_base_args(P, gr, err_word);
  const int grid = Q->grid;
  a.out_s = (bf16*)P->buf.h_s; a.out_r = (bf16*)P->buf.h_r; a.ld_out_s = s.shared_width; a.ld_out_r = s.m;
  a.use_gather = gather_mode;
  a.x_rows_ptr = (const bf16*)x_rows;
  a.band_mt = umma_band_tiles(s.d);
  if (which & 1)
    launch_kernel(dep, umma2_grouped_kernel<1>, dim3(grid), dim3(kU2Threads1), kU2SmemBytes, st,
                  P->x_rows, P->has_r ? P->x_perm : P->x_rows, Q->b1_s, Q->b1_r, a);
  if (mid && (which & 1)) cudaEventRecord(mid, st);
  a.out_s = (bf16*)P->buf.y_s; a.out_r = (bf16*)P->buf.y_r; a.ld_out_s = s.d; a.ld_out_r = s.d;
  a.band_mt = umma_band_tiles(s.shared_width > s.m ? s.shared_width : s.m);
  if (which & 2)
    launch_kernel(dep, umma2_grouped_kernel<2>, dim3(grid), dim3(kUmmaThreads), kU2SmemBytes, st, P->a2_s, P->a2_r,
                  D->wd_s, D->wd_r, a);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    snprintf(P->error, sizeof(P->error), "CTA-pair GEMM launch: %s", cudaGetErrorString(e));
    return -1;
  }
  return (which & 1) + ((which >> 1) & 1);
}

}  // namespace cmoe
