// Decode-shaped expert GEMMs (at most 64 rows per group): the contraction is turned
// around so that the WEIGHTS sit on the 128-row M side of the tcgen05 MMA and the few
// tokens on the N side (N = row count rounded up to 16).  The tensor-core time per
// 64-wide k block is then a few dozen cycles instead of the 512 a 128-row token tile
// costs, so a CTA can stream its weight rows as fast as TMA delivers them: the regime is
// HBM-bound on the active experts' weight bytes and the kernel is a weight streamer with
// deep TMA pipelines (5 x 40 KB or 8 x 24 KB in flight per SM).
//
//   MODE 4, gate/up:  Dg[n, t] = Wg[n] . x_t ,  Du[n, t] = Wu[n] . x_t  (two MMAs sharing
//       the token tile), epilogue H[t, n] = Swish(Dg) * Du           (Eq. ori_ffn_method)
//       tile = 128 neurons of one group.  The token tile is ALL rows of the group's outer
//       expert (the whole batch for a plain layer): with tokens on the N side the extra
//       columns cost almost nothing, every group shares one tiled TMA box, and a routed
//       group's epilogue simply stores the columns of the tokens that selected it.
//   MODE 5, down:     D[c, t] = Wd[c] . H_t ,  epilogue Y[t, c] = D
//       tile = 128 output channels of one group.
// With few active experts there are fewer tiles than SMs and one SM cannot pull more than
// ~100 GB/s through TMA, so a tile's K range is split into Z slices when that brings the
// unit count closer to the SM count (Z = k blocks of the tile / (all k blocks / CTAs),
// rounded down, per group).  A slice leaves its fp32 partial accumulators in a scratch slot;
// each epilogue warp takes a ticket for its 32 weight rows of the tile, and the warp that
// takes the last one adds the Z partials in slice order (a fixed order: deterministic) and
// finishes the tile.  Units are dealt to the persistent CTAs in snake order (left to right,
// then right to left), which balances long shared-expert units against short routed ones.
// Same warp roles, bounded waits and teardown as the token-major kernels.
//
// W8 = true streams FP8 (E4M3) weights, half the bytes, and multiplies them as they are:
// tcgen05.mma kind::f8f6f4 on the codes, no conversion.  The bf16 token rows (x, H) are split
// beforehand (split_rows_e4m3_kernel) into two E4M3 planes, hi = the value rounded to E4M3 and
// lo = 16 x the remainder, after a per-row power-of-two scale; a bf16 number has 8 significant
// bits and each plane carries 4, so hi + lo/16 is the value itself (exactly, down to 2^-13 of the
// row's largest magnitude).  A stage covers 128 k (128 bytes per weight row, the same TMA box
// geometry as the bf16 tiles), each k step issues one MMA per (weight plane, token plane) into
// its own accumulator columns, and the epilogue forms (hi + lo/16) x row scale x token scale.
#pragma once

#include "fp8.cuh"
#include "umma_gemm.cuh"

namespace cmoe {

constexpr int kDecMaxRows = 64;            // rows per group of the narrow kernels (every FP8 and K-splitting form)
constexpr int kDecWideRows = 128;          // rows per group of the wide bf16 kernels (NT = 128)

constexpr int kDecMaxSplit = 8;            // K slices per tile at most
constexpr int kDecMinSliceKb = 6;          // k blocks per slice at least
constexpr int kDecMaxSlots = 256;          // scratch slots for slice partials (>= CTAs)
constexpr int kDecSlotFloats = 128 * 2 * kDecMaxRows;      // 128 weight rows x (gate, up) x 64 tokens

// per group: first unit / tile / slot, split, k blocks per tile
struct DecGroup { int32_t unit0, tile0, slot0; int16_t z, kb; };
constexpr int kDecInvOff = 256 + ((kUmmaMaxGroups + 1) * (int)sizeof(DecGroup) + 15) / 16 * 16;   // per-warp token tables

// kWBytes: weight tile(s) of one stage: 128 rows x 128 bytes per plane (64 bf16 or 128 E4M3 k values);
// kXBytes: token tile(s) of one stage, NT rows of 128 bytes (W8: the hi and the lo plane);
// kStages: as many as 227 KB of shared memory hold, eight at most.
template <int MODE, bool W8, int NT> struct DecodeCfg {
  static constexpr int kWBytes = (MODE == 4 ? 2 : 1) * 128 * 128;
  static constexpr int kXBytes = (W8 ? 2 : 1) * NT * 128;
  static constexpr int kFit = (227 * 1024 - 1024 - kDecInvOff - 4 * NT * 4) / (kWBytes + kXBytes);
  static constexpr int kStages = kFit > 8 ? 8 : kFit;   // 40 KB x 5, 24 x 8 (NT 64); 48 x 4, 32 x 6 (FP8, or NT 128)
};

template <int MODE, bool W8 = false, int NT = kDecMaxRows>
constexpr int decode_smem_bytes() {
  using C = DecodeCfg<MODE, W8, NT>;
  return 1024 + C::kStages * (C::kWBytes + C::kXBytes) + kDecInvOff + 4 * NT * 4;
}
// TMEM columns: two accumulator buffers of (weight planes x token planes) x NT token columns, 256 at least
template <int MODE, bool W8, int NT> struct DecodeTmem {
  static constexpr int kNeed = 2 * (MODE == 4 ? 2 : 1) * (W8 ? 2 : 1) * NT;
  static constexpr int kCols = kNeed < 256 ? 256 : kNeed;
};

struct DecodeArgs {
  const GroupStatic* gs;
  const GroupRows* gr;
  int n_groups, n_outer, n_r;
  int d;
  bf16* out_s;           // mode 4: H_s ; mode 5: Y_s
  bf16* out_r;           // mode 4: H_r ; mode 5: Y_r
  int ld_out_s, ld_out_r;
  const int32_t* row_token;
  int32_t* err;
  float* part;           // [kDecMaxSlots][kDecSlotFloats] slice partials
  int32_t* ticket;       // [tiles][4 epilogue warps], zero between launches
  int tok_box_rows;      // rows of the token-tile TMA box (16, 32, 64 or 128): no more than the batch needs
  int tile_rows_s, tile_rows_r;   // mode 4: neurons per tile of a shared / routed group (128, or less when 128 would pad
                         // the group's width by more than 5 %: the rows past them in the 128-row MMA are dead)
  int early_units;       // plain gate/up form: tiles of the shared expert (group 0) that need nothing from the router
  int n_rows_plain;      // rows of the batch (the shared expert's rows of a plain layer)
  // W8: per-row power-of-two scales of the token planes (x or H rows), then of the FP8 weight rows
  const float* tok_scale_s;   // rows of the shared groups' token space (mode 4: x rows; mode 5: H_s rows)
  const float* tok_scale_r;   // mode 4: x rows again; mode 5: H_r rows
  const float* scale_gu; // [2][rows_w]: gate plane, then up plane, packed neuron order
  const float* scale_d;  // [n_groups][d]: per group and output channel
  long long rows_w;      // n_outer * d_ff
};

// Tile handled by CTA `cta` in its `round`-th turn: even rounds run left to right, odd
// rounds right to left.  Returns -1 past the end.
__device__ __forceinline__ int snake_tile(int round, int cta, int n_ctas, int total) {
  const int t = round * n_ctas + ((round & 1) ? n_ctas - 1 - cta : cta);
  return t < total ? t : -1;
}

// SPLIT = false is the plain form (one unit per tile, no scratch); the host picks SPLIT = true
// only when even the largest possible set of active experts leaves tiles to split.
// NT: token columns per tile at most (64, or 128 for the wide bf16 form that takes batches of 65..128 rows).
template <int MODE, bool SPLIT, bool W8 = false, int NT = kDecMaxRows>
__global__ void __launch_bounds__(kUmmaThreads, 1)
umma_decode_kernel(const __grid_constant__ CUtensorMap tm_w_s, const __grid_constant__ CUtensorMap tm_w_r,
                   const __grid_constant__ CUtensorMap tm_x_s, const __grid_constant__ CUtensorMap tm_x_r,
                   const DecodeArgs p) {
  // The plain gate/up form looks at what the preceding kernel (the router) wrote as late as it can: a CTA
  // whose first unit is a tile of the shared expert (p.early_units of them) streams that tile at once
  // and only then waits for the router, so the shared expert's weights move under the router's latency.
  constexpr bool kLazy = MODE == 4 && !SPLIT;
  if constexpr (!kLazy) grid_dep_wait();
  grid_dep_trigger();
  static_assert(NT <= kDecMaxRows || (!SPLIT && !W8), "the wide form has no K split and no FP8 planes");
  using Cfg = DecodeCfg<MODE, W8, NT>;
  constexpr int kStages = Cfg::kStages;
  constexpr int kWBytes = Cfg::kWBytes;
  constexpr int kStageBytes = kWBytes + Cfg::kXBytes;
  constexpr int kBK = W8 ? 2 * kUmmaBK : kUmmaBK;                // k per stage: 128 bytes of a weight row
  constexpr int kTmemCols = DecodeTmem<MODE, W8, NT>::kCols;
  constexpr int kBufCols = kTmemCols / 2;                        // accumulator columns per buffer
  constexpr int kUpCol = (W8 ? 2 : 1) * NT;                      // mode 4: first column of the up accumulators
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const uint32_t bars = base + kStages * kStageBytes;
  uint8_t* bars_gen = gen + kStages * kStageBytes;
  // barrier block: full[8] empty[8] acc_full[2] acc_empty[2], tmem slot, abort flag, table barrier
  const uint32_t full0 = bars, empty0 = bars + 64, accf0 = bars + 128, acce0 = bars + 144;
  const uint32_t tbl_bar = bars + 168;                           // kLazy: the unit table has been built
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars_gen + 160);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars_gen + 164);
  DecGroup* grp = reinterpret_cast<DecGroup*>(bars_gen + 256);       // SPLIT: [n_groups + 1]
  int32_t* tile_start = reinterpret_cast<int32_t*>(bars_gen + 256);  // !SPLIT: [n_groups + 1], same bytes
  int32_t* inv_tables = reinterpret_cast<int32_t*>(bars_gen + kDecInvOff);     // [4 warps][NT]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // rows of a tile of group g and the number of its tiles
  auto tile_rows = [&](const GroupStatic& g) { return MODE == 4 ? (g.is_shared ? p.tile_rows_s : p.tile_rows_r) : 128; };
  auto group_tiles = [&](int g) {
    const GroupStatic gg = p.gs[g];
    const int span = MODE == 4 ? gg.width : (gg.width > 0 ? p.d : 0), tr = tile_rows(gg);
    return p.gr[g].count > 0 ? (span + tr - 1) / tr : 0;
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(accf0 + 8 * b, 1); mbar_init(acce0 + 8 * b, 4); }
    mbar_init(tbl_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish();
  }
  if constexpr (kLazy) {
    // the table is built by the producer warp when a role first needs it (build_table below)
  } else if constexpr (!SPLIT) {
    for (int g = threadIdx.x; g < p.n_groups; g += blockDim.x) tile_start[g + 1] = group_tiles(g);
    __syncthreads();
    if (threadIdx.x == 0) {
      int run = 0;
      tile_start[0] = 0;
      for (int g = 0; g < p.n_groups; ++g) { run += tile_start[g + 1]; tile_start[g + 1] = run; }
    }
  } else {
    // per group: tile count (in .tile0 for now) and k blocks per tile
    for (int g = threadIdx.x; g < p.n_groups; g += blockDim.x) {
      grp[g].tile0 = group_tiles(g);
      grp[g].kb = (int16_t)(((MODE == 4 ? p.d : p.gs[g].width) + kBK - 1) / kBK);
    }
    __syncthreads();
    if (warp == 0) {                 // unit / tile / slot prefix sums over the groups, 32 groups per step
      int all_kb = 0;
      for (int g = lane; g < p.n_groups; g += 32) all_kb += grp[g].tile0 * grp[g].kb;
  #pragma unroll
      for (int o = 16; o > 0; o >>= 1) all_kb += __shfl_xor_sync(0xffffffffu, all_kb, o);
      int per_cta = (all_kb + (int)gridDim.x - 1) / (int)gridDim.x;    // k blocks a CTA streams if all share evenly
      if (per_cta < kDecMinSliceKb * kUmmaBK / kBK) per_cta = kDecMinSliceKb * kUmmaBK / kBK;
      // sum over split groups of tiles * z <= all_kb / per_cta <= CTAs, so the slots suffice for grids up to kDecMaxSlots
      const bool may_split = (int)gridDim.x <= kDecMaxSlots;
      int units = 0, tiles = 0, slots = 0;
      for (int g0 = 0; g0 < p.n_groups; g0 += 32) {
        const int g = g0 + lane;
        const bool in = g < p.n_groups;
        const int n_t = in ? grp[g].tile0 : 0;
        int z = in ? grp[g].kb / per_cta : 1;
        z = (z < 1 || !may_split) ? 1 : (z > kDecMaxSplit ? kDecMaxSplit : z);
        const int u = n_t * z, sl = z > 1 ? u : 0;
        int iu = u, it = n_t, is = sl;                       // inclusive scans
  #pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int au = __shfl_up_sync(0xffffffffu, iu, o), at = __shfl_up_sync(0xffffffffu, it, o),
                    as = __shfl_up_sync(0xffffffffu, is, o);
          if (lane >= o) { iu += au; it += at; is += as; }
        }
        if (in) { grp[g].unit0 = units + iu - u; grp[g].tile0 = tiles + it - n_t; grp[g].slot0 = slots + is - sl; grp[g].z = (int16_t)z; }
        units += __shfl_sync(0xffffffffu, iu, 31);
        tiles += __shfl_sync(0xffffffffu, it, 31);
        slots += __shfl_sync(0xffffffffu, is, 31);
      }
      if (lane == 0) {
        grp[p.n_groups].unit0 = units; grp[p.n_groups].tile0 = tiles; grp[p.n_groups].slot0 = slots;
        grp[p.n_groups].z = 1; grp[p.n_groups].kb = 0;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  int total_units = kLazy ? 0 : (SPLIT ? grp[p.n_groups].unit0 : tile_start[p.n_groups]);
  const int cta = blockIdx.x, n_ctas = gridDim.x;
  // kLazy: this CTA's first unit (snake round 0 = unit `cta`) is tile `cta` of the shared expert, group 0,
  // whose rows are all of the batch: nothing the router writes is needed for it
  const bool early = kLazy && cta < p.early_units;
  bool tbl_seen = !kLazy;
  // producer warp: wait for the router, count every group's tiles, publish the table
  auto build_table = [&]() {
    grid_dep_wait();
    for (int g = lane; g < p.n_groups; g += 32) tile_start[g + 1] = group_tiles(g);
    __syncwarp();
    if (lane == 0) {
      int run = 0;
      tile_start[0] = 0;
      for (int g = 0; g < p.n_groups; ++g) { run += tile_start[g + 1]; tile_start[g + 1] = run; }
      mbar_arrive(tbl_bar);
    }
    __syncwarp();
    total_units = tile_start[p.n_groups];
    tbl_seen = true;
  };
  // every other role: wait for the table (bounded), then for the router's writes
  auto await_table = [&]() -> bool {
    if (!mbar_wait(tbl_bar, 0, abort_flag, p.err, kErrWaitFull)) return false;
    grid_dep_wait();
    total_units = tile_start[p.n_groups];
    tbl_seen = true;
    return true;
  };
  auto group_rows = [&](int gidx, bool first_early) {            // rows of a group; the early unit's are known
    if (first_early) { GroupRows r; r.row0 = 0; r.count = p.n_rows_plain; return r; }
    return p.gr[gidx];
  };

  // unit -> group, tile within the group, K slice
  struct Unit { int gi, nt, z, n_z, kb0, kb1; };
  auto find_unit = [&](int uid) {
    int lo = 0, hi = p.n_groups;
    if constexpr (!SPLIT) {
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (tile_start[mid] <= uid) lo = mid; else hi = mid;
      }
      Unit u;
      u.gi = lo; u.nt = uid - tile_start[lo]; u.z = 0; u.n_z = 1; u.kb0 = 0; u.kb1 = 0;   // kb1: see k_end
      return u;
    }
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (grp[mid].unit0 <= uid) lo = mid; else hi = mid;
    }
    Unit u;
    u.gi = lo; u.n_z = grp[lo].z;
    const int local = uid - grp[lo].unit0, k_blocks = grp[lo].kb;
    if (u.n_z == 1) {
      u.nt = local; u.z = 0; u.kb0 = 0; u.kb1 = k_blocks;
    } else {
      u.nt = local / u.n_z; u.z = local - u.nt * u.n_z;
      u.kb0 = u.z * k_blocks / u.n_z;
      u.kb1 = (u.z + 1) * k_blocks / u.n_z;
    }
    return u;
  };

  Unit early_unit;
  early_unit.gi = 0; early_unit.nt = cta; early_unit.z = 0; early_unit.n_z = 1; early_unit.kb0 = 0; early_unit.kb1 = 0;
  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (whole warp)
    uint32_t it = 0;
    bool ok = true;
    for (int round = 0; ok; ++round) {
      const bool fe = early && round == 0;
      if (!fe && !tbl_seen) build_table();
      const int t = fe ? cta : snake_tile(round, cta, n_ctas, total_units);
      if (t < 0) break;
      const Unit un = fe ? early_unit : find_unit(t);
      const int gi = un.gi, nt = un.nt;
      const GroupStatic g = p.gs[gi];
      // mode 4: token rows of the group's outer expert; mode 5: the group's own H rows
      const GroupRows r = MODE == 4 ? group_rows(g.outer, fe) : p.gr[gi];
      const CUtensorMap* tw = g.is_shared ? &tm_w_s : &tm_w_r;
      const CUtensorMap* tx = g.is_shared ? &tm_x_s : &tm_x_r;
      const int j = g.is_shared ? 0 : (gi - p.n_outer) - g.outer * p.n_r;
      const int k_end = SPLIT ? un.kb1 : ((MODE == 4 ? p.d : g.width) + kBK - 1) / kBK;
      for (int kb = un.kb0; kb < k_end; ++kb, ++it) {
        const uint32_t s = it % kStages, n = it / kStages;
        if (!mbar_wait(empty0 + 8 * s, (n & 1) ^ 1, abort_flag, p.err, kErrWaitEmpty)) { ok = false; break; }
        const uint32_t fb = full0 + 8 * s;
        const uint32_t sw = base + s * kStageBytes, sx = sw + kWBytes;
        if (lane == 0) {
          const int tr = tile_rows(g);
          mbar_expect_tx(fb, (MODE == 4 ? 2 : 1) * tr * 128 + (W8 ? 2 : 1) * p.tok_box_rows * 128);
          if (MODE == 4) tma_load_3d(sw, tw, fb, kb * kBK, g.w_row0 + nt * tr, 0);   // gate rows, then the up rows behind them
          else if (g.is_shared) tma_load_3d(sw, tw, fb, kb * kBK, nt * 128, g.outer);
          else tma_load_4d(sw, tw, fb, kb * kBK, nt * 128, j, g.outer);
          if constexpr (W8) {                   // token planes [k, row, plane]: the hi rows, directly behind them the lo rows
            tma_load_3d(sx, tx, fb, kb * kBK, r.row0, 0);
            tma_load_3d(sx + p.tok_box_rows * 128, tx, fb, kb * kBK, r.row0, 1);
          } else {
            tma_load_2d(sx, tx, fb, kb * kBK, r.row0);
          }
        }
        __syncwarp();
      }
    }
    if (!ok) for (int i = 0; i < 200; ++i) __nanosleep(1000);
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int round = 0; ok; ++round) {
        const bool fe = early && round == 0;
        if (!fe && !tbl_seen && !await_table()) { ok = false; break; }
        const int t = fe ? cta : snake_tile(round, cta, n_ctas, total_units);
        if (t < 0) break;
        const Unit un = fe ? early_unit : find_unit(t);
        const int gi = un.gi;
        const GroupStatic g = p.gs[gi];
        const int n_mma = ((MODE == 4 ? group_rows(g.outer, fe).count : p.gr[gi].count) + 15) & ~15;   // columns, rounded to 16
        // W8: one MMA covers both token planes (N = hi rows + lo rows, adjacent in the stage): the decode
        // kernels are bound by the number of MMAs a tile takes (~115 cycles each at these small N), not by bytes
        const uint32_t idesc = W8 ? umma_idesc_e4m3(2 * p.tok_box_rows) : umma_idesc(n_mma);
        const uint32_t buf = round & 1, use = round >> 1;
        if (!mbar_wait(acce0 + 8 * buf, (use & 1) ^ 1, abort_flag, p.err, kErrWaitAccEmpty)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * kBufCols;
        const uint32_t up_off = (uint32_t)tile_rows(g) * 128u;          // the up plane follows the tile's gate rows
        const int k_end = SPLIT ? un.kb1 : ((MODE == 4 ? p.d : g.width) + kBK - 1) / kBK;
        for (int kb = un.kb0; kb < k_end; ++kb, ++it) {
          const uint32_t s = it % kStages, n = it / kStages;
          const uint32_t sw = base + s * kStageBytes, sx = sw + kWBytes;
          if (!mbar_wait(full0 + 8 * s, n & 1, abort_flag, p.err, kErrWaitFull)) { ok = false; break; }
          tc_fence_after();
          // four k steps of 32 bytes per 128-byte row: 16 bf16 or 32 E4M3 values each
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const uint32_t acc = (kb != un.kb0 || k != 0) ? 1u : 0u;
            const uint64_t a_g = umma_smem_desc(sw + k * 32), a_u = umma_smem_desc(sw + up_off + k * 32);
            const uint64_t b_hi = umma_smem_desc(sx + k * 32);
            if constexpr (W8) {
              umma_e4m3(d_tmem, a_g, b_hi, idesc, acc);
              if (MODE == 4) umma_e4m3(d_tmem + kUpCol, a_u, b_hi, idesc, acc);
            } else {
              umma_bf16(d_tmem, a_g, b_hi, idesc, acc);
              if (MODE == 4) umma_bf16(d_tmem + kUpCol, a_u, b_hi, idesc, acc);
            }
          }
          umma_commit(empty0 + 8 * s);
        }
        if (ok) umma_commit(accf0 + 8 * buf);
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int quad = warp & 3;
    bool ok = true;
    for (int round = 0; ok; ++round) {
      const bool fe = early && round == 0;
      if (!fe && !tbl_seen && !await_table()) { ok = false; break; }
      const int t = fe ? cta : snake_tile(round, cta, n_ctas, total_units);
      if (t < 0) break;
      const Unit un = fe ? early_unit : find_unit(t);
      const int gi = un.gi, nt = un.nt;
      const GroupStatic g = p.gs[gi];
      const GroupRows r = group_rows(gi, fe);
      const uint32_t buf = round & 1, use = round >> 1;
      if (!mbar_wait(accf0 + 8 * buf, use & 1, abort_flag, p.err, kErrWaitAccFull)) { ok = false; break; }
      tc_fence_after();
      const int tr = tile_rows(g);
      const int wr = nt * tr + quad * 32 + lane;                  // neuron (mode 4) / channel (mode 5)
      const int span = MODE == 4 ? g.width : p.d;
      const int ld = MODE == 4 ? (g.is_shared ? p.ld_out_s : p.ld_out_r) : p.d;
      bf16* dst = (g.is_shared ? p.out_s : p.out_r) + (size_t)r.row0 * ld + wr;
      const uint32_t taddr = tmem_base + buf * kBufCols + ((uint32_t)(quad * 32) << 16);
      // Columns of the accumulator: mode 5 and shared groups, the group's own rows in order;
      // routed groups in mode 4, every row of the outer expert -> position in the group or -1.
      const bool lookup = MODE == 4 && !g.is_shared;
      int32_t* inv = inv_tables + quad * NT;
      int n_cols = r.count;
      // W8: per-token scale of accumulator column c = tok_scale[c]: mode 4, the x rows of the outer expert;
      // mode 5, the group's own H rows
      const float* tok_scale = nullptr;
      if constexpr (W8) tok_scale = (g.is_shared ? p.tok_scale_s : p.tok_scale_r) + r.row0;
      if (lookup) {
        const GroupRows rs = p.gr[g.outer];
        n_cols = rs.count;
        if constexpr (W8) tok_scale = p.tok_scale_r + rs.row0;
        __syncwarp();
#pragma unroll
        for (int c = 0; c < NT; c += 32) if (c + lane < NT) inv[c + lane] = -1;
        __syncwarp();
        for (int c = lane; c < r.count; c += 32) inv[__ldg(p.row_token + r.row0 + c) - rs.row0] = c;
        __syncwarp();
      }
      const bool row_live = quad * 32 + lane < tr && wr < span;
      float sc_a = 1.0f, sc_b = 1.0f;                    // W8: power-of-two scales of this thread's weight row(s)
      if constexpr (W8) {
        if (row_live) {
          if (MODE == 4) {
            sc_a = __ldg(p.scale_gu + g.w_row0 + wr);
            sc_b = __ldg(p.scale_gu + p.rows_w + g.w_row0 + wr);
          } else {
            sc_a = __ldg(p.scale_d + (size_t)gi * p.d + wr);
          }
        }
      }
      auto finish = [&](int c, float a, float b) {       // accumulator column c of this thread's weight row
        if (row_live && c < n_cols) {
          const int pos = lookup ? inv[c] : c;
          if (pos >= 0) {
            if constexpr (W8) { const float ts = __ldg(tok_scale + c); a *= sc_a * ts; b *= sc_b * ts; }
            const float v = MODE == 4 ? a / (1.0f + __expf(-a)) * b : a;
            dst[(size_t)pos * ld] = __float2bfloat16_rn(v);
          }
        }
      };
      // 16 accumulator columns of this thread's weight row(s); W8: hi plane + lo plane / 16
      auto load16 = [&](int c0, float (&a)[16], float (&b)[16]) {
        tmem_ld16(taddr + c0, a);
        if (MODE == 4) tmem_ld16(taddr + kUpCol + c0, b);
        if constexpr (W8) {
          float al[16], bl[16];                       // the lo plane's columns follow the hi plane's tok_box_rows
          tmem_ld16(taddr + p.tok_box_rows + c0, al);
          if (MODE == 4) tmem_ld16(taddr + kUpCol + p.tok_box_rows + c0, bl);
          tmem_ld_wait();
#pragma unroll
          for (int q = 0; q < 16; ++q) {
            a[q] = fmaf(al[q], 0.0625f, a[q]);
            if (MODE == 4) b[q] = fmaf(bl[q], 0.0625f, b[q]);
          }
        } else {
          tmem_ld_wait();
        }
      };
      if (!SPLIT || un.n_z == 1) {
        for (int c0 = 0; c0 < n_cols; c0 += 16) {
          float a[16], b[16];
          load16(c0, a, b);
#pragma unroll
          for (int q = 0; q < 16; ++q) finish(c0 + q, a[q], MODE == 4 ? b[q] : 0.0f);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acce0 + 8 * buf);
      } else if constexpr (SPLIT) {
        // K slice of a split tile: park the partial sums, take this warp's ticket for the tile
        constexpr int kPlanes = MODE == 4 ? 2 : 1;
        const int slot0 = grp[gi].slot0 + nt * un.n_z;
        float* mine = p.part + (size_t)(slot0 + un.z) * kDecSlotFloats + quad * 32 + lane;
        for (int c0 = 0; c0 < n_cols; c0 += 16) {
          float a[16], b[16];
          load16(c0, a, b);
#pragma unroll
          for (int q = 0; q < 16; ++q) {
            if (c0 + q < n_cols) {
              __stcg(mine + (size_t)((c0 + q) * kPlanes) * 128, a[q]);
              if (MODE == 4) __stcg(mine + (size_t)((c0 + q) * kPlanes + 1) * 128, b[q]);
            }
          }
        }
        tc_fence_before();
        __threadfence();
        __syncwarp();
        if (lane == 0) mbar_arrive(acce0 + 8 * buf);
        int32_t* tk = p.ticket + (size_t)(grp[gi].tile0 + nt) * 4 + quad;
        int last = 0;
        if (lane == 0) last = atomicAdd(tk, 1) == un.n_z - 1;
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {
          __threadfence();
          const float* all = p.part + (size_t)slot0 * kDecSlotFloats + quad * 32 + lane;
          for (int c = 0; c < n_cols; ++c) {
            float a = 0.0f, b = 0.0f;
            for (int z = 0; z < un.n_z; ++z) {             // ascending slice order
              a += __ldcg(all + (size_t)z * kDecSlotFloats + (size_t)(c * kPlanes) * 128);
              if (MODE == 4) b += __ldcg(all + (size_t)z * kDecSlotFloats + (size_t)(c * kPlanes + 1) * 128);
            }
            finish(c, a, b);
          }
          if (lane == 0) *tk = 0;                          // ready for the next launch
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ----------------------------------------------------------------------------- host
// Both modes of one (weights, NT) family: dynamic shared memory above 48 KB has to be allowed per kernel.
template <bool W8, int NT>
inline void decode_allow_smem(cudaError_t* e) {
  auto allow = [&](auto kernel, int bytes) {
    if (*e == cudaSuccess) *e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  };
  allow(umma_decode_kernel<4, false, W8, NT>, decode_smem_bytes<4, W8, NT>());
  allow(umma_decode_kernel<5, false, W8, NT>, decode_smem_bytes<5, W8, NT>());
  if constexpr (NT <= kDecMaxRows) {
    allow(umma_decode_kernel<4, true, W8, NT>, decode_smem_bytes<4, W8, NT>());
    allow(umma_decode_kernel<5, true, W8, NT>, decode_smem_bytes<5, W8, NT>());
  }
}

// One decode GEMM: the instantiation for (mode, weights, NT), K-splitting or plain.
template <int MODE, bool W8, int NT>
inline void decode_launch(bool dep, bool split, int n_sms, cudaStream_t st, const CUtensorMap& w_s, const CUtensorMap& w_r,
                          const CUtensorMap& x_s, const CUtensorMap& x_r, const DecodeArgs& a) {
  constexpr int smem = decode_smem_bytes<MODE, W8, NT>();
  if constexpr (NT <= kDecMaxRows) {
    if (split) {
      launch_kernel(dep, umma_decode_kernel<MODE, true, W8, NT>, dim3(n_sms), dim3(kUmmaThreads), smem, st, w_s, w_r, x_s, x_r, a);
      return;
    }
  }
  launch_kernel(dep, umma_decode_kernel<MODE, false, W8, NT>, dim3(n_sms), dim3(kUmmaThreads), smem, st, w_s, w_r, x_s, x_r, a);
}

struct DecodePlan {
  bool built = false;
  float* part = nullptr;            // kDecMaxSlots slots of slice partials (caller-owned workspace)
  int32_t* ticket = nullptr;        // zeroed once; the kernels leave it zero
  CUtensorMap w_gu, w_gu_r;         // stacked gate/up rows, box 64 k x tile rows (shared, routed groups) x 2 planes
  int tile_rows_s = 128, tile_rows_r = 128;
  CUtensorMap wd_s, wd_r;           // W_down blocks, 128-channel boxes
  // token tiles come in boxes of 16, 32, 64 or 128 rows (index 0..3): a launch uses the smallest that holds
  // its rows, so that a stage carries as little besides weights as possible
  CUtensorMap x_rows[4];            // x (bound per forward for a plain layer)
  CUtensorMap h_s[4], h_r[4];       // H
  // FP8 weights (set by decode_plan_attach_fp8): codes in the packed layouts, boxes of 128 k x 128 rows;
  // E4M3 planes [2][rows][cols] of the token rows (x, H_s, H_r) with their per-row scales
  bool fp8 = false;
  CUtensorMap w_gu8, w_gu8_r, wd8_s, wd8_r;
  const float *scale_gu = nullptr, *scale_d = nullptr;
  uint8_t *xq = nullptr, *hq_s = nullptr, *hq_r = nullptr;
  float *x_scale = nullptr, *hs_scale = nullptr, *hr_scale = nullptr;
  size_t xq_rows = 0, hr_rows = 0;               // rows per plane of xq / hq_s, and of hq_r
  CUtensorMap xq_map[3], hqs_map[3], hqr_map[3]; // token boxes of 16 / 32 / 64 rows
  const void* x_ptr = nullptr;                   // x of this forward (decode_bind_x)
};

// Neurons per gate/up tile of a group of this width: 128 when that pads the width by at most 5 %, else the multiple
// of 16 in [96, 128) with the least padding (448 -> 112: four exact tiles instead of 14 % of wasted weight rows).
inline int decode_pick_tile_rows(int width) {
  if (width <= 0 || (long long)((width + 127) / 128 * 128) * 100 <= (long long)width * 105) return 128;
  int best = 128, best_pad = (width + 127) / 128 * 128;
  for (int tr = 112; tr >= 96; tr -= 16) {
    const int pad = (width + tr - 1) / tr * tr;
    if (pad < best_pad) { best = tr; best_pad = pad; }
  }
  return best;
}

inline bool decode_plan_create(UmmaPlan* P, DecodePlan* D) {
  const UmmaShape& s = P->shape;
  const UmmaBuffers& buf = P->buf;
  const size_t d = s.d, rows_w = (size_t)s.n_outer * s.d_ff;
  bool ok = true;
  D->tile_rows_s = decode_pick_tile_rows(P->has_s ? s.shared_width : 0);
  D->tile_rows_r = decode_pick_tile_rows(P->has_r ? s.m : 0);
  for (int r = 0; r < 2 && ok; ++r) {
    const cuuint64_t dims[3] = {d, rows_w, 2};
    const cuuint64_t str[2] = {d * 2, rows_w * d * 2};
    const cuuint32_t box[3] = {kUmmaBK, (cuuint32_t)(r ? D->tile_rows_r : D->tile_rows_s), 2};
    ok = umma_encode(P, r ? &D->w_gu_r : &D->w_gu, buf.w_gate_up, 3, dims, str, box, "gate/up weights (decode)");
  }
  if (ok && P->has_s) {
    const cuuint64_t dims[3] = {(cuuint64_t)s.shared_width, d, (cuuint64_t)s.n_outer};
    const cuuint64_t str[2] = {(cuuint64_t)s.shared_width * 2, d * s.d_ff * 2};
    const cuuint32_t box[3] = {kUmmaBK, 128, 1};
    ok = umma_encode(P, &D->wd_s, buf.w_down, 3, dims, str, box, "shared W_down (decode)") &&
         umma_encode_rows(P, &D->h_s[0], buf.h_s, s.max_outer_rows, s.shared_width, 16, "H shared (decode)") &&
         umma_encode_rows(P, &D->h_s[1], buf.h_s, s.max_outer_rows, s.shared_width, 32, "H shared (decode)") &&
         umma_encode_rows(P, &D->h_s[2], buf.h_s, s.max_outer_rows, s.shared_width, 64, "H shared (decode)") &&
         umma_encode_rows(P, &D->h_s[3], buf.h_s, s.max_outer_rows, s.shared_width, 128, "H shared (decode)");
  }
  if (ok && P->has_r) {
    const cuuint64_t dims[4] = {(cuuint64_t)s.m, d, (cuuint64_t)s.n_r, (cuuint64_t)s.n_outer};
    const cuuint64_t str[3] = {(cuuint64_t)s.m * 2, d * s.m * 2, d * s.d_ff * 2};
    const cuuint32_t box[4] = {kUmmaBK, 128, 1, 1};
    ok = umma_encode(P, &D->wd_r, (const bf16*)buf.w_down + (size_t)s.shared_width * d, 4, dims, str, box,
                     "routed W_down (decode)") &&
         umma_encode_rows(P, &D->h_r[0], buf.h_r, s.max_routed_rows, s.m, 16, "H routed (decode)") &&
         umma_encode_rows(P, &D->h_r[1], buf.h_r, s.max_routed_rows, s.m, 32, "H routed (decode)") &&
         umma_encode_rows(P, &D->h_r[2], buf.h_r, s.max_routed_rows, s.m, 64, "H routed (decode)") &&
         umma_encode_rows(P, &D->h_r[3], buf.h_r, s.max_routed_rows, s.m, 128, "H routed (decode)");
  }
  if (ok && buf.x_fixed)
    ok = umma_encode_rows(P, &D->x_rows[0], buf.x_fixed, s.max_outer_rows, d, 16, "outer rows of x (decode)") &&
         umma_encode_rows(P, &D->x_rows[1], buf.x_fixed, s.max_outer_rows, d, 32, "outer rows of x (decode)") &&
         umma_encode_rows(P, &D->x_rows[2], buf.x_fixed, s.max_outer_rows, d, 64, "outer rows of x (decode)") &&
         umma_encode_rows(P, &D->x_rows[3], buf.x_fixed, s.max_outer_rows, d, 128, "outer rows of x (decode)");
  if (!ok) return false;
  for (int i = 0; i < 4; ++i) {
    if (!P->has_r) { D->wd_r = D->wd_s; D->h_r[i] = D->h_s[i]; }
    if (!P->has_s) { D->wd_s = D->wd_r; D->h_s[i] = D->h_r[i]; }
  }
  cudaError_t e = cudaSuccess;
  decode_allow_smem<false, kDecMaxRows>(&e);
  decode_allow_smem<false, kDecWideRows>(&e);
  if (e != cudaSuccess) {
    snprintf(P->error, sizeof(P->error), "cudaFuncSetAttribute (decode): %s", cudaGetErrorString(e));
    return false;
  }
  D->built = true;
  return true;
}

// FP8 buffers of a quantised layer, all owned by the caller.  Weight codes in the packed layouts (maps: one
// byte per element, boxes of 128 k x 128 rows, 128-byte swizzle; d, m and the shared width must be multiples
// of 16 for the TMA strides); token planes [2][rows][cols] for x (xq_rows rows), H_s (xq_rows) and H_r (hr_rows).
struct DecodeFp8Buffers {
  const void *w_gu8, *wd8;
  const float *scale_gu, *scale_d;
  uint8_t *xq, *hq_s, *hq_r;
  float *x_scale, *hs_scale, *hr_scale;
  size_t xq_rows, hr_rows;
};

inline bool decode_plan_attach_fp8(UmmaPlan* P, DecodePlan* D, const DecodeFp8Buffers& f) {
  const UmmaShape& s = P->shape;
  const size_t d = s.d, rows_w = (size_t)s.n_outer * s.d_ff;
  auto encode8 = [&](CUtensorMap* tm, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* str,
                     const cuuint32_t* box, const char* what) {
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    const CUresult r = P->encode(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, (cuuint32_t)rank, const_cast<void*>(base), dims, str,
                                 box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
      snprintf(P->error, sizeof(P->error), "cuTensorMapEncodeTiled(%s) failed with CUresult %d", what, (int)r);
      return false;
    }
    return true;
  };
  // token planes [2][rows][cols]: box 128 k x (16 << i) rows x 1 plane
  auto encode_planes = [&](CUtensorMap* maps, const void* base, size_t rows, size_t cols, const char* what) {
    for (int i = 0; i < 3; ++i) {
      const cuuint64_t dims[3] = {cols, rows, 2};
      const cuuint64_t str[2] = {cols, rows * cols};
      const cuuint32_t box[3] = {2 * kUmmaBK, (cuuint32_t)(16 << i), 1};
      if (!encode8(&maps[i], base, 3, dims, str, box, what)) return false;
    }
    return true;
  };
  bool ok = true;
  for (int r = 0; r < 2 && ok; ++r) {
    const cuuint64_t dims[3] = {d, rows_w, 2};
    const cuuint64_t str[2] = {d, rows_w * d};
    const cuuint32_t box[3] = {2 * kUmmaBK, (cuuint32_t)(r ? D->tile_rows_r : D->tile_rows_s), 2};
    ok = encode8(r ? &D->w_gu8_r : &D->w_gu8, f.w_gu8, 3, dims, str, box, "FP8 gate/up weights");
  }
  if (ok) ok = encode_planes(D->xq_map, f.xq, f.xq_rows, d, "E4M3 planes of x");
  if (ok && P->has_s) {
    const cuuint64_t dims[3] = {(cuuint64_t)s.shared_width, d, (cuuint64_t)s.n_outer};
    const cuuint64_t str[2] = {(cuuint64_t)s.shared_width, d * s.d_ff};
    const cuuint32_t box[3] = {2 * kUmmaBK, 128, 1};
    ok = encode8(&D->wd8_s, f.wd8, 3, dims, str, box, "FP8 shared W_down") &&
         encode_planes(D->hqs_map, f.hq_s, f.xq_rows, (size_t)s.shared_width, "E4M3 planes of H shared");
  }
  if (ok && P->has_r) {
    const cuuint64_t dims[4] = {(cuuint64_t)s.m, d, (cuuint64_t)s.n_r, (cuuint64_t)s.n_outer};
    const cuuint64_t str[3] = {(cuuint64_t)s.m, d * s.m, d * s.d_ff};
    const cuuint32_t box[4] = {2 * kUmmaBK, 128, 1, 1};
    ok = encode8(&D->wd8_r, (const uint8_t*)f.wd8 + (size_t)s.shared_width * d, 4, dims, str, box, "FP8 routed W_down") &&
         encode_planes(D->hqr_map, f.hq_r, f.hr_rows, (size_t)s.m, "E4M3 planes of H routed");
  }
  if (!ok) return false;
  for (int i = 0; i < 3; ++i) {
    if (!P->has_r) { D->wd8_r = D->wd8_s; D->hqr_map[i] = D->hqs_map[i]; }
    if (!P->has_s) { D->wd8_s = D->wd8_r; D->hqs_map[i] = D->hqr_map[i]; }
  }
  cudaError_t e = cudaSuccess;
  decode_allow_smem<true, kDecMaxRows>(&e);
  if (e != cudaSuccess) {
    snprintf(P->error, sizeof(P->error), "cudaFuncSetAttribute (FP8 decode): %s", cudaGetErrorString(e));
    return false;
  }
  D->scale_gu = f.scale_gu; D->scale_d = f.scale_d;
  D->xq = f.xq; D->hq_s = f.hq_s; D->hq_r = f.hq_r;
  D->x_scale = f.x_scale; D->hs_scale = f.hs_scale; D->hr_scale = f.hr_scale;
  D->xq_rows = f.xq_rows; D->hr_rows = f.hr_rows;
  D->fp8 = true;
  return true;
}

// Index of the smallest token box (16 << index rows) that holds n_rows rows.
inline int decode_box_index(int n_rows) { return n_rows <= 16 ? 0 : (n_rows <= 32 ? 1 : (n_rows <= 64 ? 2 : 3)); }

inline bool decode_bind_x(UmmaPlan* P, DecodePlan* D, const void* x_rows, int n_rows) {
  D->x_ptr = x_rows;
  if (P->buf.x_fixed) return true;
  const int bi = decode_box_index(n_rows);
  return umma_encode_rows(P, &D->x_rows[bi], x_rows, (size_t)n_rows, (size_t)P->shape.d, 16 << bi, "x (decode)");
}

// FP8 layers: the E4M3 planes of this forward's x rows (needs nothing from the router, so it is launched first).
inline int decode_split_x(UmmaPlan* P, DecodePlan* D, int n_rows, cudaStream_t st, bool dep) {
  SplitSegment a{(const bf16*)D->x_ptr, n_rows, P->shape.d, (long long)P->shape.d, D->xq, (long long)D->xq_rows, D->x_scale};
  SplitSegment none{nullptr, 0, 0, 0, nullptr, 0, nullptr};
  launch_kernel(dep, split_rows_e4m3_kernel, dim3(n_rows), dim3(128), 0, st, a, none);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

// Both decode GEMMs; requires umma_bind_x and decode_bind_x for this forward and n_rows <=
// kDecMaxRows outer rows (kDecWideRows with bf16 weights: the wide kernels, which never split K).  The K-splitting form of a kernel is launched only when the device-side
// rule would split some group even if the largest possible set of experts were active for
// n_rows rows (fewer active experts only split more).  Returns launches or -1.
inline int decode_forward(UmmaPlan* P, DecodePlan* D, const GroupRows* gr, int n_rows, int32_t* err_word,
                          cudaStream_t st, cudaEvent_t mid, bool dep = false, bool gate_up_only = false) {
  const UmmaShape& s = P->shape;
  const long long act_s = P->has_s ? (s.n_outer < n_rows ? s.n_outer : n_rows) : 0;
  const long long all_r = (long long)s.n_outer * s.n_r, picks = (long long)n_rows * s.n_k;
  const long long act_r = P->has_r ? (all_r < picks ? all_r : picks) : 0;
  const int bk = D->fp8 ? 2 * kUmmaBK : kUmmaBK;               // k per stage, as in the kernel
  auto splits = [&](long long all_kb, int kb_max) {
    long long per_cta = (all_kb + P->n_sms - 1) / P->n_sms;
    if (per_cta < kDecMinSliceKb * kUmmaBK / bk) per_cta = kDecMinSliceKb * kUmmaBK / bk;
    return D->part != nullptr && P->n_sms <= kDecMaxSlots && kb_max / per_cta >= 2;
  };
  const int kb_d = (s.d + bk - 1) / bk, kb_s = (s.shared_width + bk - 1) / bk, kb_m = (s.m + bk - 1) / bk;
  const bool wide = n_rows > kDecMaxRows;
  const int trs = D->tile_rows_s, trr = D->tile_rows_r;
  const bool split1 = !wide && splits((act_s * ((s.shared_width + trs - 1) / trs) + act_r * ((s.m + trr - 1) / trr)) * kb_d, kb_d);
  const bool split2 = !wide && splits((long long)((s.d + 127) / 128) * (act_s * kb_s + act_r * kb_m),
                             (act_s && kb_s > kb_m) || !act_r ? kb_s : kb_m);
  DecodeArgs a{};
  a.gs = P->buf.gs_dev; a.gr = gr; a.n_groups = P->n_groups; a.n_outer = s.n_outer; a.n_r = s.n_r;
  a.d = s.d; a.row_token = P->buf.row_token; a.err = err_word;
  a.part = D->part; a.ticket = D->ticket;
  const int bi = decode_box_index(n_rows);
  a.tok_box_rows = 16 << bi;
  // plain layer: group 0 is the shared expert and its rows are the whole batch, known here
  a.tile_rows_s = trs; a.tile_rows_r = trr;
  a.early_units = (s.n_outer == 1 && P->has_s) ? (s.shared_width + trs - 1) / trs : 0;
  a.n_rows_plain = n_rows;
  a.scale_gu = D->scale_gu; a.scale_d = D->scale_d; a.rows_w = (long long)s.n_outer * s.d_ff;
  a.out_s = (bf16*)P->buf.h_s; a.out_r = (bf16*)P->buf.h_r; a.ld_out_s = s.shared_width; a.ld_out_r = s.m;
  int extra = 0;
  a.tok_scale_s = D->x_scale; a.tok_scale_r = D->x_scale;
  const int sms = P->n_sms;
  if (wide) decode_launch<4, false, kDecWideRows>(dep, false, sms, st, D->w_gu, D->w_gu_r, D->x_rows[bi], D->x_rows[bi], a);
  else if (D->fp8)          // the layer holds FP8 codes of its expert weights: stream those (half the bytes)
    decode_launch<4, true, kDecMaxRows>(dep, split1, sms, st, D->w_gu8, D->w_gu8_r, D->xq_map[bi], D->xq_map[bi], a);
  else decode_launch<4, false, kDecMaxRows>(dep, split1, sms, st, D->w_gu, D->w_gu_r, D->x_rows[bi], D->x_rows[bi], a);
  if (mid) cudaEventRecord(mid, st);
  a.out_s = (bf16*)P->buf.y_s; a.out_r = (bf16*)P->buf.y_r; a.ld_out_s = s.d; a.ld_out_r = s.d;
  if (gate_up_only) {
  } else if (wide) {
    decode_launch<5, false, kDecWideRows>(dep, false, sms, st, D->wd_s, D->wd_r, D->h_s[bi], D->h_r[bi], a);
  } else if (D->fp8) {
    // E4M3 planes of H (shared rows, then routed rows), then the down GEMM on them
    const int rows_r = P->has_r ? n_rows * s.n_k : 0, rows_s = P->has_s ? n_rows : 0;
    SplitSegment hs{(const bf16*)P->buf.h_s, rows_s, s.shared_width, (long long)s.shared_width, D->hq_s,
                    (long long)D->xq_rows, D->hs_scale};
    SplitSegment hr{(const bf16*)P->buf.h_r, rows_r, s.m, (long long)s.m, D->hq_r, (long long)D->hr_rows, D->hr_scale};
    launch_kernel(dep, split_rows_e4m3_kernel, dim3(rows_s + rows_r), dim3(128), 0, st, hs, hr);
    extra = 1;
    a.tok_scale_s = D->hs_scale; a.tok_scale_r = D->hr_scale;
    decode_launch<5, true, kDecMaxRows>(dep, split2, sms, st, D->wd8_s, D->wd8_r, D->hqs_map[bi], D->hqr_map[bi], a);
  } else {
    decode_launch<5, false, kDecMaxRows>(dep, split2, sms, st, D->wd_s, D->wd_r, D->h_s[bi], D->h_r[bi], a);
  }
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    snprintf(P->error, sizeof(P->error), "decode GEMM launch: %s", cudaGetErrorString(e));
    return -1;
  }
  return (gate_up_only ? 1 : 2) + extra;
}

}  // namespace cmoe
