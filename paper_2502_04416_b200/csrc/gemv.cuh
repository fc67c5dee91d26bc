// Expert FFN for a single token row of a plain layer (single-sequence decode).  With one row
// a tensor-core tile is almost empty and a launch is mostly ramp and tail, so the weights are
// streamed by plain 16-byte loads that bypass L1 instead: every warp of the grid has a few hundred
// bytes per lane in flight a microsecond after the launch, the multiply-adds run on the CUDA cores
// (one per weight, far below what the load stream leaves room for) and the sums are fp32.
// Whole weight rows are contiguous in the packed layouts, so a warp reads long runs of DRAM pages.
//
//   gemv_gate_up_kernel:       H[r, n] = Swish(w_gate[n] . x_r) * (w_up[n] . x_r)   (Eq. ori_ffn_method)
//       one warp per neuron of an active group, both weight rows at once; the rows r are the
//       group's rows (shared group: every token; routed group: the tokens that selected it).
//   gemv_down_combine_kernel:  out[t, c] = Y_s[t, c] + sum_j g[t, j] Y_{e_j}[t, c],  Y_e[t, c] = W_down^e[c] . H_e[t]
//       (Eq. moe_output) one warp per pair of output channels, over all active groups in group
//       order, each group's products times its row's gate (lane-level sums, one warp reduction per
//       channel at the end); fp32, one rounding: the down projection and the gate-weighted combine
//       are one launch and Y never reaches memory.
// FP8 = true streams the E4M3 codes of a quantised layer (one byte per weight) and multiplies the
// sums by the per-row power-of-two scales; the token rows stay bf16.
// The kernels are written for TT rows and instantiated for one: measured on 7B-, 8B- and 13B-shaped
// layers, two rows already run faster on the tensor-core streamers (61 vs 64, 55 vs 60, 64 vs 80 us),
// one row is faster here (40.4 vs 54.3, 37.8 vs 45.3, 50.7 vs 59.6 us per forward; with FP8 weights
// 35.0 vs 43.2, 35.0 vs 43.2, 45.6 vs 48.1).
#pragma once

#include "common.cuh"
#include "fp8.cuh"

namespace cmoe {

constexpr int kGemvMaxRows = 1;
constexpr int kGemvThreads = 256;
constexpr int kGemvWarps = kGemvThreads / 32;
constexpr int kGemvMaxGroups = 64;         // group tables in shared memory
constexpr int kGemvCH = 2;                 // output channels per warp pass of the down kernel

struct GemvArgs {
  const GroupStatic* gs;
  const GroupRows* gr;
  int n_groups, d, n_rows, n_k;
  const bf16* x;              // [n_rows, d]
  const void* w_gate_up;      // [2][rows_w][d] bf16, or E4M3 codes
  const void* w_down;         // packed [d, width] blocks (GroupStatic::wd_offset), bf16 or codes
  long long rows_w;
  const float* scale_gu;      // FP8: [2][rows_w]
  const float* scale_d;       // FP8: [n_groups][d]
  bf16* h_s;                  // [n_rows, ld_h_s]
  bf16* h_r;                  // [n_rows * n_k, ld_h_r]
  int ld_h_s, ld_h_r;
  const int32_t* row_of;      // [n_rows, n_k] -> routed row
  const float* topk_gate;     // [n_rows, n_k]
  bf16* out;                  // [n_rows, d]
};

// 16 (8) bytes that are read once: no L1 allocation, so the token rows stay cached.
__device__ __forceinline__ uint4 ld_stream16(const void* p) {
  uint4 r;
  asm("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
  return r;
}
__device__ __forceinline__ uint2 ld_stream8(const void* p) {
  uint2 r;
  asm("ld.global.nc.L1::no_allocate.v2.u32 {%0, %1}, [%2];" : "=r"(r.x), "=r"(r.y) : "l"(p));
  return r;
}

// Eight weights of one row chunk: bf16 (16 bytes) or E4M3 codes (8 bytes); as floats after unpack.
template <bool FP8> struct GemvChunk;
template <> struct GemvChunk<false> {
  uint4 raw;
  __device__ __forceinline__ void load(const void* chunk0, int chunk) { raw = ld_stream16((const uint4*)chunk0 + chunk); }
  __device__ __forceinline__ void unpack(float (&w)[8]) const {
    const uint32_t v[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) { w[2 * i] = __uint_as_float(v[i] << 16); w[2 * i + 1] = __uint_as_float(v[i] & 0xffff0000u); }
  }
};
template <> struct GemvChunk<true> {
  uint2 raw;
  __device__ __forceinline__ void load(const void* chunk0, int chunk) { raw = ld_stream8((const uint2*)chunk0 + chunk); }
  __device__ __forceinline__ void unpack(float (&w)[8]) const {
    const uint32_t v[2] = {raw.x, raw.y};
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const float2 a = e4m3x2_to_f32x2((uint16_t)(v[i] & 0xffffu)), b = e4m3x2_to_f32x2((uint16_t)(v[i] >> 16));
      w[4 * i] = a.x; w[4 * i + 1] = a.y; w[4 * i + 2] = b.x; w[4 * i + 3] = b.y;
    }
  }
};

// The groups with rows in this forward, in shared memory: what the kernels need of them, the token of
// each of their rows and its gate (1 for a shared group, g[t, j] for a routed one, 0 where there is no row).
// Every global load of the listing is independent of the others (a routed group finds its rows by looking
// at all n_rows * n_k selections), so the listing costs one memory latency.
template <int TT>
struct GemvGroups {
  int32_t n, total;                           // active groups; sum of their widths
  int32_t live[kGemvMaxGroups];
  int32_t id[kGemvMaxGroups], start[kGemvMaxGroups + 1];
  int32_t width[kGemvMaxGroups], w_row0[kGemvMaxGroups], is_shared[kGemvMaxGroups];
  int32_t row0[kGemvMaxGroups], count[kGemvMaxGroups];
  long long wd_offset[kGemvMaxGroups];
  int32_t tok[kGemvMaxGroups][TT];
  float gate[kGemvMaxGroups][TT];
};
template <int TT>
__device__ __forceinline__ void gemv_list_groups(const GemvArgs& p, GemvGroups<TT>& L) {
  const int g = threadIdx.x;
  GroupStatic gs{};
  GroupRows gr{};
  int32_t sel_row[TT * 16];
  float sel_gate[TT * 16];
  const int n_sel = p.n_rows * p.n_k;
  if (g < p.n_groups) {
    gs = p.gs[g]; gr = p.gr[g];
#pragma unroll
    for (int i = 0; i < TT * 16; ++i) {
      sel_row[i] = i < n_sel ? __ldcg(p.row_of + i) : -1;
      sel_gate[i] = i < n_sel ? __ldcg(p.topk_gate + i) : 0.0f;
    }
    L.live[g] = (gr.count > 0 && gs.width > 0) ? 1 : 0;
  }
  __syncthreads();
  if (g < p.n_groups && L.live[g]) {
    int pos = 0;
    for (int q = 0; q < g; ++q) pos += L.live[q];
    L.id[pos] = g; L.width[pos] = gs.width; L.w_row0[pos] = gs.w_row0; L.is_shared[pos] = gs.is_shared;
    L.row0[pos] = gr.row0; L.count[pos] = gr.count; L.wd_offset[pos] = gs.wd_offset;
#pragma unroll
    for (int j = 0; j < TT; ++j) {
      int t = 0;
      float gt = 0.0f;
      if (j < gr.count) {
        if (gs.is_shared) {
          t = gr.row0 + j; gt = 1.0f;
        } else {
#pragma unroll
          for (int i = 0; i < TT * 16; ++i)
            if (sel_row[i] == gr.row0 + j) { t = i / p.n_k; gt = sel_gate[i]; }
        }
      }
      L.tok[pos][j] = t; L.gate[pos][j] = gt;
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int n = 0, run = 0;
    for (int q = 0; q < p.n_groups; ++q) n += L.live[q];
    for (int a = 0; a < n; ++a) { L.start[a] = run; run += L.width[a]; }
    L.start[n] = run; L.n = n; L.total = run;
  }
  __syncthreads();
}

constexpr int kGemvEarly = 3;              // shared-expert neurons a warp may finish before the router has

template <int TT, bool FP8>
__global__ void __launch_bounds__(kGemvThreads, 4)
gemv_gate_up_kernel(const GemvArgs p) {
  __shared__ GemvGroups<TT> L;
  grid_dep_trigger();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_warps = gridDim.x * kGemvWarps, gw = blockIdx.x * kGemvWarps + warp;
  const int chunks = p.d >> 3;                         // 8 weights per chunk
  constexpr int esz = FP8 ? 1 : 2;
  // gate and up pre-activations of one neuron (packed weight row wrow) for the token rows xr[0 .. TT)
  auto neuron = [&](size_t wrow, const bf16* const (&xr)[TT], float (&g)[TT], float (&u)[TT]) {
    const char* wg = (const char*)p.w_gate_up + wrow * p.d * esz;
    const char* wu = wg + (size_t)p.rows_w * p.d * esz;
    float ag[TT], au[TT];
#pragma unroll
    for (int j = 0; j < TT; ++j) { ag[j] = 0.0f; au[j] = 0.0f; }
#pragma unroll 4
    for (int c = lane; c < chunks; c += 32) {
      GemvChunk<FP8> cg, cu;
      cg.load(wg, c);
      cu.load(wu, c);
      float fg[8], fu[8];
      cg.unpack(fg);
      cu.unpack(fu);
#pragma unroll
      for (int j = 0; j < TT; ++j) {
        float xv[8];
        load8(xr[j] + 8 * c, xv);
#pragma unroll
        for (int q = 0; q < 8; ++q) { ag[j] = fmaf(fg[q], xv[q], ag[j]); au[j] = fmaf(fu[q], xv[q], au[j]); }
      }
    }
    float sg = 1.0f, su = 1.0f;
    if constexpr (FP8) { sg = __ldg(p.scale_gu + wrow); su = __ldg(p.scale_gu + p.rows_w + wrow); }
#pragma unroll
    for (int j = 0; j < TT; ++j) { g[j] = warp_sum(ag[j]) * sg; u[j] = warp_sum(au[j]) * su; }
  };
  // Head start: group 0 of a plain layer with a shared expert is that expert, its rows are all the
  // tokens, and neither its weights nor x depend on the router.  Each warp finishes up to kGemvEarly of
  // its neurons while the router (the preceding kernel) runs, keeps the results in registers, and
  // stores them after the wait, when the previous reader of H has certainly finished.
  const GroupStatic g0 = p.gs[0];
  const int early_width = (g0.is_shared && p.n_rows <= TT) ? g0.width : 0;
  float early_h[kGemvEarly][TT];
#pragma unroll
  for (int i = 0; i < kGemvEarly; ++i) {
    const int n = gw + i * n_warps;
    if (n < early_width) {
      const bf16* xr[TT];
#pragma unroll
      for (int j = 0; j < TT; ++j) xr[j] = p.x + (size_t)(j < p.n_rows ? j : 0) * p.d;
      float g[TT], u[TT];
      neuron((size_t)(g0.w_row0 + n), xr, g, u);
#pragma unroll
      for (int j = 0; j < TT; ++j) early_h[i][j] = g[j] / (1.0f + __expf(-g[j])) * u[j];
    }
  }
  grid_dep_wait();
#pragma unroll
  for (int i = 0; i < kGemvEarly; ++i) {
    const int n = gw + i * n_warps;
    if (n < early_width && lane == 0) {
#pragma unroll
      for (int j = 0; j < TT; ++j)
        if (j < p.n_rows) p.h_s[(size_t)j * p.ld_h_s + n] = __float2bfloat16_rn(early_h[i][j]);
    }
  }
  gemv_list_groups(p, L);
  // the active groups' neurons, concatenated; group 0 comes first, so an item below early_width of the first
  // kGemvEarly rounds is one of those finished above
  int round = 0;
  for (int item = gw; item < L.total; item += n_warps, ++round) {
    if (round < kGemvEarly && item < early_width) continue;
    int lo = 0, hi = L.n;
    while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (L.start[mid] <= item) lo = mid; else hi = mid; }
    const int n = item - L.start[lo];
    const int count = L.count[lo] < TT ? L.count[lo] : TT;
    const bf16* xr[TT];
#pragma unroll
    for (int j = 0; j < TT; ++j) xr[j] = p.x + (size_t)L.tok[lo][j < count ? j : 0] * p.d;
    float g[TT], u[TT];
    neuron((size_t)(L.w_row0[lo] + n), xr, g, u);
    if (lane == 0) {
#pragma unroll
      for (int j = 0; j < TT; ++j)
        if (j < count) {
          bf16* dst = L.is_shared[lo] ? p.h_s + (size_t)(L.row0[lo] + j) * p.ld_h_s : p.h_r + (size_t)(L.row0[lo] + j) * p.ld_h_r;
          dst[n] = __float2bfloat16_rn(g[j] / (1.0f + __expf(-g[j])) * u[j]);
        }
    }
  }
}

template <int TT, bool FP8>
__global__ void __launch_bounds__(kGemvThreads, 4)
gemv_down_combine_kernel(const GemvArgs p) {
  constexpr int CH = kGemvCH, esz = FP8 ? 1 : 2;
  __shared__ GemvGroups<TT> L;
  grid_dep_wait();
  grid_dep_trigger();
  gemv_list_groups(p, L);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_warps = gridDim.x * kGemvWarps, gw = blockIdx.x * kGemvWarps + warp;
  // One pass = CH output channels; per active group one partial dot product per (channel, row), reduced over
  // the warp and added, times the row's gate, to its token's sum.
  for (int c0 = gw * CH; c0 < p.d; c0 += n_warps * CH) {
    float out_acc[CH][TT];
#pragma unroll
    for (int h = 0; h < CH; ++h)
#pragma unroll
      for (int t = 0; t < TT; ++t) out_acc[h][t] = 0.0f;
    for (int a = 0; a < L.n; ++a) {
      const int width = L.width[a], row0 = L.row0[a], count = L.count[a] < TT ? L.count[a] : TT;
      const bool is_shared = L.is_shared[a] != 0;
      const bf16* hr[TT];
#pragma unroll
      for (int j = 0; j < TT; ++j) {
        const int jj = j < count ? j : 0;
        hr[j] = is_shared ? p.h_s + (size_t)(row0 + jj) * p.ld_h_s : p.h_r + (size_t)(row0 + jj) * p.ld_h_r;
      }
      const char* w0 = (const char*)p.w_down + ((size_t)L.wd_offset[a] + (size_t)c0 * width) * esz;
      const int chunks = width >> 3;
      float acc[CH][TT];
#pragma unroll
      for (int h = 0; h < CH; ++h)
#pragma unroll
        for (int j = 0; j < TT; ++j) acc[h][j] = 0.0f;
#pragma unroll 4
      for (int c = lane; c < chunks; c += 32) {
        GemvChunk<FP8> cw[CH];
#pragma unroll
        for (int h = 0; h < CH; ++h) cw[h].load(w0 + (size_t)h * width * esz, c);    // rows c0 + h (d is even)
        float hv[TT][8];
#pragma unroll
        for (int j = 0; j < TT; ++j) load8(hr[j] + 8 * c, hv[j]);
#pragma unroll
        for (int h = 0; h < CH; ++h) {
          float fw[8];
          cw[h].unpack(fw);
#pragma unroll
          for (int j = 0; j < TT; ++j)
#pragma unroll
            for (int q = 0; q < 8; ++q) acc[h][j] = fmaf(fw[q], hv[j][q], acc[h][j]);
        }
      }
#pragma unroll
      for (int h = 0; h < CH; ++h) {
        float sc = 1.0f;
        if constexpr (FP8) sc = __ldg(p.scale_d + (size_t)L.id[a] * p.d + c0 + h);
#pragma unroll
        for (int j = 0; j < TT; ++j) {
          const float y = acc[h][j] * sc * L.gate[a][j];      // gate 0: the group has no j-th row
          const int t = L.tok[a][j];
#pragma unroll
          for (int tt = 0; tt < TT; ++tt) out_acc[h][tt] += (t == tt) ? y : 0.0f;
        }
      }
    }
#pragma unroll
    for (int h = 0; h < CH; ++h)
#pragma unroll
      for (int tt = 0; tt < TT; ++tt) {
        const float y = warp_sum(out_acc[h][tt]);
        if (lane == 0 && tt < p.n_rows) p.out[(size_t)tt * p.d + c0 + h] = __float2bfloat16_rn(y);
      }
  }
}

// Whether a plain bf16 layer's forward of n_rows rows can take this path.
struct GemvPlan { int unused; };
inline bool gemv_plan(int n_rows, int n_outer, int n_groups, int n_k, int n_r, int d, int shared_width, int m, bool has_s,
                      bool fp8, GemvPlan* out) {
  if (n_rows < 1 || n_rows > kGemvMaxRows || n_outer != 1 || n_groups > kGemvMaxGroups || n_k > 16) return false;
  const int align = fp8 ? 16 : 8;                  // 16-byte (8-byte: codes) chunks of 8 weights, rows aligned to them
  if (d % align || shared_width % align || m % align || d % kGemvCH) return false;
  (void)n_r; (void)has_s;
  out->unused = 0;
  return true;
}

// Both launches (or the first only); returns the launches made, or -1.
inline int gemv_forward(const GemvArgs& a, const GemvPlan& plan, bool fp8, int n_sms, cudaStream_t st, cudaEvent_t mid,
                        bool dep, bool gate_up_only) {
  const dim3 block(kGemvThreads);
  const dim3 grid1(4 * n_sms);
  // down + combine: a warp takes kGemvCH channels per pass; as many passes as four blocks per SM need, evenly filled
  const int warps = 4 * n_sms * kGemvWarps, pairs = a.d / kGemvCH;
  const int passes = (pairs + warps - 1) / warps;
  const dim3 grid2(((pairs + passes - 1) / passes + kGemvWarps - 1) / kGemvWarps);
#define CMOE_GEMV(TT, F8)                                                                                          \
  do {                                                                                                             \
    launch_kernel(dep, gemv_gate_up_kernel<TT, F8>, grid1, block, 0, st, a);                                       \
    if (mid) cudaEventRecord(mid, st);                                                                             \
    if (!gate_up_only) launch_kernel(dep, gemv_down_combine_kernel<TT, F8>, grid2, block, 0, st, a);               \
  } while (0)
  if (fp8) CMOE_GEMV(1, true); else CMOE_GEMV(1, false);
#undef CMOE_GEMV
  return cudaGetLastError() == cudaSuccess ? (gate_up_only ? 1 : 2) : -1;
}

}  // namespace cmoe
