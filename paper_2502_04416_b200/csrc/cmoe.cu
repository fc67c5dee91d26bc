// C-ABI library: layer construction (weight repacking into expert-contiguous
// operand layouts), the forward pass as a sequence of kernels on the caller's
// stream, and the read-back accessors.  Declarations and contracts: include/cmoe.h.
#include "../../include/cmoe.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <type_traits>
#include <vector>

#include "balance.cuh"
#include "cluster.cuh"
#include "combine.cuh"
#include "fp8.cuh"
#include "common.cuh"
#include "permute.cuh"
#include "profile.cuh"
#include "router.cuh"
#include "router_mma.cuh"
#include "simt_gemm.cuh"
#include "umma2_gemm.cuh"
#include "umma_decode.cuh"
#include "gemv.cuh"
#include "umma_gemm.cuh"

using namespace cmoe;

namespace {

thread_local char g_last_error[512] = "";

int cuda_fail(cudaError_t e, const char* what) {
  snprintf(g_last_error, sizeof(g_last_error), "%s: %s", what, cudaGetErrorString(e));
  return CMOE_ERR_CUDA;
}
int arg_fail(int code, const char* what) {
  snprintf(g_last_error, sizeof(g_last_error), "%s", what);
  return code;
}

#define CU_TRY(expr)                                          \
  do {                                                        \
    cudaError_t e_ = (expr);                                  \
    if (e_ != cudaSuccess) return cuda_fail(e_, #expr);       \
  } while (0)

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

constexpr int kPairMinRows = 256;        // outer rows from which the expert GEMMs may run on CTA pairs
constexpr int kTmaGatherMaxRows = 512;   // routed rows up to which gather4 replaces the permuted copy of x

// Bump allocator over one device allocation (base == nullptr: measure only).
struct Arena {
  char* base = nullptr;
  size_t used = 0;
  template <typename U> U* take(size_t n) {
    used = align_up(used, 256);
    U* p = base ? reinterpret_cast<U*>(base + used) : nullptr;
    used += n * sizeof(U);
    return p;
  }
};

}  // namespace

struct cmoe_layer {
  cmoe_config cfg{};
  int m = 0, n_r = 0, n_rp = 0, n_outer = 1, outer_k = 1;   // n_rp: N_r rounded up to 8
  bool hier = false;
  int device = 0;
  size_t esz = 2;
  int gemm_path = 0;
  bool chain_launches = true;
  bool umma_ok = false;

  // packed weights
  void* w_gu = nullptr;     // one allocation [2][n_outer*d_ff, d]: gate plane, then up plane
  void* wg_p = nullptr;     // [n_outer*d_ff, d]   neurons in expert order (view into w_gu)
  void* wu_p = nullptr;     // [n_outer*d_ff, d]   (view into w_gu)
  void* wd_p = nullptr;     // per outer expert: shared block [d, N_s*m], then N_r blocks [d, m]
  void* w_rep = nullptr;    // [n_outer][2*n_rp][d]: gate rows of the representatives (zero-padded to n_rp), then up rows
  void* w_router = nullptr; // [n_outer, d] (hierarchical)
  float* u = nullptr;       // [n_outer*N_r]
  float* b = nullptr;
  // FP8 copy of the expert weights (cmoe_layer_quantise_fp8): codes in the packed layouts, scales
  uint8_t *w_gu8 = nullptr, *wd8 = nullptr;
  float *scale_gu = nullptr, *scale_d = nullptr;
  void* fp8_tok = nullptr;  // E4M3 planes and scales of the token rows of a decode-sized forward (one allocation)
  bool fp8 = false;
  GroupStatic* gs = nullptr;
  std::vector<GroupStatic> gs_host;

  // workspace (one allocation)
  void* ws = nullptr;
  size_t ws_bytes = 0;
  float *scores = nullptr, *keys = nullptr, *topk_gate = nullptr;
  int32_t *topk_idx = nullptr, *row_of = nullptr, *row_token = nullptr, *counts = nullptr,
          *offsets = nullptr, *perm_scratch = nullptr;
  GroupRows* gr = nullptr;
  void *x_perm = nullptr, *h_s = nullptr, *h_r = nullptr, *y_s = nullptr, *y_r = nullptr;
  // hierarchical
  float *outer_logits = nullptr, *outer_w = nullptr;
  int32_t *outer_idx = nullptr, *outer_counts = nullptr, *outer_off = nullptr,
          *outer_row_token = nullptr, *outer_row_of = nullptr, *outer_scratch = nullptr;
  void* xo = nullptr;
  int32_t* err_word = nullptr;
  UmmaPlan umma;
  DecodePlan decode;
  Umma2Plan pair;
  float* rsk_part = nullptr;    // split-K router partial sums [slices][64 rows][64]
  int32_t* rsk_ticket = nullptr;
  float* rt_part = nullptr;     // tcgen05 router: K-slice partial sums and tickets
  int32_t* rt_ticket = nullptr;
  float* dec_part = nullptr;    // decode GEMMs: K-slice partial sums, tickets per (tile, epilogue warp)
  int32_t* dec_ticket = nullptr;
  size_t n_dec_ticket = 0, n_rt_ticket = 0;    // lengths of the ticket arrays (zeroed again after a device timeout)
  float *share = nullptr, *target = nullptr;   // utilisation of the last step / bias-update targets

  cudaStream_t last_stream = nullptr;
  int last_T = 0;
  int launches = 0;

  // staging for cmoe_ffn_forward_host (created by its first call): two device buffers each for
  // x and out, one copy stream per direction, events per buffer
  struct HostIo {
    int chunk = 0;
    void *x[2] = {nullptr, nullptr}, *out[2] = {nullptr, nullptr};
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t start = nullptr, in_done[2] = {nullptr, nullptr}, cmp_done[2] = {nullptr, nullptr},
                out_done[2] = {nullptr, nullptr};
  } hio;

  // optional per-stage CUDA-event timing: ring of (kStages + 1) events per forward
  std::vector<cudaEvent_t> ev;
  int ev_ring = 0;
  long long ev_count = 0;

  int n_groups_total() const { return n_outer + n_outer * n_r; }
  int shared_width() const { return cfg.n_shared * m; }
};

namespace {

void free_layer(cmoe_layer* L) {
  if (!L) return;
  for (cudaEvent_t e : L->ev) cudaEventDestroy(e);
  for (int b = 0; b < 2; ++b) {
    cudaFree(L->hio.x[b]); cudaFree(L->hio.out[b]);
    if (L->hio.in_done[b]) cudaEventDestroy(L->hio.in_done[b]);
    if (L->hio.cmp_done[b]) cudaEventDestroy(L->hio.cmp_done[b]);
    if (L->hio.out_done[b]) cudaEventDestroy(L->hio.out_done[b]);
  }
  if (L->hio.start) cudaEventDestroy(L->hio.start);
  if (L->hio.s_in) cudaStreamDestroy(L->hio.s_in);
  if (L->hio.s_out) cudaStreamDestroy(L->hio.s_out);
  umma_plan_destroy(&L->umma);
  cudaFree(L->w_gu8); cudaFree(L->wd8); cudaFree(L->scale_gu); cudaFree(L->scale_d); cudaFree(L->fp8_tok);
  cudaFree(L->w_gu); cudaFree(L->wd_p); cudaFree(L->w_rep);
  cudaFree(L->w_router); cudaFree(L->u); cudaFree(L->b); cudaFree(L->gs); cudaFree(L->ws);
  delete L;
}

template <typename T>
__global__ void pack_down_kernel(const T* __restrict__ w_down, const int32_t* __restrict__ perm, int d,
                                 int d_ff, int m, int shared_w, T* __restrict__ dst) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;   // packed neuron position
  const int c = blockIdx.y;
  if (n >= d_ff) return;
  const T v = w_down[(size_t)c * d_ff + perm[n]];
  size_t o;
  if (n < shared_w) {
    o = (size_t)c * shared_w + n;
  } else {
    const int j = (n - shared_w) / m, k = (n - shared_w) % m;
    o = (size_t)shared_w * d + (size_t)j * m * d + (size_t)c * m + k;
  }
  dst[o] = v;
}

int check_config(const cmoe_config& c) {
  if (c.d_model <= 0 || c.d_ff <= 0 || c.n_experts <= 0 || c.n_shared < 0 || c.top_k < 0 ||
      c.max_tokens <= 0)
    return arg_fail(CMOE_ERR_INVALID_ARG, "non-positive dimension");
  if (c.dtype != CMOE_BF16 && c.dtype != CMOE_FP32) return arg_fail(CMOE_ERR_INVALID_ARG, "dtype");
  if (c.d_model % 8) return arg_fail(CMOE_ERR_INVALID_ARG, "d_model must be a multiple of 8");
  if (c.d_ff % c.n_experts) return arg_fail(CMOE_ERR_BAD_PARTITION, "d_ff % n_experts != 0");
  if (c.n_shared > c.n_experts) return arg_fail(CMOE_ERR_INVALID_ARG, "n_shared > n_experts");
  const int n_r = c.n_experts - c.n_shared;
  if (c.top_k > n_r) return arg_fail(CMOE_ERR_INVALID_ARG, "top_k > routed experts");
  if (n_r > kMaxRouted) return arg_fail(CMOE_ERR_INVALID_ARG, "more than 32 routed experts");
  if (c.top_k > kMaxTopK) return arg_fail(CMOE_ERR_INVALID_ARG, "top_k > 8");
  return CMOE_OK;
}

int check_device() {
  int dev = 0, major = 0;
  CU_TRY(cudaGetDevice(&dev));
  CU_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
  if (major != 10) return arg_fail(CMOE_ERR_UNSUPPORTED, "device is not compute capability 10.x");
  return CMOE_OK;
}

void build_group_statics(cmoe_layer* L) {
  const int d = L->cfg.d_model, d_ff = L->cfg.d_ff, m = L->m, sw = L->shared_width();
  L->gs_host.assign(L->n_groups_total(), GroupStatic{});
  for (int i = 0; i < L->n_outer; ++i) {
    GroupStatic& s = L->gs_host[i];
    s.w_row0 = i * d_ff; s.width = sw; s.wd_offset = (int64_t)i * d * d_ff; s.is_shared = 1; s.outer = i;
    for (int j = 0; j < L->n_r; ++j) {
      GroupStatic& r = L->gs_host[L->n_outer + i * L->n_r + j];
      r.w_row0 = i * d_ff + sw + j * m; r.width = m;
      r.wd_offset = (int64_t)i * d * d_ff + (int64_t)sw * d + (int64_t)j * m * d;
      r.is_shared = 0; r.outer = i;
    }
  }
}

// Lays out the workspace; with base == nullptr only measures it.
void carve_workspace(cmoe_layer* L, char* base) {
  Arena a; a.base = base;
  const size_t T = L->cfg.max_tokens, R = T * (L->hier ? L->outer_k : 1), P = R * L->cfg.top_k;
  const size_t d = L->cfg.d_model, nr = L->n_r, G = (size_t)L->n_outer * nr, esz = L->esz;
  L->scores = a.take<float>(R * nr);
  L->keys = a.take<float>(R * nr);
  L->topk_idx = a.take<int32_t>(P);
  L->topk_gate = a.take<float>(P);
  L->row_of = a.take<int32_t>(P);
  L->row_token = a.take<int32_t>(P);
  L->counts = a.take<int32_t>(G);
  L->offsets = a.take<int32_t>(G + 1);
  L->perm_scratch = a.take<int32_t>(permute_scratch_bytes((int)R, (int)(G ? G : 1)) / 4);
  L->gr = a.take<GroupRows>(L->n_groups_total());
  L->err_word = a.take<int32_t>(1);
  L->rsk_ticket = a.take<int32_t>(kRskMaxChunks + 1);
  L->share = a.take<float>(G ? G : 1);
  L->target = a.take<float>(G ? G : 1);
  L->rsk_part = a.take<float>((size_t)kRskMaxTotalRows * kRskMaxSlices * 64);
  L->x_perm = a.take<char>(P * d * esz);
  L->h_s = a.take<char>(R * L->shared_width() * esz);
  L->h_r = a.take<char>(P * L->m * esz);
  L->y_s = a.take<char>(R * d * esz);
  L->y_r = a.take<char>(P * d * esz);
  if (L->hier) {
    L->outer_logits = a.take<float>(T * L->n_outer);
    L->outer_w = a.take<float>(T * L->outer_k);
    L->outer_idx = a.take<int32_t>(T * L->outer_k);
    L->outer_counts = a.take<int32_t>(L->n_outer);
    L->outer_off = a.take<int32_t>(L->n_outer + 1);
    L->outer_row_token = a.take<int32_t>(R);
    L->outer_row_of = a.take<int32_t>(R);
    L->outer_scratch = a.take<int32_t>(permute_scratch_bytes((int)T, L->n_outer) / 4);
    L->xo = a.take<char>(R * d * esz);
  }
  if (esz == 2) {
    // gate/up tiles hold 96 to 128 neurons (decode_pick_tile_rows): count them at the smallest height
    const size_t t1 = (size_t)L->n_outer * ((L->shared_width() + 95) / 96 + nr * ((L->m + 95) / 96));
    const size_t t2 = (size_t)L->n_groups_total() * ((d + 127) / 128);
    L->n_dec_ticket = 4 * (t1 > t2 ? t1 : t2);
    L->dec_ticket = a.take<int32_t>(L->n_dec_ticket);
    L->dec_part = a.take<float>((size_t)kDecMaxSlots * kDecSlotFloats);
  }
  if (esz == 2 && nr > 0) {
    L->n_rt_ticket = 4 * 256;
    L->rt_ticket = a.take<int32_t>(L->n_rt_ticket);
    L->rt_part = a.take<float>((size_t)256 * 64 * 128);
  }
  L->ws_bytes = align_up(a.used + 256, 256);
}

int alloc_workspace(cmoe_layer* L) {
  carve_workspace(L, nullptr);
  CU_TRY(cudaMalloc(&L->ws, L->ws_bytes));
  carve_workspace(L, static_cast<char*>(L->ws));
  CU_TRY(cudaMemset(L->ws, 0, L->ws_bytes));
  return CMOE_OK;
}

int upload_gate_params(cmoe_layer* L, const float* u, const float* b, cudaStream_t st) {
  const size_t n = (size_t)L->n_outer * L->n_r;
  if (n == 0) return CMOE_OK;
  std::vector<float> zeros(n, 0.0f);
  CU_TRY(cudaMemcpyAsync(L->u, u ? u : zeros.data(), n * sizeof(float), cudaMemcpyHostToDevice, st));
  CU_TRY(cudaMemcpyAsync(L->b, b ? b : zeros.data(), n * sizeof(float), cudaMemcpyHostToDevice, st));
  CU_TRY(cudaStreamSynchronize(st));
  return CMOE_OK;
}

int finish_layer(cmoe_layer* L, cudaStream_t st) {
  build_group_statics(L);
  CU_TRY(cudaMalloc(&L->gs, L->gs_host.size() * sizeof(GroupStatic)));
  CU_TRY(cudaMemcpyAsync(L->gs, L->gs_host.data(), L->gs_host.size() * sizeof(GroupStatic),
                         cudaMemcpyHostToDevice, st));
  int rc = alloc_workspace(L);
  if (rc != CMOE_OK) return rc;
  L->umma_ok = false;
  if (L->cfg.dtype == CMOE_BF16) {
    UmmaShape s;
    s.d = L->cfg.d_model; s.m = L->m; s.shared_width = L->shared_width(); s.d_ff = L->cfg.d_ff;
    s.n_outer = L->n_outer; s.n_r = L->n_r; s.n_rp = L->n_rp; s.n_k = L->cfg.top_k;
    s.max_outer_rows = (size_t)L->cfg.max_tokens * (L->hier ? L->outer_k : 1);
    s.max_routed_rows = s.max_outer_rows * L->cfg.top_k;
    UmmaBuffers ub;
    ub.w_gate_up = L->w_gu; ub.w_down = L->wd_p; ub.w_rep = L->w_rep;
    ub.x_fixed = L->hier ? L->xo : nullptr;
    ub.x_perm = L->x_perm;
    ub.h_s = L->h_s; ub.h_r = L->h_r; ub.y_s = L->y_s; ub.y_r = L->y_r;
    ub.gs_dev = L->gs; ub.u = L->u; ub.b = L->b;
    ub.scores = L->scores; ub.keys = L->keys; ub.topk_idx = L->topk_idx; ub.topk_gate = L->topk_gate;
    ub.row_token = L->row_token;
    rc = umma_plan_create(&L->umma, s, ub, L->n_groups_total());
    if (rc == CMOE_ERR_CUDA) return arg_fail(CMOE_ERR_CUDA, L->umma.error);
    L->umma_ok = (rc == CMOE_OK);
    if (L->umma_ok && !decode_plan_create(&L->umma, &L->decode)) return arg_fail(CMOE_ERR_CUDA, L->umma.error);
    L->decode.part = L->dec_part; L->decode.ticket = L->dec_ticket;
    L->umma.rt_part = L->rt_part; L->umma.rt_ticket = L->rt_ticket;
    if (L->umma_ok && !umma2_plan_create(&L->umma, &L->pair)) return arg_fail(CMOE_ERR_CUDA, L->umma.error);
  }
  CU_TRY(cudaStreamSynchronize(st));
  return CMOE_OK;
}

template <typename T>
int pack_weights(cmoe_layer* L, const void* w_gate, const void* w_up, const void* w_down,
                 const int32_t* perm_dev, const int32_t* rep_dev, cudaStream_t st) {
  const int d = L->cfg.d_model, d_ff = L->cfg.d_ff;
  const int row_vec = d * (int)sizeof(T) / 16;
  gather_rows_kernel<<<d_ff, 256, 0, st>>>((const uint4*)w_gate, perm_dev, d_ff, row_vec, (uint4*)L->wg_p);
  gather_rows_kernel<<<d_ff, 256, 0, st>>>((const uint4*)w_up, perm_dev, d_ff, row_vec, (uint4*)L->wu_p);
  if (L->n_r > 0) {
    gather_rows_kernel<<<L->n_r, 256, 0, st>>>((const uint4*)w_gate, rep_dev, L->n_r, row_vec,
                                               (uint4*)L->w_rep);
    gather_rows_kernel<<<L->n_r, 256, 0, st>>>((const uint4*)w_up, rep_dev, L->n_r, row_vec,
                                               (uint4*)((char*)L->w_rep + (size_t)L->n_rp * d * sizeof(T)));
  }
  dim3 grid((d_ff + 255) / 256, d);
  pack_down_kernel<T><<<grid, 256, 0, st>>>((const T*)w_down, perm_dev, d, d_ff, L->m, L->shared_width(),
                                            (T*)L->wd_p);
  CU_TRY(cudaGetLastError());
  return CMOE_OK;
}

template <typename T>
int forward_impl(cmoe_layer* L, const T* x, int n_tok, T* out, cudaStream_t st, bool gate_up_only = false) {
  const int d = L->cfg.d_model, n_r = L->n_r, n_k = L->cfg.top_k;
  const int R = n_tok * (L->hier ? L->outer_k : 1);
  const int P = R * n_k;
  const int G = L->n_outer * n_r;
  const int row_vec = d * (int)sizeof(T) / 16;
  int launches = 0;
  const T* xo = x;
  const bool use_umma = L->umma_ok && L->gemm_path != 1;     // 2: tensor, 3: tensor on CTA pairs
  cudaEvent_t* ev = (L->ev_ring && !gate_up_only) ? &L->ev[(size_t)(L->ev_count % L->ev_ring) * (CMOE_N_STAGES + 1)] : nullptr;
  auto mark = [&](int i) { if (ev) cudaEventRecord(ev[i], st); };
  mark(0);
  // bf16 layers on the tensor path chain their kernels by programmatic dependent launch (every
  // kernel after the expert router may become resident early and waits on the device for its
  // predecessor); per-stage events and the prologue of a hierarchical layer (outer router, outer
  // permutation, row copy) use ordinary launches.
  const bool dep = use_umma && !ev && L->chain_launches;

  if (L->hier) {
    if constexpr (std::is_same<T, bf16>::value) {
      outer_router_mma_kernel<8, 1><<<(n_tok + 15) / 16, 256, 0, st>>>(
          x, n_tok, d, L->n_outer, L->outer_k, (const bf16*)L->w_router, L->outer_logits, L->outer_idx,
          L->outer_w);
    } else {
      outer_router_kernel<T><<<(n_tok + 7) / 8, 256, 0, st>>>(x, n_tok, d, L->n_outer, L->outer_k,
                                                              (const T*)L->w_router, L->outer_logits,
                                                              L->outer_idx, L->outer_w);
    }
    ++launches;
    launches += launch_token_permute(L->outer_idx, n_tok, L->outer_k, L->n_outer, L->outer_counts,
                                     L->outer_off, L->outer_row_token, L->outer_row_of,
                                     L->outer_scratch, st);
    gather_rows_kernel<<<R, 256, 0, st>>>((const uint4*)x, L->outer_row_token, R, row_vec, (uint4*)L->xo);
    ++launches;
    xo = (const T*)L->xo;
  }

  // One row of a plain layer: plain-load weight streamers on the CUDA cores, the down projection and the
  // combine in one launch (automatic path only; path 2 keeps the tensor-core kernels).
  bool gemv = false;
  GemvPlan gemv_ring{};
  if constexpr (std::is_same<T, bf16>::value)
    gemv = use_umma && !L->hier && L->gemm_path == 0 &&
           gemv_plan((int)R, L->n_outer, L->n_groups_total(), n_k, n_r, d, L->shared_width(), L->m, L->cfg.n_shared > 0,
                     L->fp8, &gemv_ring);
  // Weights-on-M streaming kernels: up to 64 rows; on bf16 weights (the FP8 token planes stop at 64) the wide
  // form takes up to 128 rows.  Path 2 keeps token-major tiles from 65 rows.
  const int decode_rows = (!L->fp8 && L->gemm_path != 2) ? kDecWideRows : kDecMaxRows;
  const bool decode = use_umma && !gemv && R <= decode_rows;
  if (use_umma && !umma_bind_x(&L->umma, xo, R)) return arg_fail(CMOE_ERR_CUDA, L->umma.error);
  if (decode && !decode_bind_x(&L->umma, &L->decode, xo, R)) return arg_fail(CMOE_ERR_CUDA, L->umma.error);
  if (decode && L->fp8) {                          // E4M3 planes of the token rows: independent of the routing
    if (decode_split_x(&L->umma, &L->decode, R, st, false) < 0) return arg_fail(CMOE_ERR_CUDA, "split_rows launch failed");
    ++launches;
  }
  GroupPlanOut po;                                // the permutation also writes every group's row range
  po.gr = L->gr; po.n_outer = L->n_outer; po.n_tokens = n_tok; po.outer_off = L->hier ? L->outer_off : nullptr;
  bool perm_fused = false;                        // decode: the router's last block also permutes
  if (n_r > 0) {
    const int warps = (R + 1) / 2, blocks = (warps + 7) / 8;
    const int32_t* ooff = L->hier ? L->outer_off : nullptr;
#define CMOE_ROUTER(NACC)                                                                         \
  router_kernel<T, NACC><<<blocks, 256, 0, st>>>(xo, R, d, n_r, L->n_rp, n_k, (const T*)L->w_rep, L->u,   \
                                                 L->b, ooff, L->n_outer, L->scores, L->keys,      \
                                                 L->topk_idx, L->topk_gate)
    if constexpr (std::is_same<T, bf16>::value) {
      if (use_umma && R > kRskMaxTotalRows) {
        if (umma_router_forward(&L->umma, R, ooff, L->err_word, st) < 0)
          return arg_fail(CMOE_ERR_CUDA, L->umma.error);
      } else if (R <= kRskMaxTotalRows && d <= kRskMaxSlices * kRskSliceK) {
        // Row chunks, the grid's second dimension: 16 rows for a router with more than 8 columns, whose gate
        // logic takes a warp per row (measured: 8B-shaped layer at 32 rows 97.9 -> 95.0 us, at 128 rows
        // 118.9 -> 108.7 us); 64 rows with up to 8 columns, where the four-rows-per-warp form on 64-row chunks
        // is 1 us faster.  The last chunk's block also permutes batches of up to 128 rows (7B-shaped layer at
        // 128 rows 91.0 -> 88.9 us; at 256 rows the permutation kernels are as fast).
        const int chunk_rows = n_r > 8 ? 16 : kRskMaxRows;
        const int chunks = (R + chunk_rows - 1) / chunk_rows;
        perm_fused = G <= kRskFuseGroups && R <= 2 * kRskMaxRows && (long long)R * n_k <= 4096;
        const bool sub8 = n_r <= 8 && R > 16;                        // pays when a chunk's last block has more than 16 rows
        (sub8 ? router_splitk_kernel<true> : router_splitk_kernel<false>)
            <<<dim3((d + kRskSliceK - 1) / kRskSliceK, chunks), kRskThreads, 0, st>>>(
            xo, R, d, n_r, L->n_rp, n_k, (const bf16*)L->w_rep, L->u, L->b, ooff, L->n_outer, L->rsk_part,
            L->rsk_ticket, chunk_rows, L->scores, L->keys, L->topk_idx, L->topk_gate, perm_fused ? 1 : 0, G, L->counts,
            L->offsets, L->row_token, L->row_of, po);
      } else {
        router_mma_kernel<8, 1><<<(R + 15) / 16, 256, 0, st>>>(
            xo, R, d, n_r, L->n_rp, n_k, (const bf16*)L->w_rep, L->u, L->b, ooff, L->n_outer, L->scores,
            L->keys, L->topk_idx, L->topk_gate);
      }
    } else {
      if (2 * L->n_rp <= 16) CMOE_ROUTER(16);
      else if (2 * L->n_rp <= 32) CMOE_ROUTER(32);
      else CMOE_ROUTER(64);
    }
#undef CMOE_ROUTER
    ++launches;
    mark(1);
    if (!perm_fused)
      launches += launch_token_permute(L->topk_idx, R, n_k, G, L->counts, L->offsets, L->row_token,
                                       L->row_of, L->perm_scratch, st, po, dep);
  } else {
    mark(1);
    plan_groups_kernel<<<1, 256, 0, st>>>(L->n_outer, n_r, n_tok, L->hier ? L->outer_off : nullptr,
                                          L->counts, L->offsets, L->gr);
    ++launches;
  }
  // The tensor path gathers routed rows inside the gate/up GEMM (decode: not at all; a few rows:
  // TMA gather4; otherwise cp.async by dedicated warps); only the SIMT path reads a permuted copy of x.
  // CTA pairs (cta_group::2, 256-row tiles) move a third less operand data per flop but round every
  // group up to an even number of 128-row tiles.  Path 3 forces them; the automatic choice takes them
  // per GEMM when the padding expected for evenly loaded experts stays small (thresholds measured on
  // the paper-shaped workloads: the down GEMM gains more from pairs than the gate/up GEMM, except
  // when its K extent, the expert width, is only a few k blocks).
  int pair_mask = 0;                               // bit 0: gate/up on pairs, bit 1: down on pairs
  if (use_umma && !decode && R >= kPairMinRows) {
    if (L->gemm_path == 3) {
      pair_mask = 3;
    } else if (L->gemm_path == 0) {
      auto pad = [](double rows) {                 // tile slots on pairs / tiles on single CTAs
        const int mt = (int)((rows + 127) / 128);
        return mt > 0 ? (double)(2 * ((mt + 1) / 2)) / mt : 1.0;
      };
      const double rows_s = (double)R / L->n_outer, rows_r = G > 0 ? (double)P / G : 0.0;
      const double w_s = (double)R * L->cfg.n_shared, w_r = (double)P;
      const double ratio = (w_s + w_r) > 0 ? (pad(rows_s) * w_s + pad(rows_r) * w_r) / (w_s + w_r) : 1.0;
      if (R < 1024 && !L->hier) {
        // A few tiles per SM: operand fetch per SM is the limit, and a pair halves the weight bytes a CTA fetches,
        // but every routed group is padded to 256 rows.  Measured at 256-768 rows: pairs win with wide experts
        // (1376 neurons: 114 vs 126 us at 256 rows, 120 vs 127 at 512), single-CTA tiles with narrow ones (864:
        // 134 vs 162 us at 256 rows, 165 vs 174 at 384; 448: 113 vs 127 at 256, 151 vs 167 at 768).
        pair_mask = L->m >= 1024 ? 3 : 0;
      } else {
        if (ratio <= 1.03) pair_mask |= 1;
        if (ratio <= 1.08 && L->m >= 512) pair_mask |= 2;
      }
    }
  }
  const int gather_mode = P <= kTmaGatherMaxRows ? 1 : 2;
  if (P > 0 && !use_umma) {
    gather_rows_kernel<<<P, 256, 0, st>>>((const uint4*)xo, L->row_token, P, row_vec, (uint4*)L->x_perm);
    ++launches;
  }

  mark(2);
  if (gemv) {
    if constexpr (std::is_same<T, bf16>::value) {
      GemvArgs a{};
      a.gs = L->umma.buf.gs_dev; a.gr = L->gr; a.n_groups = L->n_groups_total(); a.d = d; a.n_rows = (int)R; a.n_k = n_k;
      a.x = xo;
      a.w_gate_up = L->fp8 ? (const void*)L->w_gu8 : (const void*)L->w_gu;
      a.w_down = L->fp8 ? (const void*)L->wd8 : (const void*)L->wd_p;
      a.rows_w = (long long)L->n_outer * L->cfg.d_ff;
      a.scale_gu = L->scale_gu; a.scale_d = L->scale_d;
      a.h_s = (bf16*)L->h_s; a.h_r = (bf16*)L->h_r; a.ld_h_s = L->shared_width(); a.ld_h_r = L->m;
      a.row_of = L->row_of; a.topk_gate = L->topk_gate;
      a.out = out;
      const int n = gemv_forward(a, gemv_ring, L->fp8, L->umma.n_sms, st, ev ? ev[3] : nullptr, dep, gate_up_only);
      if (n < 0) return arg_fail(CMOE_ERR_CUDA, "gemv launch failed");
      launches += n;
    }
    if (!gate_up_only) {                              // the second launch wrote `out`: nothing left to combine
      mark(4);
      mark(5);
      if (ev) ++L->ev_count;
      CU_TRY(cudaGetLastError());
      L->launches = launches;
      return CMOE_OK;
    }
  } else if (use_umma) {
    cudaEvent_t mid = ev ? ev[3] : nullptr;
    int n;
    if (decode) {
      n = decode_forward(&L->umma, &L->decode, L->gr, R, L->err_word, st, mid, dep, gate_up_only);
    } else {
      const int todo = gate_up_only ? 1 : 3;
      n = 0;
      for (int bit = 1; bit <= 2 && n >= 0; bit <<= 1) {          // gate/up, then down, each on its chosen tile shape
        if (!(todo & bit)) continue;
        const int k = (pair_mask & bit)
            ? umma2_forward(&L->umma, &L->pair, &L->decode, L->gr, 2, xo, L->err_word, st, mid, dep, bit)
            : umma_forward(&L->umma, L->gr, gather_mode, xo, L->err_word, st, mid, dep, bit);
        n = k < 0 ? -1 : n + k;
      }
    }
    if (n < 0) return arg_fail(CMOE_ERR_CUDA, L->umma.error);
    launches += n;
  } else {
    SimtGemmArgs<T> a;
    a.gs = L->gs; a.gr = L->gr; a.d = d;
    a.shared_width = L->shared_width(); a.routed_width = L->m;
    const int max_w = a.shared_width > a.routed_width ? a.shared_width : a.routed_width;
    a.a_shared = xo; a.a_routed = (const T*)L->x_perm;
    a.w_gate = (const T*)L->wg_p; a.w_up = (const T*)L->wu_p;
    a.c_shared = (T*)L->h_s; a.c_routed = (T*)L->h_r;
    dim3 g1((R + kSimtTile - 1) / kSimtTile, (max_w + kSimtTile - 1) / kSimtTile, L->n_groups_total());
    simt_gemm1_kernel<T><<<g1, 256, 0, st>>>(a);
    mark(3);
    if (gate_up_only) { L->launches = launches + 1; CU_TRY(cudaGetLastError()); return CMOE_OK; }
    a.a_shared = (const T*)L->h_s; a.a_routed = (const T*)L->h_r;
    a.w_gate = (const T*)L->wd_p; a.w_up = nullptr;
    a.c_shared = (T*)L->y_s; a.c_routed = (T*)L->y_r;
    dim3 g2((R + kSimtTile - 1) / kSimtTile, (d + kSimtTile - 1) / kSimtTile, L->n_groups_total());
    simt_gemm2_kernel<T><<<g2, 256, 0, st>>>(a);
    launches += 2;
  }

  if (gate_up_only) { L->launches = launches; CU_TRY(cudaGetLastError()); return CMOE_OK; }   // H_s is complete
  mark(4);
  const int per_thread = sizeof(T) == 2 ? 16 : 8;
  const int threads = d / per_thread < 256 ? ((d / per_thread + 31) / 32 * 32) : 256;
  bool fast_combine = false;
  if constexpr (sizeof(T) == 2) {
    const int th = (d / 16 + 31) / 32 * 32;
    if (!L->hier && d % 16 == 0 && th <= 1024 && n_k <= 4 && n_tok > 64) {
      fast_combine = true;
      const int sms = L->umma.n_sms > 0 ? L->umma.n_sms : 148;
      const int grid = std::min(n_tok, sms * std::max(1, 1024 / th) * 2);
      const bf16* ys = L->cfg.n_shared > 0 ? (const bf16*)L->y_s : nullptr;
      if (n_k <= 1)
        launch_kernel(dep, combine_plain_bf16_kernel<1>, dim3(grid), dim3(th), 0, st, ys, (const bf16*)L->y_r, L->topk_gate, L->row_of, n_tok, n_k, d, (bf16*)out);
      else if (n_k == 2)
        launch_kernel(dep, combine_plain_bf16_kernel<2>, dim3(grid), dim3(th), 0, st, ys, (const bf16*)L->y_r, L->topk_gate, L->row_of, n_tok, n_k, d, (bf16*)out);
      else
        launch_kernel(dep, combine_plain_bf16_kernel<4>, dim3(grid), dim3(th), 0, st, ys, (const bf16*)L->y_r, L->topk_gate, L->row_of, n_tok, n_k, d, (bf16*)out);
    }
  }
  if (!fast_combine)
  launch_kernel(dep, combine_kernel<T>, dim3(n_tok), dim3(threads), 0, st,
                L->cfg.n_shared > 0 ? (const T*)L->y_s : nullptr, (const T*)L->y_r, (const int32_t*)L->topk_idx,
                (const float*)L->topk_gate, (const int32_t*)L->row_of,
                (const int32_t*)(L->hier ? L->outer_row_of : nullptr), (const float*)(L->hier ? L->outer_w : nullptr),
                L->hier ? L->outer_k : 1, n_k, d, out);
  ++launches;
  mark(5);
  if (ev) ++L->ev_count;
  CU_TRY(cudaGetLastError());
  L->launches = launches;
  return CMOE_OK;
}

}  // namespace

extern "C" {

int cmoe_layer_create(const cmoe_config* cfg, const void* w_gate, const void* w_up,
                      const void* w_down, const int32_t* neuron_perm, const int32_t* rep_idx,
                      const float* gate_scale_u, const float* select_bias_b, void* stream,
                      cmoe_layer** out_layer) {
  if (!cfg || !w_gate || !w_up || !w_down || !neuron_perm || !out_layer)
    return arg_fail(CMOE_ERR_INVALID_ARG, "null argument");
  *out_layer = nullptr;
  int rc = check_config(*cfg);
  if (rc != CMOE_OK) return rc;
  const int d = cfg->d_model, d_ff = cfg->d_ff, m = d_ff / cfg->n_experts;
  const int n_r = cfg->n_experts - cfg->n_shared;
  if (n_r > 0 && !rep_idx) return arg_fail(CMOE_ERR_INVALID_ARG, "rep_idx is null");
  {
    std::vector<int32_t> where(d_ff, -1);          // original neuron -> packed position
    for (int i = 0; i < d_ff; ++i) {
      const int32_t n = neuron_perm[i];
      if (n < 0 || n >= d_ff || where[n] >= 0)
        return arg_fail(CMOE_ERR_BAD_PARTITION, "neuron_perm is not a permutation of [0, d_ff)");
      where[n] = i;
    }
    for (int j = 0; j < n_r; ++j) {
      const int32_t r = rep_idx[j];
      if (r < 0 || r >= d_ff || where[r] / m != cfg->n_shared + j)
        return arg_fail(CMOE_ERR_BAD_REP, "representative outside its routed expert's slice");
    }
  }
  rc = check_device();
  if (rc != CMOE_OK) return rc;

  cmoe_layer* L = new (std::nothrow) cmoe_layer();
  if (!L) return arg_fail(CMOE_ERR_INVALID_ARG, "out of host memory");
  L->cfg = *cfg; L->m = m; L->n_r = n_r; L->n_rp = (n_r + 7) / 8 * 8; L->n_outer = 1; L->outer_k = 1; L->hier = false;
  L->esz = cfg->dtype == CMOE_BF16 ? 2 : 4;
  cudaGetDevice(&L->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t *perm_dev = nullptr, *rep_dev = nullptr;
  auto fail = [&](int code) { cudaFree(perm_dev); cudaFree(rep_dev); free_layer(L); return code; };
#define TRY_OR_FAIL(expr)                                                 \
  do {                                                                    \
    cudaError_t e_ = (expr);                                              \
    if (e_ != cudaSuccess) return fail(cuda_fail(e_, #expr));             \
  } while (0)
  const size_t wbytes = (size_t)d_ff * d * L->esz;
  TRY_OR_FAIL(cudaMalloc(&L->w_gu, 2 * wbytes));
  L->wg_p = L->w_gu;
  L->wu_p = (char*)L->w_gu + wbytes;
  TRY_OR_FAIL(cudaMalloc(&L->wd_p, wbytes));
  TRY_OR_FAIL(cudaMalloc(&L->w_rep, (size_t)(n_r ? 2 * L->n_rp : 1) * d * L->esz));
  TRY_OR_FAIL(cudaMemsetAsync(L->w_rep, 0, (size_t)(n_r ? 2 * L->n_rp : 1) * d * L->esz, st));
  TRY_OR_FAIL(cudaMalloc(&L->u, (size_t)(n_r ? n_r : 1) * sizeof(float)));
  TRY_OR_FAIL(cudaMalloc(&L->b, (size_t)(n_r ? n_r : 1) * sizeof(float)));
  TRY_OR_FAIL(cudaMalloc(&perm_dev, (size_t)d_ff * sizeof(int32_t)));
  TRY_OR_FAIL(cudaMalloc(&rep_dev, (size_t)(n_r ? n_r : 1) * sizeof(int32_t)));
  TRY_OR_FAIL(cudaMemcpyAsync(perm_dev, neuron_perm, (size_t)d_ff * sizeof(int32_t),
                              cudaMemcpyHostToDevice, st));
  if (n_r)
    TRY_OR_FAIL(cudaMemcpyAsync(rep_dev, rep_idx, (size_t)n_r * sizeof(int32_t),
                                cudaMemcpyHostToDevice, st));
  rc = cfg->dtype == CMOE_BF16 ? pack_weights<bf16>(L, w_gate, w_up, w_down, perm_dev, rep_dev, st)
                               : pack_weights<float>(L, w_gate, w_up, w_down, perm_dev, rep_dev, st);
  if (rc != CMOE_OK) return fail(rc);
  rc = upload_gate_params(L, gate_scale_u, select_bias_b, st);
  if (rc != CMOE_OK) return fail(rc);
  rc = finish_layer(L, st);
  if (rc != CMOE_OK) return fail(rc);
  TRY_OR_FAIL(cudaStreamSynchronize(st));
#undef TRY_OR_FAIL
  cudaFree(perm_dev); cudaFree(rep_dev);
  *out_layer = L;
  return CMOE_OK;
}

int cmoe_hier_create(int32_t n_outer, int32_t outer_top_k, const void* w_router,
                     cmoe_layer* const* inner, int32_t max_tokens, void* stream,
                     cmoe_layer** out_layer) {
  if (!w_router || !inner || !out_layer) return arg_fail(CMOE_ERR_INVALID_ARG, "null argument");
  *out_layer = nullptr;
  if (n_outer <= 0 || n_outer > kMaxOuter || outer_top_k <= 0 || outer_top_k > n_outer ||
      outer_top_k > kMaxTopK || max_tokens <= 0)
    return arg_fail(CMOE_ERR_INVALID_ARG, "outer expert count / top-k out of range");
  for (int i = 0; i < n_outer; ++i) {
    if (!inner[i] || inner[i]->hier) return arg_fail(CMOE_ERR_INVALID_ARG, "inner layer invalid");
    const cmoe_config &a = inner[0]->cfg, &c = inner[i]->cfg;
    if (a.d_model != c.d_model || a.d_ff != c.d_ff || a.n_experts != c.n_experts ||
        a.n_shared != c.n_shared || a.top_k != c.top_k || a.dtype != c.dtype)
      return arg_fail(CMOE_ERR_INVALID_ARG, "inner layers differ in configuration");
    for (int k = 0; k < i; ++k)
      if (inner[k] == inner[i]) return arg_fail(CMOE_ERR_INVALID_ARG, "inner layer listed twice");
  }
  int rc = check_device();
  if (rc != CMOE_OK) return rc;
  cmoe_layer* L = new (std::nothrow) cmoe_layer();
  if (!L) return arg_fail(CMOE_ERR_INVALID_ARG, "out of host memory");
  L->cfg = inner[0]->cfg; L->cfg.max_tokens = max_tokens;
  L->m = inner[0]->m; L->n_r = inner[0]->n_r; L->n_rp = inner[0]->n_rp; L->esz = inner[0]->esz;
  L->n_outer = n_outer; L->outer_k = outer_top_k; L->hier = true;
  cudaGetDevice(&L->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t d = L->cfg.d_model, d_ff = L->cfg.d_ff, nr = L->n_r, esz = L->esz;
  const size_t wbytes = d_ff * d * esz, rep_bytes = 2 * (size_t)L->n_rp * d * esz;
  auto fail = [&](int code) { free_layer(L); return code; };
#define TRY_OR_FAIL(expr)                                                 \
  do {                                                                    \
    cudaError_t e_ = (expr);                                              \
    if (e_ != cudaSuccess) return fail(cuda_fail(e_, #expr));             \
  } while (0)
  TRY_OR_FAIL(cudaMalloc(&L->w_gu, 2 * wbytes * n_outer));
  L->wg_p = L->w_gu;
  L->wu_p = (char*)L->w_gu + wbytes * n_outer;
  TRY_OR_FAIL(cudaMalloc(&L->wd_p, wbytes * n_outer));
  TRY_OR_FAIL(cudaMalloc(&L->w_rep, (rep_bytes ? rep_bytes : 16) * n_outer));
  TRY_OR_FAIL(cudaMalloc(&L->w_router, (size_t)n_outer * d * esz));
  TRY_OR_FAIL(cudaMalloc(&L->u, (nr ? nr : 1) * n_outer * sizeof(float)));
  TRY_OR_FAIL(cudaMalloc(&L->b, (nr ? nr : 1) * n_outer * sizeof(float)));
  for (int i = 0; i < n_outer; ++i) {
    const cmoe_layer* S = inner[i];
    const auto D2D = cudaMemcpyDeviceToDevice;
    TRY_OR_FAIL(cudaMemcpyAsync((char*)L->wg_p + i * wbytes, S->wg_p, wbytes, D2D, st));
    TRY_OR_FAIL(cudaMemcpyAsync((char*)L->wu_p + i * wbytes, S->wu_p, wbytes, D2D, st));
    TRY_OR_FAIL(cudaMemcpyAsync((char*)L->wd_p + i * wbytes, S->wd_p, wbytes, D2D, st));
    if (nr) {
      TRY_OR_FAIL(cudaMemcpyAsync((char*)L->w_rep + i * rep_bytes, S->w_rep, rep_bytes, D2D, st));
      TRY_OR_FAIL(cudaMemcpyAsync(L->u + i * nr, S->u, nr * sizeof(float), D2D, st));
      TRY_OR_FAIL(cudaMemcpyAsync(L->b + i * nr, S->b, nr * sizeof(float), D2D, st));
    }
  }
  TRY_OR_FAIL(cudaMemcpyAsync(L->w_router, w_router, (size_t)n_outer * d * esz,
                              cudaMemcpyDeviceToDevice, st));
  rc = finish_layer(L, st);
  if (rc != CMOE_OK) return fail(rc);
  TRY_OR_FAIL(cudaStreamSynchronize(st));
#undef TRY_OR_FAIL
  for (int i = 0; i < n_outer; ++i) free_layer(inner[i]);
  *out_layer = L;
  return CMOE_OK;
}

int cmoe_ffn_forward(cmoe_layer* L, const void* x, int32_t T, void* out, void* stream) {
  if (!L) return arg_fail(CMOE_ERR_INVALID_ARG, "null layer");
  if (T < 0) return arg_fail(CMOE_ERR_INVALID_ARG, "negative token count");
  if (T == 0) { L->last_T = 0; L->launches = 0; return CMOE_OK; }
  if (!x || !out) return arg_fail(CMOE_ERR_INVALID_ARG, "null x / out");
  if (T > L->cfg.max_tokens) return arg_fail(CMOE_ERR_CAPACITY, "T exceeds max_tokens");
  if (reinterpret_cast<uintptr_t>(x) & 15) return arg_fail(CMOE_ERR_INVALID_ARG, "x must be 16-byte aligned");
  if (reinterpret_cast<uintptr_t>(out) & 31)      // the combine kernels write 32 bytes per store
    return arg_fail(CMOE_ERR_INVALID_ARG, "out must be 32-byte aligned");
  {
    const char *xa = (const char*)x, *oa = (const char*)out;
    const size_t bytes = (size_t)T * L->cfg.d_model * L->esz;
    if (xa < oa + bytes && oa < xa + bytes) return arg_fail(CMOE_ERR_INVALID_ARG, "x and out overlap");
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  L->last_stream = st;
  L->last_T = T;
  return L->cfg.dtype == CMOE_BF16 ? forward_impl<bf16>(L, (const bf16*)x, T, (bf16*)out, st)
                                   : forward_impl<float>(L, (const float*)x, T, (float*)out, st);
}

int cmoe_ffn_forward_host(cmoe_layer* L, const void* x_host, int32_t T, void* out_host, int32_t chunk_tokens,
                          void* stream) {
  if (!L) return arg_fail(CMOE_ERR_INVALID_ARG, "null layer");
  if (T < 0) return arg_fail(CMOE_ERR_INVALID_ARG, "negative token count");
  if (T == 0) { L->last_T = 0; L->launches = 0; return CMOE_OK; }
  if (!x_host || !out_host) return arg_fail(CMOE_ERR_INVALID_ARG, "null x / out");
  const size_t row_bytes = (size_t)L->cfg.d_model * L->esz;
  int chunk = chunk_tokens;
  if (chunk <= 0) {                                  // a sixteenth of the batch, in whole 128-row tiles, at least 512
    chunk = ((T + 15) / 16 + 127) / 128 * 128;
    if (chunk < 512) chunk = 512;
  }
  if (chunk > L->cfg.max_tokens) chunk = L->cfg.max_tokens;
  if (chunk > T) chunk = T;
  cmoe_layer::HostIo& h = L->hio;
  if (h.chunk < chunk) {                             // first call (or a larger chunk than before): set up the staging
    for (int b = 0; b < 2; ++b) {
      cudaFree(h.x[b]); cudaFree(h.out[b]);
      h.x[b] = h.out[b] = nullptr;
    }
    h.chunk = 0;
    for (int b = 0; b < 2; ++b) {
      CU_TRY(cudaMalloc(&h.x[b], (size_t)chunk * row_bytes));
      CU_TRY(cudaMalloc(&h.out[b], (size_t)chunk * row_bytes));
      if (!h.in_done[b]) CU_TRY(cudaEventCreateWithFlags(&h.in_done[b], cudaEventDisableTiming));
      if (!h.cmp_done[b]) CU_TRY(cudaEventCreateWithFlags(&h.cmp_done[b], cudaEventDisableTiming));
      if (!h.out_done[b]) CU_TRY(cudaEventCreateWithFlags(&h.out_done[b], cudaEventDisableTiming));
    }
    if (!h.start) CU_TRY(cudaEventCreateWithFlags(&h.start, cudaEventDisableTiming));
    if (!h.s_in) CU_TRY(cudaStreamCreateWithFlags(&h.s_in, cudaStreamNonBlocking));
    if (!h.s_out) CU_TRY(cudaStreamCreateWithFlags(&h.s_out, cudaStreamNonBlocking));
    h.chunk = chunk;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  L->last_stream = st;
  // the copies start where the caller's stream stands now
  CU_TRY(cudaEventRecord(h.start, st));
  CU_TRY(cudaStreamWaitEvent(h.s_in, h.start, 0));
  CU_TRY(cudaStreamWaitEvent(h.s_out, h.start, 0));
  int launches = 0, n_chunks = 0;
  for (int t0 = 0; t0 < T; t0 += chunk, ++n_chunks) {
    const int n = T - t0 < chunk ? T - t0 : chunk, b = n_chunks & 1;
    const char* src = static_cast<const char*>(x_host) + (size_t)t0 * row_bytes;
    char* dst = static_cast<char*>(out_host) + (size_t)t0 * row_bytes;
    if (n_chunks >= 2) CU_TRY(cudaStreamWaitEvent(h.s_in, h.cmp_done[b], 0));      // x[b] has been consumed
    CU_TRY(cudaMemcpyAsync(h.x[b], src, (size_t)n * row_bytes, cudaMemcpyHostToDevice, h.s_in));
    CU_TRY(cudaEventRecord(h.in_done[b], h.s_in));
    CU_TRY(cudaStreamWaitEvent(st, h.in_done[b], 0));
    if (n_chunks >= 2) CU_TRY(cudaStreamWaitEvent(st, h.out_done[b], 0));          // out[b] has been drained
    L->last_T = n;
    const int rc = L->cfg.dtype == CMOE_BF16 ? forward_impl<bf16>(L, (const bf16*)h.x[b], n, (bf16*)h.out[b], st)
                                             : forward_impl<float>(L, (const float*)h.x[b], n, (float*)h.out[b], st);
    if (rc != CMOE_OK) return rc;
    launches += L->launches;
    CU_TRY(cudaEventRecord(h.cmp_done[b], st));
    CU_TRY(cudaStreamWaitEvent(h.s_out, h.cmp_done[b], 0));
    CU_TRY(cudaMemcpyAsync(dst, h.out[b], (size_t)n * row_bytes, cudaMemcpyDeviceToHost, h.s_out));
    CU_TRY(cudaEventRecord(h.out_done[b], h.s_out));
  }
  for (int b = 0; b < 2 && b < n_chunks; ++b) CU_TRY(cudaStreamWaitEvent(st, h.out_done[b], 0));
  L->launches = launches;
  return CMOE_OK;
}

int cmoe_quantise_rows_fp8(const void* w, int32_t rows, int32_t cols, uint8_t* codes, float* scale, void* dequantised,
                           void* stream) {
  if (rows < 0 || cols < 0) return arg_fail(CMOE_ERR_INVALID_ARG, "negative size");
  if (rows == 0) return CMOE_OK;
  if (!w || !scale || (cols > 0 && !codes)) return arg_fail(CMOE_ERR_INVALID_ARG, "null w / codes / scale");
  quantise_rows_fp8_kernel<<<rows, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      (const bf16*)w, rows, cols, cols, codes, cols, scale, (bf16*)dequantised);
  CU_TRY(cudaGetLastError());
  return CMOE_OK;
}

int cmoe_layer_quantise_fp8(cmoe_layer* L, void* stream) {
  if (!L) return arg_fail(CMOE_ERR_INVALID_ARG, "null layer");
  if (L->fp8) return CMOE_OK;
  if (L->cfg.dtype != CMOE_BF16 || !L->umma_ok)
    return arg_fail(CMOE_ERR_UNSUPPORTED, "FP8 weights need a bf16 layer on the tensor-core path");
  if (L->cfg.d_model % 16 || L->m % 16 || L->shared_width() % 16)
    return arg_fail(CMOE_ERR_UNSUPPORTED, "FP8 weights need d_model, the expert width and the shared width to be multiples of 16");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t d = L->cfg.d_model, rows_w = (size_t)L->n_outer * L->cfg.d_ff;
  CU_TRY(cudaMalloc(&L->w_gu8, 2 * rows_w * d));
  CU_TRY(cudaMalloc(&L->wd8, rows_w * d));
  CU_TRY(cudaMalloc(&L->scale_gu, 2 * rows_w * sizeof(float)));
  CU_TRY(cudaMalloc(&L->scale_d, (size_t)L->n_groups_total() * d * sizeof(float)));
  // gate and up planes: one scale per neuron row; the bf16 rows are replaced by the dequantised values
  quantise_rows_fp8_kernel<<<(unsigned)(2 * rows_w), 256, 0, st>>>((const bf16*)L->w_gu, (int)(2 * rows_w), (int)d, (long long)d,
                                                                 L->w_gu8, (long long)d, L->scale_gu, (bf16*)L->w_gu);
  // W_down: every group's block [d, width] has one scale per output channel
  for (size_t g = 0; g < L->gs_host.size(); ++g) {
    const GroupStatic& gs = L->gs_host[g];
    if (gs.width <= 0) continue;
    bf16* blk = (bf16*)L->wd_p + gs.wd_offset;
    quantise_rows_fp8_kernel<<<(unsigned)d, 256, 0, st>>>(blk, (int)d, gs.width, (long long)gs.width, L->wd8 + gs.wd_offset,
                                                         (long long)gs.width, L->scale_d + g * d, blk);
  }
  CU_TRY(cudaGetLastError());
  CU_TRY(cudaStreamSynchronize(st));
  // token planes for batches of at most kDecMaxRows outer rows: x, H_s (that many rows), H_r (rows x N_k)
  DecodeFp8Buffers f{};
  f.w_gu8 = L->w_gu8; f.wd8 = L->wd8; f.scale_gu = L->scale_gu; f.scale_d = L->scale_d;
  f.xq_rows = kDecMaxRows;
  f.hr_rows = (size_t)kDecMaxRows * (L->cfg.top_k > 0 ? L->cfg.top_k : 1);
  {
    Arena a;
    auto carve = [&](char* base) {
      a.base = base; a.used = 0;
      f.xq = a.take<uint8_t>(2 * f.xq_rows * d);
      f.hq_s = a.take<uint8_t>(2 * f.xq_rows * (L->shared_width() > 0 ? L->shared_width() : 16));
      f.hq_r = a.take<uint8_t>(2 * f.hr_rows * L->m);
      f.x_scale = a.take<float>(f.xq_rows);
      f.hs_scale = a.take<float>(f.xq_rows);
      f.hr_scale = a.take<float>(f.hr_rows);
    };
    carve(nullptr);
    const size_t bytes = a.used + 256;
    CU_TRY(cudaMalloc(&L->fp8_tok, bytes));
    CU_TRY(cudaMemset(L->fp8_tok, 0, bytes));
    carve(static_cast<char*>(L->fp8_tok));
  }
  if (!decode_plan_attach_fp8(&L->umma, &L->decode, f))
    return arg_fail(CMOE_ERR_CUDA, L->umma.error);
  L->fp8 = true;
  return CMOE_OK;
}

int cmoe_profile_activations(cmoe_layer* L, const void* x, int32_t T, int32_t k_a, int32_t token0,
                             uint32_t* act_bits, int32_t words_per_neuron, int32_t* act_count, void* stream) {
  if (!L) return arg_fail(CMOE_ERR_INVALID_ARG, "null layer");
  if (L->hier || L->n_r != 0 || L->cfg.n_shared != L->cfg.n_experts)
    return arg_fail(CMOE_ERR_INVALID_ARG, "profiling needs a plain layer whose experts are all shared");
  if (T < 0 || token0 < 0) return arg_fail(CMOE_ERR_INVALID_ARG, "negative token count / offset");
  if (T == 0) return CMOE_OK;
  if (!x || !act_bits || !act_count) return arg_fail(CMOE_ERR_INVALID_ARG, "null x / act_bits / act_count");
  if (T > L->cfg.max_tokens) return arg_fail(CMOE_ERR_CAPACITY, "T exceeds max_tokens");
  if (k_a < 1 || k_a > L->cfg.d_ff) return arg_fail(CMOE_ERR_INVALID_ARG, "k_a outside [1, d_ff]");
  if ((long long)words_per_neuron * 32 < (long long)token0 + T)
    return arg_fail(CMOE_ERR_CAPACITY, "words_per_neuron too small for token0 + n_tokens");
  if (reinterpret_cast<uintptr_t>(x) & 15) return arg_fail(CMOE_ERR_INVALID_ARG, "x must be 16-byte aligned");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  L->last_stream = st;
  L->last_T = T;
  const int d_ff = L->cfg.d_ff;
  // a row's keys are staged in dynamic shared memory next to the kernel's static arrays; both must fit 48 KB
  if ((size_t)d_ff * L->esz + kAtopkStaticSmem > 48 * 1024)
    return arg_fail(CMOE_ERR_UNSUPPORTED, "profiling supports d_ff up to 20352 (bf16) / 10176 (fp32)");
  int rc;
  if (L->cfg.dtype == CMOE_BF16) {
    rc = forward_impl<bf16>(L, (const bf16*)x, T, nullptr, st, true);
    if (rc == CMOE_OK)
      atopk_kernel<bf16><<<T, kAtopkThreads, (size_t)d_ff * sizeof(uint16_t), st>>>((const bf16*)L->h_s, d_ff, d_ff, k_a, token0, act_bits,
                                                      words_per_neuron, act_count);
  } else {
    rc = forward_impl<float>(L, (const float*)x, T, nullptr, st, true);
    if (rc == CMOE_OK)
      atopk_kernel<float><<<T, kAtopkThreads, (size_t)d_ff * sizeof(uint32_t), st>>>((const float*)L->h_s, d_ff, d_ff, k_a, token0, act_bits,
                                                       words_per_neuron, act_count);
  }
  if (rc != CMOE_OK) return rc;
  L->launches += 1;
  CU_TRY(cudaGetLastError());
  return CMOE_OK;
}

int cmoe_select_shared(const int32_t* act_count, int32_t d_ff, int32_t n_select, int32_t* shared_idx, void* stream) {
  if (d_ff < 0 || n_select < 0 || n_select > d_ff) return arg_fail(CMOE_ERR_INVALID_ARG, "n_select outside [0, d_ff]");
  if (d_ff == 0 || n_select == 0) return CMOE_OK;
  if (!act_count || !shared_idx) return arg_fail(CMOE_ERR_INVALID_ARG, "null act_count / shared_idx");
  select_shared_kernel<<<(d_ff + 31) / 32, 256, 0, static_cast<cudaStream_t>(stream)>>>(act_count, d_ff, n_select,
                                                                                         shared_idx);
  CU_TRY(cudaGetLastError());
  return CMOE_OK;
}

namespace {
int check_cluster_args(const uint32_t* act_bits, int32_t words, int32_t q, const int32_t* neuron_idx, int32_t n,
                       int32_t n_clusters) {
  if (words < 1 || q < 1 || (long long)words * 32 < q) return arg_fail(CMOE_ERR_INVALID_ARG, "words_per_neuron * 32 < n_tokens");
  if (n < 0 || n_clusters < 1 || n_clusters > kClusterMax)
    return arg_fail(CMOE_ERR_INVALID_ARG, "n < 0 or n_clusters outside [1, 32]");
  if ((long long)q * (n > 0 ? n : 1) > 0x7fffffffLL) return arg_fail(CMOE_ERR_CAPACITY, "n_tokens * n exceeds 2^31 - 1");
  if (!act_bits || (n > 0 && !neuron_idx)) return arg_fail(CMOE_ERR_INVALID_ARG, "null act_bits / neuron_idx");
  return CMOE_OK;
}
}  // namespace

int cmoe_cluster_update(const uint32_t* act_bits, int32_t words_per_neuron, int32_t n_tokens,
                        const int32_t* neuron_idx, const int32_t* assign, int32_t n, int32_t n_clusters,
                        int32_t* centroid_count, int32_t* cluster_size, void* stream) {
  const int rc = check_cluster_args(act_bits, words_per_neuron, n_tokens, neuron_idx, n, n_clusters);
  if (rc != CMOE_OK) return rc;
  if (!centroid_count || !cluster_size || (n > 0 && !assign))
    return arg_fail(CMOE_ERR_INVALID_ARG, "null assign / centroid_count / cluster_size");
  if (n == 0) return CMOE_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cluster_reset_kernel<<<n_clusters, 256, 0, st>>>(assign, n, n_tokens, centroid_count, cluster_size);
  cluster_accumulate_kernel<<<(n + 7) / 8, 256, 0, st>>>(act_bits, words_per_neuron, n_tokens, neuron_idx, assign, n,
                                                        n_clusters, centroid_count);
  CU_TRY(cudaGetLastError());
  return CMOE_OK;
}

int cmoe_cluster_distances(const uint32_t* act_bits, int32_t words_per_neuron, int32_t n_tokens,
                           const int32_t* neuron_idx, int32_t n, const int32_t* centroid_count,
                           const int32_t* cluster_size, int32_t n_clusters, int64_t* centroid_sqnorm,
                           int64_t* scaled_sq_dist, void* stream) {
  const int rc = check_cluster_args(act_bits, words_per_neuron, n_tokens, neuron_idx, n, n_clusters);
  if (rc != CMOE_OK) return rc;
  if (!centroid_count || !cluster_size || !centroid_sqnorm || (n > 0 && !scaled_sq_dist))
    return arg_fail(CMOE_ERR_INVALID_ARG, "null centroid_count / cluster_size / centroid_sqnorm / scaled_sq_dist");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  static_assert(sizeof(long long) == sizeof(int64_t), "int64_t is long long here");
  centroid_norm_kernel<<<n_clusters, 256, 0, st>>>(centroid_count, n_tokens, reinterpret_cast<long long*>(centroid_sqnorm));
  if (n > 0)
    cluster_distance_kernel<<<(n + 7) / 8, 256, 0, st>>>(act_bits, words_per_neuron, n_tokens, neuron_idx, n,
                                                        centroid_count, cluster_size,
                                                        reinterpret_cast<const long long*>(centroid_sqnorm), n_clusters,
                                                        reinterpret_cast<long long*>(scaled_sq_dist));
  CU_TRY(cudaGetLastError());
  return CMOE_OK;
}

int cmoe_cluster_representatives(const int64_t* scaled_sq_dist, const int32_t* neuron_idx, const int32_t* assign,
                                 int32_t n, int32_t n_clusters, int32_t* rep_neuron, void* stream) {
  if (n < 0 || n_clusters < 1 || n_clusters > kClusterMax)
    return arg_fail(CMOE_ERR_INVALID_ARG, "n < 0 or n_clusters outside [1, 32]");
  if (!rep_neuron || (n > 0 && (!scaled_sq_dist || !neuron_idx || !assign)))
    return arg_fail(CMOE_ERR_INVALID_ARG, "null scaled_sq_dist / neuron_idx / assign / rep_neuron");
  cluster_representative_kernel<<<n_clusters, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      reinterpret_cast<const long long*>(scaled_sq_dist), neuron_idx, assign, n, n_clusters, rep_neuron);
  CU_TRY(cudaGetLastError());
  return CMOE_OK;
}

int cmoe_layer_set_gate_params(cmoe_layer* L, const float* u, const float* b, void* stream) {
  if (!L) return arg_fail(CMOE_ERR_INVALID_ARG, "null layer");
  return upload_gate_params(L, u, b, static_cast<cudaStream_t>(stream));
}

int cmoe_layer_get_gate_params(cmoe_layer* L, float* u, float* b, void* stream) {
  if (!L) return arg_fail(CMOE_ERR_INVALID_ARG, "null layer");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t n = (size_t)L->n_outer * L->n_r;
  if (n && u) CU_TRY(cudaMemcpyAsync(u, L->u, n * sizeof(float), cudaMemcpyDeviceToHost, st));
  if (n && b) CU_TRY(cudaMemcpyAsync(b, L->b, n * sizeof(float), cudaMemcpyDeviceToHost, st));
  CU_TRY(cudaStreamSynchronize(st));
  return CMOE_OK;
}

int cmoe_layer_update_bias(cmoe_layer* L, float gamma, const float* target_share, float* utilisation,
                           void* stream) {
  if (!L) return arg_fail(CMOE_ERR_INVALID_ARG, "null layer");
  if (!(gamma >= 0.0f)) return arg_fail(CMOE_ERR_INVALID_ARG, "gamma must be non-negative");
  const size_t n = (size_t)L->n_outer * L->n_r;
  if (n == 0 || L->cfg.top_k == 0) return arg_fail(CMOE_ERR_INVALID_ARG, "layer has no routed experts");
  if (L->last_T == 0) return arg_fail(CMOE_ERR_INVALID_ARG, "no forward has run yet");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (target_share)
    CU_TRY(cudaMemcpyAsync(L->target, target_share, n * sizeof(float), cudaMemcpyHostToDevice, st));
  bias_update_kernel<<<(L->n_outer + 7) / 8, 256, 0, st>>>(L->counts, L->n_outer, L->n_r,
                                                          target_share ? L->target : nullptr, gamma, L->b,
                                                          L->share);
  CU_TRY(cudaGetLastError());
  if (utilisation) {
    CU_TRY(cudaMemcpyAsync(utilisation, L->share, n * sizeof(float), cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaStreamSynchronize(st));
  } else if (target_share) {
    CU_TRY(cudaStreamSynchronize(st));      // the host array was read asynchronously
  }
  return CMOE_OK;
}

int cmoe_layer_set_gemm_path(cmoe_layer* L, int32_t path) {
  if (!L || path < 0 || path > 3) return arg_fail(CMOE_ERR_INVALID_ARG, "gemm path");
  if (path >= 2 && !L->umma_ok)
    return arg_fail(CMOE_ERR_INVALID_ARG, "tensor-core path not available for this layer");
  L->gemm_path = path;
  return CMOE_OK;
}

int cmoe_layer_set_launch_chaining(cmoe_layer* L, int32_t on) {
  if (!L) return arg_fail(CMOE_ERR_INVALID_ARG, "null layer");
  L->chain_launches = on != 0;
  return CMOE_OK;
}

int cmoe_layer_dims(const cmoe_layer* L, int32_t* n_routed_groups, int32_t* top_k, int32_t* n_outer,
                    int32_t* outer_top_k) {
  if (!L) return arg_fail(CMOE_ERR_INVALID_ARG, "null layer");
  if (n_routed_groups) *n_routed_groups = L->n_outer * L->n_r;
  if (top_k) *top_k = L->cfg.top_k;
  if (n_outer) *n_outer = L->hier ? L->n_outer : 0;
  if (outer_top_k) *outer_top_k = L->hier ? L->outer_k : 0;
  return CMOE_OK;
}

int cmoe_get_routing(cmoe_layer* L, float* keys, float* scores, int32_t* topk_idx, float* topk_gate,
                     int32_t* counts, int32_t* offsets, int32_t* row_token, int32_t* row_of,
                     int32_t* outer_idx, float* outer_w, int32_t* outer_row_token) {
  if (!L) return arg_fail(CMOE_ERR_INVALID_ARG, "null layer");
  cudaStream_t st = L->last_stream;
  const size_t T = L->last_T, R = T * (L->hier ? L->outer_k : 1), P = R * L->cfg.top_k;
  const size_t nr = L->n_r, G = (size_t)L->n_outer * nr;
  const auto D2H = cudaMemcpyDeviceToHost;
  if (T > 0 && nr > 0) {
    if (keys) CU_TRY(cudaMemcpyAsync(keys, L->keys, R * nr * 4, D2H, st));
    if (scores) CU_TRY(cudaMemcpyAsync(scores, L->scores, R * nr * 4, D2H, st));
    if (topk_idx && P) CU_TRY(cudaMemcpyAsync(topk_idx, L->topk_idx, P * 4, D2H, st));
    if (topk_gate && P) CU_TRY(cudaMemcpyAsync(topk_gate, L->topk_gate, P * 4, D2H, st));
    if (counts) CU_TRY(cudaMemcpyAsync(counts, L->counts, G * 4, D2H, st));
    if (offsets) CU_TRY(cudaMemcpyAsync(offsets, L->offsets, (G + 1) * 4, D2H, st));
    if (row_token && P) CU_TRY(cudaMemcpyAsync(row_token, L->row_token, P * 4, D2H, st));
    if (row_of && P) CU_TRY(cudaMemcpyAsync(row_of, L->row_of, P * 4, D2H, st));
  }
  if (T > 0 && L->hier) {
    if (outer_idx) CU_TRY(cudaMemcpyAsync(outer_idx, L->outer_idx, R * 4, D2H, st));
    if (outer_w) CU_TRY(cudaMemcpyAsync(outer_w, L->outer_w, R * 4, D2H, st));
    if (outer_row_token) CU_TRY(cudaMemcpyAsync(outer_row_token, L->outer_row_token, R * 4, D2H, st));
  }
  CU_TRY(cudaStreamSynchronize(st));
  return CMOE_OK;
}

int cmoe_layer_status(cmoe_layer* L, int32_t* device_error_word) {
  if (!L || !device_error_word) return arg_fail(CMOE_ERR_INVALID_ARG, "null argument");
  CU_TRY(cudaMemcpyAsync(device_error_word, L->err_word, 4, cudaMemcpyDeviceToHost, L->last_stream));
  CU_TRY(cudaStreamSynchronize(L->last_stream));
  if (*device_error_word == 0) return CMOE_OK;
  // A wait gave up: that forward's output is undefined and its K-slice tickets may be left part-taken.
  // Clear the error word and every ticket so that the next forward starts from a clean state.
  cudaStream_t st = L->last_stream;
  CU_TRY(cudaMemsetAsync(L->err_word, 0, 4, st));
  CU_TRY(cudaMemsetAsync(L->rsk_ticket, 0, 4 * (kRskMaxChunks + 1), st));
  if (L->dec_ticket) CU_TRY(cudaMemsetAsync(L->dec_ticket, 0, L->n_dec_ticket * 4, st));
  if (L->rt_ticket) CU_TRY(cudaMemsetAsync(L->rt_ticket, 0, L->n_rt_ticket * 4, st));
  CU_TRY(cudaStreamSynchronize(st));
  return CMOE_ERR_DEVICE_TIMEOUT;
}

int cmoe_layer_selftest_wait_timeout(cmoe_layer* L, int64_t limit_cycles, void* stream) {
  if (!L) return arg_fail(CMOE_ERR_INVALID_ARG, "null layer");
  if (limit_cycles < 1000 || limit_cycles > 2000000000LL)
    return arg_fail(CMOE_ERR_INVALID_ARG, "limit_cycles outside [1e3, 2e9]");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  L->last_stream = st;
  wait_timeout_probe_kernel<<<1, 32, 0, st>>>(L->err_word, (long long)limit_cycles);
  CU_TRY(cudaGetLastError());
  return CMOE_OK;
}

int cmoe_layer_launch_count(const cmoe_layer* L, int32_t* n_launches) {
  if (!L || !n_launches) return arg_fail(CMOE_ERR_INVALID_ARG, "null argument");
  *n_launches = L->launches;
  return CMOE_OK;
}

int cmoe_layer_enable_stage_timing(cmoe_layer* L, int32_t ring_steps) {
  if (!L || ring_steps < 0 || ring_steps > 4096) return arg_fail(CMOE_ERR_INVALID_ARG, "stage timing ring");
  for (cudaEvent_t e : L->ev) cudaEventDestroy(e);
  L->ev.clear();
  L->ev_ring = 0;
  L->ev_count = 0;
  for (int i = 0; i < ring_steps * (CMOE_N_STAGES + 1); ++i) {
    cudaEvent_t e;
    CU_TRY(cudaEventCreate(&e));
    L->ev.push_back(e);
  }
  L->ev_ring = ring_steps;
  return CMOE_OK;
}

int cmoe_layer_stage_times(cmoe_layer* L, float* ms_sum, int32_t* n_steps) {
  if (!L || !ms_sum || !n_steps) return arg_fail(CMOE_ERR_INVALID_ARG, "null argument");
  for (int s = 0; s < CMOE_N_STAGES; ++s) ms_sum[s] = 0.0f;
  *n_steps = 0;
  if (!L->ev_ring) return CMOE_OK;
  CU_TRY(cudaStreamSynchronize(L->last_stream));
  const long long n = L->ev_count < L->ev_ring ? L->ev_count : L->ev_ring;
  for (long long i = 0; i < n; ++i) {
    cudaEvent_t* ev = &L->ev[(size_t)i * (CMOE_N_STAGES + 1)];
    for (int s = 0; s < CMOE_N_STAGES; ++s) {
      float ms = 0.0f;
      CU_TRY(cudaEventElapsedTime(&ms, ev[s], ev[s + 1]));
      ms_sum[s] += ms;
    }
  }
  *n_steps = (int32_t)n;
  return CMOE_OK;
}

int cmoe_layer_destroy(cmoe_layer* L) {
  if (!L) return CMOE_OK;
  free_layer(L);
  return CMOE_OK;
}

int64_t cmoe_token_permute_scratch_bytes(int32_t n_rows, int32_t n_groups) {
  if (n_rows < 0 || n_groups <= 0) return 0;
  return permute_scratch_bytes(n_rows, n_groups);
}

int cmoe_token_permute(const int32_t* topk_idx, int32_t n_rows, int32_t n_k, int32_t n_groups,
                       int32_t* counts, int32_t* offsets, int32_t* row_token, int32_t* row_of,
                       void* scratch, int64_t scratch_bytes, void* stream) {
  if (n_rows < 0 || n_k < 0 || n_k > kMaxTopK || n_groups <= 0 || n_groups > kPermMaxGroups)
    return arg_fail(CMOE_ERR_INVALID_ARG, "permute: size out of range");
  if (!counts || !offsets || ((int64_t)n_rows * n_k > 0 && (!topk_idx || !row_token || !row_of)))
    return arg_fail(CMOE_ERR_INVALID_ARG, "permute: null pointer");
  if (n_rows > kPermChunk) {
    if (!scratch || (reinterpret_cast<uintptr_t>(scratch) & 255))
      return arg_fail(CMOE_ERR_INVALID_ARG, "permute: scratch null or not 256-byte aligned");
    if (scratch_bytes < permute_scratch_bytes(n_rows, n_groups))
      return arg_fail(CMOE_ERR_CAPACITY, "permute: scratch too small");
  }
  launch_token_permute(topk_idx, n_rows, n_k, n_groups, counts, offsets, row_token, row_of,
                       static_cast<int32_t*>(scratch), static_cast<cudaStream_t>(stream));
  CU_TRY(cudaGetLastError());
  return CMOE_OK;
}

}  // extern "C" (re-opened below)

// ---------------------------------------------------------------------------
// Token permutation for callers that cannot allocate device memory.
//
// The chunk-count matrix of the permutation lives in this fixed array instead of
// a caller-supplied buffer.  Every GPU that loads the library holds these
// kStaticPermInts * 4 bytes (1 MiB) until the process exits.  The name below is
// only meaningful to device code; the host obtains the array's device address
// once per device through cudaGetSymbolAddress and passes that to the kernels.
constexpr int64_t kStaticPermInts = 262144;   // n_chunks * n_groups may not exceed this
static __device__ __align__(256) int32_t g_static_perm_scratch[kStaticPermInts];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_perm_mutex;
int32_t* g_static_perm_addr[kMaxDevices] = {};   // device address of the array, per device

// Device address of g_static_perm_scratch on the current device (looked up once).
int static_perm_scratch(int32_t** out) {
  int dev = 0;
  CU_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return arg_fail(CMOE_ERR_INVALID_ARG, "device ordinal too large");
  std::lock_guard<std::mutex> lock(g_static_perm_mutex);
  if (!g_static_perm_addr[dev]) {
    void* p = nullptr;
    CU_TRY(cudaGetSymbolAddress(&p, g_static_perm_scratch));
    g_static_perm_addr[dev] = static_cast<int32_t*>(p);
  }
  *out = g_static_perm_addr[dev];
  return CMOE_OK;
}
}  // namespace

extern "C" {

int cmoe_token_permute_static(const int32_t* topk_idx, int32_t n_rows, int32_t n_k,
                              int32_t n_groups, int32_t* counts, int32_t* offsets,
                              int32_t* row_token, int32_t* row_of, void* stream) {
  if (n_rows < 0 || n_k < 0 || n_k > kMaxTopK || n_groups <= 0 || n_groups > kPermMaxGroups)
    return arg_fail(CMOE_ERR_INVALID_ARG, "permute: size out of range");
  if (!counts || !offsets || ((int64_t)n_rows * n_k > 0 && (!topk_idx || !row_token || !row_of)))
    return arg_fail(CMOE_ERR_INVALID_ARG, "permute: null pointer");
  const int64_t n_chunks = ((int64_t)n_rows + kPermChunk - 1) / kPermChunk;
  if (n_rows > kPermChunk && n_chunks * n_groups > kStaticPermInts)
    return arg_fail(CMOE_ERR_CAPACITY,
                    "permute (static scratch): ceil(n_rows/256) * n_groups exceeds 262144 cells");
  int32_t* scratch = nullptr;
  const int rc = static_perm_scratch(&scratch);
  if (rc != CMOE_OK) return rc;
  // Every cell the scan and scatter kernels read is first written by the count kernel of
  // the same call, so nothing left over from an earlier call needs clearing.
  launch_token_permute(topk_idx, n_rows, n_k, n_groups, counts, offsets, row_token, row_of, scratch,
                       static_cast<cudaStream_t>(stream));
  CU_TRY(cudaGetLastError());
  return CMOE_OK;
}

const char* cmoe_status_string(int status) {
  switch (status) {
    case CMOE_OK: return "ok";
    case CMOE_ERR_INVALID_ARG: return "invalid argument";
    case CMOE_ERR_BAD_PARTITION: return "neuron partition is not a permutation into equal experts";
    case CMOE_ERR_BAD_REP: return "representative neuron outside its expert";
    case CMOE_ERR_CAPACITY: return "capacity exceeded";
    case CMOE_ERR_CUDA: return "CUDA error";
    case CMOE_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case CMOE_ERR_UNSUPPORTED: return "unsupported device";
    default: return "unknown status";
  }
}

const char* cmoe_last_error(void) { return g_last_error; }

}  // extern "C"
