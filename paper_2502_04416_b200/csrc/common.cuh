// Shared device/host helpers of the cmoe library: element traits, vector
// loads, warp reductions, group descriptors.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

namespace cmoe {

constexpr int kMaxRouted = 32;   // N_r per (outer) layer: one lane per routed expert
constexpr int kMaxTopK = 8;      // N_k
constexpr int kMaxOuter = 32;    // experts of a hierarchical layer's top level

typedef __nv_bfloat16 bf16;

// Programmatic dependent launch: a kernel launched as a dependent may become resident while
// its predecessor in the stream is still running; grid_dep_wait() returns once that
// predecessor has completed and its writes are visible, so nothing it produces may be read
// (and nothing it reads may be written) before the call.  grid_dep_trigger() lets this grid's
// own dependent become resident as soon as every block has executed it.  Both are no-ops in
// a kernel that was launched the ordinary way.
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KP, typename... A>
inline cudaError_t launch_kernel(bool dependent, void (*kernel)(KP...), dim3 grid, dim3 block, size_t smem,
                                 cudaStream_t st, A&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at;
  at.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &at; cfg.numAttrs = dependent ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<A>(args)...);
}

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(bf16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_float(float v);
template <> __device__ __forceinline__ float from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_float<bf16>(float v) { return __float2bfloat16_rn(v); }

// Eight consecutive elements starting at p (p 16-byte aligned).
__device__ __forceinline__ void load8(const bf16* p, float (&v)[8]) {
  const uint4 raw = __ldg(reinterpret_cast<const uint4*>(p));
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
  const float4 a = __ldg(reinterpret_cast<const float4*>(p));
  const float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

__device__ __forceinline__ void store8(bf16* p, const float (&v)[8]) {
  uint4 raw;
  raw.x = pack_bf16x2(v[0], v[1]);
  raw.y = pack_bf16x2(v[2], v[3]);
  raw.z = pack_bf16x2(v[4], v[5]);
  raw.w = pack_bf16x2(v[6], v[7]);
  *reinterpret_cast<uint4*>(p) = raw;
}
__device__ __forceinline__ void store8(float* p, const float (&v)[8]) {
  reinterpret_cast<float4*>(p)[0] = make_float4(v[0], v[1], v[2], v[3]);
  reinterpret_cast<float4*>(p)[1] = make_float4(v[4], v[5], v[6], v[7]);
}

// Sixteen consecutive bf16 elements with one 32-byte access (p 32-byte aligned).
__device__ __forceinline__ void store16(bf16* p, const float* v) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"l"(p), "r"(pack_bf16x2(v[0], v[1])), "r"(pack_bf16x2(v[2], v[3])),
                 "r"(pack_bf16x2(v[4], v[5])), "r"(pack_bf16x2(v[6], v[7])), "r"(pack_bf16x2(v[8], v[9])),
                 "r"(pack_bf16x2(v[10], v[11])), "r"(pack_bf16x2(v[12], v[13])), "r"(pack_bf16x2(v[14], v[15]))
               : "memory");
}
__device__ __forceinline__ void load16(const bf16* p, float* v) {
  uint32_t w[8];
  asm volatile("ld.global.nc.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
               : "l"(p));
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// SiLU (Swish with beta = 1) with the accurate exponential and division.
__device__ __forceinline__ float silu_accurate(float a) { return a / (1.0f + expf(-a)); }

// Static description of one expert group (shared or routed) of a layer.
struct GroupStatic {
  int32_t w_row0;      // first row of the group's neurons in the packed W_gate / W_up
  int32_t width;       // neurons in the group: N_s*m (shared) or m (routed)
  int64_t wd_offset;   // element offset of the group's [d, width] block in the packed W_down
  int32_t is_shared;   // 1: rows come from the outer-row order; 0: from the routed-row order
  int32_t outer;       // outer expert the group belongs to (0 for a plain layer)
};

// Per-forward row range of a group, written by plan_groups_kernel.
struct GroupRows {
  int32_t row0;        // first row in the group's row space (outer rows / routed rows)
  int32_t count;       // rows in the group
};

}  // namespace cmoe
