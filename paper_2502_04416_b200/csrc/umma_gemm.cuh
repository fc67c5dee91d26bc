// Tensor-core (tcgen05 / TMEM / TMA) grouped expert GEMMs.  Placeholder: plan creation
// reports "shape not taken", so every layer runs the SIMT kernels.
#pragma once

#include "common.cuh"

namespace cmoe {

struct UmmaShape {
  int d = 0, m = 0, shared_width = 0, d_ff = 0, n_outer = 1, n_r = 0;
  size_t max_outer_rows = 0, max_routed_rows = 0;
};

struct UmmaPlan {
  char error[256] = "";
};

// 0: plan built; 1: shape not taken by this path; CMOE_ERR_CUDA (-5): a driver call failed.
inline int umma_plan_create(UmmaPlan*, const UmmaShape&, const GroupStatic*, int, const void*,
                            const void*, const void*, void*, void*, void*, void*, void*) { return 1; }
inline void umma_plan_destroy(UmmaPlan*) {}
// Enqueues both expert GEMMs; returns the number of kernels launched or -1.
inline int umma_forward(UmmaPlan*, const void*, int, int, const GroupRows*, int32_t*, cudaStream_t,
                        cudaEvent_t /*recorded between GEMM-1 and GEMM-2, may be null*/) {
  return -1;
}

}  // namespace cmoe
