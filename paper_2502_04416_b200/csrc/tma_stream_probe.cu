// Stand-alone probe (not part of libcmoe.so): how fast can CTAs stream DRAM through TMA
// boxes of 64 bf16 columns x box_rows rows when nothing else runs?  One producer thread
// keeps `stages` boxes in flight per CTA, one consumer thread frees them at once.  It
// bounds what the weight-streaming decode kernels can reach.  Build and run:
//   python -m paper_2502_04416_b200.build --probe && ./paper_2502_04416_b200/tma_stream_probe
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdio>
#include <cstdlib>
#include <vector>
#include "umma_gemm.cuh"
using namespace cmoe;

__global__ void __launch_bounds__(64, 1)
stream_kernel(const __grid_constant__ CUtensorMap tm, int box_rows, int n_kb, int n_tiles, int stages, int stage_bytes,
              unsigned long long* sink) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const uint32_t bars = base + stages * stage_bytes;
  const uint32_t full0 = bars, empty0 = bars + 128;
  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) {            // producer
    uint32_t it = 0;
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x)
      for (int kb = 0; kb < n_kb; ++kb, ++it) {
        const uint32_t s = it % stages, n = it / stages;
        for (long long spin = 0; !mbar_try_wait(empty0 + 8 * s, (n & 1) ^ 1); ++spin) if (spin > (1ll << 28)) return;
        mbar_expect_tx(full0 + 8 * s, box_rows * 128);
        tma_load_2d(base + s * stage_bytes, &tm, full0 + 8 * s, kb * 64, t * box_rows);
      }
  } else if (threadIdx.x == 32) {    // consumer
    uint32_t it = 0;
    unsigned long long acc = 0;
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x)
      for (int kb = 0; kb < n_kb; ++kb, ++it) {
        const uint32_t s = it % stages, n = it / stages;
        for (long long spin = 0; !mbar_try_wait(full0 + 8 * s, n & 1); ++spin) if (spin > (1ll << 28)) return;
        acc += *reinterpret_cast<volatile unsigned*>(smem_raw + (base - raw) + s * stage_bytes);
        mbar_arrive(empty0 + 8 * s);
      }
    if (acc == 0x123456789ull) *sink = acc;
  }
}

int main() {
  typedef CUresult (*PFN)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                          const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                          CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  void* fn = nullptr; cudaDriverEntryPointQueryResult q;
  cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
  PFN enc = (PFN)fn;
  const size_t bytes = 1ull << 30;               // 1 GiB buffer
  void* buf; cudaMalloc(&buf, bytes); cudaMemset(buf, 1, bytes);
  unsigned long long* sink; cudaMalloc(&sink, 8);
  cudaFuncSetAttribute(stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
  cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
  const int cols_list[] = {4096, 1376, 64};   // 64: every box is one contiguous 128 B x box_rows chunk
  for (int cols : cols_list)
  for (int promo = 0; promo < 2; ++promo)
  for (int box_rows : {64, 128, 256})
  for (int grid : {37, 74, 148})
  for (int stages : {4, 8, 16}) {
    const int stage_bytes = box_rows * 128;
    if (stages * stage_bytes > 200 * 1024) continue;
    const size_t rows_total = bytes / (cols * 2);
    const int n_tiles_all = rows_total / box_rows;
    // stream ~ 400 MB in total, distinct tiles
    const int n_kb = cols / 64 + (cols % 64 ? 1 : 0);
    int n_tiles = (int)(400e6 / ((double)box_rows * cols * 2));
    n_tiles = n_tiles / grid * grid; if (n_tiles > n_tiles_all) n_tiles = n_tiles_all / grid * grid;
    CUtensorMap tm;
    cuuint64_t dims[2] = {(cuuint64_t)cols, rows_total}; cuuint64_t str[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows}; cuuint32_t es[2] = {1, 1};
    CUresult r = enc(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, buf, dims, str, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, promo ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_NONE,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { printf("encode failed %d\n", (int)r); continue; }
    const int smem = 1024 + stages * stage_bytes + 512;
    float best = 1e9;
    for (int rep = 0; rep < 3; ++rep) {
      cudaMemsetAsync(buf, rep, 256 << 20);       // flush L2 with other data (first 256 MB rewritten)
      cudaEventRecord(e0);
      stream_kernel<<<grid, 64, smem>>>(tm, box_rows, n_kb, n_tiles, stages, stage_bytes, sink);
      cudaEventRecord(e1); cudaEventSynchronize(e1);
      float ms; cudaEventElapsedTime(&ms, e0, e1); if (ms < best) best = ms;
    }
    cudaError_t ce = cudaGetLastError();
    const double gb = (double)n_tiles * box_rows * cols * 2 / 1e9;
    printf("cols=%d promo=%d box_rows=%3d grid=%3d stages=%2d inflight/SM=%3dKB : %7.1f GB/s total, %6.1f GB/s per CTA (%s)\n", cols,
           promo, box_rows, grid, stages, stages * stage_bytes / 1024, gb / (best * 1e-3), gb / (best * 1e-3) / grid,
           cudaGetErrorString(ce));
  }
  return 0;
}
