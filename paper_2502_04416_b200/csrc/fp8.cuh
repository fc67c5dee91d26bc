// FP8 weight-only quantisation of the expert weights (the paper, Section 6, only states that the
// restructured FFN composes with post-training quantisation; the format is this library's choice):
// OCP E4M3 codes (bias 7, 3 mantissa bits, subnormals, largest value 448) with one power-of-two
// scale per output channel.  Because the scale is a power of two, w / scale is exact, the code
// is the round-to-nearest-even encoding of an exactly known number, and code * scale is exactly
// representable in bf16.
#pragma once

#include "common.cuh"

namespace cmoe {

// Two floats -> two E4M3 codes (round to nearest even, saturating): `lo` in bits 0..7.
__device__ __forceinline__ uint16_t f32x2_to_e4m3x2(float lo, float hi) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}
// Two E4M3 codes -> two floats (exact).
__device__ __forceinline__ float2 e4m3x2_to_f32x2(uint16_t v) {
  uint32_t h2;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(v));
  return __half22float2(*reinterpret_cast<const __half2*>(&h2));
}

// Four E4M3 codes (one 32-bit word, lowest byte first) -> four bf16 values as two packed words.
// A code's magnitude bits, shifted into a bf16's exponent / mantissa fields, read as
// 2^-120 times the code's value (also for subnormal codes, which become bf16 subnormals), so
// one exact multiplication by 2^120 finishes the conversion without a case distinction.
__device__ __forceinline__ void e4m3x4_to_bf16x4(uint32_t w, uint32_t& lo, uint32_t& hi) {
  const uint32_t a = __byte_perm(w, 0u, 0x1404);          // halfwords b0 << 8, b1 << 8
  const uint32_t b = __byte_perm(w, 0u, 0x3424);          // halfwords b2 << 8, b3 << 8
  const uint32_t ma = ((a >> 4) & 0x07F007F0u) | (a & 0x80008000u);
  const uint32_t mb = ((b >> 4) & 0x07F007F0u) | (b & 0x80008000u);
  const uint32_t two120 = 0x7B807B80u;                    // bf16 2^120, twice
  asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(lo) : "r"(ma), "r"(two120));
  asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(hi) : "r"(mb), "r"(two120));
}

// Smallest e with amax * 2^-e <= 448 = 0.875 * 2^9 (0 for amax == 0).
__device__ __forceinline__ int pow2_scale_exponent(float amax) {
  if (!(amax > 0.0f)) return 0;
  int p;
  const float f = frexpf(amax, &p);                       // amax = f * 2^p, f in [0.5, 1)
  return f <= 0.875f ? p - 9 : p - 8;
}

// One block per row of a bf16 matrix [rows, cols] (leading dimension ld elements): the row's
// scale 2^e, its E4M3 codes, and (when deq != nullptr, which may alias w) the dequantised row.
__global__ void __launch_bounds__(256)
quantise_rows_fp8_kernel(const bf16* w, int rows, int cols, long long ld, uint8_t* __restrict__ codes,
                         long long ld_codes, float* __restrict__ scale, bf16* deq) {
  const int r = blockIdx.x;
  if (r >= rows) return;
  const bf16* src = w + (size_t)r * ld;
  __shared__ float red[8];
  __shared__ float sh_amax;
  float amax = 0.0f;
  for (int c = threadIdx.x; c < cols; c += 256) {
    const float v = fabsf(__bfloat162float(src[c]));
    amax = (v > amax) ? v : amax;                          // NaN weights never raise the maximum
  }
  amax = warp_max(amax);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
  __syncthreads();
  if (threadIdx.x == 0) {
    float m = red[0];
    for (int i = 1; i < 8; ++i) m = fmaxf(m, red[i]);
    sh_amax = m;
  }
  __syncthreads();
  const int e = pow2_scale_exponent(sh_amax);
  if (threadIdx.x == 0) scale[r] = ldexpf(1.0f, e);
  uint8_t* dst = codes + (size_t)r * ld_codes;
  bf16* dq = deq ? deq + (size_t)r * ld : nullptr;
  for (int c = 2 * threadIdx.x; c < cols; c += 512) {
    const float v0 = ldexpf(__bfloat162float(src[c]), -e);
    const bool two = c + 1 < cols;
    const float v1 = two ? ldexpf(__bfloat162float(src[c + 1]), -e) : 0.0f;
    const uint16_t q = f32x2_to_e4m3x2(v0, v1);
    dst[c] = (uint8_t)(q & 0xFF);
    if (two) dst[c + 1] = (uint8_t)(q >> 8);
    if (dq) {
      const float2 back = e4m3x2_to_f32x2(q);
      dq[c] = __float2bfloat16_rn(ldexpf(back.x, e));
      if (two) dq[c + 1] = __float2bfloat16_rn(ldexpf(back.y, e));
    }
  }
}

// Splits bf16 rows into two E4M3 planes for the FP8 tensor-core path: with the row's power-of-two
// scale 2^e (largest magnitude brought to at most 448), hi = E4M3(v / 2^e) and lo = E4M3(16 (v / 2^e - hi)).
// A bf16 value has 8 significant bits, hi keeps the top 4 and the remainder is a multiple of the
// value's last place not above 8 of them, so lo holds it exactly unless it falls below E4M3's range
// (values under 2^-13 of the row's maximum): v = (hi + lo / 16) 2^e.  One block per row.
__device__ __forceinline__ void split_row_e4m3(const bf16* __restrict__ row, int cols, uint8_t* __restrict__ h,
                                               uint8_t* __restrict__ l, float* __restrict__ scale_out) {
  __shared__ float red[4];
  float amax = 0.0f;
  for (int c = 8 * threadIdx.x; c < cols; c += 8 * 128) {
    float v[8];
    load8(row + c, v);
#pragma unroll
    for (int q = 0; q < 8; ++q) { const float a = fabsf(v[q]); amax = (a > amax) ? a : amax; }
  }
  amax = warp_max(amax);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
  __syncthreads();
  const int e = pow2_scale_exponent(fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3])));
  if (threadIdx.x == 0) *scale_out = ldexpf(1.0f, e);
  for (int c = 8 * threadIdx.x; c < cols; c += 8 * 128) {
    float v[8];
    load8(row + c, v);
    uint32_t hw[2], lw[2];
#pragma unroll
    for (int q = 0; q < 8; q += 2) {
      const float v0 = ldexpf(v[q], -e), v1 = ldexpf(v[q + 1], -e);
      const uint16_t hq = f32x2_to_e4m3x2(v0, v1);
      const float2 back = e4m3x2_to_f32x2(hq);
      const uint16_t lq = f32x2_to_e4m3x2((v0 - back.x) * 16.0f, (v1 - back.y) * 16.0f);
      hw[q >> 2] = (q & 2) ? (hw[q >> 2] | ((uint32_t)hq << 16)) : (uint32_t)hq;
      lw[q >> 2] = (q & 2) ? (lw[q >> 2] | ((uint32_t)lq << 16)) : (uint32_t)lq;
    }
    *reinterpret_cast<uint2*>(h + c) = make_uint2(hw[0], hw[1]);
    *reinterpret_cast<uint2*>(l + c) = make_uint2(lw[0], lw[1]);
  }
}

// One segment of rows: src [rows, cols] bf16 (leading dimension ld) -> planes [2][plane_rows][cols], scales [rows].
struct SplitSegment {
  const bf16* src;
  int rows, cols;
  long long ld;
  uint8_t* planes;
  long long plane_rows;
  float* scale;
};

// Blocks 0 .. a.rows-1 split the rows of segment a, the next b.rows blocks those of segment b (b.rows may be 0).
__global__ void __launch_bounds__(128) split_rows_e4m3_kernel(const SplitSegment a, const SplitSegment b) {
  grid_dep_wait();
  grid_dep_trigger();
  int r = blockIdx.x;
  const SplitSegment& sg = r < a.rows ? a : b;
  if (r >= a.rows) r -= a.rows;
  if (r >= sg.rows) return;
  uint8_t* hi = sg.planes + (size_t)r * sg.cols;
  split_row_e4m3(sg.src + (size_t)r * sg.ld, sg.cols, hi, hi + (size_t)sg.plane_rows * sg.cols, sg.scale + r);
}

}  // namespace cmoe
