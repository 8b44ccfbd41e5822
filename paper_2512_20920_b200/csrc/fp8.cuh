// FP8 (e4m3) operands for the routed experts' products: per-row quantisation kernels.
//
//   scale[r] = max_c |x[r, c]| / 448      (1 for an all-zero row)
//   code[r, c] = e4m3(x[r, c] / scale[r]) round to nearest even, saturating at +-448
//
// all in fp32, so that a reference that rounds the same fp32 quotient the same way produces the same codes.
// A product of two operands quantised this way is  scale_a[m] * scale_b[n] * sum_k code_a[m,k] code_b[n,k];
// the two factors are applied in the product's epilogue.
#pragma once

#include <cuda_fp8.h>

#include "common.cuh"

namespace revffn {

constexpr float E4M3_MAX = 448.f;

__device__ __forceinline__ uint2 e4m3_pack8(const float* f, float scale) {
  uint32_t w[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const __nv_fp8x2_storage_t lo =
        __nv_cvt_float2_to_fp8x2(make_float2(f[4 * h] / scale, f[4 * h + 1] / scale), __NV_SATFINITE, __NV_E4M3);
    const __nv_fp8x2_storage_t hi =
        __nv_cvt_float2_to_fp8x2(make_float2(f[4 * h + 2] / scale, f[4 * h + 3] / scale), __NV_SATFINITE, __NV_E4M3);
    w[h] = (uint32_t)lo | ((uint32_t)hi << 16);
  }
  return make_uint2(w[0], w[1]);
}

// One block per output row.  row_map == NULL: out[r] = quantised in[r].  row_map != NULL (the permutation into the
// padded expert-major row space): out[r] = quantised in[row_map[r]], zeros with scale 1 for padding rows
// (row_map[r] < 0); rows at or beyond *rows_total are skipped.  width a multiple of 8, at most 8 * blockDim.x.
__global__ void __launch_bounds__(256)
quantize_rows_e4m3_kernel(const bf16* __restrict__ in, int64_t ld_in, const int32_t* __restrict__ row_map,
                          const int32_t* __restrict__ rows_total, int width, uint8_t* __restrict__ out,
                          float* __restrict__ scale) {
  __shared__ float red[32];
  const int row = blockIdx.x;
  if (rows_total && row >= *rows_total) return;
  int src = row;
  if (row_map) src = row_map[row];
  const int c = threadIdx.x * 8;
  float f[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) f[i] = 0.f;
  if (src >= 0 && c < width) {
    Vec8<bf16> v;
    v.load(in + (int64_t)src * ld_in + c);
    v.get(f);
  }
  float amax = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(f[i]));
  // block maximum (all threads take part, also those beyond the row's width)
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
  __syncthreads();
  amax = (threadIdx.x & 31) < (blockDim.x >> 5) ? red[threadIdx.x & 31] : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  const float s = amax > 0.f ? amax / E4M3_MAX : 1.f;
  if (threadIdx.x == 0) scale[row] = s;
  if (c < width) *reinterpret_cast<uint2*>(out + (int64_t)row * width + c) = e4m3_pack8(f, s);
}

inline cudaError_t launch_quantize_rows(const bf16* in, int64_t ld_in, const int32_t* row_map, const int32_t* rows_total,
                                        int64_t rows, int width, uint8_t* out, float* scale, cudaStream_t st) {
  if (rows <= 0) return cudaSuccess;
  if (width % 8 != 0 || width > 8 * 256) return cudaErrorInvalidValue;
  quantize_rows_e4m3_kernel<<<(unsigned)rows, 256, 0, st>>>(in, ld_in, row_map, rows_total, width, out, scale);
  return cudaGetLastError();
}

}  // namespace revffn
