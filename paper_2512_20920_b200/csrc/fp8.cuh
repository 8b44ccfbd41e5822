// FP8 (e4m3) operands for the routed experts' products: per-row quantisation kernels.
//
//   scale[r] = max_c |x[r, c]| / 448      (1 for an all-zero row)
//   code[r, c] = e4m3(x[r, c] * (1 / scale[r])) round to nearest even, saturating at +-448
//                (one correctly rounded reciprocal per row, one multiplication per element: a division per
//                element made the kernel ALU-bound at three times its memory time)
//
// all in fp32, so that a reference that rounds the same fp32 quotient the same way produces the same codes.
// A product of two operands quantised this way is  scale_a[m] * scale_b[n] * sum_k code_a[m,k] code_b[n,k];
// the two factors are applied in the product's epilogue.
#pragma once

#include <cuda_fp8.h>

#include "common.cuh"

namespace revffn {

constexpr float E4M3_MAX = 448.f;

__device__ __forceinline__ uint2 e4m3_pack8(const float* f, float inv) {
  uint32_t w[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const __nv_fp8x2_storage_t lo =
        __nv_cvt_float2_to_fp8x2(make_float2(__fmul_rn(f[4 * h], inv), __fmul_rn(f[4 * h + 1], inv)), __NV_SATFINITE, __NV_E4M3);
    const __nv_fp8x2_storage_t hi =
        __nv_cvt_float2_to_fp8x2(make_float2(__fmul_rn(f[4 * h + 2], inv), __fmul_rn(f[4 * h + 3], inv)), __NV_SATFINITE, __NV_E4M3);
    w[h] = (uint32_t)lo | ((uint32_t)hi << 16);
  }
  return make_uint2(w[0], w[1]);
}

// One warp per output row (8 rows per block); a lane keeps its up to eight 16-byte pieces of the row in registers
// between the maximum and the conversion, so the row is read once and nothing goes through shared memory.
// row_map == NULL: out[r] = quantised in[r].  row_map != NULL (the permutation into the padded expert-major row
// space): out[r] = quantised in[row_map[r]], zeros with scale 1 for padding rows (row_map[r] < 0); rows at or beyond
// *rows_total are skipped.  width a multiple of 8, at most 2048.
__global__ void __launch_bounds__(256)
quantize_rows_e4m3_kernel(const bf16* __restrict__ in, int64_t ld_in, const int32_t* __restrict__ row_map,
                          const int32_t* __restrict__ rows_total, int64_t rows, int width, uint8_t* __restrict__ out,
                          float* __restrict__ scale) {
  const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows || (rows_total && row >= *rows_total)) return;
  int64_t src = row;
  if (row_map) src = row_map[row];
  Vec8<bf16> v[8];
  float amax = 0.f;
#pragma unroll
  for (int it = 0; it < 8; ++it) {
    const int c = it * 256 + lane * 8;
    v[it].zero();
    if (src >= 0 && c < width) v[it].load(in + src * ld_in + c);
  }
#pragma unroll
  for (int it = 0; it < 8; ++it) {
    float f[8];
    v[it].get(f);
#pragma unroll
    for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(f[i]));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  const float s = amax > 0.f ? amax / E4M3_MAX : 1.f;
  const float inv = 1.f / s;
  if (lane == 0) scale[row] = s;
#pragma unroll
  for (int it = 0; it < 8; ++it) {
    const int c = it * 256 + lane * 8;
    if (c < width) {
      float f[8];
      v[it].get(f);
      *reinterpret_cast<uint2*>(out + row * width + c) = e4m3_pack8(f, inv);
    }
  }
}

inline cudaError_t launch_quantize_rows(const bf16* in, int64_t ld_in, const int32_t* row_map, const int32_t* rows_total,
                                        int64_t rows, int width, uint8_t* out, float* scale, cudaStream_t st) {
  if (rows <= 0) return cudaSuccess;
  if (width % 8 != 0 || width > 2048) return cudaErrorInvalidValue;
  quantize_rows_e4m3_kernel<<<(unsigned)ceil_div(rows, 8), 256, 0, st>>>(in, ld_in, row_map, rows_total, rows, width, out, scale);
  return cudaGetLastError();
}

}  // namespace revffn
