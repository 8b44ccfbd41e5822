// Attention coupling branch (Eq. 1): the steps of Attn_pt that are not plain matrix products.
//
//   rope_table        (cos, sin)(s * theta^(-2i/hd)) for every position and rotated pair, from fp64
//   to_heads          token-major [T, n*hd] (+ bias, + rotation) -> head-major [B, n, S_pad, hd]
//   from_heads        head-major -> token-major, optionally with the opposite rotation (backward)
//   softmax_causal    P = softmax(scale * scores) over keys 0..s of query position s
//   dsoftmax_causal   dS = scale * P * (dP - <P, dP>)
//   attn_tables       row-block -> key/value group table and group offsets for the grouped products
//
// Head-major buffers pad every (sequence, head) to S_pad = round_up(S, ROW_PAD) rows, so that a
// 128-row tile of a grouped product never spans two heads; the padding rows are kept at zero.
#pragma once

#include "common.cuh"

namespace revffn {

__global__ void rope_table_kernel(int S, int hd, double theta, float2* __restrict__ cs) {
  const int half = hd / 2;
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= S * half) return;
  int s = idx / half, i = idx % half;
  double ang = (double)s * pow(theta, -2.0 * (double)i / (double)hd);
  double sn, c;
  sincos(ang, &sn, &c);
  cs[idx] = make_float2((float)c, (float)sn);
}

// RMSNorm of both streams in one launch: warp w < tokens normalises row w of x1, the others row w - tokens of x2;
// output rows in that order (the layout the shared P_up product reads).  Same arithmetic as rmsnorm_fwd_kernel.
template <typename T>
__global__ void rmsnorm2_fwd_kernel(const float* __restrict__ x1, const float* __restrict__ x2, int64_t ld,
                                    const float* __restrict__ gamma, float eps, int tokens, int h, T* __restrict__ n_out,
                                    float* __restrict__ r_out) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp >= 2 * tokens) return;
  const float* row = warp < tokens ? x1 + (int64_t)warp * ld : x2 + (int64_t)(warp - tokens) * ld;
  float ss = 0.f;
  for (int i = lane * 4; i < h; i += 128) {
    float4 v = *reinterpret_cast<const float4*>(row + i);
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = warp_sum(ss);
  const float r = rsqrtf(ss / (float)h + eps);
  if (lane == 0) r_out[warp] = r;
  T* out = n_out + (int64_t)warp * h;
  for (int i = lane * 4; i < h; i += 128) {
    float4 v = *reinterpret_cast<const float4*>(row + i);
    float4 g = make_float4(1.f, 1.f, 1.f, 1.f);
    if (gamma) g = *reinterpret_cast<const float4*>(gamma + i);
    out[i + 0] = from_f32<T>(v.x * r * g.x);
    out[i + 1] = from_f32<T>(v.y * r * g.y);
    out[i + 2] = from_f32<T>(v.z * r * g.z);
    out[i + 3] = from_f32<T>(v.w * r * g.w);
  }
}

// One block per token.  in: [T, ld_in] with n heads of hd columns; out: [B, n, S_pad, hd].
template <typename TIn, typename T>
__global__ void to_heads_kernel(const TIn* __restrict__ in, int64_t ld_in, const float* __restrict__ bias,
                                const float2* __restrict__ cs, int S, int Sp, int n, int hd, T* __restrict__ out) {
  const int t = blockIdx.x, b = t / S, s = t % S, half = hd / 2;
  const TIn* row = in + (int64_t)t * ld_in;
  for (int p = threadIdx.x; p < n * half; p += blockDim.x) {
    const int head = p / half, i = p % half;
    const int c0 = head * hd + i, c1 = c0 + half;
    float x0 = to_f32(row[c0]), x1 = to_f32(row[c1]);
    if (bias) { x0 += bias[c0]; x1 += bias[c1]; }
    float y0 = x0, y1 = x1;
    if (cs) {
      const float2 r = cs[s * half + i];
      y0 = x0 * r.x - x1 * r.y;
      y1 = x1 * r.x + x0 * r.y;
    }
    T* o = out + (((int64_t)b * n + head) * Sp + s) * hd;
    o[i] = from_f32<T>(y0);
    o[i + half] = from_f32<T>(y1);
  }
}

// One block per token.  in: [B, n, S_pad, hd]; out: [T, ld_out] at column col0.  sign = -1 undoes the
// rotation of to_heads (the transpose of a rotation), cs == NULL copies.
template <typename TIn, typename T>
__global__ void from_heads_kernel(const TIn* __restrict__ in, const float2* __restrict__ cs, float sign, int S, int Sp,
                                  int n, int hd, T* __restrict__ out, int64_t ld_out, int col0) {
  const int t = blockIdx.x, b = t / S, s = t % S, half = hd / 2;
  T* row = out + (int64_t)t * ld_out + col0;
  for (int p = threadIdx.x; p < n * half; p += blockDim.x) {
    const int head = p / half, i = p % half;
    const TIn* src = in + (((int64_t)b * n + head) * Sp + s) * hd;
    float x0 = to_f32(src[i]), x1 = to_f32(src[i + half]);
    float y0 = x0, y1 = x1;
    if (cs) {
      const float2 r = cs[s * half + i];
      const float sn = sign * r.y;
      y0 = x0 * r.x - x1 * sn;
      y1 = x1 * r.x + x0 * sn;
    }
    row[head * hd + i] = from_f32<T>(y0);
    row[head * hd + i + half] = from_f32<T>(y1);
  }
}

// The same two layout changes with 16-byte accesses, for head widths whose half is a multiple of 8: a thread takes 8
// consecutive columns i .. i+7 of a head's first half and their partners i + hd/2 ..; a block covers
// blockDim.x / (n * hd / 16) tokens.
template <typename TIn, typename T>
__global__ void to_heads_vec_kernel(const TIn* __restrict__ in, int64_t ld_in, const float* __restrict__ bias,
                                    const float2* __restrict__ cs, int tokens, int S, int Sp, int n, int hd, T* __restrict__ out) {
  const int half = hd / 2, units = n * half / 8;
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int t = (int)(gid / units), u = (int)(gid % units);
  if (t >= tokens) return;
  const int head = u / (half / 8), i = (u % (half / 8)) * 8;
  const int b = t / S, s = t % S, c0 = head * hd + i, c1 = c0 + half;
  Vec8<TIn> v0, v1;
  v0.load(in + (int64_t)t * ld_in + c0);
  v1.load(in + (int64_t)t * ld_in + c1);
  float x0[8], x1[8], y0[8], y1[8];
  v0.get(x0); v1.get(x1);
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    if (bias) { x0[e] += bias[c0 + e]; x1[e] += bias[c1 + e]; }
    y0[e] = x0[e]; y1[e] = x1[e];
    if (cs) {
      const float2 r = cs[s * half + i + e];
      y0[e] = x0[e] * r.x - x1[e] * r.y;
      y1[e] = x1[e] * r.x + x0[e] * r.y;
    }
  }
  T* o = out + (((int64_t)b * n + head) * Sp + s) * hd + i;
  Vec8<T> w0, w1;
  w0.set(y0); w1.set(y1);
  w0.store(o); w1.store(o + half);
}

template <typename TIn, typename T>
__global__ void from_heads_vec_kernel(const TIn* __restrict__ in, const float2* __restrict__ cs, float sign, int tokens, int S,
                                      int Sp, int n, int hd, T* __restrict__ out, int64_t ld_out, int col0) {
  const int half = hd / 2, units = n * half / 8;
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int t = (int)(gid / units), u = (int)(gid % units);
  if (t >= tokens) return;
  const int head = u / (half / 8), i = (u % (half / 8)) * 8;
  const int b = t / S, s = t % S;
  const TIn* src = in + (((int64_t)b * n + head) * Sp + s) * hd + i;
  Vec8<TIn> v0, v1;
  v0.load(src); v1.load(src + half);
  float x0[8], x1[8], y0[8], y1[8];
  v0.get(x0); v1.get(x1);
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    y0[e] = x0[e]; y1[e] = x1[e];
    if (cs) {
      const float2 r = cs[s * half + i + e];
      const float sn = sign * r.y;
      y0[e] = x0[e] * r.x - x1[e] * sn;
      y1[e] = x1[e] * r.x + x0[e] * sn;
    }
  }
  T* o = out + (int64_t)t * ld_out + col0 + head * hd + i;
  Vec8<T> w0, w1;
  w0.set(y0); w1.set(y1);
  w0.store(o); w1.store(o + half);
}

template <typename TIn, typename T>
inline cudaError_t launch_to_heads(const TIn* in, int64_t ld_in, const float* bias, const float2* cs, int tokens, int S, int Sp,
                                   int n, int hd, T* out, cudaStream_t st) {
  if (tokens <= 0) return cudaSuccess;
  if ((hd / 2) % 8 == 0 && ld_in % 8 == 0) {
    const int64_t threads = (int64_t)tokens * (n * (hd / 2) / 8);
    to_heads_vec_kernel<TIn, T><<<(unsigned)ceil_div(threads, 256), 256, 0, st>>>(in, ld_in, bias, cs, tokens, S, Sp, n, hd, out);
  } else {
    to_heads_kernel<TIn, T><<<tokens, 256, 0, st>>>(in, ld_in, bias, cs, S, Sp, n, hd, out);
  }
  return cudaGetLastError();
}

template <typename TIn, typename T>
inline cudaError_t launch_from_heads(const TIn* in, const float2* cs, float sign, int tokens, int S, int Sp, int n, int hd, T* out,
                                     int64_t ld_out, int col0, cudaStream_t st) {
  if (tokens <= 0) return cudaSuccess;
  if ((hd / 2) % 8 == 0 && ld_out % 8 == 0 && col0 % 8 == 0) {
    const int64_t threads = (int64_t)tokens * (n * (hd / 2) / 8);
    from_heads_vec_kernel<TIn, T><<<(unsigned)ceil_div(threads, 256), 256, 0, st>>>(in, cs, sign, tokens, S, Sp, n, hd, out,
                                                                                    ld_out, col0);
  } else {
    from_heads_kernel<TIn, T><<<tokens, 256, 0, st>>>(in, cs, sign, S, Sp, n, hd, out, ld_out, col0);
  }
  return cudaGetLastError();
}

// One warp per row of the score matrix; row = (sequence, head, s) with s < S_pad.  Keys j <= s take part;
// the rest of the row, and every padding row, is written as zero (later products read whole rows).
template <typename T>
__global__ void softmax_causal_kernel(const float* __restrict__ sc, int S, int Sp, float scale_log2e, int64_t rows,
                                      T* __restrict__ P) {
  const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  const int s = (int)(row % Sp);
  const float* x = sc + row * Sp;
  T* p = P + row * Sp;
  if (s >= S) {
    for (int j = lane; j < Sp; j += 32) p[j] = from_f32<T>(0.f);
    return;
  }
  const int n = s + 1;
  float m = -INFINITY;
  for (int j = lane; j < n; j += 32) m = fmaxf(m, x[j]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  float sum = 0.f;
  for (int j = lane; j < n; j += 32) sum += exp2f((x[j] - m) * scale_log2e);
  sum = warp_sum(sum);
  const float inv = 1.f / sum;
  for (int j = lane; j < Sp; j += 32) p[j] = from_f32<T>(j < n ? exp2f((x[j] - m) * scale_log2e) * inv : 0.f);
}

// Softmax backward for one row: dS = scale * P * (dP - sum_j P_j dP_j), zero beyond the causal range.
template <typename T>
__global__ void dsoftmax_causal_kernel(const T* __restrict__ P, const float* __restrict__ dP, int S, int Sp, float scale,
                                       int64_t rows, T* __restrict__ dS) {
  const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  const int s = (int)(row % Sp);
  const T* p = P + row * Sp;
  const float* g = dP + row * Sp;
  T* o = dS + row * Sp;
  if (s >= S) {
    for (int j = lane; j < Sp; j += 32) o[j] = from_f32<T>(0.f);
    return;
  }
  const int n = s + 1;
  float dot = 0.f;
  for (int j = lane; j < n; j += 32) dot += to_f32(p[j]) * g[j];
  dot = warp_sum(dot);
  for (int j = lane; j < Sp; j += 32) o[j] = from_f32<T>(j < n ? scale * to_f32(p[j]) * (g[j] - dot) : 0.f);
}

// tile_group[i] = key/value group (sequence * n_kv_heads + kv head) of the i-th 128-row block of the
// head-major query rows; group_off[g] = first query row of group g; rows_total[0] = all rows.
__global__ void attn_tables_kernel(int n_tiles, int tiles_per_head, int rep, int n_groups, int rows_per_group,
                                   int32_t* __restrict__ tile_group, int32_t* __restrict__ group_off,
                                   int32_t* __restrict__ rows_total) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n_tiles) tile_group[i] = (i / tiles_per_head) / rep;
  if (i <= n_groups) group_off[i] = i * rows_per_group;
  if (i == 0) { rows_total[0] = n_tiles * ROW_PAD; rows_total[1] = 0; }
}

// out[t, :] = in[t, :] for fp32 streams with row strides (dx1 starts as dy1).
__global__ void copy_stream_kernel(const float* __restrict__ in, int64_t ld_in, int tokens, int h, float* __restrict__ out,
                                   int64_t ld_out) {
  int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i >= (int64_t)tokens * h) return;
  int t = (int)(i / h), c = (int)(i % h);
  *reinterpret_cast<float4*>(out + (int64_t)t * ld_out + c) = *reinterpret_cast<const float4*>(in + (int64_t)t * ld_in + c);
}

}  // namespace revffn
