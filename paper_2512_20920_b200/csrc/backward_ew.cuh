// Element-wise and reduction kernels of the backward pass (everything that is
// not a matrix product).  Notation follows the forward pass: u = P_up(n),
// z = sum_s g_s f_s(u) + sgate * S, F = P_down(z).
#pragma once

#include "common.cuh"

namespace revffn {

// Gb = T(G): the upstream gradient as a GEMM operand.
template <typename T>
__global__ void cast_stream_kernel(const float* __restrict__ g, int64_t ld, int tokens, int h, T* __restrict__ out) {
  int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i >= (int64_t)tokens * h) return;
  int t = (int)(i / h), c = (int)(i % h);
  float4 v = *reinterpret_cast<const float4*>(g + (int64_t)t * ld + c);
  T* o = out + i;
  o[0] = from_f32<T>(v.x); o[1] = from_f32<T>(v.y); o[2] = from_f32<T>(v.z); o[3] = from_f32<T>(v.w);
}

// Shared-expert gate:  z += sgate * S.
//   dsg[t] = <dZ_t, S_t>;  dS[t] = sgate_t * dZ_t;  dl[t] = dsg * sgate (1 - sgate)
// One block per token.
template <typename T>
__global__ void shared_gate_bwd_kernel(const T* __restrict__ dZ, const T* __restrict__ S,
                                       const float* __restrict__ sgate, int width, T* __restrict__ dS,
                                       float* __restrict__ dl) {
  __shared__ float red[32];
  int t = blockIdx.x;
  float sg = sgate[t];
  float dot = 0.f;
  for (int c = threadIdx.x * 8; c < width; c += blockDim.x * 8) {
    Vec8<T> a, b;
    float fa[8], fb[8];
    a.load(dZ + (int64_t)t * width + c); a.get(fa);
    b.load(S + (int64_t)t * width + c); b.get(fb);
#pragma unroll
    for (int i = 0; i < 8; ++i) { dot += fa[i] * fb[i]; fa[i] *= sg; }
    a.set(fa);
    a.store(dS + (int64_t)t * width + c);
  }
  dot = block_sum(dot, red);
  if (threadIdx.x == 0) dl[t] = dot * sg * (1.f - sg);
}

// Gate backward (softmax over the selected logits):
//   dg[t,s]  = sum_j dg_part[row(t,s), j]              (fixed order)
//   dsel[t,s] = g[t,s] * (dg[t,s] - sum_s' g[t,s'] dg[t,s'])
// written per (token, slot) and per padded row.
__global__ void router_bwd_kernel(const float* __restrict__ dg_part, int dg_ld, int n_part,
                                  const float* __restrict__ gate, const int32_t* __restrict__ tok_row,
                                  int tokens, int k, float* __restrict__ tok_dl, float* __restrict__ row_dl) {
  int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= tokens) return;
  float dg[8], g[8], mix = 0.f;
  for (int s = 0; s < k; ++s) {
    int row = tok_row[(int64_t)t * k + s];      // -1: entry with an out-of-range expert index, contributes nothing
    float acc = 0.f;
    if (row >= 0)
      for (int j = 0; j < n_part; ++j) acc += dg_part[(int64_t)row * dg_ld + j];
    dg[s] = acc;
    g[s] = row >= 0 ? gate[(int64_t)t * k + s] : 0.f;
    mix += g[s] * acc;
  }
  for (int s = 0; s < k; ++s) {
    float v = g[s] * (dg[s] - mix);
    tok_dl[(int64_t)t * k + s] = v;
    const int row = tok_row[(int64_t)t * k + s];
    if (row >= 0) row_dl[row] = v;
  }
}

// Gate backward when the gates are entries of the softmax over all experts (no renormalisation):
//   dg[t,s] as above;  c = sum_s p[t, e_s] dg[t,s];  dL[t,j] = p[t,j] * ([j = e_s] dg[t,s] - c) for every j.
// dL is written as a GEMM operand [T, ld_dl] (columns E .. ld_dl-1 zero).
template <typename T>
__global__ void router_bwd_dense_kernel(const float* __restrict__ dg_part, int dg_ld, int n_part,
                                        const float* __restrict__ prob, const int32_t* __restrict__ idx,
                                        const int32_t* __restrict__ tok_row, int tokens, int k, int E, int ld_dl,
                                        T* __restrict__ dl_out) {
  int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= tokens) return;
  float dg[8];
  int ex[8];
  const float* p = prob + (int64_t)t * E;
  float c = 0.f;
  for (int s = 0; s < k; ++s) {
    int row = tok_row[(int64_t)t * k + s];      // -1: entry with an out-of-range expert index, contributes nothing
    float acc = 0.f;
    if (row >= 0)
      for (int j = 0; j < n_part; ++j) acc += dg_part[(int64_t)row * dg_ld + j];
    dg[s] = acc;
    ex[s] = row >= 0 ? idx[(int64_t)t * k + s] : -1;
    if (row >= 0) c += p[ex[s]] * acc;
  }
  T* o = dl_out + (int64_t)t * ld_dl;
  for (int j = 0; j < ld_dl; ++j) {
    float v = 0.f;
    if (j < E) {
      float sel = 0.f;
      for (int s = 0; s < k; ++s)
        if (ex[s] == j) sel = dg[s];
      v = p[j] * (sel - c);
    }
    o[j] = from_f32<T>(v);
  }
}

// Router weight gradient from the permuted layout:
//   dW_r[e, c] (+)= sum_{rows of e} row_dl[row] * Up[row, c];  db_r[e] (+)= sum row_dl[row]
// grid (ceil(d / blockDim), E); each thread owns one column.
template <typename T>
__global__ void router_wgrad_kernel(const T* __restrict__ Up, const float* __restrict__ row_dl,
                                    const int32_t* __restrict__ expert_off, const int32_t* __restrict__ expert_cnt,
                                    int d, int accumulate, float* __restrict__ dWr, float* __restrict__ dbr) {
  int e = blockIdx.y;
  int c = blockIdx.x * blockDim.x + threadIdx.x;
  int r0 = expert_off[e], n = expert_cnt[e];
  if (c < d && dWr) {
    float acc = 0.f;
    for (int r = r0; r < r0 + n; ++r) acc += row_dl[r] * to_f32(Up[(int64_t)r * d + c]);
    float* o = dWr + (int64_t)e * d + c;
    *o = (accumulate ? *o : 0.f) + acc;
  }
  if (c == 0 && dbr) {
    float acc = 0.f;
    for (int r = r0; r < r0 + n; ++r) acc += row_dl[r];
    dbr[e] = (accumulate ? dbr[e] : 0.f) + acc;
  }
}

// Column reduction with a per-row weight, two passes (deterministic):
//   part[b, c] = sum_{t in strip b} w[t] * X[t, c]      (colsum_partial)
//   out[c] (+)= sum_b part[b, c]                        (colsum_final)
// Used for d w_sgate = sum_t dl[t] u_t (and, with w == NULL meaning all ones, for plain column sums).
// V = 4: a thread takes four consecutive columns with one 8- or 16-byte load per row (cols and ldx multiples of 4,
// X 16-byte aligned); V = 1: any shape.
template <typename T, int V>
__global__ void colsum_partial_kernel(const T* __restrict__ X, int64_t ldx, const float* __restrict__ w,
                                      int rows, int cols, int strip, float* __restrict__ part) {
  int c = (blockIdx.x * blockDim.x + threadIdx.x) * V;
  int b = blockIdx.y;
  if (c >= cols) return;
  int t0 = b * strip, t1 = min(rows, t0 + strip);
  float acc[V];
#pragma unroll
  for (int v = 0; v < V; ++v) acc[v] = 0.f;
#pragma unroll 8
  for (int t = t0; t < t1; ++t) {
    const float wt = w ? w[t] : 1.f;
    const T* px = X + (int64_t)t * ldx + c;
    if constexpr (V == 4 && sizeof(T) == 2) {
      const uint2 raw = *reinterpret_cast<const uint2*>(px);
      const __nv_bfloat162* hp = reinterpret_cast<const __nv_bfloat162*>(&raw);
      const float2 a = __bfloat1622float2(hp[0]), b2 = __bfloat1622float2(hp[1]);
      acc[0] += wt * a.x; acc[1] += wt * a.y; acc[2] += wt * b2.x; acc[3] += wt * b2.y;
    } else if constexpr (V == 4) {
      const float4 a = *reinterpret_cast<const float4*>(px);
      acc[0] += wt * a.x; acc[1] += wt * a.y; acc[2] += wt * a.z; acc[3] += wt * a.w;
    } else {
      acc[0] += wt * to_f32(px[0]);
    }
  }
#pragma unroll
  for (int v = 0; v < V; ++v) part[(int64_t)b * cols + c + v] = acc[v];
}

template <typename T>
inline cudaError_t launch_colsum_partial(const T* X, int64_t ldx, const float* w, int rows, int cols, int strip, int n_strips,
                                         float* part, cudaStream_t st) {
  if (cols % 4 == 0 && ldx % 4 == 0 && (reinterpret_cast<uintptr_t>(X) & 15u) == 0) {
    dim3 grid((unsigned)ceil_div(cols, 4 * 128), (unsigned)n_strips);
    colsum_partial_kernel<T, 4><<<grid, 128, 0, st>>>(X, ldx, w, rows, cols, strip, part);
  } else {
    dim3 grid((unsigned)ceil_div(cols, 256), (unsigned)n_strips);
    colsum_partial_kernel<T, 1><<<grid, 256, 0, st>>>(X, ldx, w, rows, cols, strip, part);
  }
  return cudaGetLastError();
}

// Launch with COLSUM_FINAL_COLS columns per block of 256 threads: 8 threads share a column, each adds every 8th
// strip in ascending order, and the 8 sums are added in a fixed order.
constexpr int COLSUM_FINAL_COLS = 32;
__global__ void __launch_bounds__(256)
colsum_final_kernel(const float* __restrict__ part, int n_strips, int cols, int accumulate, float* __restrict__ out) {
  __shared__ float red[8][COLSUM_FINAL_COLS];
  const int cl = threadIdx.x % COLSUM_FINAL_COLS, g = threadIdx.x / COLSUM_FINAL_COLS;
  const int c = blockIdx.x * COLSUM_FINAL_COLS + cl;
  float acc = 0.f;
  if (c < cols)
    for (int b = g; b < n_strips; b += 8) acc += part[(int64_t)b * cols + c];
  red[g][cl] = acc;
  __syncthreads();
  if (g == 0 && c < cols) {
    float v = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) v += red[i][cl];
    out[c] = (accumulate ? out[c] : 0.f) + v;
  }
}

// dU[t, :] = sum_s dUp[tok_row[t,s], :] + dUsh[t, :] + sum_s tok_dl[t,s] * W_r[idx[t,s], :]
//            + dl[t] * w_sgate[:]
// fp32 sums in a fixed order.  A block owns DU_COLS columns and every (gridDim.x)-th group of eight tokens; a
// warp takes one token at a time, a lane eight columns, and the k + 1 streamed row pieces of a token are
// requested before the first is used.  The grid is sized to the blocks that are resident at once (one wave).
// (Fetching a token's indices one token ahead cost registers, hence resident warps, and measured 20 % slower.)
// The router rows are the same few for every token: the block keeps its column slab of W_r in shared memory
// (n_experts x DU_COLS elements, when that fits 48 KB) instead of fetching k more rows per token from the L2,
// where those fetches cost as much time as the streamed rows.  K = k at compile time; K = 0 takes k <= 8 at run
// time.  dUr (dense gates): the router term arrives as one more streamed row, dL[t, :] W_r.
constexpr int DU_COLS = 256;
constexpr size_t DU_SLAB_MAX = 48 * 1024;

template <typename T, int K>
__global__ void __launch_bounds__(256)
du_reduce_kernel(const T* __restrict__ dUp, const int32_t* __restrict__ tok_row,
                 const int32_t* __restrict__ idx, const float* __restrict__ tok_dl, int k_rt,
                 const T* __restrict__ dUsh, const T* __restrict__ w_router, int n_experts, int slab,
                 const float* __restrict__ dl, const T* __restrict__ w_sgate,
                 const T* __restrict__ dUr, int width, int tokens, T* __restrict__ dU) {
  extern __shared__ __align__(16) uint8_t du_smem[];
  T* wsl = reinterpret_cast<T*>(du_smem);                  // [n_experts][DU_COLS] when slab != 0
  constexpr int KS = K ? K : 8;
  const int k = K ? K : k_rt;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int c = blockIdx.y * DU_COLS + lane * 8;
  const bool col_ok = c < width;
  const bool router_rows = dUr == nullptr;
  if (slab && router_rows) {
    for (int i = threadIdx.x; i < n_experts * (DU_COLS / 8); i += blockDim.x) {
      const int e = i / (DU_COLS / 8), piece = i % (DU_COLS / 8);
      const int col = blockIdx.y * DU_COLS + piece * 8;
      Vec8<T> v;
      if (col < width) v.load(w_router + (int64_t)e * width + col); else v.zero();
      v.store(wsl + e * DU_COLS + piece * 8);
    }
    __syncthreads();
  }
  if (!col_ok) return;
  float sgv[8];
  {
    Vec8<T> v;
    if (dUsh) v.load(w_sgate + c); else v.zero();
    v.get(sgv);
  }
  for (int64_t t = (int64_t)blockIdx.x * 8 + warp; t < tokens; t += (int64_t)gridDim.x * 8) {
    int ex[KS];
    float dls[KS];
    Vec8<T> v[KS], vsh, vr;
#pragma unroll
    for (int s = 0; s < KS; ++s) {
      const int r = s < k ? tok_row[t * k + s] : -1;      // -1: entry with an out-of-range expert index, skipped
      ex[s] = r >= 0 ? idx[t * k + s] : -1;
      dls[s] = (r >= 0 && router_rows) ? tok_dl[t * k + s] : 0.f;
      if (r >= 0) v[s].load(dUp + (int64_t)r * width + c); else v[s].zero();
    }
    const float dlt = dUsh ? dl[t] : 0.f;
    if (dUsh) vsh.load(dUsh + t * width + c); else vsh.zero();
    if (dUr) vr.load(dUr + t * width + c); else vr.zero();
    float acc[8], f[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
#pragma unroll
    for (int s = 0; s < KS; ++s) {
      v[s].get(f);
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] += f[i];
    }
    vsh.get(f);
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] += f[i];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] += dlt * sgv[i];
    vr.get(f);
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] += f[i];
    if (router_rows) {
#pragma unroll
      for (int s = 0; s < KS; ++s) {
        if (ex[s] < 0) continue;                           // warp-uniform
        Vec8<T> w;
        if (slab) w.load(wsl + ex[s] * DU_COLS + lane * 8);
        else w.load(w_router + (int64_t)ex[s] * width + c);
        w.get(f);
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] += dls[s] * f[i];
      }
    }
    vr.set(acc);
    vr.store(dU + t * width + c);
  }
}

template <typename T>
inline cudaError_t launch_du_reduce(const T* dUp, const int32_t* tok_row, const int32_t* idx, const float* tok_dl,
                                    int k, const T* dUsh, const T* w_router, int n_experts, const float* dl,
                                    const T* w_sgate, const T* dUr, int width, int tokens, T* dU, cudaStream_t st) {
  if (tokens <= 0) return cudaSuccess;
  const int col_slabs = (width + DU_COLS - 1) / DU_COLS;
  size_t smem = (size_t)n_experts * DU_COLS * sizeof(T);
  const int slab = (dUr == nullptr && smem <= DU_SLAB_MAX) ? 1 : 0;
  if (!slab) smem = 0;
  cudaError_t e = cudaSuccess;
#define REVFFN_DU_CASE(KK)                                                                                           \
  {                                                                                                                  \
    int wave = 0;                                                                                                    \
    e = resident_blocks(du_reduce_kernel<T, KK>, 256, smem, &wave);                                                  \
    if (e != cudaSuccess) return e;                                                                                  \
    const int groups = (tokens + 7) / 8;                                                                             \
    const dim3 grid(std::max(1, std::min(groups, wave / col_slabs)), col_slabs);                                     \
    du_reduce_kernel<T, KK><<<grid, 256, smem, st>>>(dUp, tok_row, idx, tok_dl, k, dUsh, w_router, n_experts, slab,  \
                                                     dl, w_sgate, dUr, width, tokens, dU);                           \
  }
  switch (k) {
    case 1: REVFFN_DU_CASE(1); break;
    case 2: REVFFN_DU_CASE(2); break;
    case 4: REVFFN_DU_CASE(4); break;
    default: REVFFN_DU_CASE(0); break;
  }
#undef REVFFN_DU_CASE
  return cudaGetLastError();
}

// RMSNorm backward, rows:  q = gamma * dn;  dy = r q - y r^3 <q, y> / h;  dY1 += dy.
// One warp per token.  norm NONE: dY1 += dn.
__global__ void rmsnorm_bwd_rows_kernel(const float* __restrict__ dn, const float* __restrict__ y, int64_t ld,
                                        const float* __restrict__ gamma, const float* __restrict__ r,
                                        int norm_none, int tokens, int h, float* __restrict__ dy1, int64_t ld_dy) {
  int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  int lane = threadIdx.x & 31;
  if (warp >= tokens) return;
  const float* dn_row = dn + (int64_t)warp * h;
  const float* y_row = y + (int64_t)warp * ld;
  float* o = dy1 + (int64_t)warp * ld_dy;
  if (norm_none) {
    for (int i = lane; i < h; i += 32) o[i] += dn_row[i];
    return;
  }
  float dot = 0.f;
  for (int i = lane; i < h; i += 32) dot += (gamma ? gamma[i] : 1.f) * dn_row[i] * y_row[i];
  dot = warp_sum(dot);
  float rt = r[warp];
  float coef = rt * rt * rt * dot / (float)h;
  for (int i = lane; i < h; i += 32) {
    float q = (gamma ? gamma[i] : 1.f) * dn_row[i];
    o[i] += rt * q - y_row[i] * coef;
  }
}

// dgamma partials: part[b, c] = sum_{t in strip b} dn[t, c] * y[t, c] * r[t]; four columns per thread (h and ld are
// multiples of 4, both arrays 16-byte aligned)
__global__ void dgamma_partial_kernel(const float* __restrict__ dn, const float* __restrict__ y, int64_t ld,
                                      const float* __restrict__ r, int tokens, int h, int strip,
                                      float* __restrict__ part) {
  int c = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
  int b = blockIdx.y;
  if (c >= h) return;
  int t0 = b * strip, t1 = min(tokens, t0 + strip);
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
  for (int t = t0; t < t1; ++t) {
    const float4 a = *reinterpret_cast<const float4*>(dn + (int64_t)t * h + c);
    const float4 v = *reinterpret_cast<const float4*>(y + (int64_t)t * ld + c);
    const float rt = r[t];
    acc.x += a.x * v.x * rt; acc.y += a.y * v.y * rt; acc.z += a.z * v.z * rt; acc.w += a.w * v.w * rt;
  }
  *reinterpret_cast<float4*>(part + (int64_t)b * h + c) = acc;
}
inline cudaError_t launch_dgamma_partial(const float* dn, const float* y, int64_t ld, const float* r, int tokens, int h, int strip,
                                         int n_strips, float* part, cudaStream_t st) {
  dim3 grid((unsigned)ceil_div(h, 4 * 128), (unsigned)n_strips);
  dgamma_partial_kernel<<<grid, 128, 0, st>>>(dn, y, ld, r, tokens, h, strip, part);
  return cudaGetLastError();
}

}  // namespace revffn
