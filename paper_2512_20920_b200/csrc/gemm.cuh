// One description of every matrix product on the path, the per-element
// epilogue arithmetic shared by both back ends, and the plain CUDA-core
// back end (used for fp32 weights and as the on-device cross-check of the
// tcgen05 back end).
//
//   C[m, n] = sum_k A(m, k) * B(n, k)
//
// Operand storage
//   a_mn_major = 0: A is [M, K] row-major (K contiguous), lda = row stride
//   a_mn_major = 1: A is [K, M] row-major (M contiguous), lda = row stride,
//                   columns a_col0 .. a_col0+M-1 of that buffer
//   b_mn_major likewise for B ([N, K] or [K, N], column offset b_col0).
// B concatenation
//   CONCAT_N: two products with the same A: acc0 against B0, acc1 against B1
//             (gate and up projections of a SwiGLU pair)
//   CONCAT_K: K = 2*Kh; k < Kh multiplies B0(n, k), k >= Kh multiplies B1(n, k-Kh)
// Grouping
//   GROUP_M: rows of A/C live in the padded expert-major row space; the 128-row
//            tile i belongs to expert tile_group[i]; B/C1 are offset by
//            expert * b_group_stride; rows >= *rows_total are not touched.
//            With tok_chunks the tcgen05 back end may work such a product transposed:
//            weights on the MMA M side, an expert's real rows (to a multiple of 32) on
//            the N side, so that padding rows cost no tensor-core time.
//   GROUP_K: one product per expert e over the rows group_off[e]..group_off[e+1]
//            as the K range (weight gradients); output offset e * c_group_stride.
//            With group_cnt the range may stop at the first 64-row boundary past the
//            expert's real rows: what follows is zero padding.
//            Without group_off the n_groups ranges are equal slices of K (a multiple of 64 rows
//            each, the last one ends at K): a dense weight gradient split over K, whose n_groups
//            partial results are added by splitk_reduce_kernel.
#pragma once

#include "common.cuh"

namespace revffn {

enum { EPI_STORE = 0, EPI_SWIGLU = 1, EPI_ROWSCALE = 2, EPI_COUPLE = 3, EPI_DSWIGLU = 4, EPI_WGRAD = 5, EPI_HEADS = 6 };
enum { CONCAT_NONE = 0, CONCAT_N = 1, CONCAT_K = 2 };
enum { GROUP_NONE = 0, GROUP_M = 1, GROUP_K = 2 };

// Update rule of a fused optimiser step (EPI_WGRAD with upd_w set).  kind 0: W <- W - lr g.  kind 1: Adam with
// decoupled weight decay, m <- b1 m + (1 - b1) g, v <- b2 v + (1 - b2) g^2,
// W <- W - lr (m / c1 / (sqrt(v / c2) + eps) + wd W), c1 = 1 - b1^t, c2 = 1 - b2^t.
// The host passes the reciprocals 1 / c1, 1 / c2.
struct UpdRule { int kind; float lr, b1, b2, eps, inv_c1, inv_c2, wd; };

// One element of the step: returns the new weight; for Adam also rewrites the element's two moments.
// The square root and the quotient use the hardware approximations (rsqrt, rcp: about 2 ulp, far inside every
// tolerance of the update): with correctly rounded divisions and square root the element cost about a hundred
// instructions and the experts' weight-gradient epilogue became arithmetic-bound (4 ms for dW_gate|dW_up).
__device__ __forceinline__ float upd_step(const UpdRule& r, float w, float g, float* mom, float* var) {
  if (r.kind == 0) return w - r.lr * g;
  const float m = r.b1 * *mom + (1.f - r.b1) * g;
  const float v = r.b2 * *var + (1.f - r.b2) * g * g;
  *mom = m;
  *var = v;
  const float vh = v * r.inv_c2;
  const float root = vh > 0.f ? vh * __frsqrt_rn(vh) : 0.f;
  return w - r.lr * (__fdividef(m * r.inv_c1, root + r.eps) + r.wd * w);
}

struct GemmProblem {
  int M, N, K;
  int a_mn_major, b_mn_major;
  int concat;
  int epilogue;
  int out_f32;        // EPI_STORE: write fp32 instead of T
  int accumulate;     // EPI_WGRAD: add to C
  const void* A; const void* B0; const void* B1;
  int64_t lda, ldb;
  void* C; void* C1;  // C1: SWIGLU -> optional [M, 2N] pre-activations a|b
  int64_t ldc, ldc1;
  const float* rowscale;                       // ROWSCALE / SWIGLU (scales H) / DSWIGLU (scales dH) (NULL = 1)
  const float* resid; int64_t ld_resid; float resid_sign;   // COUPLE: C = resid + sign * acc (fp32)
  void* ab; int64_t ld_ab;                     // DSWIGLU: [M, 2N] a|b in, da|db out (in place)
  float* dg_part; int dg_ld;                   // DSWIGLU: per (row, n-tile) partial of <acc, H>
  int group_mode, n_groups;
  const int32_t* group_off; const int32_t* tile_group; const int32_t* rows_total;
  const int4* tok_chunks;                      // GROUP_M, optional: (expert, first row, rows, -) runs of real rows; count at rows_total[1]
  const int32_t* group_cnt;                    // GROUP_K, optional: real rows per group (the rest up to the next offset is zero padding)
  int64_t b_group_stride, c_group_stride;
  int a_col0, b_col0;
  // EPI_WGRAD, two outputs from one product: rows >= split_m of (every group's) M belong to C2, which is laid out
  // like C with M replaced by split_m (M must be 2 * split_m); 0 = one output.  Used for dW_gate | dW_up, whose
  // A operand is the one [rows, 2I] buffer da|db.
  void* C2; int split_m;
  // EPI_WGRAD, fused SGD step: instead of writing the gradient g to C, update the weight it belongs to in place,
  // W <- W - upd_lr * g (W of the operand type, same layout as C; upd_w2 goes with C2's rows).  With a master
  // copy (fp32, same layout) the step is taken there and W receives the rounded result.  C / C2 may then be NULL.
  // upd.kind 1 (Adam): upd_mom / upd_var (fp32, same layout, and their second-output twins) hold the moment
  // estimates, which are updated in place as well.
  void* upd_w; void* upd_w2; float* upd_m; float* upd_m2; UpdRule upd;
  float* upd_mom; float* upd_mom2; float* upd_var; float* upd_var2;
  // tcgen05 back end, fp8 operands (both K-major): A and B hold e4m3 codes, one byte per element; the accumulator
  // is multiplied by a_scale[row] * b_scale[(group * N +) column] before the epilogue's own arithmetic
  // (b_scale1: the second matrix of an N-concatenated pair).  lda / ldb / K count elements (= bytes).
  int fp8; const float* a_scale; const float* b_scale0; const float* b_scale1;
  int no_pair;        // tcgen05 back end: never pair CTAs for this product
  long long dbg_wait_cycles;   // tcgen05 back end, tests: bound on every device-side wait (0 = default)
  int dbg_starve;              // tcgen05 back end, tests (needs no_pair): no operand loads are issued
  int dbg_split_loads;         // tcgen05 back end, measurements: 0 the kernel's own choice, 1 two load threads, 2 one
  int dbg_mn_boxes;            // tcgen05 back end, tests: MN-major operands through 64 x 64 boxes of 2-D maps (the fallback form)
  // EPI_HEADS (tcgen05 back end, dense products only): the N columns are heads of 128; C receives, head-major
  // [sequence, head, hm_Sp, 128], the product plus hm_bias, with the pairs (i, i + 64) of a head turned by the
  // angle of hm_cs[position, i] (cos, sin) when hm_cs is given.  Row m is position m % hm_S of sequence m / hm_S.
  const float* hm_bias; const float2* hm_cs; int hm_S, hm_Sp;
  int* status;
};

// --------------------------------------------------------------------------
// Epilogue arithmetic (fp32), shared by both back ends.
// --------------------------------------------------------------------------
__device__ __forceinline__ float swiglu_f(float a, float b) { return a * sigmoid_f(a) * b; }

// SwiGLU backward for one element.  dh = dL/dH; returns H and writes da, db.
__device__ __forceinline__ float dswiglu_f(float a, float b, float dh, float& da, float& db) {
  float s = sigmoid_f(a);
  float si = a * s;
  da = dh * b * (s * (1.f + a * (1.f - s)));
  db = dh * si;
  return si * b;
}

// --------------------------------------------------------------------------
// CUDA-core back end: 64x64 tile, 256 threads, 4x4 outputs per thread, BK = 16.
// Element loads go through generic accessors, bounds-checked; slow but plain.
// --------------------------------------------------------------------------
constexpr int SIMT_BM = 64, SIMT_BN = 64, SIMT_BK = 16;

// Rows of K per slice when a dense product is split into n equal K ranges (whole 64-row K steps).
__host__ __device__ inline int64_t split_k_rows(int64_t K, int n) { return round_up(ceil_div(K, n), 64); }

// Sum of the n partial results of a K-split weight gradient, slices in ascending order (fixed order), then what
// the product's own epilogue would have done with the sum: write it, add it to the gradient buffer, or take the
// fused SGD step on the weight (and its master copy).
template <typename T>
__global__ void splitk_reduce_kernel(const float* __restrict__ part, int n, int64_t count, float* __restrict__ out,
                                     int accumulate, T* __restrict__ W, float* __restrict__ master, UpdRule rule,
                                     float* __restrict__ mom, float* __restrict__ var) {
  const int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i >= count) return;
  float4 v = *reinterpret_cast<const float4*>(part + i);
  for (int s = 1; s < n; ++s) {
    const float4 u = *reinterpret_cast<const float4*>(part + (int64_t)s * count + i);
    v.x += u.x; v.y += u.y; v.z += u.z; v.w += u.w;
  }
  if (W) {
    float w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) w[j] = master ? master[i + j] : to_f32(W[i + j]);
    const float g[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) w[j] = upd_step(rule, w[j], g[j], mom ? mom + i + j : nullptr, var ? var + i + j : nullptr);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (master) master[i + j] = w[j];
      W[i + j] = from_f32<T>(w[j]);
    }
  } else {
    float4* o = reinterpret_cast<float4*>(out + i);
    if (accumulate) { const float4 old = *o; v.x += old.x; v.y += old.y; v.z += old.z; v.w += old.w; }
    *o = v;
  }
}

template <typename T>
__device__ __forceinline__ float simt_load_a(const GemmProblem& p, int m, int64_t k, int m_lim, int64_t k_lim) {
  if (m >= m_lim || k >= k_lim) return 0.f;
  const T* A = reinterpret_cast<const T*>(p.A);
  return p.a_mn_major ? to_f32(A[k * p.lda + p.a_col0 + m]) : to_f32(A[(int64_t)m * p.lda + k]);
}

template <typename T>
__device__ __forceinline__ float simt_load_b(const GemmProblem& p, const T* B, int n, int64_t k, int64_t k_lim) {
  if (n >= p.N || k >= k_lim) return 0.f;
  return p.b_mn_major ? to_f32(B[k * p.ldb + p.b_col0 + n]) : to_f32(B[(int64_t)n * p.ldb + k]);
}

template <typename T>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const GemmProblem p) {
  __shared__ float As[SIMT_BK][SIMT_BM + 1];
  __shared__ float Bs0[SIMT_BK][SIMT_BN + 1];
  __shared__ float Bs1[SIMT_BK][SIMT_BN + 1];
  __shared__ float red[SIMT_BM][17];

  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const int n0 = blockIdx.x * SIMT_BN;
  int m0 = blockIdx.y * SIMT_BM;
  int group = 0;
  int m_lim = p.M;
  int64_t k_begin = 0, k_end = p.K;
  if (p.group_mode == GROUP_M) {
    int total = *p.rows_total;
    if (m0 >= total) return;
    group = p.tile_group[m0 / ROW_PAD];
    m_lim = total;
  } else if (p.group_mode == GROUP_K) {
    group = blockIdx.z;
    if (p.group_off) {
      k_begin = p.group_off[group];
      k_end = p.group_off[group + 1];
    } else {
      const int64_t slice = split_k_rows(p.K, p.n_groups);
      k_begin = group * slice;
      k_end = k_begin + slice < p.K ? k_begin + slice : p.K;
      if (k_begin > k_end) k_begin = k_end;
    }
  }
  const T* B0 = reinterpret_cast<const T*>(p.B0);
  const T* B1 = reinterpret_cast<const T*>(p.B1);
  if (p.group_mode == GROUP_M) {
    B0 += (int64_t)group * p.b_group_stride;
    if (B1) B1 += (int64_t)group * p.b_group_stride;
  }
  const int64_t k_half = (p.concat == CONCAT_K) ? (k_end / 2) : k_end;
  const bool dual = (p.concat == CONCAT_N);

  float acc0[4][4], acc1[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) { acc0[i][j] = 0.f; acc1[i][j] = 0.f; }

  for (int64_t k0 = k_begin; k0 < k_end; k0 += SIMT_BK) {
    for (int i = tid; i < SIMT_BK * SIMT_BM; i += 256) {
      int kk, mm;
      if (p.a_mn_major) { kk = i / SIMT_BM; mm = i % SIMT_BM; } else { mm = i / SIMT_BK; kk = i % SIMT_BK; }
      As[kk][mm] = simt_load_a<T>(p, m0 + mm, k0 + kk, m_lim, k_end);
    }
    for (int i = tid; i < SIMT_BK * SIMT_BN; i += 256) {
      int kk, nn;
      if (p.b_mn_major) { kk = i / SIMT_BN; nn = i % SIMT_BN; } else { nn = i / SIMT_BK; kk = i % SIMT_BK; }
      int64_t k = k0 + kk;
      float v0, v1 = 0.f;
      if (p.concat == CONCAT_K) {
        v0 = (k < k_half) ? simt_load_b<T>(p, B0, n0 + nn, k, k_half)
                          : simt_load_b<T>(p, B1, n0 + nn, k - k_half, k_half);
      } else {
        v0 = simt_load_b<T>(p, B0, n0 + nn, k, k_end);
        if (dual) v1 = simt_load_b<T>(p, B1, n0 + nn, k, k_end);
      }
      Bs0[kk][nn] = v0;
      Bs1[kk][nn] = v1;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < SIMT_BK; ++kk) {
      float a[4], b0[4], b1[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) { b0[j] = Bs0[kk][tx * 4 + j]; b1[j] = Bs1[kk][tx * 4 + j]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc0[i][j] += a[i] * b0[j];
          if (dual) acc1[i][j] += a[i] * b1[j];
        }
    }
    __syncthreads();
  }

  // epilogue
  float dg_local[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int m = m0 + ty * 4 + i;
    bool m_ok = m < m_lim;
    float rs = (p.rowscale && m_ok) ? p.rowscale[m] : 1.f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int n = n0 + tx * 4 + j;
      if (!m_ok || n >= p.N) continue;
      float v = acc0[i][j];
      switch (p.epilogue) {
        case EPI_STORE:
          if (p.out_f32) reinterpret_cast<float*>(p.C)[(int64_t)m * p.ldc + n] = v;
          else reinterpret_cast<T*>(p.C)[(int64_t)m * p.ldc + n] = from_f32<T>(v);
          break;
        case EPI_SWIGLU: {
          float w = acc1[i][j];
          reinterpret_cast<T*>(p.C)[(int64_t)m * p.ldc + n] = from_f32<T>(rs * swiglu_f(v, w));
          if (p.C1) {
            T* ab = reinterpret_cast<T*>(p.C1) + (int64_t)m * p.ldc1;
            ab[n] = from_f32<T>(v);
            ab[p.N + n] = from_f32<T>(w);
          }
        } break;
        case EPI_ROWSCALE:
          reinterpret_cast<T*>(p.C)[(int64_t)m * p.ldc + n] = from_f32<T>(rs * v);
          break;
        case EPI_COUPLE:
          reinterpret_cast<float*>(p.C)[(int64_t)m * p.ldc + n] =
              p.resid[(int64_t)m * p.ld_resid + n] + p.resid_sign * v;
          break;
        case EPI_DSWIGLU: {
          T* ab = reinterpret_cast<T*>(p.ab) + (int64_t)m * p.ld_ab;
          float a = to_f32(ab[n]), b = to_f32(ab[p.N + n]);
          float da, db;
          float H = dswiglu_f(a, b, rs * v, da, db);
          ab[n] = from_f32<T>(da);
          ab[p.N + n] = from_f32<T>(db);
          dg_local[i] += v * H;
        } break;
        case EPI_WGRAD: {
          // element index inside the output this row belongs to (first or second, see split_m)
          const bool second = p.split_m > 0 && m >= p.split_m;
          const int64_t at = (int64_t)group * p.c_group_stride + (int64_t)(second ? m - p.split_m : m) * p.ldc + n;
          T* W = reinterpret_cast<T*>(second ? p.upd_w2 : p.upd_w);
          if (W) {
            float* master = second ? p.upd_m2 : p.upd_m;
            float* mom = second ? p.upd_mom2 : p.upd_mom;
            float* var = second ? p.upd_var2 : p.upd_var;
            const float w_new = upd_step(p.upd, master ? master[at] : to_f32(W[at]), v, mom ? mom + at : nullptr,
                                         var ? var + at : nullptr);
            if (master) master[at] = w_new;
            W[at] = from_f32<T>(w_new);
          } else {
            float* o = reinterpret_cast<float*>(second ? p.C2 : p.C) + at;
            *o = (p.accumulate ? *o : 0.f) + v;
          }
        } break;
      }
    }
  }
  if (p.epilogue == EPI_DSWIGLU && p.dg_part) {
#pragma unroll
    for (int i = 0; i < 4; ++i) red[ty * 4 + i][tx] = dg_local[i];
    __syncthreads();
    if (tid < SIMT_BM) {
      int m = m0 + tid;
      if (m < m_lim) {
        float s = 0.f;
        for (int j = 0; j < 16; ++j) s += red[tid][j];
        p.dg_part[(int64_t)m * p.dg_ld + blockIdx.x] = s;
      }
    }
  }
}

// Number of per-row dg partials the SIMT back end writes for N columns.
inline int simt_dg_parts(int N) { return (int)ceil_div(N, SIMT_BN); }

template <typename T>
inline cudaError_t launch_gemm_simt(const GemmProblem& p, cudaStream_t stream) {
  if (p.M <= 0 || p.N <= 0) return cudaSuccess;
  dim3 grid((unsigned)ceil_div(p.N, SIMT_BN), (unsigned)ceil_div(p.M, SIMT_BM),
            p.group_mode == GROUP_K ? (unsigned)p.n_groups : 1u);
  gemm_simt_kernel<T><<<grid, 256, 0, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace revffn
