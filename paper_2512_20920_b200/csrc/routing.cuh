// Norm, router (logits, top-k, gates), permutation maps, gather and combine.
//
// Forward steps of MLP(Norm(Y1)) in Eq. 2 that are not matrix products:
//   rmsnorm_fwd        n = y * r * gamma, r = (mean(y^2)+eps)^-1/2
//   fold_router        W_rc = [W_r; w_sgate] * W_up   (so logits come straight from n)
//   router_topk        logits (fp64), top-k, softmax over the selected k, shared sigmoid gate
//   map_*              stable counting sort of (token, slot) pairs by expert -> padded rows
//   gather_rows        Up[row] = U[token(row)]
//   combine_rows       Z[t] = sum_s O[row(t,s)] + sgate_t * S[t]
#pragma once

#include <mutex>

#include "common.cuh"

namespace revffn {

// ---------------------------------------------------------------------------
// RMSNorm forward.  One warp per token; fp32 math; output in T plus r[t].
// norm_kind NONE: n = y, r = 1.
// ---------------------------------------------------------------------------
template <typename T>
__global__ void rmsnorm_fwd_kernel(const float* __restrict__ y, int64_t ld, const float* __restrict__ gamma,
                                   float eps, int norm_none, int tokens, int h,
                                   T* __restrict__ n_out, float* __restrict__ r_out) {
  int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  int lane = threadIdx.x & 31;
  if (warp >= tokens) return;
  const float* row = y + (int64_t)warp * ld;
  float r = 1.0f;
  if (!norm_none) {
    float ss = 0.f;
    for (int i = lane * 4; i < h; i += 128) {
      float4 v = *reinterpret_cast<const float4*>(row + i);
      ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
    ss = warp_sum(ss);
    r = rsqrtf(ss / (float)h + eps);
  }
  if (lane == 0) r_out[warp] = r;
  T* out = n_out + (int64_t)warp * h;
  for (int i = lane * 4; i < h; i += 128) {
    float4 v = *reinterpret_cast<const float4*>(row + i);
    float4 g = make_float4(1.f, 1.f, 1.f, 1.f);
    if (gamma && !norm_none) g = *reinterpret_cast<const float4*>(gamma + i);
    out[i + 0] = from_f32<T>(v.x * r * g.x);
    out[i + 1] = from_f32<T>(v.y * r * g.y);
    out[i + 2] = from_f32<T>(v.z * r * g.z);
    out[i + 3] = from_f32<T>(v.w * r * g.w);
  }
}

// ---------------------------------------------------------------------------
// Fold the router (and the shared-expert gate vector) through P_up:
//   W_rc[e, i] = sum_j W_r'[e, j] * W_up[j, i],   W_r' = [W_r; w_sgate]  ((E+1) x d)
// fp64 accumulation and output, so that logits = W_rc * n differ from the
// two-step definition only by fp64 rounding and the routing decision is
// reproducible against a higher-precision reference.
// Block = FD_I columns i x FD_E rows e x FD_S slices of j (512 threads).  W_up is staged
// through shared memory in chunks of FD_J rows (16-byte loads, the next chunk in flight
// while the current one is summed); the rows' weights are staged as doubles.  A thread
// owns one column, one slice (FD_J / FD_S consecutive j of every chunk) and FD_E
// accumulators; the slices are added in ascending order at the end (fixed order).
// ---------------------------------------------------------------------------
constexpr int FD_E = 4;     // rows of W_r' per block
constexpr int FD_J = 64;    // j-chunk staged per iteration
constexpr int FD_I = 128;   // columns per block
constexpr int FD_S = 4;     // j-slices per chunk
constexpr int FD_THREADS = FD_I * FD_S;

template <typename T>
__global__ void __launch_bounds__(FD_THREADS)
fold_router_kernel(const T* __restrict__ w_router, const T* __restrict__ w_sgate,
                   const T* __restrict__ w_up, int E, int d, int h, double* __restrict__ w_rc) {
  constexpr int PER16 = 16 / (int)sizeof(T);                  // elements per 16-byte piece
  constexpr int ROW_PIECES = FD_I / PER16;                    // pieces per staged row
  constexpr int N_PIECES = FD_J * ROW_PIECES / FD_THREADS;    // pieces per thread and chunk
  constexpr int SL = FD_J / FD_S;                             // rows per slice
  __shared__ __align__(16) double wr_s[FD_J][FD_E];
  __shared__ __align__(16) T up_s[FD_J][FD_I];
  static_assert(sizeof(T) * FD_J * FD_I >= sizeof(double) * FD_S * FD_E * FD_I, "slice sums reuse the W_up stage");
  double (*red)[FD_E][FD_I] = reinterpret_cast<double (*)[FD_E][FD_I]>(&up_s[0][0]);   // used after the last chunk
  const int tid = threadIdx.x;
  const int col = tid % FD_I, sl = tid / FD_I;
  const int i0 = blockIdx.x * FD_I;
  const int e0 = blockIdx.y * FD_E;
  double acc[FD_E];
#pragma unroll
  for (int a = 0; a < FD_E; ++a) acc[a] = 0.0;

  uint4 pre[N_PIECES];
  float pre_w = 0.f;
  auto prefetch = [&](int j0) {
#pragma unroll
    for (int q = 0; q < N_PIECES; ++q) {
      int piece = tid + q * FD_THREADS;
      int jj = piece / ROW_PIECES, c = (piece % ROW_PIECES) * PER16;
      pre[q] = make_uint4(0u, 0u, 0u, 0u);
      if (j0 + jj < d && i0 + c < h)      // h is a multiple of 8: a piece never straddles the edge
        pre[q] = *reinterpret_cast<const uint4*>(w_up + (int64_t)(j0 + jj) * h + i0 + c);
    }
    if (tid < FD_E * FD_J) {
      int ee = tid / FD_J, jj = tid % FD_J;
      int e = e0 + ee, j = j0 + jj;
      const T* src = (e < E) ? (w_router + (int64_t)e * d) : (e == E ? w_sgate : nullptr);
      pre_w = (src != nullptr && j < d) ? to_f32(src[j]) : 0.f;
    }
  };
  prefetch(0);
  for (int j0 = 0; j0 < d; j0 += FD_J) {
    __syncthreads();
#pragma unroll
    for (int q = 0; q < N_PIECES; ++q) {
      int piece = tid + q * FD_THREADS;
      int jj = piece / ROW_PIECES, c = (piece % ROW_PIECES) * PER16;
      *reinterpret_cast<uint4*>(&up_s[jj][c]) = pre[q];
    }
    if (tid < FD_E * FD_J) wr_s[tid % FD_J][tid / FD_J] = (double)pre_w;
    __syncthreads();
    if (j0 + FD_J < d) prefetch(j0 + FD_J);
#pragma unroll
    for (int q = 0; q < SL; ++q) {      // rows past d were staged as zeros
      const int jj = sl * SL + q;
      double b = (double)to_f32(up_s[jj][col]);
      const double2* w2 = reinterpret_cast<const double2*>(wr_s[jj]);
#pragma unroll
      for (int a = 0; a < FD_E / 2; ++a) {
        double2 w = w2[a];
        acc[2 * a] += w.x * b;
        acc[2 * a + 1] += w.y * b;
      }
    }
  }
  __syncthreads();      // every slice has finished reading the stage
#pragma unroll
  for (int a = 0; a < FD_E; ++a) red[sl][a][col] = acc[a];
  __syncthreads();
  if (sl == 0 && i0 + col < h) {
#pragma unroll
    for (int a = 0; a < FD_E; ++a) {
      double v = red[0][a][col];
#pragma unroll
      for (int q = 1; q < FD_S; ++q) v += red[q][a][col];
      if (e0 + a <= E) w_rc[(int64_t)(e0 + a) * h + i0 + col] = v;
    }
  }
}

template <typename T>
inline cudaError_t launch_fold_router(const T* w_router, const T* w_sgate, const T* w_up, int E, int d, int h,
                                      double* w_rc, cudaStream_t st) {
  dim3 grid((unsigned)ceil_div(h, FD_I), (unsigned)ceil_div(E + 1, FD_E));
  fold_router_kernel<T><<<grid, FD_THREADS, 0, st>>>(w_router, w_sgate, w_up, E, d, h, w_rc);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// The same fold on the fp64 tensor-core path, K split across blocks.
//   fold_router_mma_kernel: block (x: 64 columns i, y: 64 rows e, z: slice of rows j) computes the slice's
//     part[z][e][i] = sum_{j in slice z} W_r'[e, j] * W_up[j, i] with mma.sync m8n8k4 (warp = 16 rows x
//     32 columns as 2 x 4 fragments).
//   fold_router_reduce_kernel: W_rc[e][i] = sum_z part[z][e][i], z ascending (fixed order).
// Needs FOLD_SLICES * (E+1) * h doubles of scratch, which the workspace has; the entry point that may
// not use a workspace keeps the FMA kernel above.
// ---------------------------------------------------------------------------
constexpr int FOLD_SLICES = 16;        // upper bound on the K slices
constexpr int FM_J_BYTES = 256;        // a slice is this many bytes of a W_r' row: 128 rows j in bf16, 64 in fp32
template <typename T> __host__ __device__ constexpr int fold_slice_rows() { return FM_J_BYTES / (int)sizeof(T); }
constexpr int FM_PAD = 8;              // elements of padding per staged row (keeps rows 16-byte aligned)

__device__ __forceinline__ void fold_dmma(double& d0, double& d1, double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
               : "+d"(d0), "+d"(d1) : "d"(a), "d"(b));
}

// The block's whole operand slices are fetched with 16-byte loads that are all in flight together
// (one memory round trip), kept in shared memory in their storage type, and widened to fp64 as the
// fragments are read.
template <typename T>
__global__ void __launch_bounds__(256)
fold_router_mma_kernel(const T* __restrict__ w_router, const T* __restrict__ w_sgate, const T* __restrict__ w_up,
                       int E, int d, int h, double* __restrict__ part) {
  constexpr int PER16 = 16 / (int)sizeof(T);
  constexpr int FM_J = fold_slice_rows<T>();
  constexpr int LDA = FM_J + FM_PAD, LDB = 64 + FM_PAD;
  __shared__ __align__(16) T as[64 * LDA];       // W_r' slice  [e][j]
  __shared__ __align__(16) T bs[FM_J * LDB];     // W_up slice  [j][i]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int i0 = blockIdx.x * 64, e0 = blockIdx.y * 64, jb = blockIdx.z * FM_J;
  const int EP = E + 1;
  const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
  // d and h are multiples of 8, so a 16-byte piece never straddles the end of a row
  for (int piece = tid; piece < 64 * (FM_J / PER16); piece += 256) {
    const int ee = piece / (FM_J / PER16), jj = (piece % (FM_J / PER16)) * PER16;
    const int e = e0 + ee, j = jb + jj;
    const T* src = (e < E) ? (w_router + (int64_t)e * d) : (e == E ? w_sgate : nullptr);
    *reinterpret_cast<uint4*>(&as[ee * LDA + jj]) =
        (src != nullptr && j < d) ? *reinterpret_cast<const uint4*>(src + j) : zero4;
  }
  for (int piece = tid; piece < FM_J * (64 / PER16); piece += 256) {
    const int jj = piece / (64 / PER16), ii = (piece % (64 / PER16)) * PER16;
    const int j = jb + jj, i = i0 + ii;
    *reinterpret_cast<uint4*>(&bs[jj * LDB + ii]) =
        (j < d && i < h) ? *reinterpret_cast<const uint4*>(w_up + (int64_t)j * h + i) : zero4;
  }
  __syncthreads();
  const int wm = warp >> 1, wn = warp & 1, fr = lane >> 2, fc = lane & 3;
  double acc[2][4][2];
#pragma unroll
  for (int a = 0; a < 2; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) { acc[a][b][0] = 0.0; acc[a][b][1] = 0.0; }
#pragma unroll 4
  for (int kk = 0; kk < FM_J; kk += 4) {
    double af[2], bf[4];
#pragma unroll
    for (int a = 0; a < 2; ++a) af[a] = (double)to_f32(as[(wm * 16 + a * 8 + fr) * LDA + kk + fc]);
#pragma unroll
    for (int b = 0; b < 4; ++b) bf[b] = (double)to_f32(bs[(kk + fc) * LDB + wn * 32 + b * 8 + fr]);
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) fold_dmma(acc[a][b][0], acc[a][b][1], af[a], bf[b]);
  }
  double* out = part + (int64_t)blockIdx.z * EP * h;
#pragma unroll
  for (int a = 0; a < 2; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b)
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const int e = e0 + wm * 16 + a * 8 + fr;
        const int i = i0 + wn * 32 + b * 8 + 2 * fc + c;
        if (e < EP && i < h) out[(int64_t)e * h + i] = acc[a][b][c];
      }
}

__global__ void fold_router_reduce_kernel(const double* __restrict__ part, int n_slices, int64_t n,
                                          double* __restrict__ w_rc) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  double v = part[i];
  for (int z = 1; z < n_slices; ++z) v += part[(int64_t)z * n + i];
  w_rc[i] = v;
}

// Returns cudaErrorInvalidValue when d needs more slices than the scratch holds (the caller then uses the FMA kernel).
template <typename T>
inline cudaError_t launch_fold_router_mma(const T* w_router, const T* w_sgate, const T* w_up, int E, int d, int h,
                                          double* part, double* w_rc, cudaStream_t st) {
  const int n_slices = (int)ceil_div(d, fold_slice_rows<T>());
  if (n_slices > FOLD_SLICES) return cudaErrorInvalidValue;
  dim3 grid((unsigned)ceil_div(h, 64), (unsigned)ceil_div(E + 1, 64), (unsigned)n_slices);
  fold_router_mma_kernel<T><<<grid, 256, 0, st>>>(w_router, w_sgate, w_up, E, d, h, part);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const int64_t n = (int64_t)(E + 1) * h;
  fold_router_reduce_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, st>>>(part, n_slices, n, w_rc);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Router: logits in fp64 from the fp32 stream, top-k by warp shuffles, gates.
//   block = 256 threads, RT_TOK tokens per block.
//   phase 1: L[t, e] = r_t <W_rc[e], y_t * gamma> (+ b_r[e]) for e < E; row E is the
//            shared gate.  The product runs on the fp64 tensor-core path
//            (mma.sync m8n8k4): y*gamma (fp64, [token][i]) and W_rc ([expert][i]) are
//            staged chunk-wise in shared memory, each warp owns a 16-token x 16-expert
//            block of the 32 x 64 tile as 2 x 2 fragments.  (Blocks of 64 tokens with 16 x 32
//            per warp read fewer operand values per instruction, but a batch of 8192 tokens
//            then fills the GPU with one block of 8 warps per SM, which cannot hide the
//            latency of its own loads: 32-token blocks, two or three to an SM, took the kernel
//            from 0.106 to 0.083 ms.)  (A register-tiled DFMA version of the same product
//            spent its time on shared-memory operand reads: 8 values per 16 FMAs.)
//            The staging threads also sum y^2 (fp64), which gives
//            r_t = (mean(y_t^2)+eps)^-1/2; the scale is applied to the finished sums.
//   phase 2: per token, k rounds of warp arg-max (ties -> lowest index), softmax
//            over the k selected logits, sigmoid of the shared-gate logit.
// idx_in != NULL: expert sets are taken from it (gates are still recomputed).
// prob_out != NULL: gates are the selected entries of the softmax over ALL experts (not
// renormalised), and that softmax is written to prob_out[T, E].
// ---------------------------------------------------------------------------
constexpr int RT_TOK = 32;   // tokens per block
constexpr int RT_KC = 32;    // k-chunk
constexpr int RT_EC = 64;    // experts per pass
constexpr int RT_LD = RT_KC + 4;    // row stride (doubles) of both staged chunks: rows 4 doubles apart modulo 16 banks,
                                    // so the 8 rows x 4 columns a fragment load touches fall on distinct banks

// D (8x8) += A (8x4, row-major fragment) * B (4x8, column-major fragment), fp64.
// Lane l holds A[l/4][l%4], B[l%4][l/4] and D[l/4][2*(l%4) + {0,1}].
__device__ __forceinline__ void dmma_8x8x4(double& d0, double& d1, double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
               : "+d"(d0), "+d"(d1) : "d"(a), "d"(b));
}

__global__ void __launch_bounds__(256)
router_topk_kernel(const float* __restrict__ y, int64_t ld, const float* __restrict__ gamma, float eps,
                   int norm_none, const double* __restrict__ w_rc, const float* __restrict__ b_router,
                   int tokens, int h, int E, int k, int has_shared, const int32_t* __restrict__ idx_in,
                   int32_t* __restrict__ idx_out, float* __restrict__ gate_out, float* __restrict__ sgate_out,
                   int32_t* __restrict__ idx_user, float* __restrict__ prob_out, int* __restrict__ status,
                   int check_finite) {
  extern __shared__ __align__(16) double smem_d[];
  const int EP = E + 1;                       // logits per token incl. the shared-gate row
  double* ns = smem_d;                        // [RT_TOK][RT_LD]  stream chunk, one row per token
  double* ws = ns + RT_TOK * RT_LD;           // [RT_EC][RT_LD]   W_rc chunk, one row per expert
  double* rs = ws + RT_EC * RT_LD;            // [RT_TOK]
  double* Ls = rs + RT_TOK;                   // [RT_TOK][EP]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int t0 = blockIdx.x * RT_TOK;

  // phase 1: logits.  Warp (wm, wn) owns tokens 16 wm .. +15 and experts e0 + 16 wn .. +15.
  const int wm = warp >> 2, wn = warp & 3;
  constexpr int NY = RT_TOK * RT_KC / 4 / 256;      // float4 pieces of the stream chunk per thread
  static_assert(NY >= 1 && RT_TOK * RT_KC / 4 % 256 == 0, "stream chunk must split evenly over the block");
  const int fr = lane >> 2, fc = lane & 3;          // fragment row / column of this lane
  for (int e0 = 0; e0 < EP; e0 += RT_EC) {
    double acc[2][2][2];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int b = 0; b < 2; ++b) { acc[a][b][0] = 0.0; acc[a][b][1] = 0.0; }
    // Register prefetch: the global loads of chunk c+1 are in flight while chunk c is summed.
    //   y:    RT_TOK x RT_KC floats  = NY float4 per thread (token tt, 4 consecutive i)
    //   W_rc: RT_EC x RT_KC doubles  = 4 double2 per thread (expert ee, 2 consecutive i)
    float4 py[NY];
    double2 pw[4];
    double ss[NY];                  // sum of y^2 over this thread's 4-column strip of its token(s)
#pragma unroll
    for (int q = 0; q < NY; ++q) ss[q] = 0.0;
    auto prefetch = [&](int k0) {
#pragma unroll
      for (int q = 0; q < NY; ++q) {
        int idx = tid + q * 256;
        int tt = idx / (RT_KC / 4), kq = (idx % (RT_KC / 4)) * 4;
        int t = t0 + tt, i = k0 + kq;
        py[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (t < tokens && i < h) py[q] = *reinterpret_cast<const float4*>(y + (int64_t)t * ld + i);   // h % 4 == 0
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        int idx = tid + q * 256;
        int ee = idx / (RT_KC / 2), kq = (idx % (RT_KC / 2)) * 2;
        int e = e0 + ee, i = k0 + kq;
        pw[q] = make_double2(0.0, 0.0);
        if (e < EP && i < h) pw[q] = *reinterpret_cast<const double2*>(w_rc + (int64_t)e * h + i);   // h % 2 == 0
      }
    };
    prefetch(0);
    for (int k0 = 0; k0 < h; k0 += RT_KC) {
#pragma unroll
      for (int q = 0; q < NY; ++q) {
        int idx = tid + q * 256;
        int tt = idx / (RT_KC / 4), kq = (idx % (RT_KC / 4)) * 4;
        int i = k0 + kq;
        float4 g = make_float4(1.f, 1.f, 1.f, 1.f);
        if (gamma && !norm_none && i < h) g = *reinterpret_cast<const float4*>(gamma + i);
        const double v0 = (double)py[q].x, v1 = (double)py[q].y, v2 = (double)py[q].z, v3 = (double)py[q].w;
        ss[q] += v0 * v0; ss[q] += v1 * v1; ss[q] += v2 * v2; ss[q] += v3 * v3;
        double2* dst = reinterpret_cast<double2*>(ns + tt * RT_LD + kq);
        dst[0] = make_double2(v0 * (double)g.x, v1 * (double)g.y);
        dst[1] = make_double2(v2 * (double)g.z, v3 * (double)g.w);
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        int idx = tid + q * 256;
        int ee = idx / (RT_KC / 2), kq = (idx % (RT_KC / 2)) * 2;
        *reinterpret_cast<double2*>(ws + ee * RT_LD + kq) = pw[q];
      }
      __syncthreads();
      if (k0 + RT_KC < h) prefetch(k0 + RT_KC);
      const double* ap = ns + (wm * 16 + fr) * RT_LD + fc;
      const double* bp = ws + (wn * 16 + fr) * RT_LD + fc;
#pragma unroll
      for (int kk = 0; kk < RT_KC; kk += 4) {
        double af[2], bf[2];
#pragma unroll
        for (int a = 0; a < 2; ++a) af[a] = ap[a * 8 * RT_LD + kk];
#pragma unroll
        for (int b = 0; b < 2; ++b) bf[b] = bp[b * 8 * RT_LD + kk];
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
          for (int b = 0; b < 2; ++b) dmma_8x8x4(acc[a][b][0], acc[a][b][1], af[a], bf[b]);
      }
      __syncthreads();
    }
    // r per token: the 8 threads that staged one token hold its strips (lanes 8m .. 8m+7)
#pragma unroll
    for (int q = 0; q < NY; ++q) {
      double v = ss[q];
      v += __shfl_xor_sync(0xffffffffu, v, 1);
      v += __shfl_xor_sync(0xffffffffu, v, 2);
      v += __shfl_xor_sync(0xffffffffu, v, 4);
      if ((tid & 7) == 0) rs[tid / 8 + q * 32] = norm_none ? 1.0 : 1.0 / sqrt(v / (double)h + (double)eps);
    }
    __syncthreads();
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int b = 0; b < 2; ++b)
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const int tt = wm * 16 + a * 8 + fr;
          const int e = e0 + wn * 16 + b * 8 + 2 * fc + c;
          if (e < EP) {
            double v = acc[a][b][c] * rs[tt];
            if (e < E && b_router) v += (double)b_router[e];
            Ls[tt * EP + e] = v;
          }
        }
  }
  __syncthreads();

  // phase 2: top-k and gates; one warp per token
  for (int tt = warp; tt < RT_TOK; tt += 8) {
    int t = t0 + tt;
    if (t >= tokens) continue;
    const double* L = Ls + tt * EP;
    double sel[8];
    int seli[8];
    if (check_finite) {
      // a NaN or infinite logit (non-finite input or weight) makes the selection meaningless: report it
      bool bad = false;
      for (int e = lane; e < EP; e += 32) bad |= !isfinite(L[e]);
      if (__any_sync(0xffffffffu, bad) && lane == 0) set_status(status, REVFFN_ERR_NONFINITE);
    }
    if (idx_in) {
      // Expert sets from the caller.  An index outside [0, E) is reported and kept as -1: the
      // permutation maps skip such an entry, and its gate weight is zero.
#pragma unroll
      for (int s = 0; s < 8; ++s)
        if (s < k) {
          const int e = idx_in[(int64_t)t * k + s];
          const bool in_range = (unsigned)e < (unsigned)E;
          if (!in_range && lane == 0) set_status(status, REVFFN_ERR_INDEX);
          seli[s] = in_range ? e : -1;
          sel[s] = in_range ? L[e] : __longlong_as_double(0xfff0000000000000LL);
        }
    } else {
      // candidates of this lane: e = lane + 32 j
      unsigned taken = 0u;                    // bit j set: candidate j already selected
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        if (s >= k) break;
        double best = __longlong_as_double(0xfff0000000000000LL);   // -inf
        int besti = 0x7fffffff;
        for (int j = 0; lane + 32 * j < E; ++j) {
          if (taken & (1u << j)) continue;
          double v = L[lane + 32 * j];
          if (v != v) v = __longlong_as_double(0xfff0000000000000LL);   // NaN orders as -inf: the comparisons below stay a
                                                                        // total order and every lane names the same winner
          int e = lane + 32 * j;
          if (v > best || (v == best && e < besti) || besti == 0x7fffffff) { best = v; besti = e; }
        }
        // warp arg-max: larger value wins, equal values -> lower index
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          double ov = __shfl_xor_sync(0xffffffffu, best, o);
          int oi = __shfl_xor_sync(0xffffffffu, besti, o);
          bool take = (oi != 0x7fffffff) && (besti == 0x7fffffff || ov > best || (ov == best && oi < besti));
          if (take) { best = ov; besti = oi; }
        }
        sel[s] = best; seli[s] = besti;
        if ((besti & 31) == lane) taken |= 1u << (besti >> 5);
      }
    }
    // gates: lane s < k takes slot s, lane k the shared gate.  The softmax runs in fp32 on the fp64
    // differences to the largest selected logit (the decision above is fp64; the weights are fp32 outputs).
    double m = sel[0], mine = sel[0];
    int mine_i = seli[0];
#pragma unroll
    for (int s = 1; s < 8; ++s) {
      if (s < k) {
        m = fmax(m, sel[s]);
        if (lane == s) { mine = sel[s]; mine_i = seli[s]; }
      }
    }
    float den;
    if (prob_out) {
      // softmax over all E logits (no renormalisation of the selected ones): largest logit and the sum of
      // exponentials over every expert; the probabilities are kept for the backward pass
      double ma = __longlong_as_double(0xfff0000000000000LL);
      for (int e = lane; e < E; e += 32) ma = fmax(ma, L[e]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ma = fmax(ma, __shfl_xor_sync(0xffffffffu, ma, o));
      m = ma;
      float sa = 0.f;
      for (int e = lane; e < E; e += 32) sa += expf((float)(L[e] - ma));
      den = warp_sum(sa);
      for (int e = lane; e < E; e += 32) prob_out[(int64_t)t * E + e] = expf((float)(L[e] - ma)) / den;
    }
    float x = 0.f;
    if (lane < k) x = (float)(mine - m);
    else if (lane == k) x = (float)(-L[E]);
    const float ev = expf(x);
    if (!prob_out) {
      den = (lane < k) ? ev : 0.f;
      den += __shfl_xor_sync(0xffffffffu, den, 1);
      den += __shfl_xor_sync(0xffffffffu, den, 2);
      den += __shfl_xor_sync(0xffffffffu, den, 4);      // k <= 8: lanes 0..7 hold the sum
    }
    if (lane < k) {
      idx_out[(int64_t)t * k + lane] = mine_i;
      if (idx_user) idx_user[(int64_t)t * k + lane] = mine_i;
      gate_out[(int64_t)t * k + lane] = ev / den;
    } else if (lane == k) {
      sgate_out[t] = has_shared ? 1.f / (1.f + ev) : 0.f;
    }
  }
}

inline size_t router_smem_bytes(int E) {
  return sizeof(double) * ((size_t)(RT_TOK + RT_EC) * RT_LD + RT_TOK + (size_t)RT_TOK * (E + 1));
}

// Raises the kernel's dynamic shared-memory limit when the logits of a block do not
// fit the default 48 KB (once per device), then launches.
inline cudaError_t launch_router_topk(const float* y, int64_t ld, const float* gamma, float eps, int norm_none,
                                      const double* w_rc, const float* b_router, int tokens, int h, int E, int k,
                                      int has_shared, const int32_t* idx_in, int32_t* idx_out, float* gate_out,
                                      float* sgate_out, int32_t* idx_user, float* prob_out, int* status,
                                      int check_finite, cudaStream_t st) {
  static size_t raised[64] = {0};
  static std::mutex mu;
  const size_t smem = router_smem_bytes(E);
  if (smem > 48 * 1024) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (raised[dev] < smem) {
      e = cudaFuncSetAttribute(router_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      raised[dev] = smem;
    }
  }
  router_topk_kernel<<<(unsigned)ceil_div(tokens, RT_TOK), 256, smem, st>>>(
      y, ld, gamma, eps, norm_none, w_rc, b_router, tokens, h, E, k, has_shared, idx_in, idx_out, gate_out,
      sgate_out, idx_user, prob_out, status, check_finite);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Permutation maps: stable counting sort of the T*k (token, slot) entries by
// expert, each expert's segment padded to a multiple of ROW_PAD rows.
//   map_rank:   per chunk of MAP_CHUNK tokens, rank of each entry among the
//               chunk's entries of the same expert (entry order = token-major)
//   map_scan:   per expert totals, padded offsets, per-chunk bases, tile->expert
//   map_assign: row of each entry; row -> token; row -> gate weight
// ---------------------------------------------------------------------------
// An entry outside [0, E) (possible only in expert sets handed in by the caller) matches no expert: it gets
// no rank and no row, map_assign marks it with row -1, and every later step skips it.  It is reported once here.
__global__ void map_rank_kernel(const int32_t* __restrict__ idx, int tokens, int k, int E,
                                int32_t* __restrict__ local_rank, int32_t* __restrict__ chunk_cnt,
                                int* __restrict__ status) {
  extern __shared__ int32_t sm_i[];
  int chunk = blockIdx.x;
  int64_t e0 = (int64_t)chunk * MAP_CHUNK * k;
  int n = (int)min((int64_t)MAP_CHUNK * k, (int64_t)tokens * k - e0);
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const int e = idx[e0 + i];
    sm_i[i] = e;
    if ((unsigned)e >= (unsigned)E) set_status(status, REVFFN_ERR_INDEX);
  }
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    int c = 0;
    for (int i = 0; i < n; ++i)
      if (sm_i[i] == e) { local_rank[e0 + i] = c; ++c; }
    chunk_cnt[(int64_t)chunk * E + e] = c;
  }
}

constexpr int TOK_CHUNK = 256;   // most token rows of one expert in one N-side tile

__global__ void map_scan_kernel(const int32_t* __restrict__ chunk_cnt, int n_chunks, int E,
                                int32_t* __restrict__ chunk_base, int32_t* __restrict__ expert_cnt,
                                int32_t* __restrict__ expert_off, int32_t* __restrict__ tile_group,
                                int32_t* __restrict__ rows_total, int max_tiles, int4* __restrict__ tok_chunks,
                                int max_chunks) {
  extern __shared__ int32_t sm_i[];          // [E+1] padded offsets
  // Per expert, the exclusive prefix sum of its chunk counts: a warp per expert, 32 chunks per round, so the
  // dependent loads of a round are one round trip (a thread per expert walking its chunks one by one spent a
  // memory latency per chunk).
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  for (int e = warp; e < E; e += n_warps) {
    int run = 0;
    for (int c0 = 0; c0 < n_chunks; c0 += 32) {
      const int c = c0 + lane;
      const int v = c < n_chunks ? chunk_cnt[(int64_t)c * E + e] : 0;
      int incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += u;
      }
      if (c < n_chunks) chunk_base[(int64_t)c * E + e] = run + incl - v;
      run += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) expert_cnt[e] = run;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int off = 0;
    for (int e = 0; e < E; ++e) {
      sm_i[e] = off;
      off += (int)round_up(expert_cnt[e], ROW_PAD);
    }
    sm_i[E] = off;
    rows_total[0] = off;
    // Token chunks for the products that put tokens on the MMA N side: per expert, runs of up to
    // TOK_CHUNK rows covering its real rows rounded up to 32 (the rounding stays inside the expert's
    // zero padding).  Entry = (expert, first row, rows, 0); the count goes to rows_total[1].
    // (Runs of equal length, 3 x 192 instead of 256 + 256 + 64 for 546 rows, stay within 2 % either way: the two
    // products that use the table measured 2 % faster alone and the whole step 1-2 % slower.)
    int nc = 0;
    for (int e = 0; e < E; ++e) {
      const int n = (int)round_up(expert_cnt[e], 32);
      for (int r = 0; r < n && nc < max_chunks; r += TOK_CHUNK)
        tok_chunks[nc++] = make_int4(e, sm_i[e] + r, min(TOK_CHUNK, n - r), 0);
    }
    rows_total[1] = nc;
  }
  __syncthreads();
  for (int e = threadIdx.x; e <= E; e += blockDim.x) expert_off[e] = sm_i[e];
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    for (int t = sm_i[e] / ROW_PAD; t < sm_i[e + 1] / ROW_PAD && t < max_tiles; ++t) tile_group[t] = e;
  }
}

__global__ void map_assign_kernel(const int32_t* __restrict__ idx, const float* __restrict__ gate,
                                  const int32_t* __restrict__ local_rank, const int32_t* __restrict__ chunk_base,
                                  const int32_t* __restrict__ expert_off, int tokens, int k, int E,
                                  int32_t* __restrict__ tok_row, int32_t* __restrict__ row_tok,
                                  float* __restrict__ row_gate) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (int64_t)tokens * k) return;
  int t = (int)(i / k);
  int e = idx[i];
  if ((unsigned)e >= (unsigned)E) { tok_row[i] = -1; return; }      // reported by map_rank
  int chunk = t / MAP_CHUNK;
  int row = expert_off[e] + chunk_base[(int64_t)chunk * E + e] + local_rank[i];
  tok_row[i] = row;
  row_tok[row] = t;
  row_gate[row] = gate[i];
}

// ---------------------------------------------------------------------------
// Gather rows into the padded expert-major layout:
//   out[row, :] = src[row_tok[row], :]   (zeros for padding rows)
// One block per row, 16-byte accesses.  Rows at or beyond *rows_total are skipped.
// ---------------------------------------------------------------------------
template <typename T>
__global__ void gather_rows_kernel(const T* __restrict__ src, int64_t ld_src, const int32_t* __restrict__ row_tok,
                                   const int32_t* __restrict__ rows_total, int width, T* __restrict__ out) {
  int row = blockIdx.x;
  if (row >= *rows_total) return;
  int t = row_tok[row];
  T* o = out + (int64_t)row * width;
  Vec8<T> v;
  for (int c = threadIdx.x * 8; c < width; c += blockDim.x * 8) {
    if (t >= 0) v.load(src + (int64_t)t * ld_src + c); else v.zero();
    v.store(o + c);
  }
}

// ---------------------------------------------------------------------------
// Combine: Z[t, :] = sum_{s<k} O[tok_row[t,s], :] + sgate[t] * S[t, :]
// fp32 sums in slot order (fixed, so forward and inverse agree bit for bit).
// One warp per token, eight tokens per block; each lane walks the row in 256-element strides with all k + 1
// row pieces of a stride requested before the first is used (K = k at compile time; K = 0 takes k <= 8 at run
// time and pays for eight slots).  Many short blocks: a one-wave grid striding over the tokens measured 12 %
// slower.
// ---------------------------------------------------------------------------
constexpr int COMBINE_TOKENS = 8;      // tokens (warps) per block

template <typename T, int K>
__global__ void __launch_bounds__(32 * COMBINE_TOKENS)
combine_rows_kernel(const T* __restrict__ O, const int32_t* __restrict__ tok_row, int k_rt,
                    const T* __restrict__ S, const float* __restrict__ sgate, int width, int tokens,
                    T* __restrict__ Z) {
  constexpr int KS = K ? K : 8;
  const int k = K ? K : k_rt;
  const int lane = threadIdx.x & 31;
  const int64_t t = (int64_t)blockIdx.x * COMBINE_TOKENS + (threadIdx.x >> 5);
  if (t >= tokens) return;
  const T* rows[KS];
#pragma unroll
  for (int s = 0; s < KS; ++s) {
    const int r = s < k ? tok_row[t * k + s] : -1;      // -1: entry with an out-of-range expert index
    rows[s] = r >= 0 ? O + (int64_t)r * width : nullptr;
  }
  const float sg = S ? sgate[t] : 0.f;
  const T* srow = S ? S + t * width : nullptr;
  T* zrow = Z + t * width;
  for (int c = lane * 8; c < width; c += 256) {
    Vec8<T> v[KS], vs;
#pragma unroll
    for (int s = 0; s < KS; ++s) {
      if (rows[s]) v[s].load(rows[s] + c); else v[s].zero();
    }
    if (srow) vs.load(srow + c); else vs.zero();
    float acc[8], f[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
#pragma unroll
    for (int s = 0; s < KS; ++s) {
      v[s].get(f);
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] += f[i];
    }
    vs.get(f);
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] += sg * f[i];
    vs.set(acc);
    vs.store(zrow + c);
  }
}

template <typename T>
inline cudaError_t launch_combine_rows(const T* O, const int32_t* tok_row, int k, const T* S, const float* sgate,
                                       int width, int tokens, T* Z, cudaStream_t st) {
  if (tokens <= 0) return cudaSuccess;
  const int blocks = (int)ceil_div(tokens, COMBINE_TOKENS), th = 32 * COMBINE_TOKENS;
  switch (k) {
    case 1: combine_rows_kernel<T, 1><<<blocks, th, 0, st>>>(O, tok_row, k, S, sgate, width, tokens, Z); break;
    case 2: combine_rows_kernel<T, 2><<<blocks, th, 0, st>>>(O, tok_row, k, S, sgate, width, tokens, Z); break;
    case 4: combine_rows_kernel<T, 4><<<blocks, th, 0, st>>>(O, tok_row, k, S, sgate, width, tokens, Z); break;
    default: combine_rows_kernel<T, 0><<<blocks, th, 0, st>>>(O, tok_row, k, S, sgate, width, tokens, Z); break;
  }
  return cudaGetLastError();
}

}  // namespace revffn
