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
// ---------------------------------------------------------------------------
template <typename T>
__global__ void fold_router_kernel(const T* __restrict__ w_router, const T* __restrict__ w_sgate,
                                   const T* __restrict__ w_up, int E, int d, int h,
                                   double* __restrict__ w_rc) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  int e = blockIdx.y;
  if (i >= h) return;
  const T* wr = (e < E) ? (w_router + (int64_t)e * d) : w_sgate;
  double acc = 0.0;
  if (wr != nullptr) {
    for (int j = 0; j < d; ++j) acc += (double)to_f32(wr[j]) * (double)to_f32(w_up[(int64_t)j * h + i]);
  }
  w_rc[(int64_t)e * h + i] = acc;
}

// ---------------------------------------------------------------------------
// Router: logits in fp64 from the fp32 stream, top-k by warp shuffles, gates.
//   block = 256 threads, RT_TOK tokens per block.
//   phase 1: r per token (fp64) and n = y*r*gamma (fp64) staged chunk-wise
//   phase 2: L[t, e] = <W_rc[e], n_t> (+ b_r[e]) for e < E; row E is the shared gate
//   phase 3: per token, k rounds of warp arg-max (ties -> lowest index), softmax
//            over the k selected logits, sigmoid of the shared-gate logit.
// idx_in != NULL: expert sets are taken from it (gates are still recomputed).
// ---------------------------------------------------------------------------
constexpr int RT_TOK = 32;   // tokens per block
constexpr int RT_KC = 32;    // k-chunk
constexpr int RT_EC = 64;    // experts per pass

__global__ void __launch_bounds__(256)
router_topk_kernel(const float* __restrict__ y, int64_t ld, const float* __restrict__ gamma, float eps,
                   int norm_none, const double* __restrict__ w_rc, const float* __restrict__ b_router,
                   int tokens, int h, int E, int k, int has_shared, const int32_t* __restrict__ idx_in,
                   int32_t* __restrict__ idx_out, float* __restrict__ gate_out, float* __restrict__ sgate_out,
                   int32_t* __restrict__ idx_user) {
  extern __shared__ double smem_d[];
  const int EP = E + 1;                       // logits per token incl. the shared-gate row
  double* Ls = smem_d;                        // [RT_TOK][EP]
  double* ns = Ls + RT_TOK * EP;              // [RT_TOK][RT_KC + 1]
  double* ws = ns + RT_TOK * (RT_KC + 1);     // [RT_EC][RT_KC + 1]
  double* rs = ws + RT_EC * (RT_KC + 1);      // [RT_TOK]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int t0 = blockIdx.x * RT_TOK;

  // phase 1: r per token
  for (int tt = warp; tt < RT_TOK; tt += 8) {
    int t = t0 + tt;
    double r = 1.0;
    if (t < tokens && !norm_none) {
      const float* row = y + (int64_t)t * ld;
      double ss = 0.0;
      for (int i = lane; i < h; i += 32) { double v = (double)row[i]; ss += v * v; }
      ss = warp_sum(ss);
      r = 1.0 / sqrt(ss / (double)h + (double)eps);
    }
    if (lane == 0) rs[tt] = r;
  }
  __syncthreads();

  // phase 2: logits
  const int tx = tid & 15, ty = tid >> 4;     // 16 x 16 threads: 2 tokens x 4 experts each
  for (int e0 = 0; e0 < EP; e0 += RT_EC) {
    double acc[2][4];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) acc[a][b] = 0.0;
    for (int k0 = 0; k0 < h; k0 += RT_KC) {
      // stage n chunk: RT_TOK x RT_KC
      for (int idx = tid; idx < RT_TOK * RT_KC; idx += 256) {
        int tt = idx / RT_KC, kk = idx % RT_KC;
        int t = t0 + tt, i = k0 + kk;
        double v = 0.0;
        if (t < tokens && i < h) {
          v = (double)y[(int64_t)t * ld + i] * rs[tt];
          if (gamma && !norm_none) v *= (double)gamma[i];
        }
        ns[tt * (RT_KC + 1) + kk] = v;
      }
      for (int idx = tid; idx < RT_EC * RT_KC; idx += 256) {
        int ee = idx / RT_KC, kk = idx % RT_KC;
        int e = e0 + ee, i = k0 + kk;
        ws[ee * (RT_KC + 1) + kk] = (e < EP && i < h) ? w_rc[(int64_t)e * h + i] : 0.0;
      }
      __syncthreads();
#pragma unroll 4
      for (int kk = 0; kk < RT_KC; ++kk) {
        double nv0 = ns[(ty * 2 + 0) * (RT_KC + 1) + kk];
        double nv1 = ns[(ty * 2 + 1) * (RT_KC + 1) + kk];
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          double wv = ws[(tx * 4 + b) * (RT_KC + 1) + kk];
          acc[0][b] += nv0 * wv;
          acc[1][b] += nv1 * wv;
        }
      }
      __syncthreads();
    }
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        int e = e0 + tx * 4 + b;
        if (e < EP) {
          double v = acc[a][b];
          if (e < E && b_router) v += (double)b_router[e];
          Ls[(ty * 2 + a) * EP + e] = v;
        }
      }
  }
  __syncthreads();

  // phase 3: top-k and gates; one warp per token, 4 tokens per warp
  for (int tt = warp; tt < RT_TOK; tt += 8) {
    int t = t0 + tt;
    if (t >= tokens) continue;
    const double* L = Ls + tt * EP;
    double sel[8];
    int seli[8];
    if (idx_in) {
      for (int s = 0; s < k; ++s) { seli[s] = idx_in[(int64_t)t * k + s]; sel[s] = L[seli[s]]; }
    } else {
      // candidates of this lane: e = lane + 32 j
      unsigned taken = 0u;                    // bit j set: candidate j already selected
      for (int s = 0; s < k; ++s) {
        double best = __longlong_as_double(0xfff0000000000000LL);   // -inf
        int besti = 0x7fffffff;
        for (int j = 0; lane + 32 * j < E; ++j) {
          if (taken & (1u << j)) continue;
          double v = L[lane + 32 * j];
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
    if (lane == 0) {
      double m = sel[0];
      for (int s = 1; s < k; ++s) m = fmax(m, sel[s]);
      double den = 0.0, ex[8];
      for (int s = 0; s < k; ++s) { ex[s] = exp(sel[s] - m); den += ex[s]; }
      for (int s = 0; s < k; ++s) {
        idx_out[(int64_t)t * k + s] = seli[s];
        if (idx_user) idx_user[(int64_t)t * k + s] = seli[s];
        gate_out[(int64_t)t * k + s] = (float)(ex[s] / den);
      }
      sgate_out[t] = has_shared ? (float)(1.0 / (1.0 + exp(-L[E]))) : 0.f;
    }
  }
}

inline size_t router_smem_bytes(int E) {
  return sizeof(double) * ((size_t)RT_TOK * (E + 1) + RT_TOK * (RT_KC + 1) + RT_EC * (RT_KC + 1) + RT_TOK);
}

// ---------------------------------------------------------------------------
// Permutation maps: stable counting sort of the T*k (token, slot) entries by
// expert, each expert's segment padded to a multiple of ROW_PAD rows.
//   map_rank:   per chunk of MAP_CHUNK tokens, rank of each entry among the
//               chunk's entries of the same expert (entry order = token-major)
//   map_scan:   per expert totals, padded offsets, per-chunk bases, tile->expert
//   map_assign: row of each entry; row -> token; row -> gate weight
// ---------------------------------------------------------------------------
__global__ void map_rank_kernel(const int32_t* __restrict__ idx, int tokens, int k, int E,
                                int32_t* __restrict__ local_rank, int32_t* __restrict__ chunk_cnt) {
  extern __shared__ int32_t sm_i[];
  int chunk = blockIdx.x;
  int64_t e0 = (int64_t)chunk * MAP_CHUNK * k;
  int n = (int)min((int64_t)MAP_CHUNK * k, (int64_t)tokens * k - e0);
  for (int i = threadIdx.x; i < n; i += blockDim.x) sm_i[i] = idx[e0 + i];
  __syncthreads();
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    int c = 0;
    for (int i = 0; i < n; ++i)
      if (sm_i[i] == e) { local_rank[e0 + i] = c; ++c; }
    chunk_cnt[(int64_t)chunk * E + e] = c;
  }
}

__global__ void map_scan_kernel(const int32_t* __restrict__ chunk_cnt, int n_chunks, int E,
                                int32_t* __restrict__ chunk_base, int32_t* __restrict__ expert_cnt,
                                int32_t* __restrict__ expert_off, int32_t* __restrict__ tile_group,
                                int32_t* __restrict__ rows_total, int max_tiles) {
  extern __shared__ int32_t sm_i[];          // [E+1] padded offsets
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    int run = 0;
    for (int c = 0; c < n_chunks; ++c) {
      chunk_base[(int64_t)c * E + e] = run;
      run += chunk_cnt[(int64_t)c * E + e];
    }
    expert_cnt[e] = run;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int off = 0;
    for (int e = 0; e < E; ++e) {
      sm_i[e] = off;
      off += (int)round_up(expert_cnt[e], ROW_PAD);
    }
    sm_i[E] = off;
    *rows_total = off;
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
// `extra` (optional) adds more per-token terms: used by the backward pass.
// ---------------------------------------------------------------------------
template <typename T>
__global__ void combine_rows_kernel(const T* __restrict__ O, const int32_t* __restrict__ tok_row, int k,
                                    const T* __restrict__ S, const float* __restrict__ sgate, int width,
                                    T* __restrict__ Z) {
  int t = blockIdx.x;
  int rows[8];
  for (int s = 0; s < k; ++s) rows[s] = tok_row[(int64_t)t * k + s];
  float sg = S ? sgate[t] : 0.f;
  for (int c = threadIdx.x * 8; c < width; c += blockDim.x * 8) {
    float acc[8], f[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
    Vec8<T> v;
    for (int s = 0; s < k; ++s) {
      v.load(O + (int64_t)rows[s] * width + c);
      v.get(f);
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] += f[i];
    }
    if (S) {
      v.load(S + (int64_t)t * width + c);
      v.get(f);
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] += sg * f[i];
    }
    v.set(acc);
    v.store(Z + (int64_t)t * width + c);
  }
}

}  // namespace revffn
