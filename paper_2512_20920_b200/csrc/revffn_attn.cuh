// C ABI, workspace planner and launch sequences of the attention coupling branch (Eq. 1).
// See include/revffn_attn.h for the contract of every entry point.  Included at the end of
// revffn_moe.cu: it uses that file's launch accounting, error macros and GEMM back ends.
//
// Attention core: forward and inverse run it as one tcgen05 kernel (flash_attn.cuh) that never
// writes the score matrix.  The backward pass, and the CUDA-core cross-check path, materialise it:
// scores = Q K^T as one grouped product over all heads (fp32), a row kernel turns it into the
// causal softmax P (operand type), O = P V is a second grouped product; then dP = dO V^T, the row
// kernel for dS, dV = P^T dO and dK = dS^T Q as grouped weight-gradient-style products, dQ = dS K.
#pragma once

#include "../../include/revffn_attn.h"
#include "attn.cuh"
#include "flash_attn.cuh"

namespace revffn {

struct AttnLayout {
  Buf status, rows_total, tile_group, group_off, cs, n12, r12, u12, raw, qh, kh, vh, lse, sc, p, oh, o, a;
  size_t fwd_bytes = 0;
  Buf dyb, da, dob, doh, ds, dqh, dkh, dvh, dq, dkv, du12, dn12, part, lse_d;
  size_t bwd_bytes = 0;
  int T = 0, h = 0, hd = 0, d_kv = 0, Sp = 0, n_tiles = 0, groups = 0, strips = 0;
  int64_t rows = 0, kv_rows = 0;
};

static AttnLayout plan_attn(const revffn_attn_desc& D) {
  AttnLayout L;
  const size_t ts = D.weight_dtype == REVFFN_BF16 ? 2 : 4;
  const int64_t B = D.batch, S = D.seq_len, d = D.d_model, h = d / 2, nh = D.n_heads, nkv = D.n_kv_heads;
  const int64_t T = B * S, hd = d / nh, dkv = nkv * hd, Sp = round_up(S, ROW_PAD);
  L.T = (int)T; L.h = (int)h; L.hd = (int)hd; L.d_kv = (int)dkv; L.Sp = (int)Sp;
  L.rows = B * nh * Sp; L.kv_rows = B * nkv * Sp;
  L.n_tiles = (int)(L.rows / ROW_PAD);
  L.groups = (int)(B * nkv);
  L.strips = (int)ceil_div(2 * T > 0 ? 2 * T : 1, STRIP);
  size_t off = 0;
  auto take = [&](Buf& b, size_t bytes) {
    b.off = off; b.bytes = bytes;
    off += (size_t)round_up((int64_t)(bytes > 0 ? bytes : 1), 256);
  };
  take(L.status, 256);
  take(L.rows_total, 256);
  take(L.tile_group, (size_t)L.n_tiles * 4);
  take(L.group_off, (size_t)(L.groups + 1) * 4);
  take(L.cs, (size_t)S * (hd / 2) * 8);
  take(L.n12, (size_t)2 * T * h * ts);
  take(L.r12, (size_t)2 * T * 4);
  take(L.u12, (size_t)2 * T * d * ts);
  take(L.raw, (size_t)T * d * 4);
  take(L.qh, (size_t)L.rows * hd * ts);
  take(L.kh, (size_t)L.kv_rows * hd * ts);
  take(L.vh, (size_t)L.kv_rows * hd * ts);
  take(L.lse, (size_t)L.rows * 4);
  take(L.sc, (size_t)L.rows * Sp * 4);
  take(L.p, (size_t)L.rows * Sp * ts);
  take(L.oh, (size_t)L.rows * hd * ts);
  take(L.o, (size_t)T * d * ts);
  take(L.a, (size_t)T * d * ts);
  L.fwd_bytes = off;
  take(L.dyb, (size_t)T * h * ts);
  take(L.da, (size_t)T * d * ts);
  take(L.dob, (size_t)T * d * ts);
  take(L.doh, (size_t)L.rows * hd * ts);
  take(L.ds, (size_t)L.rows * Sp * ts);
  take(L.dqh, (size_t)L.rows * hd * 4);
  take(L.dkh, (size_t)L.kv_rows * hd * 4);
  take(L.dvh, (size_t)L.kv_rows * hd * 4);
  take(L.dq, (size_t)T * d * ts);
  take(L.dkv, (size_t)T * 2 * dkv * ts);
  take(L.du12, (size_t)2 * T * d * ts);
  take(L.dn12, (size_t)2 * T * h * 4);
  take(L.part, (size_t)L.strips * d * 4);
  take(L.lse_d, (size_t)L.rows * 8);
  L.bwd_bytes = off;
  return L;
}

static int validate_attn_desc(const revffn_attn_desc* D) {
  if (!D) return REVFFN_ERR_NULL;
  if (D->batch < 0 || D->seq_len < 1 || D->d_model <= 0 || (D->d_model & 1)) return REVFFN_ERR_SHAPE;
  if (D->n_heads < 1 || D->d_model % D->n_heads) return REVFFN_ERR_SHAPE;
  if (D->n_kv_heads < 1 || D->n_heads % D->n_kv_heads) return REVFFN_ERR_SHAPE;
  if (D->weight_dtype != REVFFN_F32 && D->weight_dtype != REVFFN_BF16) return REVFFN_ERR_SHAPE;
  const int h = D->d_model / 2, hd = D->d_model / D->n_heads;
  if (hd & 1) return REVFFN_ERR_SHAPE;
  if (D->weight_dtype == REVFFN_BF16) {
    if (h % 128 || D->d_model % 128 || hd % 128) return REVFFN_ERR_SHAPE;
  } else if (h % 8 || D->d_model % 8 || hd % 8) {
    return REVFFN_ERR_SHAPE;
  }
  if (!(D->rope_theta > 0.f)) return REVFFN_ERR_SHAPE;
  if (D->flags & ~(REVFFN_FLAG_FORCE_SIMT | REVFFN_FLAG_REUSE_ACTIVATIONS)) return REVFFN_ERR_UNSUPPORTED;
  if (D->ld_stream < h || (D->ld_stream % 4)) return REVFFN_ERR_ALIGN;
  const int64_t Sp = round_up(D->seq_len, ROW_PAD);
  if ((int64_t)D->batch * D->n_heads * Sp > (int64_t)1 << 30 || (int64_t)D->batch * D->seq_len > (int64_t)1 << 28)
    return REVFFN_ERR_SHAPE;
  return REVFFN_OK;
}

static int validate_attn_weights(const revffn_attn_weights* w) {
  if (!w) return REVFFN_ERR_NULL;
  if (!w->w_up || !w->w_down || !w->w_q || !w->w_k || !w->w_v || !w->w_o) return REVFFN_ERR_NULL;
  const void* ps[] = {w->norm_gamma, w->w_up, w->w_down, w->w_q, w->w_k, w->w_v, w->w_o, w->b_q, w->b_k, w->b_v};
  for (const void* p : ps)
    if (p && !aligned16(p)) return REVFFN_ERR_ALIGN;
  return REVFFN_OK;
}

template <typename T>
struct ACtx {
  revffn_attn_desc D;
  revffn_attn_weights W;
  AttnLayout L;
  char* ws;
  cudaStream_t st;
  bool tc;
  template <typename U> U* p(const Buf& b) const { return reinterpret_cast<U*>(ws + b.off); }
};

template <typename T>
static int a_gemm(const ACtx<T>& c, GemmProblem p, int tag) {
  p.status = c.template p<int>(c.L.status);
  ProfScope ps(tag, c.st);
  if constexpr (std::is_same<T, bf16>::value) {
    if (c.tc) return launch_gemm_tc(p, c.st);
  }
  return launch_gemm_simt<T>(p, c.st) == cudaSuccess ? REVFFN_OK : REVFFN_ERR_CUDA;
}

// Tables of the grouped products, the rotary table, and zeroed padding rows of the head-major buffers.
template <typename T>
static int a_setup(const ACtx<T>& c, bool backward) {
  const revffn_attn_desc& D = c.D;
  const AttnLayout& L = c.L;
  cudaStream_t st = c.st;
  const int n_tab = L.n_tiles > L.groups + 1 ? L.n_tiles : L.groups + 1;
  { ProfScope ps(TG_A_TABLES, st);
  attn_tables_kernel<<<(unsigned)ceil_div(n_tab, 256), 256, 0, st>>>(
      L.n_tiles, L.Sp / ROW_PAD, D.n_heads / D.n_kv_heads, L.groups, (D.n_heads / D.n_kv_heads) * L.Sp,
      c.template p<int32_t>(L.tile_group), c.template p<int32_t>(L.group_off), c.template p<int32_t>(L.rows_total));
  }
  CK(cudaGetLastError());
  { ProfScope ps(TG_A_TABLES, st);
  rope_table_kernel<<<(unsigned)ceil_div((int64_t)D.seq_len * (L.hd / 2), 256), 256, 0, st>>>(
      D.seq_len, L.hd, (double)D.rope_theta, c.template p<float2>(L.cs));
  }
  CK(cudaGetLastError());
  if (L.Sp != D.seq_len) {
    CK(cudaMemsetAsync(c.ws + L.qh.off, 0, L.qh.bytes, st));
    CK(cudaMemsetAsync(c.ws + L.kh.off, 0, L.kh.bytes, st));
    CK(cudaMemsetAsync(c.ws + L.vh.off, 0, L.vh.bytes, st));
    if (backward) CK(cudaMemsetAsync(c.ws + L.doh.off, 0, L.doh.bytes, st));
  }
  return REVFFN_OK;
}

// n = Norm(x), u = n W_up^T for one stream (side 0: query stream, side 1: key/value stream).
template <typename T>
static int a_norm_up(const ACtx<T>& c, const float* x, int side) {
  const revffn_attn_desc& D = c.D;
  const AttnLayout& L = c.L;
  const int Tn = L.T, d = D.d_model, h = L.h;
  T* n = c.template p<T>(L.n12) + (int64_t)side * Tn * h;
  { ProfScope ps(TG_NORM, c.st);
  rmsnorm_fwd_kernel<T><<<(unsigned)ceil_div((int64_t)Tn * 32, 128), 128, 0, c.st>>>(
      x, D.ld_stream, c.W.norm_gamma, D.norm_eps, 0, Tn, h, n, c.template p<float>(L.r12) + (int64_t)side * Tn);
  }
  CK(cudaGetLastError());
  GemmProblem p = blank_problem();
  p.M = Tn; p.N = d; p.K = h;
  p.A = n; p.lda = h;
  p.B0 = c.W.w_up; p.ldb = h;
  p.epilogue = EPI_STORE; p.C = c.template p<T>(L.u12) + (int64_t)side * Tn * d; p.ldc = d;
  return a_gemm(c, p, TG_PUP);
}

// heads = to_heads(u W^T + bias [, rotated])
template <typename T>
static int a_project(const ACtx<T>& c, int side, const void* W, const float* bias, int n, bool rotate, T* heads) {
  const revffn_attn_desc& D = c.D;
  const AttnLayout& L = c.L;
  const int Tn = L.T, d = D.d_model;
  GemmProblem p = blank_problem();
  p.M = Tn; p.N = n * L.hd; p.K = d;
  p.A = c.template p<T>(L.u12) + (int64_t)side * Tn * d; p.lda = d;
  p.B0 = W; p.ldb = d;
  if constexpr (std::is_same<T, bf16>::value) {
    if (c.tc && L.hd == 128) {
      // bias, rotation and the head-major layout happen in the product's epilogue: no fp32 round trip
      p.epilogue = EPI_HEADS; p.C = heads;
      p.hm_bias = bias; p.hm_cs = rotate ? c.template p<float2>(L.cs) : nullptr; p.hm_S = D.seq_len; p.hm_Sp = L.Sp;
      return a_gemm(c, p, TG_A_QKV);
    }
  }
  p.epilogue = EPI_STORE; p.out_f32 = 1; p.C = c.template p<float>(L.raw); p.ldc = n * L.hd;
  CKR(a_gemm(c, p, TG_A_QKV));
  { ProfScope ps(TG_A_HEADS, c.st);
  CK((launch_to_heads<float, T>(c.template p<float>(L.raw), (int64_t)n * L.hd, bias,
                                rotate ? c.template p<float2>(L.cs) : nullptr, Tn, D.seq_len, L.Sp, n, L.hd, heads, c.st)));
  }
  return REVFFN_OK;
}

template <typename T>
static GemmProblem a_grouped_rows(const ACtx<T>& c) {
  const AttnLayout& L = c.L;
  GemmProblem p = blank_problem();
  p.M = (int)L.rows;
  p.group_mode = GROUP_M; p.n_groups = L.groups; p.b_group_stride = (int64_t)L.Sp * L.hd;
  p.group_off = c.template p<int32_t>(L.group_off); p.tile_group = c.template p<int32_t>(L.tile_group);
  p.rows_total = c.template p<int32_t>(L.rows_total);
  return p;
}

// O (token-major) from the head-major q, k, v.  need_p: the backward pass reads P afterwards, so the score
// matrix is materialised; otherwise the tcgen05 back end runs the attention core as one kernel.
template <typename T>
static int a_core(const ACtx<T>& c, bool need_p, bool keep_o32 = false) {
  const revffn_attn_desc& D = c.D;
  const AttnLayout& L = c.L;
  if constexpr (std::is_same<T, bf16>::value) {
    if (c.tc && !need_p && L.hd == FA_HD) {
      ProfScope ps(TG_A_FLASH, c.st);
      return launch_flash_fwd(c.template p<bf16>(L.qh), c.template p<bf16>(L.kh), c.template p<bf16>(L.vh), D.batch,
                              D.n_heads, D.n_kv_heads, D.seq_len, L.Sp, c.template p<bf16>(L.o), D.d_model,
                              c.template p<float>(L.lse), keep_o32 ? c.template p<float>(L.sc) : nullptr,
                              c.template p<int>(L.status), c.st);
    }
  }
  {
    GemmProblem p = a_grouped_rows(c);   // scores = Q K^T
    p.N = L.Sp; p.K = L.hd;
    p.A = c.template p<T>(L.qh); p.lda = L.hd;
    p.B0 = c.template p<T>(L.kh); p.ldb = L.hd;
    p.epilogue = EPI_STORE; p.out_f32 = 1; p.C = c.template p<float>(L.sc); p.ldc = L.Sp;
    CKR(a_gemm(c, p, TG_A_SCORES));
  }
  { ProfScope ps(TG_A_SOFTMAX, c.st);
  softmax_causal_kernel<T><<<(unsigned)ceil_div(L.rows * 32, 256), 256, 0, c.st>>>(
      c.template p<float>(L.sc), D.seq_len, L.Sp, 1.4426950408889634f / sqrtf((float)L.hd), L.rows, c.template p<T>(L.p));
  }
  CK(cudaGetLastError());
  {
    GemmProblem p = a_grouped_rows(c);   // O = P V
    p.N = L.hd; p.K = L.Sp;
    p.A = c.template p<T>(L.p); p.lda = L.Sp;
    p.B0 = c.template p<T>(L.vh); p.ldb = L.hd; p.b_mn_major = 1;
    p.epilogue = EPI_STORE; p.C = c.template p<T>(L.oh); p.ldc = L.hd;
    CKR(a_gemm(c, p, TG_A_PV));
  }
  { ProfScope ps(TG_A_HEADS, c.st);
  CK((launch_from_heads<T, T>(c.template p<T>(L.oh), nullptr, 1.f, L.T, D.seq_len, L.Sp, D.n_heads, L.hd,
                              c.template p<T>(L.o), D.d_model, 0, c.st)));
  }
  return REVFFN_OK;
}

// a = O W_o^T
template <typename T>
static int a_wo(const ACtx<T>& c) {
  const int d = c.D.d_model;
  GemmProblem p = blank_problem();
  p.M = c.L.T; p.N = d; p.K = d;
  p.A = c.template p<T>(c.L.o); p.lda = d;
  p.B0 = c.W.w_o; p.ldb = d;
  p.epilogue = EPI_STORE; p.C = c.template p<T>(c.L.a); p.ldc = d;
  return a_gemm(c, p, TG_A_WO);
}

// P_down fused with the coupling: out = resid + sign * (a W_down^T)
template <typename T>
static int a_couple(const ACtx<T>& c, const float* resid, float sign, float* out) {
  const int d = c.D.d_model;
  GemmProblem p = blank_problem();
  p.M = c.L.T; p.N = c.L.h; p.K = d;
  p.A = c.template p<T>(c.L.a); p.lda = d;
  p.B0 = c.W.w_down; p.ldb = d;
  p.epilogue = EPI_COUPLE; p.resid = resid; p.ld_resid = c.D.ld_stream; p.resid_sign = sign;
  p.C = out; p.ldc = c.D.ld_stream;
  return a_gemm(c, p, TG_PDOWN);
}

template <typename T>
static int a_kv_side(const ACtx<T>& c, const float* x2) {
  CKR(a_norm_up(c, x2, 1));
  CKR(a_project(c, 1, c.W.w_k, c.W.b_k, c.D.n_kv_heads, true, c.template p<T>(c.L.kh)));
  return a_project(c, 1, c.W.w_v, c.W.b_v, c.D.n_kv_heads, false, c.template p<T>(c.L.vh));
}

template <typename T>
static int a_query_side(const ACtx<T>& c, const float* x1, bool need_p, bool keep_o32 = false) {
  CKR(a_norm_up(c, x1, 0));
  CKR(a_project(c, 0, c.W.w_q, c.W.b_q, c.D.n_heads, true, c.template p<T>(c.L.qh)));
  CKR(a_core(c, need_p, keep_o32));
  return a_wo(c);
}

// Forward pass: both streams are known at once, so the norm and P_up run over the 2T rows together.
template <typename T>
static int a_forward(const ACtx<T>& c, const float* x1, const float* x2, float* y1) {
  const revffn_attn_desc& D = c.D;
  const AttnLayout& L = c.L;
  CKR(a_setup(c, false));
  { ProfScope ps(TG_NORM, c.st);
  rmsnorm2_fwd_kernel<T><<<(unsigned)ceil_div((int64_t)2 * L.T * 32, 128), 128, 0, c.st>>>(
      x1, x2, D.ld_stream, c.W.norm_gamma, D.norm_eps, L.T, L.h, c.template p<T>(L.n12), c.template p<float>(L.r12));
  }
  CK(cudaGetLastError());
  {
    GemmProblem p = blank_problem();
    p.M = 2 * L.T; p.N = D.d_model; p.K = L.h;
    p.A = c.template p<T>(L.n12); p.lda = L.h;
    p.B0 = c.W.w_up; p.ldb = L.h;
    p.epilogue = EPI_STORE; p.C = c.template p<T>(L.u12); p.ldc = D.d_model;
    CKR(a_gemm(c, p, TG_PUP));
  }
  CKR(a_project(c, 1, c.W.w_k, c.W.b_k, D.n_kv_heads, true, c.template p<T>(L.kh)));
  CKR(a_project(c, 1, c.W.w_v, c.W.b_v, D.n_kv_heads, false, c.template p<T>(L.vh)));
  CKR(a_project(c, 0, c.W.w_q, c.W.b_q, D.n_heads, true, c.template p<T>(L.qh)));
  CKR(a_core(c, false));
  CKR(a_wo(c));
  return a_couple(c, x1, 1.f, y1);
}

template <typename T>
static int a_inverse(const ACtx<T>& c, const float* y1, const float* x2, float* x1, int n_iter) {
  const AttnLayout& L = c.L;
  if (n_iter == 0) {
    if (x1 != y1) {
      copy_stream_kernel<<<(unsigned)ceil_div((int64_t)L.T * L.h, 4 * 256), 256, 0, c.st>>>(y1, c.D.ld_stream, L.T, L.h, x1,
                                                                                            c.D.ld_stream);
      ++g_prof.launches;
      CK(cudaGetLastError());
    }
    return REVFFN_OK;
  }
  CKR(a_setup(c, false));
  CKR(a_kv_side(c, x2));
  const float* cur = y1;
  for (int it = 0; it < n_iter; ++it) {
    CKR(a_query_side(c, cur, false));
    CKR(a_couple(c, y1, -1.f, x1));
    cur = x1;
  }
  return REVFFN_OK;
}

template <typename T>
static int a_backward(const ACtx<T>& c, const float* x1, const float* x2, const float* dy1, float* dx1, float* dx2,
                      const revffn_attn_grads& G) {
  const revffn_attn_desc& D = c.D;
  const AttnLayout& L = c.L;
  const int Tn = L.T, d = D.d_model, h = L.h, hd = L.hd, dkv = L.d_kv, Sp = L.Sp;
  const int acc = G.accumulate ? 1 : 0;
  cudaStream_t st = c.st;

  // recompute the branch's intermediates (Sec. 3.1: nothing was cached)
  // REUSE: an inverse call (at least one iteration) on this workspace with the same x2 and weights has left the
  // tables and the key/value side (n2, u2, k, v head-major) behind; only the query side is evaluated again
  const bool reuse_kv = (D.flags & REVFFN_FLAG_REUSE_ACTIVATIONS) != 0;
  if (!reuse_kv) CKR(a_setup(c, true));
  else if (L.Sp != D.seq_len) CK(cudaMemsetAsync(c.ws + L.doh.off, 0, L.doh.bytes, st));
  // tcgen05 back end: the attention core runs fused in both directions and P is never written;
  // otherwise the score matrix is materialised and the gradient pass reads P from memory
  bool fused = false;
  if constexpr (std::is_same<T, bf16>::value) fused = c.tc && hd == FA_HD;
  if (!reuse_kv) CKR(a_kv_side(c, x2));
  CKR(a_query_side(c, x1, !fused, fused));      // fused: the score buffer holds the unrounded output instead

  auto wgrad = [&](float* out, int M, int N, const void* A, int64_t lda, int a_col0, const void* B, int64_t ldb,
                   int K, int accumulate) -> int {
    GemmProblem p = blank_problem();
    p.M = M; p.N = N; p.K = K;
    p.a_mn_major = 1; p.b_mn_major = 1;
    p.A = A; p.lda = lda; p.a_col0 = a_col0;
    p.B0 = B; p.ldb = ldb;
    p.epilogue = EPI_WGRAD; p.accumulate = accumulate;
    p.C = out; p.ldc = N;
    return a_gemm(c, p, TG_A_WGRAD);
  };
  auto dgrad = [&](int tag, int M, int N, int K, const void* A, int64_t lda, const void* W, int64_t ldw, void* C,
                   bool f32) -> int {
    GemmProblem p = blank_problem();   // C = A W  with W stored [K, N]
    p.M = M; p.N = N; p.K = K;
    p.A = A; p.lda = lda;
    p.B0 = W; p.ldb = ldw; p.b_mn_major = 1;
    p.epilogue = EPI_STORE; p.out_f32 = f32 ? 1 : 0; p.C = C; p.ldc = N;
    return a_gemm(c, p, tag);
  };
  const int strip = STRIP;      // rows per partial sum of the two-pass column reductions
  auto colsum = [&](const T* X, int64_t ldx, int cols, float* out) -> int {
    const int strips = (int)ceil_div(Tn, strip);
    { ProfScope ps(TG_A_BIAS, st);
    CK(launch_colsum_partial<T>(X, ldx, nullptr, Tn, cols, strip, strips, c.template p<float>(L.part), st));
    }
    { ProfScope ps(TG_A_BIAS, st);
    colsum_final_kernel<<<(unsigned)ceil_div(cols, COLSUM_FINAL_COLS), 256, 0, st>>>(c.template p<float>(L.part), strips, cols, acc, out);
    }
    CK(cudaGetLastError());
    return REVFFN_OK;
  };

  // P_down and W_o backward
  { ProfScope ps(TG_CAST, st);
  cast_stream_kernel<T><<<(unsigned)ceil_div((int64_t)Tn * h, 4 * 256), 256, 0, st>>>(dy1, D.ld_stream, Tn, h,
                                                                                      c.template p<T>(L.dyb));
  }
  CK(cudaGetLastError());
  if (G.w_down) CKR(wgrad(G.w_down, h, d, c.template p<T>(L.dyb), h, 0, c.template p<T>(L.a), d, Tn, acc));
  CKR(dgrad(TG_A_DGRAD, Tn, d, h, c.template p<T>(L.dyb), h, c.W.w_down, d, c.template p<T>(L.da), false));
  if (G.w_o) CKR(wgrad(G.w_o, d, d, c.template p<T>(L.da), d, 0, c.template p<T>(L.o), d, Tn, acc));
  if (fused) {
    GemmProblem p = blank_problem();   // dO = da W_o, written head-major by the product's epilogue
    p.M = Tn; p.N = d; p.K = d;
    p.A = c.template p<T>(L.da); p.lda = d;
    p.B0 = c.W.w_o; p.ldb = d; p.b_mn_major = 1;
    p.epilogue = EPI_HEADS; p.C = c.template p<T>(L.doh); p.hm_S = D.seq_len; p.hm_Sp = Sp;
    CKR(a_gemm(c, p, TG_A_DGRAD));
  } else {
    CKR(dgrad(TG_A_DGRAD, Tn, d, d, c.template p<T>(L.da), d, c.W.w_o, d, c.template p<T>(L.dob), false));
    { ProfScope ps(TG_A_HEADS, st);
    CK((launch_to_heads<T, T>(c.template p<T>(L.dob), d, nullptr, nullptr, Tn, D.seq_len, Sp, D.n_heads, hd,
                              c.template p<T>(L.doh), st)));
    }
  }

  // attention core backward
  if (fused) {
    if constexpr (std::is_same<T, bf16>::value) {
      { ProfScope ps(TG_A_SOFTMAX, st);
      attn_rowdot_kernel<<<(unsigned)ceil_div(L.rows * 32, 256), 256, 0, st>>>(
          c.template p<float>(L.sc), c.template p<bf16>(L.doh), c.template p<float>(L.lse), D.seq_len, Sp, L.rows,
          1.f / sqrtf((float)hd), c.template p<float2>(L.lse_d));
      }
      CK(cudaGetLastError());
      { ProfScope ps(TG_A_FLASH, st);
      // the two launches also undo the rotation and write dq and dk|dv token-major in the operand type
      CKR(launch_flash_bwd(c.template p<bf16>(L.qh), c.template p<bf16>(L.kh), c.template p<bf16>(L.vh),
                           c.template p<bf16>(L.doh), c.template p<float2>(L.lse_d), c.template p<float2>(L.cs), D.batch,
                           D.n_heads, D.n_kv_heads, D.seq_len, Sp, c.template p<bf16>(L.dq), d, c.template p<bf16>(L.dkv),
                           2 * (int64_t)dkv, dkv, c.template p<int>(L.status), st));
      ++g_prof.launches;
      }
    }
  } else {
    {
      GemmProblem p = a_grouped_rows(c);   // dP = dO V^T
      p.N = Sp; p.K = hd;
      p.A = c.template p<T>(L.doh); p.lda = hd;
      p.B0 = c.template p<T>(L.vh); p.ldb = hd;
      p.epilogue = EPI_STORE; p.out_f32 = 1; p.C = c.template p<float>(L.sc); p.ldc = Sp;
      CKR(a_gemm(c, p, TG_A_DP));
    }
    { ProfScope ps(TG_A_SOFTMAX, st);
    dsoftmax_causal_kernel<T><<<(unsigned)ceil_div(L.rows * 32, 256), 256, 0, st>>>(
        c.template p<T>(L.p), c.template p<float>(L.sc), D.seq_len, Sp, 1.f / sqrtf((float)hd), L.rows, c.template p<T>(L.ds));
    }
    CK(cudaGetLastError());
    auto kv_grad = [&](const T* A, const T* Bm, float* out) -> int {
      GemmProblem p = blank_problem();   // out[g] = A_g^T B_g over the query rows of key/value group g
      p.M = Sp; p.N = hd; p.K = (int)L.rows;
      p.a_mn_major = 1; p.b_mn_major = 1;
      p.A = A; p.lda = Sp;
      p.B0 = Bm; p.ldb = hd;
      p.epilogue = EPI_WGRAD; p.accumulate = 0;
      p.C = out; p.ldc = hd; p.c_group_stride = (int64_t)Sp * hd;
      p.group_mode = GROUP_K; p.n_groups = L.groups; p.group_off = c.template p<int32_t>(L.group_off);
      return a_gemm(c, p, TG_A_DKV);
    };
    CKR(kv_grad(c.template p<T>(L.p), c.template p<T>(L.doh), c.template p<float>(L.dvh)));    // dV = P^T dO
    CKR(kv_grad(c.template p<T>(L.ds), c.template p<T>(L.qh), c.template p<float>(L.dkh)));    // dK = dS^T Q
    {
      GemmProblem p = a_grouped_rows(c);   // dQ = dS K
      p.N = hd; p.K = Sp;
      p.A = c.template p<T>(L.ds); p.lda = Sp;
      p.B0 = c.template p<T>(L.kh); p.ldb = hd; p.b_mn_major = 1;
      p.epilogue = EPI_STORE; p.out_f32 = 1; p.C = c.template p<float>(L.dqh); p.ldc = hd;
      CKR(a_gemm(c, p, TG_A_DQ));
    }
  }
  if (!fused) {
    // back to token-major; the rotation is undone by its transpose
    { ProfScope ps(TG_A_HEADS, st);
    CK((launch_from_heads<float, T>(c.template p<float>(L.dqh), c.template p<float2>(L.cs), -1.f, Tn, D.seq_len, Sp,
                                    D.n_heads, hd, c.template p<T>(L.dq), d, 0, st)));
    }
    { ProfScope ps(TG_A_HEADS, st);
    CK((launch_from_heads<float, T>(c.template p<float>(L.dkh), c.template p<float2>(L.cs), -1.f, Tn, D.seq_len, Sp,
                                    D.n_kv_heads, hd, c.template p<T>(L.dkv), 2 * (int64_t)dkv, 0, st)));
    }
    { ProfScope ps(TG_A_HEADS, st);
    CK((launch_from_heads<float, T>(c.template p<float>(L.dvh), nullptr, 1.f, Tn, D.seq_len, Sp, D.n_kv_heads, hd,
                                    c.template p<T>(L.dkv), 2 * (int64_t)dkv, dkv, st)));
    }
  }

  // q/k/v projections backward
  const T* u1 = c.template p<T>(L.u12);
  const T* u2 = u1 + (int64_t)Tn * d;
  if (G.b_q) CKR(colsum(c.template p<T>(L.dq), d, d, G.b_q));
  if (G.b_k) CKR(colsum(c.template p<T>(L.dkv), 2 * (int64_t)dkv, dkv, G.b_k));
  if (G.b_v) CKR(colsum(c.template p<T>(L.dkv) + dkv, 2 * (int64_t)dkv, dkv, G.b_v));
  if (G.w_q) CKR(wgrad(G.w_q, d, d, c.template p<T>(L.dq), d, 0, u1, d, Tn, acc));
  if (G.w_k) CKR(wgrad(G.w_k, dkv, d, c.template p<T>(L.dkv), 2 * (int64_t)dkv, 0, u2, d, Tn, acc));
  if (G.w_v) CKR(wgrad(G.w_v, dkv, d, c.template p<T>(L.dkv), 2 * (int64_t)dkv, dkv, u2, d, Tn, acc));
  T* du1 = c.template p<T>(L.du12);
  T* du2 = du1 + (int64_t)Tn * d;
  CKR(dgrad(TG_A_DGRAD, Tn, d, d, c.template p<T>(L.dq), d, c.W.w_q, d, du1, false));
  {
    GemmProblem p = blank_problem();   // dU2 = dK W_k + dV W_v
    p.M = Tn; p.N = d; p.K = 2 * dkv;
    p.A = c.template p<T>(L.dkv); p.lda = 2 * (int64_t)dkv;
    p.B0 = c.W.w_k; p.B1 = c.W.w_v; p.ldb = d; p.b_mn_major = 1; p.concat = CONCAT_K;
    p.epilogue = EPI_STORE; p.C = du2; p.ldc = d;
    CKR(a_gemm(c, p, TG_A_DGRAD));
  }

  // P_up and the norm, both streams at once where the rows are independent
  if (G.w_up) CKR(wgrad(G.w_up, d, h, du1, d, 0, c.template p<T>(L.n12), h, 2 * Tn, acc));
  CKR(dgrad(TG_DN, 2 * Tn, h, d, du1, d, c.W.w_up, h, c.template p<float>(L.dn12), true));
  if (dx1 != dy1) {
    copy_stream_kernel<<<(unsigned)ceil_div((int64_t)Tn * h, 4 * 256), 256, 0, st>>>(dy1, D.ld_stream, Tn, h, dx1,
                                                                                     D.ld_stream);
    ++g_prof.launches;
    CK(cudaGetLastError());
  }
  const float* dn1 = c.template p<float>(L.dn12);
  const float* dn2 = dn1 + (int64_t)Tn * h;
  const float* r1 = c.template p<float>(L.r12);
  const float* r2 = r1 + Tn;
  { ProfScope ps(TG_NORM_BWD, st);
  rmsnorm_bwd_rows_kernel<<<(unsigned)ceil_div((int64_t)Tn * 32, 128), 128, 0, st>>>(dn1, x1, D.ld_stream, c.W.norm_gamma, r1,
                                                                                     0, Tn, h, dx1, D.ld_stream);
  }
  CK(cudaGetLastError());
  { ProfScope ps(TG_NORM_BWD, st);
  rmsnorm_bwd_rows_kernel<<<(unsigned)ceil_div((int64_t)Tn * 32, 128), 128, 0, st>>>(dn2, x2, D.ld_stream, c.W.norm_gamma, r2,
                                                                                     0, Tn, h, dx2, D.ld_stream);
  }
  CK(cudaGetLastError());
  if (G.norm_gamma) {
    const int strips = (int)ceil_div(Tn, strip);
    for (int side = 0; side < 2; ++side) {
      { ProfScope ps(TG_DGAMMA, st);
      CK(launch_dgamma_partial(side ? dn2 : dn1, side ? x2 : x1, D.ld_stream, side ? r2 : r1, Tn, h, strip, strips,
                               c.template p<float>(L.part), st));
      }
      { ProfScope ps(TG_DGAMMA, st);
      colsum_final_kernel<<<(unsigned)ceil_div(h, COLSUM_FINAL_COLS), 256, 0, st>>>(c.template p<float>(L.part), strips, h,
                                                                      side ? 1 : acc, G.norm_gamma);
      }
      CK(cudaGetLastError());
    }
  }
  return REVFFN_OK;
}

enum APass { APASS_FWD = 3, APASS_INV = 4, APASS_BWD = 5 };

template <typename T>
static int a_dispatch(APass pass, const revffn_attn_desc& D, const revffn_attn_weights& W, const AttnLayout& L, void* ws,
                      cudaStream_t st, const float* in1, const float* x2, const float* dy1, float* out1, float* dx2,
                      int n_iter, const revffn_attn_grads* G) {
  ACtx<T> c;
  c.D = D; c.W = W; c.L = L; c.ws = reinterpret_cast<char*>(ws); c.st = st;
  g_prof.pass = (int)pass;
  c.tc = std::is_same<T, bf16>::value && !(D.flags & REVFFN_FLAG_FORCE_SIMT);
  if (c.tc) CKR(tc_prepare());
  CK(cudaMemsetAsync(c.ws + L.status.off, 0, L.status.bytes, st));
  if (L.T == 0) return REVFFN_OK;
  if (pass == APASS_FWD) return a_forward(c, in1, x2, out1);
  if (pass == APASS_INV) return a_inverse(c, in1, x2, out1, n_iter);
  return a_backward(c, in1, x2, dy1, out1, dx2, *G);
}

static int a_entry(APass pass, const revffn_attn_desc* desc, const revffn_attn_weights* w, const float* in1,
                   const float* x2, const float* dy1, float* out1, float* dx2, int n_iter,
                   const revffn_attn_grads* grads, void* ws, size_t ws_bytes, void* cuda_stream) {
  CKR(validate_attn_desc(desc));
  CKR(validate_attn_weights(w));
  if (!ws) return REVFFN_ERR_NULL;
  if (n_iter < 0) return REVFFN_ERR_SHAPE;
  const bool bwd = pass == APASS_BWD;
  if (bwd && !grads) return REVFFN_ERR_NULL;
  if ((int64_t)desc->batch * desc->seq_len > 0 && (!in1 || !x2 || !out1 || (bwd && (!dy1 || !dx2)))) return REVFFN_ERR_NULL;
  if (!aligned16(in1) || !aligned16(x2) || !aligned16(dy1) || !aligned16(out1) || !aligned16(dx2) ||
      (reinterpret_cast<uintptr_t>(ws) & 255u))
    return REVFFN_ERR_ALIGN;
  if (grads) {
    const float* gs[] = {grads->norm_gamma, grads->w_up, grads->w_down, grads->w_q, grads->w_k, grads->w_v,
                         grads->w_o, grads->b_q, grads->b_k, grads->b_v};
    for (const float* g : gs)
      if (g && !aligned16(g)) return REVFFN_ERR_ALIGN;
  }
  AttnLayout L = plan_attn(*desc);
  if (ws_bytes < (bwd ? L.bwd_bytes : L.fwd_bytes)) return REVFFN_ERR_WORKSPACE;
  CKR(check_device());
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (desc->weight_dtype == REVFFN_BF16)
    return a_dispatch<bf16>(pass, *desc, *w, L, ws, st, in1, x2, dy1, out1, dx2, n_iter, grads);
  return a_dispatch<float>(pass, *desc, *w, L, ws, st, in1, x2, dy1, out1, dx2, n_iter, grads);
}

}  // namespace revffn

extern "C" {

int revffn_attn_workspace_size(const revffn_attn_desc* desc, size_t* fwd_bytes, size_t* bwd_bytes) {
  int r = revffn::validate_attn_desc(desc);
  if (r != REVFFN_OK) return r;
  revffn::AttnLayout L = revffn::plan_attn(*desc);
  if (fwd_bytes) *fwd_bytes = L.fwd_bytes;
  if (bwd_bytes) *bwd_bytes = L.bwd_bytes;
  return REVFFN_OK;
}

int revffn_attn_forward(const revffn_attn_desc* desc, const revffn_attn_weights* w, const float* x1, const float* x2,
                        float* y1, void* ws, size_t ws_bytes, void* cuda_stream) {
  return revffn::a_entry(revffn::APASS_FWD, desc, w, x1, x2, nullptr, y1, nullptr, 0, nullptr, ws, ws_bytes, cuda_stream);
}

int revffn_attn_inverse(const revffn_attn_desc* desc, const revffn_attn_weights* w, const float* y1, const float* x2,
                        float* x1, int32_t n_iter, void* ws, size_t ws_bytes, void* cuda_stream) {
  if (n_iter > 1 && x1 == y1) return REVFFN_ERR_UNSUPPORTED;
  return revffn::a_entry(revffn::APASS_INV, desc, w, y1, x2, nullptr, x1, nullptr, n_iter, nullptr, ws, ws_bytes,
                         cuda_stream);
}

int revffn_attn_backward(const revffn_attn_desc* desc, const revffn_attn_weights* w, const float* x1, const float* x2,
                         const float* dy1, float* dx1, float* dx2_inout, const revffn_attn_grads* grads, void* ws,
                         size_t ws_bytes, void* cuda_stream) {
  return revffn::a_entry(revffn::APASS_BWD, desc, w, x1, x2, dy1, dx1, dx2_inout, 0, grads, ws, ws_bytes, cuda_stream);
}

int revffn_attn_status(const void* ws, void* cuda_stream, int32_t* device_status) {
  return revffn_moe_status(ws, cuda_stream, device_status);
}

}  // extern "C"
