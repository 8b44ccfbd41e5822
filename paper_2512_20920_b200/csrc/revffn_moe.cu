// C ABI, workspace planner and launch sequences of the RevFFN MoE coupling branch.
// See include/revffn_moe.h for the contract of every entry point.

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <type_traits>
#include <string>
#include <vector>

#include "common.cuh"
#include "../../include/revffn_debug.h"
#include "routing.cuh"
#include "backward_ew.cuh"
#include "gemm.cuh"
#include "gemm_tcgen05.cuh"
#include "fp8.cuh"

namespace revffn {


// ---------------------------------------------------------------------------
// Launch accounting and optional per-kernel timing (CUDA events on the caller's
// stream around each launch).  Off by default; revffn_prof_enable switches it.
// ---------------------------------------------------------------------------
enum Tag {
  TG_NORM, TG_FOLD, TG_ROUTER, TG_MAP, TG_PUP, TG_GATHER, TG_EXP_GATEUP, TG_EXP_DOWN, TG_SH_GATEUP, TG_SH_DOWN,
  TG_COMBINE, TG_PDOWN, TG_CAST, TG_DZ, TG_WG_PDOWN, TG_SHGATE_BWD, TG_SH_DH, TG_WG_SH_DOWN, TG_SH_DU,
  TG_WG_SH_GATE, TG_WG_SH_UP, TG_WG_SH_GATEUP, TG_WG_SGATE, TG_GATHER_DZ, TG_EXP_DH, TG_EXP_DU, TG_WG_EXP_DOWN, TG_WG_EXP_GATE,
  TG_WG_EXP_UP, TG_WG_EXP_GATEUP, TG_ROUTER_BWD, TG_WG_ROUTER, TG_DU_REDUCE, TG_DN, TG_WG_PUP, TG_NORM_BWD, TG_DGAMMA,
  // attention coupling branch
  TG_A_TABLES, TG_A_QKV, TG_A_HEADS, TG_A_SCORES, TG_A_SOFTMAX, TG_A_PV, TG_A_WO, TG_A_WGRAD, TG_A_DGRAD, TG_A_BIAS,
  TG_A_DP, TG_A_DKV, TG_A_DQ, TG_A_FLASH, TG_COUNT
};
static const char* kTagNames[TG_COUNT] = {
    "rmsnorm_fwd", "fold_router", "router_topk", "permute_maps", "gemm_p_up", "gather_u", "gemm_expert_gate_up_swiglu",
    "gemm_expert_down_scale", "gemm_shared_gate_up_swiglu", "gemm_shared_down", "combine", "gemm_p_down_couple",
    "cast_dy2", "gemm_dz", "wgrad_p_down", "shared_gate_bwd", "gemm_shared_dh_dswiglu", "wgrad_shared_down",
    "gemm_shared_du", "wgrad_shared_gate", "wgrad_shared_up", "wgrad_shared_gate_up", "wgrad_shared_sgate", "gather_dz",
    "gemm_expert_dh_dswiglu", "gemm_expert_du", "wgrad_expert_down", "wgrad_expert_gate", "wgrad_expert_up", "wgrad_expert_gate_up",
    "router_bwd", "wgrad_router", "du_reduce", "gemm_dn", "wgrad_p_up", "rmsnorm_bwd", "dgamma",
    "attn_tables", "gemm_qkv", "attn_heads", "gemm_scores", "attn_softmax", "gemm_pv", "gemm_w_o", "attn_wgrad",
    "attn_dgrad", "attn_bias_grad", "gemm_dp", "gemm_dk_dv", "gemm_dq", "flash_attention"};
constexpr int N_PASSES = 6;
static const char* kPassNames[N_PASSES] = {"fwd", "inv", "bwd", "attn_fwd", "attn_inv", "attn_bwd"};

struct Profiler {
  bool on = false;
  int pass = 0;
  std::vector<cudaEvent_t> pool;
  size_t used = 0;
  struct Rec { int slot; size_t e; };
  std::vector<Rec> recs;
  long long launches = 0;
};
static Profiler g_prof;

struct ProfScope {
  cudaStream_t st;
  bool active;
  ProfScope(int tag, cudaStream_t s) : st(s), active(false) {
    ++g_prof.launches;
    if (!g_prof.on) return;
    while (g_prof.pool.size() < g_prof.used + 2) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) return;
      g_prof.pool.push_back(e);
    }
    cudaEventRecord(g_prof.pool[g_prof.used], st);
    g_prof.recs.push_back({g_prof.pass * TG_COUNT + tag, g_prof.used});
    active = true;
  }
  ~ProfScope() {
    if (!active) return;
    cudaEventRecord(g_prof.pool[g_prof.used + 1], st);
    g_prof.used += 2;
  }
};

// ---------------------------------------------------------------------------
// Workspace layout
// ---------------------------------------------------------------------------
struct Buf { size_t off = 0, bytes = 0; };
constexpr int MAX_GUARDS = 80;
constexpr int GUARD_BYTES = 256;

struct WsLayout {
  // forward / inverse
  Buf status, rows_total, w_rc, w_rc_part, n, r, idx, gates, sgate, prob, local_rank, chunk_cnt, chunk_base, expert_cnt,
      expert_off, tile_group, tok_chunks, tok_row, row_tok, row_gate, u, up, hmid, o, hs, s, z, upq, up_scale, hq, h_scale;
  int max_chunks = 0;
  size_t fwd_bytes = 0;
  size_t saved_bytes = 0;   // fwd region + SwiGLU pre-activations: what a saved evaluation consists of
  // backward only
  Buf ab, abs, gb, dz, ds, dl, dop, dg_part, tok_dl, row_dl, dlf, dur, dup, dush, du, dn, part, ksplit;
  int ld_dlf = 0;
  size_t bwd_bytes = 0;
  int64_t rows_pad = 0;   // upper bound on padded rows
  int n_chunks = 0, max_tiles = 0, dg_ld = 0, strips = 0;
  // REVFFN_FLAG_DEBUG_CHECKS: a guard zone of GUARD_BYTES follows every buffer
  int n_guards = 0;
  size_t guard_off[MAX_GUARDS];
};

constexpr int STRIP = 32;    // tokens per strip in two-pass column reductions
constexpr int SPLIT_K_MAX = 4;   // most K slices of a dense weight gradient

static WsLayout plan_workspace(const revffn_moe_desc& D) {
  WsLayout L;
  const size_t ts = D.weight_dtype == REVFFN_BF16 ? 2 : 4;
  const int64_t T = D.tokens, d = D.d_model, h = d / 2, E = D.n_experts, k = D.top_k, I = D.d_expert,
                Is = D.d_shared;
  L.rows_pad = max_padded_rows(T, (int)k, (int)E);
  L.n_chunks = (int)ceil_div(T > 0 ? T : 1, MAP_CHUNK);
  L.max_tiles = (int)(L.rows_pad / ROW_PAD);
  L.dg_ld = (int)ceil_div(I, SIMT_BN);
  L.strips = (int)ceil_div(T > 0 ? T : 1, STRIP);
  const int64_t Rp = L.rows_pad;
  size_t off = 0;
  const bool guards = (D.flags & REVFFN_FLAG_DEBUG_CHECKS) != 0;
  auto take = [&](Buf& b, size_t bytes) {
    b.off = off; b.bytes = bytes;
    off += (size_t)round_up((int64_t)(bytes > 0 ? bytes : 1), 256);
    if (guards && L.n_guards < MAX_GUARDS) {
      L.guard_off[L.n_guards++] = off;
      off += GUARD_BYTES;
    }
  };
  take(L.status, 256);
  take(L.rows_total, 256);
  take(L.w_rc, (size_t)(E + 1) * h * 8);
  take(L.w_rc_part, (size_t)FOLD_SLICES * (E + 1) * h * 8);
  take(L.n, (size_t)T * h * ts);
  take(L.r, (size_t)T * 4);
  take(L.idx, (size_t)T * k * 4);
  take(L.gates, (size_t)T * k * 4);
  take(L.sgate, (size_t)T * 4);
  take(L.prob, (D.flags & REVFFN_FLAG_GATE_SOFTMAX_ALL) ? (size_t)T * E * 4 : 0);
  take(L.local_rank, (size_t)T * k * 4);
  take(L.chunk_cnt, (size_t)L.n_chunks * E * 4);
  take(L.chunk_base, (size_t)L.n_chunks * E * 4);
  take(L.expert_cnt, (size_t)E * 4);
  take(L.expert_off, (size_t)(E + 1) * 4);
  take(L.tile_group, (size_t)L.max_tiles * 4);
  L.max_chunks = (int)(ceil_div(T * k, TOK_CHUNK) + E);
  take(L.tok_chunks, (size_t)L.max_chunks * 16);
  take(L.tok_row, (size_t)T * k * 4);
  take(L.row_tok, (size_t)Rp * 4);
  take(L.row_gate, (size_t)Rp * 4);
  take(L.u, (size_t)T * d * ts);
  take(L.up, (size_t)Rp * d * ts);
  take(L.hmid, (size_t)Rp * I * ts);
  take(L.o, (size_t)Rp * d * ts);
  take(L.hs, (size_t)T * Is * ts);
  take(L.s, (size_t)T * d * ts);
  take(L.z, (size_t)T * d * ts);
  // REVFFN_FLAG_FP8_EXPERTS: e4m3 copies of the permuted u rows and of g*H with their row scales
  const bool fp8 = (D.flags & REVFFN_FLAG_FP8_EXPERTS) != 0;
  take(L.upq, fp8 ? (size_t)Rp * d : 0);
  take(L.up_scale, fp8 ? (size_t)Rp * 4 : 0);
  take(L.hq, fp8 ? (size_t)Rp * I : 0);
  take(L.h_scale, fp8 ? (size_t)Rp * 4 : 0);
  L.fwd_bytes = off;
  take(L.ab, (size_t)Rp * 2 * I * ts);
  take(L.abs, (size_t)T * 2 * Is * ts);
  L.saved_bytes = off;
  take(L.gb, (size_t)T * h * ts);
  take(L.dz, (size_t)T * d * ts);
  take(L.ds, (size_t)T * d * ts);
  take(L.dl, (size_t)T * 4);
  take(L.dop, (size_t)Rp * d * ts);
  take(L.dg_part, (size_t)Rp * L.dg_ld * 4);
  take(L.tok_dl, (size_t)T * k * 4);
  take(L.row_dl, (size_t)Rp * 4);
  L.ld_dlf = (int)round_up(E, 64);
  const bool dense_gate = (D.flags & REVFFN_FLAG_GATE_SOFTMAX_ALL) != 0;
  take(L.dlf, dense_gate ? (size_t)T * L.ld_dlf * ts : 0);
  take(L.dur, dense_gate ? (size_t)T * d * ts : 0);
  take(L.dup, (size_t)Rp * d * ts);
  take(L.dush, (size_t)T * d * ts);
  take(L.du, (size_t)T * d * ts);
  take(L.dn, (size_t)T * h * 4);
  take(L.part, (size_t)L.strips * d * 4);
  take(L.ksplit, (size_t)SPLIT_K_MAX * d * h * 4);      // partial sums of the adapters' K-split weight gradients
  L.bwd_bytes = off;
  return L;
}

static int validate_desc(const revffn_moe_desc* D) {
  if (!D) return REVFFN_ERR_NULL;
  if (D->tokens < 0 || D->d_model <= 0 || (D->d_model & 1)) return REVFFN_ERR_SHAPE;
  if (D->top_k < 1 || D->top_k > 8 || D->n_experts < D->top_k || D->n_experts > 256) return REVFFN_ERR_SHAPE;
  if (D->d_expert <= 0 || D->d_shared < 0) return REVFFN_ERR_SHAPE;
  if (D->weight_dtype != REVFFN_F32 && D->weight_dtype != REVFFN_BF16) return REVFFN_ERR_SHAPE;
  if (D->norm_kind != REVFFN_NORM_RMS && D->norm_kind != REVFFN_NORM_NONE) return REVFFN_ERR_SHAPE;
  const int h = D->d_model / 2;
  const int mult = D->weight_dtype == REVFFN_BF16 ? 128 : 8;
  if (h % mult || D->d_model % mult || D->d_expert % mult || D->d_shared % mult) return REVFFN_ERR_SHAPE;
  if (D->ld_stream < h || (D->ld_stream % 4)) return REVFFN_ERR_ALIGN;
  if ((int64_t)D->tokens * D->top_k > (int64_t)1 << 28) return REVFFN_ERR_SHAPE;
  if (D->flags & REVFFN_FLAG_FP8_EXPERTS) {
    if (D->weight_dtype != REVFFN_BF16 || (D->flags & (REVFFN_FLAG_FORCE_SIMT | REVFFN_FLAG_SAVE_ACTIVATIONS | REVFFN_FLAG_REUSE_ACTIVATIONS)) ||
        D->d_model > 2048 || D->d_expert > 2048 || D->d_model % 256 != 0)
      return REVFFN_ERR_UNSUPPORTED;
  }
  return REVFFN_OK;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Routing record: [T*k] int32 indices | [T*k] float gates | [T] float shared gate, parts 16-byte aligned.
struct RecordLayout { size_t gates_off, sgate_off, bytes; };
static RecordLayout record_layout(const revffn_moe_desc& D) {
  RecordLayout r;
  const size_t tk = (size_t)D.tokens * D.top_k * 4;
  r.gates_off = (size_t)round_up((int64_t)tk, 16);
  r.sgate_off = r.gates_off + (size_t)round_up((int64_t)tk, 16);
  r.bytes = r.sgate_off + (size_t)round_up((int64_t)D.tokens * 4, 16);
  return r;
}
// Bytes between the index arrays (or routing records) of consecutive layers of a stack.
static size_t routing_stride(const revffn_moe_desc& D) {
  return (D.flags & REVFFN_FLAG_ROUTING_RECORD) ? record_layout(D).bytes : (size_t)D.tokens * D.top_k * 4;
}

static int validate_weights(const revffn_moe_desc& D, const revffn_moe_weights* w) {
  if (!w) return REVFFN_ERR_NULL;
  if (!w->w_up || !w->w_down || !w->w_router || !w->w_gate || !w->w_upx || !w->w_downx) return REVFFN_ERR_NULL;
  if (D.d_shared > 0 && (!w->ws_gate || !w->ws_up || !w->ws_down || !w->ws_sgate)) return REVFFN_ERR_NULL;
  if ((D.flags & REVFFN_FLAG_FP8_EXPERTS) && (!w->q_gate || !w->q_upx || !w->q_downx || !w->s_gate || !w->s_upx || !w->s_downx))
    return REVFFN_ERR_NULL;
  {
    const void* qs[] = {w->q_gate, w->q_upx, w->q_downx, w->s_gate, w->s_upx, w->s_downx};
    for (const void* q : qs)
      if (q && !aligned16(q)) return REVFFN_ERR_ALIGN;
  }
  const void* ps[] = {w->norm_gamma, w->w_up, w->w_down, w->w_router, w->b_router, w->w_gate, w->w_upx,
                      w->w_downx, w->ws_gate, w->ws_up, w->ws_down, w->ws_sgate};
  for (const void* p : ps)
    if (p && !aligned16(p)) return REVFFN_ERR_ALIGN;
  return REVFFN_OK;
}

static int check_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return REVFFN_ERR_CUDA;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return REVFFN_ERR_CUDA;
  return major == 10 ? REVFFN_OK : REVFFN_ERR_ARCH;
}

#define CK(expr)                                   \
  do {                                             \
    cudaError_t e_ = (expr);                       \
    if (e_ != cudaSuccess) return REVFFN_ERR_CUDA; \
  } while (0)
#define CKR(expr)                  \
  do {                             \
    int r_ = (expr);               \
    if (r_ != REVFFN_OK) return r_; \
  } while (0)

// ---------------------------------------------------------------------------
// Guard zones between the workspace's buffers (REVFFN_FLAG_DEBUG_CHECKS): filled with a
// position-dependent pattern when a pass starts, verified when it ends.  A kernel that
// writes past the end of its buffer lands in one of them.
// ---------------------------------------------------------------------------
struct GuardTable { int n; unsigned long long off[MAX_GUARDS]; };

__device__ __forceinline__ uint32_t guard_word(int zone, int i) { return 0xC0DE0000u ^ (uint32_t)(zone * 64 + i) * 2654435761u; }

__global__ void guard_fill_kernel(char* __restrict__ ws, const GuardTable g) {
  const int z = blockIdx.x, i = threadIdx.x;
  reinterpret_cast<uint32_t*>(ws + g.off[z])[i] = guard_word(z, i);
}
__global__ void guard_check_kernel(const char* __restrict__ ws, const GuardTable g, int* __restrict__ status) {
  const int z = blockIdx.x, i = threadIdx.x;
  if (reinterpret_cast<const uint32_t*>(ws + g.off[z])[i] != guard_word(z, i)) set_status(status, REVFFN_ERR_CANARY);
}

// Guards that lie inside the first `limit` bytes of the workspace (a forward pass may own only fwd_bytes).
static GuardTable guard_table(const WsLayout& L, size_t limit) {
  GuardTable g;
  g.n = 0;
  for (int i = 0; i < L.n_guards; ++i)
    if (L.guard_off[i] + GUARD_BYTES <= limit) g.off[g.n++] = L.guard_off[i];
  return g;
}
static int guards_fill(const WsLayout& L, size_t limit, char* ws, cudaStream_t st) {
  const GuardTable g = guard_table(L, limit);
  if (g.n == 0) return REVFFN_OK;
  guard_fill_kernel<<<g.n, GUARD_BYTES / 4, 0, st>>>(ws, g);
  return cudaGetLastError() == cudaSuccess ? REVFFN_OK : REVFFN_ERR_CUDA;
}
static int guards_check(const WsLayout& L, size_t limit, char* ws, cudaStream_t st) {
  const GuardTable g = guard_table(L, limit);
  if (g.n == 0) return REVFFN_OK;
  guard_check_kernel<<<g.n, GUARD_BYTES / 4, 0, st>>>(ws, g, reinterpret_cast<int*>(ws + L.status.off));
  return cudaGetLastError() == cudaSuccess ? REVFFN_OK : REVFFN_ERR_CUDA;
}

// ---------------------------------------------------------------------------
// Launch context
// ---------------------------------------------------------------------------
// A second stream per device for launches that do not depend on what the caller's stream is doing at that point
// (the shared expert beside the routed experts, the weight gradients beside the chain of input gradients).  The
// matrix products are persistent kernels of one CTA per SM and equal tiles, so most of them end with a partly
// empty last round of tiles; a kernel from the other stream starts on the SMs that fall idle there.  Ordering is by
// events from a small ring (a wait refers to the record that preceded it, so an event can be recorded again while
// an older wait is still pending).  Created on first use.
struct Overlap {
  cudaStream_t side = nullptr;
  cudaEvent_t ev[64];
  std::atomic<unsigned> next{0};
  bool made = false;
  cudaEvent_t mark(cudaStream_t s, cudaError_t* e) {       // an event that follows everything queued on s so far
    cudaEvent_t x = ev[next.fetch_add(1) & 63u];
    *e = cudaEventRecord(x, s);
    return x;
  }
};

static Overlap* overlap_state() {
  static Overlap state[64];
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  Overlap& o = state[dev];
  if (!o.made) {
    for (auto& x : o.ev)
      if (cudaEventCreateWithFlags(&x, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaStreamCreateWithFlags(&o.side, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    o.made = true;
  }
  return &o;
}

template <typename T>
struct Ctx {
  revffn_moe_desc D;
  revffn_moe_weights W;
  WsLayout L;
  char* ws;
  cudaStream_t st;
  Overlap* ov = nullptr;   // non-null: the second stream is in use for this call
  // what is queued on `to` from now on follows everything queued on `from` so far (no-op without the second stream)
  int order(cudaStream_t from, cudaStream_t to) const {
    if (!ov || from == to) return REVFFN_OK;
    cudaError_t e;
    cudaEvent_t x = ov->mark(from, &e);
    if (e != cudaSuccess || cudaStreamWaitEvent(to, x, 0) != cudaSuccess) return REVFFN_ERR_CUDA;
    return REVFFN_OK;
  }
  cudaStream_t side() const { return ov ? ov->side : st; }
  bool tc;   // tcgen05 back end for the matrix products
  template <typename U> U* p(const Buf& b) const { return reinterpret_cast<U*>(ws + b.off); }
  int T_() const { return D.tokens; }
};

template <typename T>
static int run_gemm(const Ctx<T>& c, GemmProblem p, int tag) {
  p.status = c.template p<int>(c.L.status);
  ProfScope ps(tag, c.st);
  if constexpr (std::is_same<T, bf16>::value) {
    if (c.tc) return launch_gemm_tc(p, c.st);
  }
  return launch_gemm_simt<T>(p, c.st) == cudaSuccess ? REVFFN_OK : REVFFN_ERR_CUDA;
}

template <typename T>
static int dg_parts(const Ctx<T>& c, int N) {
  if constexpr (std::is_same<T, bf16>::value) {
    if (c.tc) return tc_dg_parts(N);
  }
  return simt_dg_parts(N);
}

static GemmProblem blank_problem() {
  GemmProblem p;
  memset(&p, 0, sizeof(p));
  p.resid_sign = 1.f;
  return p;
}

// ---------------------------------------------------------------------------
// F = MLP(Norm(Y1)) up to z (the input of P_down).  save_ab keeps the SwiGLU
// pre-activations for the backward pass.
// ---------------------------------------------------------------------------
template <typename T>
static int run_branch(const Ctx<T>& c, const float* y1, const int32_t* idx_in, int32_t* idx_user, bool save_ab) {
  const revffn_moe_desc& D = c.D;
  const WsLayout& L = c.L;
  const int Tn = D.tokens, d = D.d_model, h = d / 2, E = D.n_experts, k = D.top_k, I = D.d_expert, Is = D.d_shared;
  const int norm_none = D.norm_kind == REVFFN_NORM_NONE;
  cudaStream_t st = c.st;
  cudaStream_t rt = c.side();      // router and permutation maps (the caller's stream without the second stream)
  const T* w_up = reinterpret_cast<const T*>(c.W.w_up);
  CKR(c.order(st, rt));

  // Norm
  { ProfScope ps(TG_NORM, st);
  rmsnorm_fwd_kernel<T><<<(unsigned)ceil_div((int64_t)Tn * 32, 128), 128, 0, st>>>(
      y1, D.ld_stream, c.W.norm_gamma, D.norm_eps, norm_none, Tn, h, c.template p<T>(L.n), c.template p<float>(L.r));
  }
  CK(cudaGetLastError());

  // Router: fold through P_up, logits, top-k, gates -- or everything from a routing record.  The router reads y1
  // and the permutation maps read the router's result: neither needs the norm or P_up, so with the second stream
  // they run beside those two.
  const bool records = (D.flags & REVFFN_FLAG_ROUTING_RECORD) != 0;
  const bool gate_all = (D.flags & REVFFN_FLAG_GATE_SOFTMAX_ALL) != 0;
  const RecordLayout R = record_layout(D);
  if (idx_in && records && !gate_all) {
    const char* rec = reinterpret_cast<const char*>(idx_in);
    const size_t tk = (size_t)Tn * k * 4;
    CK(cudaMemcpyAsync(c.ws + L.idx.off, rec, tk, cudaMemcpyDeviceToDevice, rt));
    CK(cudaMemcpyAsync(c.ws + L.gates.off, rec + R.gates_off, tk, cudaMemcpyDeviceToDevice, rt));
    CK(cudaMemcpyAsync(c.ws + L.sgate.off, rec + R.sgate_off, (size_t)Tn * 4, cudaMemcpyDeviceToDevice, rt));
  } else {
    if (!(D.flags & REVFFN_FLAG_ROUTER_FOLDED)) {     // else the folded router of an earlier call is still in the workspace
    ProfScope ps(TG_FOLD, rt);
    if (d <= FOLD_SLICES * fold_slice_rows<T>()) {
      CK(launch_fold_router_mma<T>(reinterpret_cast<const T*>(c.W.w_router), reinterpret_cast<const T*>(c.W.ws_sgate),
                                   w_up, E, d, h, c.template p<double>(L.w_rc_part), c.template p<double>(L.w_rc), rt));
      ++g_prof.launches;      // two kernels under one timing scope: the slice products and their sum
    } else {
      CK(launch_fold_router<T>(reinterpret_cast<const T*>(c.W.w_router), reinterpret_cast<const T*>(c.W.ws_sgate), w_up,
                               E, d, h, c.template p<double>(L.w_rc), rt));
    }
    }
    { ProfScope ps(TG_ROUTER, rt);
    CK(launch_router_topk(y1, D.ld_stream, c.W.norm_gamma, D.norm_eps, norm_none, c.template p<double>(L.w_rc),
                          c.W.b_router, Tn, h, E, k, Is > 0 ? 1 : 0, idx_in, c.template p<int32_t>(L.idx),
                          c.template p<float>(L.gates), c.template p<float>(L.sgate), idx_user,
                          gate_all ? c.template p<float>(L.prob) : nullptr, c.template p<int>(L.status),
                          (D.flags & REVFFN_FLAG_DEBUG_CHECKS) ? 1 : 0, rt));
    }
    if (idx_user && records) {      // complete the record the kernel has started with the indices
      char* rec = reinterpret_cast<char*>(idx_user);
      CK(cudaMemcpyAsync(rec + R.gates_off, c.ws + L.gates.off, (size_t)Tn * k * 4, cudaMemcpyDeviceToDevice, rt));
      CK(cudaMemcpyAsync(rec + R.sgate_off, c.ws + L.sgate.off, (size_t)Tn * 4, cudaMemcpyDeviceToDevice, rt));
    }
  }

  // Permutation maps
  CK(cudaMemsetAsync(c.ws + L.row_tok.off, 0xFF, L.row_tok.bytes, rt));
  CK(cudaMemsetAsync(c.ws + L.row_gate.off, 0, L.row_gate.bytes, rt));
  { ProfScope ps(TG_MAP, rt);
  map_rank_kernel<<<L.n_chunks, 256, (size_t)MAP_CHUNK * k * 4, rt>>>(
      c.template p<int32_t>(L.idx), Tn, k, E, c.template p<int32_t>(L.local_rank), c.template p<int32_t>(L.chunk_cnt),
      c.template p<int>(L.status));
  }
  CK(cudaGetLastError());
  { ProfScope ps(TG_MAP, rt);
  map_scan_kernel<<<1, 256, (size_t)(E + 1) * 4, rt>>>(
      c.template p<int32_t>(L.chunk_cnt), L.n_chunks, E, c.template p<int32_t>(L.chunk_base),
      c.template p<int32_t>(L.expert_cnt), c.template p<int32_t>(L.expert_off), c.template p<int32_t>(L.tile_group),
      c.template p<int32_t>(L.rows_total), L.max_tiles, c.template p<int4>(L.tok_chunks), L.max_chunks);
  }
  CK(cudaGetLastError());
  { ProfScope ps(TG_MAP, rt);
  map_assign_kernel<<<(unsigned)ceil_div((int64_t)Tn * k, 256), 256, 0, rt>>>(
      c.template p<int32_t>(L.idx), c.template p<float>(L.gates), c.template p<int32_t>(L.local_rank),
      c.template p<int32_t>(L.chunk_base), c.template p<int32_t>(L.expert_off), Tn, k, E,
      c.template p<int32_t>(L.tok_row), c.template p<int32_t>(L.row_tok), c.template p<float>(L.row_gate));
  }
  CK(cudaGetLastError());

  // P_up: U = N W_up^T
  {
    GemmProblem p = blank_problem();
    p.M = Tn; p.N = d; p.K = h;
    p.A = c.template p<T>(L.n); p.lda = h;
    p.B0 = w_up; p.ldb = h;
    p.epilogue = EPI_STORE; p.C = c.template p<T>(L.u); p.ldc = d;
    CKR(run_gemm(c, p, TG_PUP));
  }
  CKR(c.order(rt, st));            // the permutation needs the maps
  // The shared expert needs u and nothing else of this pass: on the second stream it runs beside the routed experts.
  Ctx<T> cs = c;
  cs.st = c.side();
  if (Is > 0) CKR(c.order(st, cs.st));

  const bool fp8 = (D.flags & REVFFN_FLAG_FP8_EXPERTS) != 0;
  if constexpr (std::is_same<T, bf16>::value) {
    if (fp8) {
      // Routed experts on e4m3 operands: the permutation quantises the u rows as it gathers them, the first
      // product's epilogue applies the scales before the SwiGLU, g*H is quantised row by row, and the down
      // projection (tokens on the MMA N side) applies its scales before it stores.
      { ProfScope ps(TG_GATHER, st);
      CK(launch_quantize_rows(c.template p<bf16>(L.u), d, c.template p<int32_t>(L.row_tok), c.template p<int32_t>(L.rows_total),
                              L.rows_pad, d, c.template p<uint8_t>(L.upq), c.template p<float>(L.up_scale), st));
      }
      {
        GemmProblem p = blank_problem();
        p.M = (int)L.rows_pad; p.N = I; p.K = d;
        p.fp8 = 1; p.A = c.template p<uint8_t>(L.upq); p.lda = d; p.a_scale = c.template p<float>(L.up_scale);
        p.B0 = c.W.q_gate; p.B1 = c.W.q_upx; p.ldb = d; p.concat = CONCAT_N;
        p.b_scale0 = c.W.s_gate; p.b_scale1 = c.W.s_upx;
        p.group_mode = GROUP_M; p.n_groups = E; p.b_group_stride = (int64_t)I * d;
        p.group_off = c.template p<int32_t>(L.expert_off); p.tile_group = c.template p<int32_t>(L.tile_group);
        p.rows_total = c.template p<int32_t>(L.rows_total);
        p.epilogue = EPI_SWIGLU; p.C = c.template p<T>(L.hmid); p.ldc = I;
        p.rowscale = c.template p<float>(L.row_gate);
        CKR(run_gemm(c, p, TG_EXP_GATEUP));
      }
      { ProfScope ps(TG_GATHER, st);
      CK(launch_quantize_rows(c.template p<bf16>(L.hmid), I, nullptr, c.template p<int32_t>(L.rows_total), L.rows_pad, I,
                              c.template p<uint8_t>(L.hq), c.template p<float>(L.h_scale), st));
      }
      {
        GemmProblem p = blank_problem();
        p.M = (int)L.rows_pad; p.N = d; p.K = I;
        p.fp8 = 1; p.A = c.template p<uint8_t>(L.hq); p.lda = I; p.a_scale = c.template p<float>(L.h_scale);
        p.B0 = c.W.q_downx; p.ldb = I; p.b_scale0 = c.W.s_downx;
        p.group_mode = GROUP_M; p.n_groups = E; p.b_group_stride = (int64_t)d * I;
        p.group_off = c.template p<int32_t>(L.expert_off); p.tile_group = c.template p<int32_t>(L.tile_group);
        p.rows_total = c.template p<int32_t>(L.rows_total);
        p.tok_chunks = c.template p<int4>(L.tok_chunks);
        p.epilogue = EPI_STORE;
        p.C = c.template p<T>(L.o); p.ldc = d;
        CKR(run_gemm(c, p, TG_EXP_DOWN));
      }
    }
  }
  if (!fp8) {
    // Permute: Up[row] = U[token(row)]
    { ProfScope ps(TG_GATHER, st);
    gather_rows_kernel<T><<<(unsigned)L.rows_pad, 256, 0, st>>>(c.template p<T>(L.u), d, c.template p<int32_t>(L.row_tok),
                                                                c.template p<int32_t>(L.rows_total), d,
                                                                c.template p<T>(L.up));
    }
    CK(cudaGetLastError());
  
    // Routed experts: H' = g * silu(Up Wg^T) * (Up Wu^T);  O = H' Wd^T.  The row's gate weight g goes onto H in
    // the first product's epilogue: the second then needs no scaling, and the backward pass finds in H' exactly the
    // operand its down-projection weight gradient takes (dW_d = dO^T (g H)).
    {
      GemmProblem p = blank_problem();
      p.M = (int)L.rows_pad; p.N = I; p.K = d;
      p.A = c.template p<T>(L.up); p.lda = d;
      p.B0 = c.W.w_gate; p.B1 = c.W.w_upx; p.ldb = d; p.concat = CONCAT_N;
      p.group_mode = GROUP_M; p.n_groups = E; p.b_group_stride = (int64_t)I * d;
      p.group_off = c.template p<int32_t>(L.expert_off); p.tile_group = c.template p<int32_t>(L.tile_group);
      p.rows_total = c.template p<int32_t>(L.rows_total);
      p.epilogue = EPI_SWIGLU; p.C = c.template p<T>(L.hmid); p.ldc = I;
      p.rowscale = c.template p<float>(L.row_gate);
      if (save_ab) { p.C1 = c.template p<T>(L.ab); p.ldc1 = 2 * (int64_t)I; }
      CKR(run_gemm(c, p, TG_EXP_GATEUP));
    }
    {
      GemmProblem p = blank_problem();
      p.M = (int)L.rows_pad; p.N = d; p.K = I;
      p.A = c.template p<T>(L.hmid); p.lda = I;
      p.B0 = c.W.w_downx; p.ldb = I;
      p.group_mode = GROUP_M; p.n_groups = E; p.b_group_stride = (int64_t)d * I;
      p.group_off = c.template p<int32_t>(L.expert_off); p.tile_group = c.template p<int32_t>(L.tile_group);
      p.rows_total = c.template p<int32_t>(L.rows_total);
      p.tok_chunks = c.template p<int4>(L.tok_chunks);
      p.epilogue = EPI_STORE;
      p.C = c.template p<T>(L.o); p.ldc = d;
      CKR(run_gemm(c, p, TG_EXP_DOWN));
    }
  }

  // Shared expert: S = (silu(U Wsg^T) * (U Wsu^T)) Wsd^T
  if (Is > 0) {
    GemmProblem p = blank_problem();
    p.M = Tn; p.N = Is; p.K = d;
    p.A = c.template p<T>(L.u); p.lda = d;
    p.B0 = c.W.ws_gate; p.B1 = c.W.ws_up; p.ldb = d; p.concat = CONCAT_N;
    p.epilogue = EPI_SWIGLU; p.C = c.template p<T>(L.hs); p.ldc = Is;
    if (save_ab) { p.C1 = c.template p<T>(L.abs); p.ldc1 = 2 * (int64_t)Is; }
    CKR(run_gemm(cs, p, TG_SH_GATEUP));
    GemmProblem q = blank_problem();
    q.M = Tn; q.N = d; q.K = Is;
    q.A = c.template p<T>(L.hs); q.lda = Is;
    q.B0 = c.W.ws_down; q.ldb = Is;
    q.epilogue = EPI_STORE; q.C = c.template p<T>(L.s); q.ldc = d;
    CKR(run_gemm(cs, q, TG_SH_DOWN));
    CKR(c.order(cs.st, st));
  }

  // Combine: Z[t] = sum_s O[row(t,s)] + sgate_t S[t]
  if (Tn > 0) {
    { ProfScope ps(TG_COMBINE, st);
    CK(launch_combine_rows<T>(c.template p<T>(L.o), c.template p<int32_t>(L.tok_row), k,
                              Is > 0 ? c.template p<T>(L.s) : nullptr, c.template p<float>(L.sgate), d, Tn,
                              c.template p<T>(L.z), st));
    }
    CK(cudaGetLastError());
  }
  return REVFFN_OK;
}

// P_down fused with the coupling: out = resid + sign * (Z W_down^T)
template <typename T>
static int run_couple(const Ctx<T>& c, const float* resid, float sign, float* out) {
  const int d = c.D.d_model, h = d / 2;
  GemmProblem p = blank_problem();
  p.M = c.D.tokens; p.N = h; p.K = d;
  p.A = c.template p<T>(c.L.z); p.lda = d;
  p.B0 = c.W.w_down; p.ldb = d;
  p.epilogue = EPI_COUPLE; p.resid = resid; p.ld_resid = c.D.ld_stream; p.resid_sign = sign;
  p.C = out; p.ldc = c.D.ld_stream;
  return run_gemm(c, p, TG_PDOWN);
}

// A fused optimiser step as the gradient pass sees it: which matrices (REVFFN_UPD_* bits, bit i = entry i of the
// arrays), the rule, and per matrix the optional fp32 master copy and, for Adam, the two moment buffers.
struct UpdateSpec {
  uint32_t mask = 0;
  UpdRule rule = {};
  float* master[8] = {};
  float* mom[8] = {};
  float* var[8] = {};
};

static UpdateSpec spec_from_sgd(const revffn_moe_sgd& s) {
  UpdateSpec u;
  u.mask = s.mask;
  u.rule.kind = 0;
  u.rule.lr = s.lr;
  float* m[8] = {s.m_w_up, s.m_w_down, s.m_w_gate, s.m_w_upx, s.m_w_downx, s.m_ws_gate, s.m_ws_up, s.m_ws_down};
  for (int i = 0; i < 8; ++i) u.master[i] = m[i];
  return u;
}

static int spec_from_adam(const revffn_moe_adam& a, UpdateSpec* u) {
  if (a.step < 1 || !(a.beta1 >= 0.f && a.beta1 < 1.f) || !(a.beta2 >= 0.f && a.beta2 < 1.f) || !(a.eps > 0.f)) return REVFFN_ERR_SHAPE;
  u->mask = a.mask;
  u->rule.kind = 1;
  u->rule.lr = a.lr; u->rule.b1 = a.beta1; u->rule.b2 = a.beta2; u->rule.eps = a.eps; u->rule.wd = a.weight_decay;
  u->rule.inv_c1 = (float)(1.0 / (1.0 - pow((double)a.beta1, (double)a.step)));
  u->rule.inv_c2 = (float)(1.0 / (1.0 - pow((double)a.beta2, (double)a.step)));
  for (int i = 0; i < 8; ++i) {
    u->master[i] = a.master[i]; u->mom[i] = a.mom[i]; u->var[i] = a.var[i];
    if ((a.mask & (1u << i)) && (!a.mom[i] || !a.var[i])) return REVFFN_ERR_NULL;
  }
  return REVFFN_OK;
}

template <typename T>
static int run_backward(const Ctx<T>& c, const float* y1, const float* dy2, float* dy1, const revffn_moe_grads& G,
                        const UpdateSpec* sgd, const int32_t* idx_in) {
  const revffn_moe_desc& D = c.D;
  const WsLayout& L = c.L;
  const int Tn = D.tokens, d = D.d_model, h = d / 2, E = D.n_experts, k = D.top_k, I = D.d_expert, Is = D.d_shared;
  const int norm_none = D.norm_kind == REVFFN_NORM_NONE;
  const int acc = G.accumulate ? 1 : 0;
  cudaStream_t st = c.st;
  const int Rp = (int)L.rows_pad;

  if (!(D.flags & REVFFN_FLAG_REUSE_ACTIVATIONS)) CKR(run_branch(c, y1, idx_in, nullptr, true));

  // One weight gradient: `out` receives it (fp32), or, when the fused SGD step covers this weight (its bit in
  // sgd->mask), the weight W itself is updated tile by tile in the product's epilogue and no gradient is stored.
  // out2 / W2 / master2: second output of a product whose M is two stacked weights (gate | up of the experts).
  const uint32_t upd_mask = sgd ? sgd->mask : 0u;
  Ctx<T> cw = c;
  cw.st = c.side();
  auto wgrad = [&](int tag, uint32_t bit, float* out, const void* W, float* master, int M, int N, const void* A, int64_t lda,
                   int a_col0, const void* B, int64_t ldb, bool grouped, int64_t cstride, float* out2 = nullptr,
                   const void* W2 = nullptr, float* master2 = nullptr) -> int {
    const bool upd = (upd_mask & bit) != 0;
    if (!upd && !out) return REVFFN_OK;      // frozen: neither gradient nor update wanted
    int wi = 0;                              // index of this matrix in the update's arrays
    while (wi < 7 && !((bit >> wi) & 1u)) ++wi;
    // Nothing later in this pass reads a weight gradient (or an updated weight): the product goes to the second
    // stream, after everything queued so far (its operands, and every product that reads the weight it may update).
    CKR(c.order(st, cw.st));
    GemmProblem p = blank_problem();
    p.M = M; p.N = N; p.K = grouped ? Rp : Tn;   // grouped: bound on rows, the range comes from group_off
    p.a_mn_major = 1; p.b_mn_major = 1;
    p.A = A; p.lda = lda; p.a_col0 = a_col0;
    p.B0 = B; p.ldb = ldb;
    p.epilogue = EPI_WGRAD; p.accumulate = acc;
    p.ldc = N; p.c_group_stride = cstride;
    if (upd) {
      p.upd_w = const_cast<void*>(W); p.upd_m = master; p.upd = sgd->rule;
      p.upd_w2 = const_cast<void*>(W2); p.upd_m2 = master2;
      p.upd_mom = sgd->mom[wi]; p.upd_var = sgd->var[wi];
      if (W2) { p.upd_mom2 = sgd->mom[wi + 1]; p.upd_var2 = sgd->var[wi + 1]; }    // gate | up: neighbouring bits
    } else {
      p.C = out; p.C2 = out2;
    }
    if (out2 || W2) p.split_m = M / 2;
    if (grouped) {
      p.group_mode = GROUP_K; p.n_groups = E;
      p.group_off = c.template p<int32_t>(L.expert_off);
      p.group_cnt = c.template p<int32_t>(L.expert_cnt);
    }
    // A dense weight gradient with few output tiles (the adapters': 32 tiles of 256 x 256) leaves most of the GPU
    // idle while every tile walks all T tokens.  Split K over the tokens into as many slices as fill the GPU, write
    // the partial results to the workspace and add them in a second, fixed-order pass, which also does what the
    // epilogue would have done (store, accumulate or the fused update).
    int n_split = 1;
    if constexpr (std::is_same<T, bf16>::value) {
      if (c.tc && !grouped && !p.split_m) {
        const int64_t tiles = ceil_div(M, 2 * TC_BM) * ceil_div(N, 256);
        const int pairs = tc_state().n_sms / 2;
        n_split = (int)std::min<int64_t>(SPLIT_K_MAX, pairs / (tiles > 0 ? tiles : 1));
        if ((size_t)n_split * M * N * 4 > L.ksplit.bytes || Tn < 64 * 8 * n_split || (M * (int64_t)N) % 4 != 0 || M % TC_BM != 0) n_split = 1;
      }
    }
    if (n_split <= 1) return run_gemm(cw, p, tag);
    p.group_mode = GROUP_K; p.n_groups = n_split; p.group_off = nullptr;
    p.C = c.template p<float>(L.ksplit); p.C2 = nullptr; p.c_group_stride = (int64_t)M * N; p.accumulate = 0;
    p.upd_w = nullptr; p.upd_m = nullptr; p.upd_mom = nullptr; p.upd_var = nullptr;
    CKR(run_gemm(cw, p, tag));
    {
      ProfScope ps(tag, cw.st);
      const int64_t count = (int64_t)M * N;
      splitk_reduce_kernel<T><<<(unsigned)ceil_div(count, 4 * 256), 256, 0, cw.st>>>(
          c.template p<float>(L.ksplit), n_split, count, out, acc, upd ? reinterpret_cast<T*>(const_cast<void*>(W)) : nullptr,
          upd ? master : nullptr, upd ? sgd->rule : UpdRule{}, upd ? sgd->mom[wi] : nullptr, upd ? sgd->var[wi] : nullptr);
    }
    CK(cudaGetLastError());
    return REVFFN_OK;
  };
  struct Masters { float *m_w_up, *m_w_down, *m_w_gate, *m_w_upx, *m_w_downx, *m_ws_gate, *m_ws_up, *m_ws_down; };
  const Masters S = sgd ? Masters{sgd->master[0], sgd->master[1], sgd->master[2], sgd->master[3], sgd->master[4],
                                  sgd->master[5], sgd->master[6], sgd->master[7]}
                        : Masters{};

  // P_down backward: dZ = G W_down;  dW_down = G^T Z
  { ProfScope ps(TG_CAST, st);
  cast_stream_kernel<T><<<(unsigned)ceil_div((int64_t)Tn * h, 4 * 256), 256, 0, st>>>(dy2, D.ld_stream, Tn, h,
                                                                                      c.template p<T>(L.gb));
  }
  CK(cudaGetLastError());
  {
    GemmProblem p = blank_problem();
    p.M = Tn; p.N = d; p.K = h;
    p.A = c.template p<T>(L.gb); p.lda = h;
    p.B0 = c.W.w_down; p.ldb = d; p.b_mn_major = 1;
    p.epilogue = EPI_STORE; p.C = c.template p<T>(L.dz); p.ldc = d;
    CKR(run_gemm(c, p, TG_DZ));
  }
  CKR(wgrad(TG_WG_PDOWN, REVFFN_UPD_W_DOWN, G.w_down, c.W.w_down, S.m_w_down, h, d, c.template p<T>(L.gb), h, 0,
            c.template p<T>(L.z), d, false, 0));

  // Shared expert backward
  if (Is > 0) {
    { ProfScope ps(TG_SHGATE_BWD, st);
    shared_gate_bwd_kernel<T><<<Tn, 256, 0, st>>>(c.template p<T>(L.dz), c.template p<T>(L.s),
                                                  c.template p<float>(L.sgate), d, c.template p<T>(L.ds),
                                                  c.template p<float>(L.dl));
    }
    CK(cudaGetLastError());
    {
      GemmProblem p = blank_problem();   // dH_s = dS Ws_d, then SwiGLU backward in place on a|b
      p.M = Tn; p.N = Is; p.K = d;
      p.A = c.template p<T>(L.ds); p.lda = d;
      p.B0 = c.W.ws_down; p.ldb = Is; p.b_mn_major = 1;
      p.epilogue = EPI_DSWIGLU; p.ab = c.template p<T>(L.abs); p.ld_ab = 2 * (int64_t)Is;
      CKR(run_gemm(c, p, TG_SH_DH));
    }
    CKR(wgrad(TG_WG_SH_DOWN, REVFFN_UPD_WS_DOWN, G.ws_down, c.W.ws_down, S.m_ws_down, d, Is, c.template p<T>(L.ds), d, 0,
              c.template p<T>(L.hs), Is, false, 0));
    {
      GemmProblem p = blank_problem();   // dU_sh = da Ws_g + db Ws_u
      p.M = Tn; p.N = d; p.K = 2 * Is;
      p.A = c.template p<T>(L.abs); p.lda = 2 * (int64_t)Is;
      p.B0 = c.W.ws_gate; p.B1 = c.W.ws_up; p.ldb = d; p.b_mn_major = 1; p.concat = CONCAT_K;
      p.epilogue = EPI_STORE; p.C = c.template p<T>(L.dush); p.ldc = d;
      CKR(run_gemm(c, p, TG_SH_DU));
    }
    {
      // as for the routed experts below: da|db is one buffer and both gradients read u, so when both are wanted in
      // the same form they are one product with M = 2 I_s and two outputs (352 instead of 2 x 176 output tiles of
      // 256 x 256 at the benchmark shape: 4.8 instead of 2 x 2.4 waves of 74 CTA pairs)
      const bool ug = (upd_mask & REVFFN_UPD_WS_GATE) != 0, uu = (upd_mask & REVFFN_UPD_WS_UP) != 0;
      if ((ug && uu) || (!ug && !uu && G.ws_gate && G.ws_up)) {
        CKR(wgrad(TG_WG_SH_GATEUP, REVFFN_UPD_WS_GATE, G.ws_gate, c.W.ws_gate, S.m_ws_gate, 2 * Is, d, c.template p<T>(L.abs),
                  2 * (int64_t)Is, 0, c.template p<T>(L.u), d, false, 0, G.ws_up, c.W.ws_up, S.m_ws_up));
      } else {
        CKR(wgrad(TG_WG_SH_GATE, REVFFN_UPD_WS_GATE, G.ws_gate, c.W.ws_gate, S.m_ws_gate, Is, d, c.template p<T>(L.abs),
                  2 * (int64_t)Is, 0, c.template p<T>(L.u), d, false, 0));
        CKR(wgrad(TG_WG_SH_UP, REVFFN_UPD_WS_UP, G.ws_up, c.W.ws_up, S.m_ws_up, Is, d, c.template p<T>(L.abs), 2 * (int64_t)Is, Is,
                  c.template p<T>(L.u), d, false, 0));
      }
    }
    if (G.ws_sgate) {
      // a leaf like the matrix gradients: second stream (which also owns the column-sum scratch `part`: every
      // user of it, this one, the router bias and the norm scale, is queued there, in order)
      CKR(c.order(st, cw.st));
      { ProfScope ps(TG_WG_SGATE, cw.st);
      CK(launch_colsum_partial<T>(c.template p<T>(L.u), d, c.template p<float>(L.dl), Tn, d, STRIP, L.strips,
                                  c.template p<float>(L.part), cw.st));
      }
      { ProfScope ps(TG_WG_SGATE, cw.st);
      colsum_final_kernel<<<(unsigned)ceil_div(d, COLSUM_FINAL_COLS), 256, 0, cw.st>>>(c.template p<float>(L.part), L.strips, d, acc,
                                                                      G.ws_sgate);
      }
      CK(cudaGetLastError());
    }
  }

  // Routed experts backward
  { ProfScope ps(TG_GATHER_DZ, st);
  gather_rows_kernel<T><<<(unsigned)Rp, 256, 0, st>>>(c.template p<T>(L.dz), d, c.template p<int32_t>(L.row_tok),
                                                      c.template p<int32_t>(L.rows_total), d, c.template p<T>(L.dop));
  }
  CK(cudaGetLastError());
  const int n_part = dg_parts(c, I);
  {
    GemmProblem p = blank_problem();   // dH' = dO Wd; SwiGLU backward in place on a|b; dg partials
    p.M = Rp; p.N = I; p.K = d;
    p.A = c.template p<T>(L.dop); p.lda = d;
    p.B0 = c.W.w_downx; p.ldb = I; p.b_mn_major = 1;
    p.group_mode = GROUP_M; p.n_groups = E; p.b_group_stride = (int64_t)d * I;
    p.group_off = c.template p<int32_t>(L.expert_off); p.tile_group = c.template p<int32_t>(L.tile_group);
    p.rows_total = c.template p<int32_t>(L.rows_total);
    p.epilogue = EPI_DSWIGLU; p.ab = c.template p<T>(L.ab); p.ld_ab = 2 * (int64_t)I;
    p.rowscale = c.template p<float>(L.row_gate);
    p.dg_part = c.template p<float>(L.dg_part); p.dg_ld = L.dg_ld;
    CKR(run_gemm(c, p, TG_EXP_DH));
  }
  {
    GemmProblem p = blank_problem();   // dUp = da Wg + db Wu
    p.M = Rp; p.N = d; p.K = 2 * I;
    p.A = c.template p<T>(L.ab); p.lda = 2 * (int64_t)I;
    p.B0 = c.W.w_gate; p.B1 = c.W.w_upx; p.ldb = d; p.b_mn_major = 1; p.concat = CONCAT_K;
    p.group_mode = GROUP_M; p.n_groups = E; p.b_group_stride = (int64_t)I * d;
    p.group_off = c.template p<int32_t>(L.expert_off); p.tile_group = c.template p<int32_t>(L.tile_group);
    p.rows_total = c.template p<int32_t>(L.rows_total);
    p.tok_chunks = c.template p<int4>(L.tok_chunks);
    p.epilogue = EPI_STORE; p.C = c.template p<T>(L.dup); p.ldc = d;
    CKR(run_gemm(c, p, TG_EXP_DU));
  }
  CKR(wgrad(TG_WG_EXP_DOWN, REVFFN_UPD_W_DOWNX, G.w_downx, c.W.w_downx, S.m_w_downx, d, I, c.template p<T>(L.dop), d, 0,
            c.template p<T>(L.hmid), I, true, (int64_t)d * I));
  {
    // dW_gate and dW_up share their B operand (the permuted u rows) and their A operand is one buffer da|db:
    // when both are wanted in the same form they are one product with M = 2I and two outputs.
    const bool ug = (upd_mask & REVFFN_UPD_W_GATE) != 0, uu = (upd_mask & REVFFN_UPD_W_UPX) != 0;
    if ((ug && uu) || (!ug && !uu && G.w_gate && G.w_upx)) {
      CKR(wgrad(TG_WG_EXP_GATEUP, REVFFN_UPD_W_GATE, G.w_gate, c.W.w_gate, S.m_w_gate, 2 * I, d, c.template p<T>(L.ab),
                2 * (int64_t)I, 0, c.template p<T>(L.up), d, true, (int64_t)I * d, G.w_upx, c.W.w_upx, S.m_w_upx));
    } else {
      CKR(wgrad(TG_WG_EXP_GATE, REVFFN_UPD_W_GATE, G.w_gate, c.W.w_gate, S.m_w_gate, I, d, c.template p<T>(L.ab), 2 * (int64_t)I, 0,
                c.template p<T>(L.up), d, true, (int64_t)I * d));
      CKR(wgrad(TG_WG_EXP_UP, REVFFN_UPD_W_UPX, G.w_upx, c.W.w_upx, S.m_w_upx, I, d, c.template p<T>(L.ab), 2 * (int64_t)I, I,
                c.template p<T>(L.up), d, true, (int64_t)I * d));
    }
  }

  // Gate / router backward
  const bool dense_gate = (D.flags & REVFFN_FLAG_GATE_SOFTMAX_ALL) != 0;
  if (!dense_gate) {
    { ProfScope ps(TG_ROUTER_BWD, st);
    router_bwd_kernel<<<(unsigned)ceil_div(Tn, 128), 128, 0, st>>>(
        c.template p<float>(L.dg_part), L.dg_ld, n_part, c.template p<float>(L.gates), c.template p<int32_t>(L.tok_row),
        Tn, k, c.template p<float>(L.tok_dl), c.template p<float>(L.row_dl));
    }
    CK(cudaGetLastError());
    if (G.w_router || G.b_router) {
      dim3 grid((unsigned)ceil_div(d, 256), (unsigned)E);
      CKR(c.order(st, cw.st));
      { ProfScope ps(TG_WG_ROUTER, cw.st);
      router_wgrad_kernel<T><<<grid, 256, 0, cw.st>>>(c.template p<T>(L.up), c.template p<float>(L.row_dl),
                                                   c.template p<int32_t>(L.expert_off), c.template p<int32_t>(L.expert_cnt),
                                                   d, acc, G.w_router, G.b_router);
      }
      CK(cudaGetLastError());
    }
  } else {
    // every logit carries a gradient: dL is a dense [T, E] matrix and its products are matrix products
    { ProfScope ps(TG_ROUTER_BWD, st);
    router_bwd_dense_kernel<T><<<(unsigned)ceil_div(Tn, 128), 128, 0, st>>>(
        c.template p<float>(L.dg_part), L.dg_ld, n_part, c.template p<float>(L.prob), c.template p<int32_t>(L.idx),
        c.template p<int32_t>(L.tok_row), Tn, k, E, L.ld_dlf, c.template p<T>(L.dlf));
    }
    CK(cudaGetLastError());
    {
      GemmProblem p = blank_problem();   // dU_r = dL W_r
      p.M = Tn; p.N = d; p.K = E;
      p.A = c.template p<T>(L.dlf); p.lda = L.ld_dlf;
      p.B0 = c.W.w_router; p.ldb = d; p.b_mn_major = 1;
      p.epilogue = EPI_STORE; p.C = c.template p<T>(L.dur); p.ldc = d;
      CKR(run_gemm(c, p, TG_ROUTER_BWD));
    }
    if (G.w_router)
      CKR(wgrad(TG_WG_ROUTER, 0u, G.w_router, nullptr, nullptr, E, d, c.template p<T>(L.dlf), L.ld_dlf, 0, c.template p<T>(L.u), d,
                false, 0));
    if (G.b_router) {
      CKR(c.order(st, cw.st));
      { ProfScope ps(TG_WG_ROUTER, cw.st);
      CK(launch_colsum_partial<T>(c.template p<T>(L.dlf), L.ld_dlf, nullptr, Tn, E, STRIP, L.strips,
                                  c.template p<float>(L.part), cw.st));
      }
      { ProfScope ps(TG_WG_ROUTER, cw.st);
      colsum_final_kernel<<<(unsigned)ceil_div(E, COLSUM_FINAL_COLS), 256, 0, cw.st>>>(c.template p<float>(L.part), L.strips, E, acc,
                                                                      G.b_router);
      }
      CK(cudaGetLastError());
    }
  }

  // dU, then P_up backward and the norm
  { ProfScope ps(TG_DU_REDUCE, st);
  CK(launch_du_reduce<T>(c.template p<T>(L.dup), c.template p<int32_t>(L.tok_row), c.template p<int32_t>(L.idx),
                         c.template p<float>(L.tok_dl), k, Is > 0 ? c.template p<T>(L.dush) : nullptr,
                         reinterpret_cast<const T*>(c.W.w_router), E, c.template p<float>(L.dl),
                         reinterpret_cast<const T*>(c.W.ws_sgate), dense_gate ? c.template p<T>(L.dur) : nullptr, d,
                         Tn, c.template p<T>(L.du), st));
  }
  CK(cudaGetLastError());
  {
    GemmProblem p = blank_problem();   // dN = dU W_up  (fp32 out)
    p.M = Tn; p.N = h; p.K = d;
    p.A = c.template p<T>(L.du); p.lda = d;
    p.B0 = c.W.w_up; p.ldb = h; p.b_mn_major = 1;
    p.epilogue = EPI_STORE; p.out_f32 = 1; p.C = c.template p<float>(L.dn); p.ldc = h;
    CKR(run_gemm(c, p, TG_DN));
  }
  CKR(wgrad(TG_WG_PUP, REVFFN_UPD_W_UP, G.w_up, c.W.w_up, S.m_w_up, d, h, c.template p<T>(L.du), d, 0, c.template p<T>(L.n), h,
            false, 0));
  { ProfScope ps(TG_NORM_BWD, st);
  rmsnorm_bwd_rows_kernel<<<(unsigned)ceil_div((int64_t)Tn * 32, 128), 128, 0, st>>>(
      c.template p<float>(L.dn), y1, D.ld_stream, c.W.norm_gamma, c.template p<float>(L.r), norm_none, Tn, h, dy1,
      D.ld_stream);
  }
  CK(cudaGetLastError());
  if (G.norm_gamma) {
    if (norm_none) {
      if (!acc) CK(cudaMemsetAsync(G.norm_gamma, 0, (size_t)h * 4, st));
    } else {
      CKR(c.order(st, cw.st));
      { ProfScope ps(TG_DGAMMA, cw.st);
      CK(launch_dgamma_partial(c.template p<float>(L.dn), y1, D.ld_stream, c.template p<float>(L.r), Tn, h, STRIP, L.strips,
                               c.template p<float>(L.part), cw.st));
      }
      { ProfScope ps(TG_DGAMMA, cw.st);
      colsum_final_kernel<<<(unsigned)ceil_div(h, COLSUM_FINAL_COLS), 256, 0, cw.st>>>(c.template p<float>(L.part), L.strips, h, acc,
                                                                      G.norm_gamma);
      }
      CK(cudaGetLastError());
    }
  }
  CKR(c.order(cw.st, st));      // the caller's stream ends after the weight gradients too
  return REVFFN_OK;
}

// ---------------------------------------------------------------------------
// Entry-point plumbing
// ---------------------------------------------------------------------------
enum Pass { PASS_FWD, PASS_INV, PASS_BWD };

template <typename T>
static int dispatch(Pass pass, const revffn_moe_desc& D, const revffn_moe_weights& W, const WsLayout& L, void* ws,
                    cudaStream_t st, const float* y1, const float* in2, float* out, const revffn_moe_grads* G,
                    const UpdateSpec* sgd, const int32_t* idx_in, int32_t* idx_out) {
  Ctx<T> c;
  c.D = D; c.W = W; c.L = L; c.ws = reinterpret_cast<char*>(ws); c.st = st;
  g_prof.pass = (int)pass;
  c.tc = std::is_same<T, bf16>::value && !(D.flags & REVFFN_FLAG_FORCE_SIMT);
  // second stream: every call on the tcgen05 back end (at 512 tokens, where the launches are short, the step still
  // gains 13 %), never while the per-launch profiler is on (its events bracket launches on one stream)
  if (c.tc && !g_prof.on && !(D.flags & REVFFN_FLAG_SINGLE_STREAM)) {
    c.ov = overlap_state();
    if (!c.ov) return REVFFN_ERR_CUDA;
  }
  if (c.tc) CKR(tc_prepare());
  if (!(D.flags & REVFFN_FLAG_KEEP_STATUS)) CK(cudaMemsetAsync(c.ws + L.status.off, 0, L.status.bytes, st));
  if (D.tokens == 0) return REVFFN_OK;   // empty batch: nothing to compute, gradients untouched
  const bool big_ws = pass == PASS_BWD || (D.flags & REVFFN_FLAG_SAVE_ACTIVATIONS);
  const size_t ws_limit = big_ws ? L.bwd_bytes : L.fwd_bytes;
  if (L.n_guards) CKR(guards_fill(L, ws_limit, c.ws, st));
  if (pass == PASS_BWD) {
    CKR(run_backward(c, y1, in2, out, *G, sgd, idx_in));
  } else {
    CKR(run_branch(c, y1, idx_in, idx_out, (D.flags & REVFFN_FLAG_SAVE_ACTIVATIONS) != 0));
    CKR(run_couple(c, in2, pass == PASS_FWD ? 1.f : -1.f, out));
  }
  if (L.n_guards) CKR(guards_check(L, ws_limit, c.ws, st));
  return REVFFN_OK;
}

static int entry(Pass pass, const revffn_moe_desc* desc, const revffn_moe_weights* w, const float* y1,
                 const float* in2, float* out, const revffn_moe_grads* grads, const int32_t* idx_in,
                 int32_t* idx_out, void* ws, size_t ws_bytes, void* cuda_stream, const UpdateSpec* sgd = nullptr) {
  CKR(validate_desc(desc));
  CKR(validate_weights(*desc, w));
  if (!ws) return REVFFN_ERR_NULL;
  if (pass == PASS_BWD && !grads) return REVFFN_ERR_NULL;
  if (pass == PASS_BWD && (desc->flags & REVFFN_FLAG_FP8_EXPERTS)) return REVFFN_ERR_UNSUPPORTED;      // gradients are taken on the bf16 path
  if (desc->tokens > 0 && (!y1 || !in2 || !out)) return REVFFN_ERR_NULL;
  if (!aligned16(y1) || !aligned16(in2) || !aligned16(out) || (reinterpret_cast<uintptr_t>(ws) & 255u))
    return REVFFN_ERR_ALIGN;
  if ((reinterpret_cast<uintptr_t>(idx_in) | reinterpret_cast<uintptr_t>(idx_out)) &
      ((desc->flags & REVFFN_FLAG_ROUTING_RECORD) ? 15u : 3u))
    return REVFFN_ERR_ALIGN;
  if (sgd) {
    if (sgd->mask & ~REVFFN_UPD_ALL) return REVFFN_ERR_SHAPE;
    if (desc->d_shared == 0 && (sgd->mask & (REVFFN_UPD_WS_GATE | REVFFN_UPD_WS_UP | REVFFN_UPD_WS_DOWN))) return REVFFN_ERR_NULL;
    for (int i = 0; i < 8; ++i)
      if (!aligned16(sgd->master[i]) || !aligned16(sgd->mom[i]) || !aligned16(sgd->var[i])) return REVFFN_ERR_ALIGN;
    // a weight is either updated in place or has its gradient written, not both
    const float* gs8[] = {grads->w_up, grads->w_down, grads->w_gate, grads->w_upx, grads->w_downx, grads->ws_gate,
                          grads->ws_up, grads->ws_down};
    for (int i = 0; i < 8; ++i)
      if ((sgd->mask & (1u << i)) && gs8[i]) return REVFFN_ERR_UNSUPPORTED;
  }
  if (grads) {
    const float* gs[] = {grads->norm_gamma, grads->w_up, grads->w_down, grads->w_router, grads->b_router,
                         grads->w_gate, grads->w_upx, grads->w_downx, grads->ws_gate, grads->ws_up,
                         grads->ws_down, grads->ws_sgate};
    for (const float* g : gs)
      if (g && !aligned16(g)) return REVFFN_ERR_ALIGN;
  }
  WsLayout L = plan_workspace(*desc);
  const bool big_ws = pass == PASS_BWD || (desc->flags & REVFFN_FLAG_SAVE_ACTIVATIONS);
  if (ws_bytes < (big_ws ? L.bwd_bytes : L.fwd_bytes)) return REVFFN_ERR_WORKSPACE;
  CKR(check_device());
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (desc->weight_dtype == REVFFN_BF16)
    return dispatch<bf16>(pass, *desc, *w, L, ws, st, y1, in2, out, grads, sgd, idx_in, idx_out);
  return dispatch<float>(pass, *desc, *w, L, ws, st, y1, in2, out, grads, sgd, idx_in, idx_out);
}

// ---------------------------------------------------------------------------
// Routing without any allocation.  The folded router matrix, which the regular
// entry points keep in the caller's workspace, lives in a fixed array inside
// the library's own device image instead.
// ---------------------------------------------------------------------------
static __device__ __align__(256) double g_route_scratch[REVFFN_ROUTE_NOALLOC_MAX_ELEMS];

// Device address of g_route_scratch, looked up once per device.  In host code the
// symbol itself is only a handle, not something a kernel may dereference.
static double* route_scratch_ptr(int* err) {
  static double* ptr[64] = {nullptr};
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { *err = REVFFN_ERR_CUDA; return nullptr; }
  if (!ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_route_scratch) != cudaSuccess || !p) { *err = REVFFN_ERR_CUDA; return nullptr; }
    ptr[dev] = reinterpret_cast<double*>(p);
  }
  *err = REVFFN_OK;
  return ptr[dev];
}

template <typename T>
static int route_noalloc_launch(const revffn_moe_desc& D, const revffn_moe_weights& W, const float* y1,
                                double* w_rc, int32_t* idx, float* gates, float* sgate, cudaStream_t st) {
  const int d = D.d_model, h = d / 2, E = D.n_experts;
  const int norm_none = D.norm_kind == REVFFN_NORM_NONE;
  CK(launch_fold_router<T>(reinterpret_cast<const T*>(W.w_router), reinterpret_cast<const T*>(W.ws_sgate),
                           reinterpret_cast<const T*>(W.w_up), E, d, h, w_rc, st));
  CK(launch_router_topk(y1, D.ld_stream, W.norm_gamma, D.norm_eps, norm_none, w_rc, W.b_router, D.tokens, h, E,
                        D.top_k, D.d_shared > 0 ? 1 : 0, nullptr, idx, gates, sgate, nullptr, nullptr, nullptr, 0, st));
  g_prof.launches += 2;
  return REVFFN_OK;
}

}  // namespace revffn

using namespace revffn;

extern "C" {

int revffn_moe_workspace_size(const revffn_moe_desc* desc, size_t* fwd_bytes, size_t* bwd_bytes) {
  int r = validate_desc(desc);
  if (r != REVFFN_OK) return r;
  WsLayout L = plan_workspace(*desc);
  if (fwd_bytes) *fwd_bytes = L.fwd_bytes;
  if (bwd_bytes) *bwd_bytes = L.bwd_bytes;
  return REVFFN_OK;
}

int revffn_moe_forward(const revffn_moe_desc* desc, const revffn_moe_weights* w, const float* y1, const float* x2,
                       float* y2, int32_t* topk_idx_out, void* ws, size_t ws_bytes, void* cuda_stream) {
  return entry(PASS_FWD, desc, w, y1, x2, y2, nullptr, nullptr, topk_idx_out, ws, ws_bytes, cuda_stream);
}

int revffn_moe_inverse(const revffn_moe_desc* desc, const revffn_moe_weights* w, const float* y1, const float* y2,
                       float* x2, const int32_t* topk_idx_in, void* ws, size_t ws_bytes, void* cuda_stream) {
  return entry(PASS_INV, desc, w, y1, y2, x2, nullptr, topk_idx_in, nullptr, ws, ws_bytes, cuda_stream);
}

int revffn_moe_backward(const revffn_moe_desc* desc, const revffn_moe_weights* w, const float* y1, const float* dy2,
                        float* dy1_inout, const revffn_moe_grads* grads, const int32_t* topk_idx_in, void* ws,
                        size_t ws_bytes, void* cuda_stream) {
  return entry(PASS_BWD, desc, w, y1, dy2, dy1_inout, grads, topk_idx_in, nullptr, ws, ws_bytes, cuda_stream);
}

int revffn_moe_backward_sgd(const revffn_moe_desc* desc, const revffn_moe_weights* w, const float* y1, const float* dy2,
                            float* dy1_inout, const revffn_moe_grads* grads, const revffn_moe_sgd* sgd,
                            const int32_t* topk_idx_in, void* ws, size_t ws_bytes, void* cuda_stream) {
  if (!sgd) return REVFFN_ERR_NULL;
  const UpdateSpec u = spec_from_sgd(*sgd);
  return entry(PASS_BWD, desc, w, y1, dy2, dy1_inout, grads, topk_idx_in, nullptr, ws, ws_bytes, cuda_stream, &u);
}

int revffn_moe_backward_adam(const revffn_moe_desc* desc, const revffn_moe_weights* w, const float* y1, const float* dy2,
                             float* dy1_inout, const revffn_moe_grads* grads, const revffn_moe_adam* adam,
                             const int32_t* topk_idx_in, void* ws, size_t ws_bytes, void* cuda_stream) {
  if (!adam) return REVFFN_ERR_NULL;
  UpdateSpec u;
  CKR(spec_from_adam(*adam, &u));
  return entry(PASS_BWD, desc, w, y1, dy2, dy1_inout, grads, topk_idx_in, nullptr, ws, ws_bytes, cuda_stream, &u);
}

int revffn_moe_quantize_experts(const revffn_moe_desc* desc, const revffn_moe_weights* w, void* cuda_stream) {
  int r = validate_desc(desc);
  if (r != REVFFN_OK) return r;
  if (!w || !w->w_gate || !w->w_upx || !w->w_downx || !w->q_gate || !w->q_upx || !w->q_downx || !w->s_gate || !w->s_upx || !w->s_downx)
    return REVFFN_ERR_NULL;
  if (desc->weight_dtype != REVFFN_BF16 || desc->d_model > 2048 || desc->d_expert > 2048) return REVFFN_ERR_UNSUPPORTED;
  const void* ps[] = {w->w_gate, w->w_upx, w->w_downx, w->q_gate, w->q_upx, w->q_downx, w->s_gate, w->s_upx, w->s_downx};
  for (const void* p : ps)
    if (!aligned16(p)) return REVFFN_ERR_ALIGN;
  r = check_device();
  if (r != REVFFN_OK) return r;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  const int64_t E = desc->n_experts, I = desc->d_expert, d = desc->d_model;
  auto q = [&](const void* in, int64_t rows, int width, const void* out, const float* scale) {
    return launch_quantize_rows(reinterpret_cast<const bf16*>(in), width, nullptr, nullptr, rows, width,
                                reinterpret_cast<uint8_t*>(const_cast<void*>(out)), const_cast<float*>(scale), st);
  };
  CK(q(w->w_gate, E * I, (int)d, w->q_gate, w->s_gate));
  CK(q(w->w_upx, E * I, (int)d, w->q_upx, w->s_upx));
  CK(q(w->w_downx, E * d, (int)I, w->q_downx, w->s_downx));
  g_prof.launches += 3;
  return REVFFN_OK;
}

int revffn_moe_status(const void* ws, void* cuda_stream, int32_t* device_status) {
  if (!ws || !device_status) return REVFFN_ERR_NULL;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(device_status, ws, sizeof(int32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return REVFFN_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return REVFFN_ERR_CUDA;
  return REVFFN_OK;
}

const char* revffn_strerror(int code) {
  switch (code) {
    case REVFFN_OK: return "ok";
    case REVFFN_ERR_NULL: return "a required pointer is NULL";
    case REVFFN_ERR_SHAPE: return "descriptor violates a shape constraint";
    case REVFFN_ERR_ALIGN: return "pointer or stride not 16-byte aligned";
    case REVFFN_ERR_WORKSPACE: return "workspace too small";
    case REVFFN_ERR_ARCH: return "device is not compute capability 10.x (sm_100a)";
    case REVFFN_ERR_CUDA: return "CUDA call failed";
    case REVFFN_ERR_DEVICE_WAIT: return "a bounded device-side wait expired";
    case REVFFN_ERR_UNSUPPORTED: return "not supported";
    case REVFFN_ERR_NOALLOC_LIMIT: return "problem exceeds the fixed scratch of the no-allocation entry point";
    case REVFFN_ERR_INDEX: return "an expert index supplied by the caller is out of range";
    case REVFFN_ERR_CANARY: return "a guard zone between workspace buffers was overwritten";
    case REVFFN_ERR_NONFINITE: return "a router logit is not finite";
    default: return "unknown error";
  }
}

int revffn_moe_ws_lookup(const revffn_moe_desc* desc, const char* name, size_t* offset, size_t* bytes) {
  int r = validate_desc(desc);
  if (r != REVFFN_OK) return r;
  if (!name) return REVFFN_ERR_NULL;
  WsLayout L = plan_workspace(*desc);
  struct { const char* n; const Buf* b; } tab[] = {
      {"status", &L.status}, {"rows_total", &L.rows_total}, {"w_rc", &L.w_rc}, {"n", &L.n}, {"r", &L.r},
      {"idx", &L.idx}, {"gates", &L.gates}, {"sgate", &L.sgate}, {"expert_cnt", &L.expert_cnt},
      {"expert_off", &L.expert_off}, {"tile_group", &L.tile_group}, {"tok_row", &L.tok_row},
      {"row_tok", &L.row_tok}, {"row_gate", &L.row_gate}, {"u", &L.u}, {"up", &L.up}, {"hmid", &L.hmid},
      {"o", &L.o}, {"hs", &L.hs}, {"s", &L.s}, {"z", &L.z}, {"ab", &L.ab}, {"abs", &L.abs}, {"gb", &L.gb},
      {"dz", &L.dz}, {"ds", &L.ds}, {"dl", &L.dl}, {"dop", &L.dop}, {"dg_part", &L.dg_part},
      {"tok_dl", &L.tok_dl}, {"row_dl", &L.row_dl}, {"prob", &L.prob}, {"dlf", &L.dlf}, {"dup", &L.dup}, {"dush", &L.dush}, {"du", &L.du},
      {"dn", &L.dn}};
  for (auto& t : tab)
    if (strcmp(t.n, name) == 0) {
      if (offset) *offset = t.b->off;
      if (bytes) *bytes = t.b->bytes;
      return REVFFN_OK;
    }
  if (strncmp(name, "guard", 5) == 0 && name[5] >= '0' && name[5] <= '9') {
    const int i = atoi(name + 5);
    if (i < L.n_guards) {
      if (offset) *offset = L.guard_off[i];
      if (bytes) *bytes = GUARD_BYTES;
      return REVFFN_OK;
    }
  }
  return REVFFN_ERR_UNSUPPORTED;
}

// Events that order the copy streams against the compute stream in revffn_moe_step_host, the upload stream
// of the pipelined form and its call counter (created on first use, per device; no timing).
struct StepState {
  cudaEvent_t ev[10];            // 0..6 plain form; pipelined form: 0 inputs A, 1 inputs B, 2..4 passes done, 8/9 set free
  cudaStream_t upload = nullptr; // pipelined form: host -> device copies
  unsigned calls = 0;            // pipelined form: parity selects the staging set
  bool made = false;
};

static StepState* step_state(int* err) {
  static StepState state[64];
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { *err = REVFFN_ERR_CUDA; return nullptr; }
  StepState& s = state[dev];
  if (!s.made) {
    for (int i = 0; i < 10; ++i)
      if (cudaEventCreateWithFlags(&s.ev[i], cudaEventDisableTiming) != cudaSuccess) { *err = REVFFN_ERR_CUDA; return nullptr; }
    if (cudaStreamCreateWithFlags(&s.upload, cudaStreamNonBlocking) != cudaSuccess) { *err = REVFFN_ERR_CUDA; return nullptr; }
    s.made = true;
  }
  *err = REVFFN_OK;
  return &s;
}

// The pipelined form of revffn_moe_step_host (REVFFN_FLAG_STEP_PIPELINED): two sets of staging slots used in
// turn, uploads on a stream of the library's own, downloads on the caller's copy stream, and no join of the
// copy stream into the compute stream, so that the uploads of one call run beside the passes of the call before
// it and its downloads beside the passes of the call after it.
static int step_host_pipelined(const revffn_moe_desc* desc, const revffn_moe_weights* w, const revffn_moe_grads* grads,
                               const float* y1_host, const float* x2_host, const float* dy2_host, float* y2_host,
                               float* x2_rec_host, float* dy1_host, char* staging, size_t slot, size_t n, void* ws,
                               size_t ws_bytes, cudaStream_t st, cudaStream_t cs) {
  int r = REVFFN_OK;
  StepState* S = step_state(&r);
  if (r != REVFFN_OK) return r;
  const unsigned set = S->calls++ & 1u;
  cudaStream_t up = S->upload;
  cudaEvent_t ev_free = S->ev[8 + set];
  char* sp = staging + (size_t)set * 6 * slot;
  float* y1 = reinterpret_cast<float*>(sp);
  float* x2 = reinterpret_cast<float*>(sp + slot);
  float* dy2 = reinterpret_cast<float*>(sp + 2 * slot);
  float* y2 = reinterpret_cast<float*>(sp + 3 * slot);
  float* x2r = reinterpret_cast<float*>(sp + 4 * slot);
  float* dy1 = reinterpret_cast<float*>(sp + 5 * slot);
  revffn_moe_desc d_fwd = *desc, d_inv = *desc, d_bwd = *desc;
  d_fwd.flags &= ~REVFFN_FLAG_STEP_PIPELINED;
  d_inv.flags = d_fwd.flags | REVFFN_FLAG_SAVE_ACTIVATIONS | REVFFN_FLAG_KEEP_STATUS | REVFFN_FLAG_ROUTER_FOLDED;
  d_bwd.flags = d_fwd.flags | REVFFN_FLAG_REUSE_ACTIVATIONS | REVFFN_FLAG_KEEP_STATUS;
  // this set's slots are free once the call before the previous one has sent its last result to the host
  CK(cudaStreamWaitEvent(up, ev_free, 0));
  CK(cudaStreamWaitEvent(st, ev_free, 0));
  if (n > 0) {
    CK(cudaMemcpyAsync(y1, y1_host, n, cudaMemcpyHostToDevice, up));
    CK(cudaMemcpyAsync(x2, x2_host, n, cudaMemcpyHostToDevice, up));
  }
  CK(cudaEventRecord(S->ev[0], up));
  if (n > 0) {
    CK(cudaMemcpyAsync(dy2, dy2_host, n, cudaMemcpyHostToDevice, up));
    CK(cudaMemsetAsync(dy1, 0, n, st));
  }
  CK(cudaEventRecord(S->ev[1], up));
  CK(cudaStreamWaitEvent(st, S->ev[0], 0));
  CKR(revffn_moe_forward(&d_fwd, w, y1, x2, y2, nullptr, ws, ws_bytes, st));
  CK(cudaEventRecord(S->ev[2], st));
  CK(cudaStreamWaitEvent(cs, S->ev[2], 0));
  if (n > 0) CK(cudaMemcpyAsync(y2_host, y2, n, cudaMemcpyDeviceToHost, cs));
  CKR(revffn_moe_inverse(&d_inv, w, y1, y2, x2r, nullptr, ws, ws_bytes, st));
  CK(cudaEventRecord(S->ev[3], st));
  CK(cudaStreamWaitEvent(cs, S->ev[3], 0));
  if (n > 0) CK(cudaMemcpyAsync(x2_rec_host, x2r, n, cudaMemcpyDeviceToHost, cs));
  CK(cudaStreamWaitEvent(st, S->ev[1], 0));
  CKR(revffn_moe_backward(&d_bwd, w, y1, dy2, dy1, grads, nullptr, ws, ws_bytes, st));
  CK(cudaEventRecord(S->ev[4], st));
  CK(cudaStreamWaitEvent(cs, S->ev[4], 0));
  if (n > 0) CK(cudaMemcpyAsync(dy1_host, dy1, n, cudaMemcpyDeviceToHost, cs));
  CK(cudaEventRecord(ev_free, cs));
  return REVFFN_OK;
}

int revffn_moe_step_host(const revffn_moe_desc* desc, const revffn_moe_weights* w, const revffn_moe_grads* grads,
                         const float* y1_host, const float* x2_host, const float* dy2_host, float* y2_host,
                         float* x2_rec_host, float* dy1_host, void* staging, size_t staging_bytes, void* ws,
                         size_t ws_bytes, void* cuda_stream, void* copy_stream) {
  int r = validate_desc(desc);
  if (r != REVFFN_OK) return r;
  if (!y1_host || !x2_host || !dy2_host || !y2_host || !x2_rec_host || !dy1_host || !staging) return REVFFN_ERR_NULL;
  const int h = desc->d_model / 2;
  if (desc->ld_stream != h) return REVFFN_ERR_SHAPE;
  const size_t n = (size_t)desc->tokens * h * sizeof(float);
  const size_t slot = (size_t)round_up((int64_t)(n > 0 ? n : 1), 256);
  const bool pipelined = (desc->flags & REVFFN_FLAG_STEP_PIPELINED) != 0;
  if (staging_bytes < (pipelined ? 12 : 6) * slot || (reinterpret_cast<uintptr_t>(staging) & 255u)) return REVFFN_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  cudaStream_t cs = reinterpret_cast<cudaStream_t>(copy_stream);
  const bool two = copy_stream != nullptr && cs != st;
  if (pipelined) {
    if (!two) return REVFFN_ERR_UNSUPPORTED;      // the downloads need a stream of their own
    return step_host_pipelined(desc, w, grads, y1_host, x2_host, dy2_host, y2_host, x2_rec_host, dy1_host,
                               reinterpret_cast<char*>(staging), slot, n, ws, ws_bytes, st, cs);
  }
  if (!two) cs = st;
  cudaEvent_t* ev = nullptr;
  if (two) {
    StepState* S = step_state(&r);
    if (r != REVFFN_OK) return r;
    ev = S->ev;
  }
  char* sp = reinterpret_cast<char*>(staging);
  float* y1 = reinterpret_cast<float*>(sp);
  float* x2 = reinterpret_cast<float*>(sp + slot);
  float* dy2 = reinterpret_cast<float*>(sp + 2 * slot);
  float* y2 = reinterpret_cast<float*>(sp + 3 * slot);
  float* x2r = reinterpret_cast<float*>(sp + 4 * slot);
  float* dy1 = reinterpret_cast<float*>(sp + 5 * slot);
  // the inverse and the gradient pass share one evaluation of the branch
  // the status word is cleared once (by the first forward call); every later pass keeps it, so that
  // revffn_moe_status reports the first device-side error of the whole step
  revffn_moe_desc d_inv = *desc, d_bwd = *desc;
  d_inv.flags |= REVFFN_FLAG_SAVE_ACTIVATIONS | REVFFN_FLAG_KEEP_STATUS | REVFFN_FLAG_ROUTER_FOLDED;
  d_bwd.flags |= REVFFN_FLAG_REUSE_ACTIVATIONS | REVFFN_FLAG_KEEP_STATUS;
  // With a copy stream, what a pass does not need right away travels beside the passes: the second half of
  // the tokens comes in while the forward pass works on the first half (tokens are independent through the
  // branch, so two half-batch forward calls give the same y2), dy2 comes in during forward and inverse, y2 goes
  // out during the inverse pass, the reconstructed x2 during backward.
  const int32_t T0 = (two && desc->tokens >= 2048) ? (desc->tokens / 2 / 8) * 8 : desc->tokens;   // first part
  const size_t n0 = (size_t)T0 * h * sizeof(float);
  if (two) {
    CK(cudaEventRecord(ev[0], st));            // everything queued on the compute stream so far (earlier steps
    CK(cudaStreamWaitEvent(cs, ev[0], 0));     // may still use the staging buffers)
  }
  if (n > 0) {
    CK(cudaMemcpyAsync(y1, y1_host, n0, cudaMemcpyHostToDevice, cs));
    CK(cudaMemcpyAsync(x2, x2_host, n0, cudaMemcpyHostToDevice, cs));
    if (two) CK(cudaEventRecord(ev[1], cs));   // first part of y1, x2 on the device
    if (n > n0) {
      CK(cudaMemcpyAsync(reinterpret_cast<char*>(y1) + n0, reinterpret_cast<const char*>(y1_host) + n0, n - n0,
                         cudaMemcpyHostToDevice, cs));
      CK(cudaMemcpyAsync(reinterpret_cast<char*>(x2) + n0, reinterpret_cast<const char*>(x2_host) + n0, n - n0,
                         cudaMemcpyHostToDevice, cs));
    }
    if (two) CK(cudaEventRecord(ev[2], cs));   // all of y1, x2 on the device
    CK(cudaMemcpyAsync(dy2, dy2_host, n, cudaMemcpyHostToDevice, cs));
    CK(cudaMemsetAsync(dy1, 0, n, st));
  }
  if (two) CK(cudaEventRecord(ev[3], cs));     // dy2 is on the device
  if (two && T0 < desc->tokens) {
    revffn_moe_desc d_a = *desc, d_b = *desc;
    d_a.tokens = T0;
    d_b.tokens = desc->tokens - T0;
    d_b.flags |= REVFFN_FLAG_KEEP_STATUS | REVFFN_FLAG_ROUTER_FOLDED;
    CK(cudaStreamWaitEvent(st, ev[1], 0));
    CKR(revffn_moe_forward(&d_a, w, y1, x2, y2, nullptr, ws, ws_bytes, cuda_stream));
    CK(cudaStreamWaitEvent(st, ev[2], 0));
    CKR(revffn_moe_forward(&d_b, w, y1 + (size_t)T0 * h, x2 + (size_t)T0 * h, y2 + (size_t)T0 * h, nullptr, ws, ws_bytes,
                           cuda_stream));
  } else {
    if (two) CK(cudaStreamWaitEvent(st, ev[2], 0));
    CKR(revffn_moe_forward(desc, w, y1, x2, y2, nullptr, ws, ws_bytes, cuda_stream));
  }
  if (two) {
    CK(cudaEventRecord(ev[4], st));
    CK(cudaStreamWaitEvent(cs, ev[4], 0));
  }
  if (n > 0) CK(cudaMemcpyAsync(y2_host, y2, n, cudaMemcpyDeviceToHost, cs));
  CKR(revffn_moe_inverse(&d_inv, w, y1, y2, x2r, nullptr, ws, ws_bytes, cuda_stream));
  if (two) {
    CK(cudaEventRecord(ev[5], st));
    CK(cudaStreamWaitEvent(cs, ev[5], 0));
  }
  if (n > 0) CK(cudaMemcpyAsync(x2_rec_host, x2r, n, cudaMemcpyDeviceToHost, cs));
  if (two) CK(cudaStreamWaitEvent(st, ev[3], 0));
  CKR(revffn_moe_backward(&d_bwd, w, y1, dy2, dy1, grads, nullptr, ws, ws_bytes, cuda_stream));
  if (n > 0) CK(cudaMemcpyAsync(dy1_host, dy1, n, cudaMemcpyDeviceToHost, st));
  if (two) {
    CK(cudaEventRecord(ev[6], cs));            // the compute stream's completion covers the copy stream's work
    CK(cudaStreamWaitEvent(st, ev[6], 0));
  }
  return REVFFN_OK;
}

int revffn_moe_routing_record_bytes(const revffn_moe_desc* desc, size_t* bytes) {
  int r = validate_desc(desc);
  if (r != REVFFN_OK) return r;
  if (!bytes) return REVFFN_ERR_NULL;
  *bytes = record_layout(*desc).bytes;
  return REVFFN_OK;
}

int revffn_moe_saved_size(const revffn_moe_desc* desc, size_t* bytes) {
  int r = validate_desc(desc);
  if (r != REVFFN_OK) return r;
  if (!bytes) return REVFFN_ERR_NULL;
  *bytes = plan_workspace(*desc).saved_bytes;
  return REVFFN_OK;
}

// One cache slot of the activation-caching stack: the layer's input stream (rows of
// ld_stream floats, as in the caller's buffer) followed by a full workspace.
static size_t stack_stream_slot(const revffn_moe_desc& D) {
  return (size_t)round_up((int64_t)(D.tokens > 0 ? D.tokens : 1) * D.ld_stream * (int64_t)sizeof(float), 256);
}

int revffn_moe_stack_cache_stride(const revffn_moe_desc* desc, size_t* bytes) {
  int r = validate_desc(desc);
  if (r != REVFFN_OK) return r;
  if (!bytes) return REVFFN_ERR_NULL;
  *bytes = stack_stream_slot(*desc) + plan_workspace(*desc).bwd_bytes;
  return REVFFN_OK;
}

int revffn_moe_stack_forward(const revffn_moe_desc* desc, const revffn_moe_weights* weights, int32_t n_blocks,
                             float* stream_a, float* stream_b, int32_t* topk_idx, void* cache, size_t cache_bytes,
                             void* ws, size_t ws_bytes, void* cuda_stream) {
  int r = validate_desc(desc);
  if (r != REVFFN_OK) return r;
  if (n_blocks < 0) return REVFFN_ERR_SHAPE;
  if (n_blocks > 0 && !weights) return REVFFN_ERR_NULL;
  size_t stride = 0;
  revffn_moe_stack_cache_stride(desc, &stride);
  if (cache && (cache_bytes < stride * (size_t)n_blocks || (reinterpret_cast<uintptr_t>(cache) & 255u)))
    return REVFFN_ERR_WORKSPACE;
  const size_t slot = stack_stream_slot(*desc);
  const size_t idx_stride = routing_stride(*desc);     // bytes
  const size_t ws_need = plan_workspace(*desc).bwd_bytes;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  revffn_moe_desc d = *desc;
  if (cache) d.flags |= REVFFN_FLAG_SAVE_ACTIVATIONS;
  // Without a cache all layers share `ws`: its status word is cleared here, once, and every layer keeps it, so
  // that it reports the first device-side error of the whole sweep (a later layer would otherwise erase it).
  // With a cache every layer runs in, and reports through, its own slot; the shared workspace reads "no error".
  if (ws && ws_bytes >= 256) CK(cudaMemsetAsync(ws, 0, 256, st));
  if (!cache) d.flags |= REVFFN_FLAG_KEEP_STATUS;
  for (int l = 0; l < n_blocks; ++l) {
    float* P = (l & 1) ? stream_b : stream_a;
    float* R = (l & 1) ? stream_a : stream_b;
    void* lws = ws;
    size_t lws_bytes = ws_bytes;
    if (cache) {
      char* c = reinterpret_cast<char*>(cache) + (size_t)l * stride;
      if (desc->tokens > 0)   // the layer's input stream is overwritten two layers later: keep a copy
        CK(cudaMemcpy2DAsync(c, (size_t)desc->ld_stream * 4, P, (size_t)desc->ld_stream * 4,
                             (size_t)(desc->d_model / 2) * 4, (size_t)desc->tokens, cudaMemcpyDeviceToDevice, st));
      lws = c + slot;
      lws_bytes = ws_need;
    }
    CKR(revffn_moe_forward(&d, &weights[l], P, R, R, topk_idx ? reinterpret_cast<int32_t*>(reinterpret_cast<char*>(topk_idx) + (size_t)l * idx_stride) : nullptr, lws,
                           lws_bytes, cuda_stream));
  }
  return REVFFN_OK;
}

int revffn_moe_stack_backward(const revffn_moe_desc* desc, const revffn_moe_weights* weights, int32_t n_blocks,
                              float* stream_a, float* stream_b, float* grad_a, float* grad_b,
                              const revffn_moe_grads* grads, const int32_t* topk_idx, void* cache,
                              size_t cache_bytes, void* ws, size_t ws_bytes, void* cuda_stream) {
  return revffn_moe_stack_backward_sgd(desc, weights, n_blocks, stream_a, stream_b, grad_a, grad_b, grads, nullptr, topk_idx,
                                       cache, cache_bytes, ws, ws_bytes, cuda_stream);
}

static int stack_backward_impl(const revffn_moe_desc* desc, const revffn_moe_weights* weights, int32_t n_blocks,
                               float* stream_a, float* stream_b, float* grad_a, float* grad_b,
                               const revffn_moe_grads* grads, const revffn_moe_sgd* sgd, const revffn_moe_adam* adam,
                               const int32_t* topk_idx, void* cache, size_t cache_bytes, void* ws, size_t ws_bytes,
                               void* cuda_stream);

int revffn_moe_stack_backward_sgd(const revffn_moe_desc* desc, const revffn_moe_weights* weights, int32_t n_blocks,
                                  float* stream_a, float* stream_b, float* grad_a, float* grad_b,
                                  const revffn_moe_grads* grads, const revffn_moe_sgd* sgd, const int32_t* topk_idx,
                                  void* cache, size_t cache_bytes, void* ws, size_t ws_bytes, void* cuda_stream) {
  return stack_backward_impl(desc, weights, n_blocks, stream_a, stream_b, grad_a, grad_b, grads, sgd, nullptr, topk_idx,
                             cache, cache_bytes, ws, ws_bytes, cuda_stream);
}

int revffn_moe_stack_backward_adam(const revffn_moe_desc* desc, const revffn_moe_weights* weights, int32_t n_blocks,
                                   float* stream_a, float* stream_b, float* grad_a, float* grad_b,
                                   const revffn_moe_grads* grads, const revffn_moe_adam* adam, const int32_t* topk_idx,
                                   void* cache, size_t cache_bytes, void* ws, size_t ws_bytes, void* cuda_stream) {
  return stack_backward_impl(desc, weights, n_blocks, stream_a, stream_b, grad_a, grad_b, grads, nullptr, adam, topk_idx,
                             cache, cache_bytes, ws, ws_bytes, cuda_stream);
}

static int stack_backward_impl(const revffn_moe_desc* desc, const revffn_moe_weights* weights, int32_t n_blocks,
                               float* stream_a, float* stream_b, float* grad_a, float* grad_b,
                               const revffn_moe_grads* grads, const revffn_moe_sgd* sgd, const revffn_moe_adam* adam,
                               const int32_t* topk_idx, void* cache, size_t cache_bytes, void* ws, size_t ws_bytes,
                               void* cuda_stream) {
  int r = validate_desc(desc);
  if (r != REVFFN_OK) return r;
  if (n_blocks < 0) return REVFFN_ERR_SHAPE;
  if (n_blocks > 0 && (!weights || !grads)) return REVFFN_ERR_NULL;
  size_t stride = 0;
  revffn_moe_stack_cache_stride(desc, &stride);
  if (cache && (cache_bytes < stride * (size_t)n_blocks || (reinterpret_cast<uintptr_t>(cache) & 255u)))
    return REVFFN_ERR_WORKSPACE;
  const size_t slot = stack_stream_slot(*desc);
  const size_t idx_stride = routing_stride(*desc);     // bytes
  const size_t ws_need = plan_workspace(*desc).bwd_bytes;
  revffn_moe_desc d_inv = *desc, d_bwd = *desc;
  d_inv.flags |= REVFFN_FLAG_SAVE_ACTIVATIONS | REVFFN_FLAG_KEEP_STATUS;
  // with a cache the slot's word still holds what the layer's forward pass reported: keep it as well
  d_bwd.flags |= REVFFN_FLAG_REUSE_ACTIVATIONS | REVFFN_FLAG_KEEP_STATUS;
  if (ws && ws_bytes >= 256) CK(cudaMemsetAsync(ws, 0, 256, reinterpret_cast<cudaStream_t>(cuda_stream)));
  for (int l = n_blocks - 1; l >= 0; --l) {
    float* P = (l & 1) ? stream_b : stream_a;
    float* R = (l & 1) ? stream_a : stream_b;
    float* gP = (l & 1) ? grad_b : grad_a;
    float* gR = (l & 1) ? grad_a : grad_b;
    const int32_t* idx =
        topk_idx ? reinterpret_cast<const int32_t*>(reinterpret_cast<const char*>(topk_idx) + (size_t)l * idx_stride) : nullptr;
    UpdateSpec u;
    if (sgd) u = spec_from_sgd(sgd[l]);
    if (adam) CKR(spec_from_adam(adam[l], &u));
    if (cache) {
      char* c = reinterpret_cast<char*>(cache) + (size_t)l * stride;
      CKR(entry(PASS_BWD, &d_bwd, &weights[l], reinterpret_cast<const float*>(c), gR, gP, &grads[l], idx, nullptr, c + slot,
                ws_need, cuda_stream, (sgd || adam) ? &u : nullptr));
    } else {
      // the layer's weights are read for the last time in this step by these two calls (inverse, then the
      // gradient pass, whose weight-gradient products come after every product that reads the same weight),
      // so a fused update of layer l cannot disturb any other layer's reconstruction
      CKR(revffn_moe_inverse(&d_inv, &weights[l], P, R, R, idx, ws, ws_bytes, cuda_stream));
      CKR(entry(PASS_BWD, &d_bwd, &weights[l], P, gR, gP, &grads[l], idx, nullptr, ws, ws_bytes, cuda_stream,
                (sgd || adam) ? &u : nullptr));
    }
  }
  return REVFFN_OK;
}

int revffn_moe_route_noalloc(const revffn_moe_desc* desc, const revffn_moe_weights* w, const float* y1,
                             int32_t* topk_idx_out, float* gates_out, float* sgate_out, void* cuda_stream) {
  int r = validate_desc(desc);
  if (r != REVFFN_OK) return r;
  r = validate_weights(*desc, w);
  if (r != REVFFN_OK) return r;
  if (desc->tokens > 0 && (!y1 || !topk_idx_out || !gates_out || !sgate_out)) return REVFFN_ERR_NULL;
  if (!aligned16(y1) || !aligned16(topk_idx_out)) return REVFFN_ERR_ALIGN;
  if (desc->flags & REVFFN_FLAG_GATE_SOFTMAX_ALL) return REVFFN_ERR_UNSUPPORTED;   // needs the softmax over all E logits
  const int64_t need = (int64_t)(desc->n_experts + 1) * (desc->d_model / 2);
  if (need > REVFFN_ROUTE_NOALLOC_MAX_ELEMS) return REVFFN_ERR_NOALLOC_LIMIT;
  r = check_device();
  if (r != REVFFN_OK) return r;
  if (desc->tokens == 0) return REVFFN_OK;
  double* scratch = route_scratch_ptr(&r);     // first call on a device resolves the array's address
  if (r != REVFFN_OK) return r;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (desc->weight_dtype == REVFFN_BF16)
    return route_noalloc_launch<bf16>(*desc, *w, y1, scratch, topk_idx_out, gates_out, sgate_out, st);
  return route_noalloc_launch<float>(*desc, *w, y1, scratch, topk_idx_out, gates_out, sgate_out, st);
}

int revffn_dbg_check_guards(const revffn_moe_desc* desc, void* ws, size_t ws_bytes, void* cuda_stream) {
  int r = validate_desc(desc);
  if (r != REVFFN_OK) return r;
  if (!ws) return REVFFN_ERR_NULL;
  if (!(desc->flags & REVFFN_FLAG_DEBUG_CHECKS)) return REVFFN_ERR_UNSUPPORTED;
  WsLayout L = plan_workspace(*desc);
  if (ws_bytes < L.fwd_bytes) return REVFFN_ERR_WORKSPACE;
  return guards_check(L, ws_bytes < L.bwd_bytes ? L.fwd_bytes : L.bwd_bytes, reinterpret_cast<char*>(ws),
                      reinterpret_cast<cudaStream_t>(cuda_stream));
}

int revffn_prof_enable(int on) {
  int prev = g_prof.on ? 1 : 0;
  g_prof.on = on != 0;
  g_prof.recs.clear();
  g_prof.used = 0;
  return prev;
}

long long revffn_prof_launches(void) { return g_prof.launches; }

int revffn_prof_num_slots(void) { return N_PASSES * TG_COUNT; }

const char* revffn_prof_slot_name(int slot) {
  static char buf[N_PASSES * TG_COUNT][64];
  if (slot < 0 || slot >= N_PASSES * TG_COUNT) return "";
  snprintf(buf[slot], sizeof(buf[slot]), "%s/%s", kPassNames[slot / TG_COUNT], kTagNames[slot % TG_COUNT]);
  return buf[slot];
}

int revffn_prof_collect(float* ms, int32_t* count, int n_slots) {
  if (!ms || !count) return REVFFN_ERR_NULL;
  for (int i = 0; i < n_slots; ++i) { ms[i] = 0.f; count[i] = 0; }
  for (const auto& rec : g_prof.recs) {
    if (rec.e + 1 >= g_prof.pool.size()) continue;
    if (cudaEventSynchronize(g_prof.pool[rec.e + 1]) != cudaSuccess) return REVFFN_ERR_CUDA;
    float t = 0.f;
    if (cudaEventElapsedTime(&t, g_prof.pool[rec.e], g_prof.pool[rec.e + 1]) != cudaSuccess) return REVFFN_ERR_CUDA;
    if (rec.slot >= 0 && rec.slot < n_slots) { ms[rec.slot] += t; count[rec.slot] += 1; }
  }
  g_prof.recs.clear();
  g_prof.used = 0;
  return REVFFN_OK;
}

int revffn_dbg_gemm(const revffn_dbg_gemm_args* a, int32_t* status_word_dev, void* cuda_stream) {
  if (!a) return REVFFN_ERR_NULL;
  int r = check_device();
  if (r != REVFFN_OK) return r;
  GemmProblem p = blank_problem();
  p.M = a->M; p.N = a->N; p.K = a->K;
  p.a_mn_major = a->a_mn_major; p.b_mn_major = a->b_mn_major;
  p.concat = a->concat; p.epilogue = a->epilogue; p.out_f32 = a->out_f32; p.accumulate = a->accumulate;
  p.A = a->A; p.B0 = a->B0; p.B1 = a->B1; p.lda = a->lda; p.ldb = a->ldb;
  p.C = a->C; p.C1 = a->C1; p.ldc = a->ldc; p.ldc1 = a->ldc1;
  p.rowscale = a->rowscale; p.resid = a->resid; p.ld_resid = a->ld_resid; p.resid_sign = a->resid_sign;
  p.ab = a->ab; p.ld_ab = a->ld_ab; p.dg_part = a->dg_part; p.dg_ld = a->dg_ld;
  p.group_mode = a->group_mode; p.n_groups = a->n_groups;
  p.group_off = a->group_off; p.tile_group = a->tile_group; p.rows_total = a->rows_total;
  p.b_group_stride = a->b_group_stride; p.c_group_stride = a->c_group_stride;
  p.a_col0 = a->a_col0; p.b_col0 = a->b_col0;
  p.tok_chunks = reinterpret_cast<const int4*>(a->tok_chunks); p.no_pair = a->no_pair;
  p.dbg_wait_cycles = a->wait_cycles; p.dbg_starve = a->starve_operands; p.dbg_split_loads = a->split_loads; p.dbg_mn_boxes = a->mn_boxes;
  p.status = status_word_dev;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (a->use_simt) return launch_gemm_simt<bf16>(p, st) == cudaSuccess ? REVFFN_OK : REVFFN_ERR_CUDA;
  r = tc_prepare();
  if (r != REVFFN_OK) return r;
  return launch_gemm_tc(p, st);
}

}  // extern "C"

#include "revffn_attn.cuh"
#include "revffn_block.cuh"
