/*
 * revffn_attn.h -- C ABI of the B200 (sm_100a) library for the attention coupling
 * branch of a RevFFN block.
 *
 * The block (paper Sec. 3.1) splits the hidden state H = [X1, X2] into two streams of
 * width h = d/2.  This header covers the first update (Eq. 1) and what reversible
 * back-propagation needs from it:
 *
 *   forward   Y1 = X1 + Attn(Norm(X1), Norm(X2), Norm(X2))                 (Eq. 1)
 *   inverse   X1 = Y1 - Attn(Norm(X1), Norm(X2), Norm(X2)), solved by fixed-point
 *             iteration started from X1 = Y1 (Sec. 3.1 inverse pass; the paper runs one
 *             iteration, the caller chooses the number)
 *   backward  dX1 = dY1 + J1^T dY1,  dX2 += J2^T dY1 and the weight gradients, with the
 *             intermediates recomputed from X1 and X2 instead of cached (Sec. 2, Sec. 3.1)
 *
 * with  Attn(a, b, b) = P_down( Attn_pt( P_up(a), P_up(b), P_up(b) ) )      (Sec. 3.2)
 * where P_up: R^h -> R^d and P_down: R^d -> R^h are bias-free linear adapters (one P_up
 * serves query, key and value) and Attn_pt is the base model's attention evaluated in the
 * d-wide space with the queries taken from the first argument and keys and values from the
 * second: q/k/v projections with bias, rotary position embedding on q and k (the pairs
 * (i, i + hd/2) of a head turn by pos * theta^(-2i/hd)), causal softmax attention per head
 * with scale hd^(-1/2), n_kv_heads key/value heads shared by groups of query heads, and a
 * bias-free output projection.  Norm is RMSNorm over the h-wide stream with one learnable
 * scale that serves both streams.
 *
 * Conventions: those of revffn_moe.h (device pointers unless marked host, row-major
 * [out, in] matrices, 16-byte alignment, caller-owned buffers and workspace, everything
 * enqueued on the caller's stream, negative revffn_error on failure with nothing
 * launched).  Tokens are batch-major: token t = b * seq_len + s is position s of sequence
 * b, and sequences do not attend to each other.
 */
#ifndef REVFFN_ATTN_H_
#define REVFFN_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#include "revffn_moe.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Branch descriptor.  Shape constraints (else REVFFN_ERR_SHAPE):
 *   batch >= 0, seq_len >= 1; d_model even; n_heads >= 1 divides d_model; n_kv_heads >= 1
 *   divides n_heads; head_dim = d_model / n_heads is even.
 *   weight_dtype REVFFN_F32 : h, d and head_dim multiples of 8.
 *   weight_dtype REVFFN_BF16: h and d multiples of 128, head_dim 128 (TMA / tcgen05 tiles).
 * flags: REVFFN_FLAG_FORCE_SIMT; REVFFN_FLAG_REUSE_ACTIVATIONS on a backward call (below).
 */
typedef struct {
  int32_t batch, seq_len;       /* T = batch * seq_len tokens                              */
  int32_t d_model, n_heads, n_kv_heads;
  int32_t weight_dtype;         /* REVFFN_F32 | REVFFN_BF16                                */
  float norm_eps;
  float rope_theta;             /* base of the rotary embedding                            */
  int64_t ld_stream;            /* row stride of the fp32 streams, elements                */
  uint32_t flags;
} revffn_attn_desc;

/* Weights of the branch (Sec. 3.2 adapters; Attn_pt of the base model).  d_kv = n_kv_heads * head_dim. */
typedef struct {
  const float* norm_gamma; /* [h] fp32 RMSNorm scale, NULL = ones  */
  const void* w_up;        /* [d, h]    P_up                        */
  const void* w_down;      /* [h, d]    P_down                      */
  const void* w_q;         /* [d, d]                                */
  const void* w_k;         /* [d_kv, d]                             */
  const void* w_v;         /* [d_kv, d]                             */
  const void* w_o;         /* [d, d]                                */
  const float* b_q;        /* [d]    fp32, NULL = no bias           */
  const float* b_k;        /* [d_kv] fp32, NULL = no bias           */
  const float* b_v;        /* [d_kv] fp32, NULL = no bias           */
} revffn_attn_weights;

/* Weight-gradient outputs, fp32, same shapes as the weights.  A NULL member is skipped
 * (Sec. 3.3: stage 1 trains only the adapters).  accumulate != 0 adds to the buffers. */
typedef struct {
  float *norm_gamma, *w_up, *w_down, *w_q, *w_k, *w_v, *w_o, *b_q, *b_k, *b_v;
  int32_t accumulate;
} revffn_attn_grads;

/* Bytes of workspace forward/inverse (fwd_bytes) and backward (bwd_bytes) need.  Both
 * out-pointers are host pointers and may be NULL.  (Planner; no paper counterpart.) */
int revffn_attn_workspace_size(const revffn_attn_desc* desc, size_t* fwd_bytes, size_t* bwd_bytes);

/*
 * Eq. 1:  y1[t] = x1[t] + Attn(Norm(x1), Norm(x2), Norm(x2))[t].
 *   x1, x2  in  fp32 [T, h] (stride ld_stream);  y1 out, may alias x1.
 *   ws / ws_bytes workspace of at least fwd_bytes, 256-byte aligned.
 */
int revffn_attn_forward(const revffn_attn_desc* desc, const revffn_attn_weights* w,
                        const float* x1, const float* x2, float* y1,
                        void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Sec. 3.1 inverse pass:  x1 <- y1;  n_iter times  x1 <- y1 - Attn(Norm(x1), Norm(x2), Norm(x2)).
 * The key/value side does not depend on the iterate and is evaluated once.  n_iter >= 0
 * (0 copies y1); x1 out must not alias y1 when n_iter > 1 (every iteration reads y1).
 */
int revffn_attn_inverse(const revffn_attn_desc* desc, const revffn_attn_weights* w,
                        const float* y1, const float* x2, float* x1, int32_t n_iter,
                        void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Backward of Eq. 1 by recomputation: given x1, x2 and dy1 = dL/dY1,
 *   dx1[t]        = dy1[t] + J1^T dy1      (fp32 [T, h]; may alias dy1)
 *   dx2_inout[t] += J2^T dy1               (the gradient that reaches x2 through keys and values)
 *   grads->X (+)= dL/dX                    for every non-NULL member.
 * ws must hold at least bwd_bytes.
 * With REVFFN_FLAG_REUSE_ACTIVATIONS the call takes the key/value side (which depends on x2 and the
 * weights only) from the workspace, where a revffn_attn_inverse call with n_iter >= 1, the same x2,
 * weights and descriptor has left it, and evaluates only the query side again: in reversible
 * back-propagation the inverse pass of a block runs right before its gradient pass.
 */
int revffn_attn_backward(const revffn_attn_desc* desc, const revffn_attn_weights* w,
                         const float* x1, const float* x2, const float* dy1,
                         float* dx1, float* dx2_inout, const revffn_attn_grads* grads,
                         void* ws, size_t ws_bytes, void* cuda_stream);

/* Synchronise the stream and copy the workspace's device status word to *device_status
 * (host pointer): 0 or a negative revffn_error.  (No paper counterpart.) */
int revffn_attn_status(const void* ws, void* cuda_stream, int32_t* device_status);

#ifdef __cplusplus
}
#endif

#endif /* REVFFN_ATTN_H_ */
