/*
 * revffn_moe.h -- C ABI of the B200 (sm_100a) library for the MoE coupling
 * branch of a RevFFN block.
 *
 * The block (paper Sec. 3.1) splits the hidden state H = [X1, X2] into two
 * streams of width h = d/2 and updates them in a coupled way.  This library
 * implements the second update (Eq. 2) and what reversible back-propagation
 * needs from it:
 *
 *   forward   Y2 = X2 + MLP(Norm(Y1))                         (Eq. 2)
 *   inverse   X2 = Y2 - MLP(Norm(Y1))                         (Sec. 3.1, inverse pass)
 *   backward  dY1 += J^T dY2 and the weight gradients, with the intermediates
 *             recomputed from Y1 instead of cached            (Sec. 2, Sec. 3.1)
 *
 * with  MLP(y) = P_down( MLP_pt( P_up(y) ) )                  (Sec. 3.2)
 * where P_up: R^h -> R^d and P_down: R^d -> R^h are bias-free linear adapters
 * and MLP_pt is the base model's sparse MoE block evaluated in the d-wide
 * space: a linear router, top-k selection (ties to the lower expert index),
 * softmax over the k selected logits, routed SwiGLU experts, and an optional
 * SwiGLU shared expert scaled by sigmoid(<w_sgate, u>).  Norm is RMSNorm over
 * the h-wide stream with a learnable scale.
 *
 * Conventions
 *   - T tokens (batch*seq flattened), d = d_model, h = d/2, E experts, k = top_k,
 *     I = d_expert, I_s = d_shared.
 *   - Every pointer is a DEVICE pointer unless its comment says "host".
 *   - Matrices are row-major [out, in], contiguous, 16-byte aligned.  Streams
 *     (y1, x2, y2, dy2, dy1) are fp32 [T, h] with row stride ld_stream elements
 *     (h for packed streams, d for views into an interleaved [X1, X2] tensor).
 *   - The caller owns every buffer including the workspace.  The library
 *     allocates no device memory and never synchronises, except
 *     revffn_moe_status, which synchronises the given stream.
 *   - Work is enqueued on the caller's CUDA stream (cudaStream_t passed as
 *     void*), and the call is asynchronous on it: what the caller queues on that
 *     stream afterwards follows everything of the call.  Inside a call on the
 *     tcgen05 back end, launches that nothing later in the pass depends on run on a second stream that the library creates per device
 *     on its first call (with a ring of events that order it against the
 *     caller's stream); REVFFN_FLAG_SINGLE_STREAM keeps every launch on the
 *     caller's stream.  The results are the same bits either way.  The pipelined
 *     host step (REVFFN_FLAG_STEP_PIPELINED) owns one more stream, for uploads.
 *     Calls that share a workspace must be ordered on one stream, and calls on
 *     one device must not be made from two host threads at once.
 *   - Return value: REVFFN_OK (0) or a negative revffn_error.  On an error
 *     return nothing has been launched.  Device-side problems (a bounded wait
 *     that expired, an expert index out of range) set a status word in the
 *     workspace, first error wins; each forward/inverse/backward call clears it
 *     when it starts unless REVFFN_FLAG_KEEP_STATUS is set, so revffn_moe_status
 *     reports the most recent call.  The entry points that chain several passes
 *     on one workspace (the stack, the host step) clear it once and report the
 *     first error of the whole chain.
 *   - Expert indices handed in by the caller (topk_idx_in, routing records, the
 *     stack's topk_idx) must lie in [0, E).  An entry outside that range is not
 *     used: its (token, slot) pair contributes nothing, the status word becomes
 *     REVFFN_ERR_INDEX, and no access leaves the buffers.
 *   - One device per process at a time is the tested configuration.  Per-device
 *     set-up (kernel attributes, the SM count) is done on the first call on each
 *     device under a lock; the profiler of revffn_debug.h is not thread-safe.
 */
#ifndef REVFFN_MOE_H_
#define REVFFN_MOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  REVFFN_OK = 0,
  REVFFN_ERR_NULL = -1,         /* a required pointer is NULL                       */
  REVFFN_ERR_SHAPE = -2,        /* descriptor violates a stated shape constraint    */
  REVFFN_ERR_ALIGN = -3,        /* a pointer or stride is not 16-byte aligned       */
  REVFFN_ERR_WORKSPACE = -4,    /* workspace smaller than revffn_moe_workspace_size */
  REVFFN_ERR_ARCH = -5,         /* current device is not compute capability 10.x    */
  REVFFN_ERR_CUDA = -6,         /* a CUDA runtime/driver call failed                */
  REVFFN_ERR_DEVICE_WAIT = -7,  /* status word: a bounded device-side wait expired  */
  REVFFN_ERR_UNSUPPORTED = -8,  /* valid request that this build does not implement */
  REVFFN_ERR_NOALLOC_LIMIT = -9, /* revffn_moe_route_noalloc: problem exceeds its fixed scratch */
  REVFFN_ERR_INDEX = -10,       /* status word: a caller-supplied expert index is outside [0, E)   */
  REVFFN_ERR_CANARY = -11,      /* status word (DEBUG_CHECKS): a guard word between workspace buffers was overwritten */
  REVFFN_ERR_NONFINITE = -12    /* status word (DEBUG_CHECKS): a router logit is NaN or infinite    */
} revffn_error;

enum { REVFFN_F32 = 0, REVFFN_BF16 = 1 };          /* weight_dtype                    */
enum { REVFFN_NORM_RMS = 0, REVFFN_NORM_NONE = 1 }; /* norm_kind                       */

/* flags */
#define REVFFN_FLAG_FORCE_SIMT 1u  /* run bf16 GEMMs on the plain CUDA-core kernels (cross-check) */
/* Sharing one evaluation of the branch between two passes.  In a reversible stack the
 * backward sweep visits a block twice with the same y1: first the inverse pass (Sec. 3.1)
 * to recover x2, then the gradient pass, which by the method recomputes the branch's
 * intermediates.  Both evaluate MLP(Norm(y1)); with these two flags the second call reads
 * what the first one left in the workspace instead of computing it again.  The same pair
 * of flags gives the activation-caching variant that the reversible design is compared
 * against: forward with SAVE into a workspace kept per block, backward with REUSE.
 *   SAVE_ACTIVATIONS   forward / inverse: ws must hold bwd_bytes; the SwiGLU
 *                      pre-activations are kept next to the other intermediates.
 *   REUSE_ACTIVATIONS  backward: ws still holds everything a forward / inverse call with
 *                      SAVE_ACTIVATIONS wrote for the same y1, weights and descriptor; the
 *                      recomputation is skipped.  The backward pass overwrites some of it,
 *                      so one saved evaluation serves one backward call.               */
#define REVFFN_FLAG_SAVE_ACTIVATIONS 2u
#define REVFFN_FLAG_REUSE_ACTIVATIONS 4u
/* Gate weights without renormalisation: g_e = softmax(L over all E experts)_e for the k selected
 * experts (they sum to less than 1 unless k == E), instead of the softmax over the k selected
 * logits.  The same experts are selected.  In the backward pass every logit then receives a
 * gradient (through the softmax denominator), not only the selected ones.  Set the flag on every
 * pass of a block alike. */
#define REVFFN_FLAG_GATE_SOFTMAX_ALL 8u
/* Routing records.  With this flag topk_idx_out / topk_idx_in (and the stack's topk_idx, per layer) point
 * to a routing record of revffn_moe_routing_record_bytes bytes instead of the bare index array: the
 * [T, k] int32 expert indices, then (each part starting on a 16-byte boundary) the [T, k] fp32 gate
 * weights and the [T] fp32 shared-expert gate.  forward writes the whole record; inverse and backward,
 * given one, take routing AND gate values from it and run no router at all: the inverse then subtracts
 * exactly the branch the forward pass added even when y1 itself is a reconstruction that differs from
 * the original by rounding (Sec. 3.1 recomputes the router; this remembers 4(2k+1) bytes per token
 * instead).  Combined with REVFFN_FLAG_GATE_SOFTMAX_ALL only the indices of the record are used. */
#define REVFFN_FLAG_ROUTING_RECORD 16u
/* Keep the status word: the call does not clear the workspace's status word when it starts, so
 * that several calls chained on one workspace report the FIRST device-side error of the chain
 * (clear the word once, with a call that does not carry the flag or with a memset of the first
 * 4 bytes of the workspace, then read it after the last call).  The stack and host-step entry
 * points use it for their inner calls. */
#define REVFFN_FLAG_KEEP_STATUS 32u
/* Debug checks (the stand-in for a memory checker): every sub-buffer of the workspace is followed
 * by a 256-byte guard zone that the call fills with a pattern when it starts and verifies when it
 * ends (REVFFN_ERR_CANARY in the status word names an overrun), and the router raises
 * REVFFN_ERR_NONFINITE for a NaN or infinite logit.  The workspace is larger with the flag set
 * (ask revffn_moe_workspace_size with the same flags) and every pass runs two more small kernels.
 * Range checks of caller-supplied expert indices are always on (REVFFN_ERR_INDEX). */
#define REVFFN_FLAG_DEBUG_CHECKS 64u
/* The router folded through P_up (an (E+1) x h fp64 matrix that forward / inverse / backward derive
 * from w_router, ws_sgate and w_up at the start of each call) is still in this workspace from an
 * earlier call with the same weights: skip that step.  The paper freezes the router (Sec. 3.3) and the
 * adapters change once per optimiser step, so within a training step every pass after the first may
 * set the flag.  The caller vouches that the three tensors are unchanged since that call and that no
 * call with another descriptor has used the workspace in between. */
#define REVFFN_FLAG_ROUTER_FOLDED 128u
/* FP8 routed experts (forward and inverse passes; bf16 weights only; no paper counterpart: a variant of the
 * arithmetic of MLP_pt's routed experts).  The three products of the routed experts take e4m3 operands with fp32
 * accumulation: each token row of u and of g*H is scaled by max|row| / 448 and rounded to e4m3 on the fly, and the
 * expert weights come quantised per output row from revffn_moe_quantize_experts (the q_* / s_* members of
 * revffn_moe_weights; the bf16 weights stay the master copy).  Three bits of mantissa put the branch output about
 * 4 % (relative L2) away from the bf16 evaluation; forward and inverse still add and subtract bit-identical
 * branches.  Not with REVFFN_FLAG_FORCE_SIMT, SAVE/REUSE_ACTIVATIONS or in revffn_moe_backward
 * (REVFFN_ERR_UNSUPPORTED): gradients are taken on the bf16 path. */
#define REVFFN_FLAG_FP8_EXPERTS 256u
/* revffn_moe_step_host only: the pipelined form described there (two staging sets used in turn, results
 * complete when the copy stream completes).  Other entry points ignore it. */
#define REVFFN_FLAG_STEP_PIPELINED 512u
/* Keep every launch of the call on cuda_stream.  Without it, calls on the tcgen05 back end put launches that nothing later in the pass depends on (the shared expert beside the routed experts, the weight
 * gradients beside the input gradients) on a second stream that the library creates per device on first use,
 * ordered against cuda_stream by events; cuda_stream still ends after everything of the call, and the results
 * are the same bits either way. */
#define REVFFN_FLAG_SINGLE_STREAM 1024u

/*
 * Block descriptor.  Shape constraints (else REVFFN_ERR_SHAPE):
 *   tokens >= 0; d_model even; 1 <= top_k <= 8; top_k <= n_experts <= 256;
 *   d_shared >= 0 (0 = no shared expert).
 *   weight_dtype REVFFN_F32 : every width (h, d, I, I_s) a multiple of 8.
 *   weight_dtype REVFFN_BF16: every width a multiple of 128 (TMA / tcgen05 tiles).
 * With REVFFN_F32 all weights are float and every intermediate is fp32; with
 * REVFFN_BF16 weights are bfloat16, GEMM operands are bf16 with fp32
 * accumulation, and routing is still decided in higher precision from the
 * fp32 stream.
 */
typedef struct {
  int32_t tokens, d_model, n_experts, top_k, d_expert, d_shared;
  int32_t weight_dtype;
  int32_t norm_kind;
  float norm_eps;
  int64_t ld_stream;
  uint32_t flags;
} revffn_moe_desc;

/* Weights of one block (Sec. 3.2 adapters; MLP_pt of the base model). */
typedef struct {
  const float* norm_gamma; /* [h] fp32 RMSNorm scale, NULL = ones                       */
  const void* w_up;        /* [d, h]   P_up                                              */
  const void* w_down;      /* [h, d]   P_down                                            */
  const void* w_router;    /* [E, d]                                                     */
  const float* b_router;   /* [E] fp32 router bias or NULL                               */
  const void* w_gate;      /* [E, I, d] expert gate projections                          */
  const void* w_upx;       /* [E, I, d] expert up projections                            */
  const void* w_downx;     /* [E, d, I] expert down projections                          */
  const void* ws_gate;     /* [I_s, d] shared expert (all four NULL iff d_shared == 0)   */
  const void* ws_up;       /* [I_s, d]                                                   */
  const void* ws_down;     /* [d, I_s]                                                   */
  const void* ws_sgate;    /* [d]      shared-expert sigmoid gate                        */
  /* REVFFN_FLAG_FP8_EXPERTS only (NULL otherwise): e4m3 codes and fp32 per-output-row scales of the expert
   * weights, written by revffn_moe_quantize_experts from the bf16 weights above. */
  const void* q_gate;      /* [E, I, d] e4m3                                             */
  const void* q_upx;       /* [E, I, d] e4m3                                             */
  const void* q_downx;     /* [E, d, I] e4m3                                             */
  const float* s_gate;     /* [E, I] fp32                                                */
  const float* s_upx;      /* [E, I] fp32                                                */
  const float* s_downx;    /* [E, d] fp32                                                */
} revffn_moe_weights;

/*
 * Weight-gradient outputs, fp32, same shapes as the weights.  Any member may be
 * NULL: that gradient is skipped (Sec. 3.3: stage 1 trains only the adapters,
 * stage 2 the experts and adapters, the router stays frozen).  accumulate != 0
 * adds to the buffers' contents instead of overwriting them.
 */
typedef struct {
  float *norm_gamma, *w_up, *w_down, *w_router, *b_router, *w_gate, *w_upx, *w_downx,
        *ws_gate, *ws_up, *ws_down, *ws_sgate;
  int32_t accumulate;
} revffn_moe_grads;

/* Bytes of workspace forward/inverse (fwd_bytes) and backward (bwd_bytes) need.
 * Both out-pointers are host pointers and may be NULL.  (Planner; no paper counterpart.) */
int revffn_moe_workspace_size(const revffn_moe_desc* desc, size_t* fwd_bytes, size_t* bwd_bytes);

/*
 * Eq. 2:  y2[t] = x2[t] + MLP(Norm(y1[t])).
 *   y1, x2  in   fp32 [T, h] (stride ld_stream);  y2 out, may alias x2.
 *   topk_idx_out  optional int32 [T, k]: selected experts per token in
 *                 descending-logit order.
 *   ws / ws_bytes workspace of at least fwd_bytes, 256-byte aligned.
 */
int revffn_moe_forward(const revffn_moe_desc* desc, const revffn_moe_weights* w,
                       const float* y1, const float* x2, float* y2,
                       int32_t* topk_idx_out, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Sec. 3.1 inverse pass:  x2[t] = y2[t] - MLP(Norm(y1[t])).  The branch is
 * recomputed with the same kernels and reduction orders as the forward pass, so
 * the subtracted term is bit-identical to the one that was added.
 *   topk_idx_in   optional int32 [T, k]: reuse these expert sets instead of
 *                 re-selecting them (gate weights are still recomputed).
 *   x2 out, may alias y2.
 */
int revffn_moe_inverse(const revffn_moe_desc* desc, const revffn_moe_weights* w,
                       const float* y1, const float* y2, float* x2,
                       const int32_t* topk_idx_in, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Backward of Eq. 2 by recomputation (Sec. 2 "Reversible Networks", Sec. 3.1):
 * given y1 and dy2 = dL/dY2, recompute the branch's intermediates, then
 *   dy1_inout[t] += J^T dy2[t]      (fp32 [T, h], stride ld_stream)
 *   grads->X (+)= dL/dX             for every non-NULL member.
 * dL/dX2 equals dy2 and is not written.  The router may be frozen (its
 * gradient pointers NULL) but the gradient through the gate values still
 * reaches dy1.  ws must hold at least bwd_bytes.
 */
int revffn_moe_backward(const revffn_moe_desc* desc, const revffn_moe_weights* w,
                        const float* y1, const float* dy2, float* dy1_inout,
                        const revffn_moe_grads* grads, const int32_t* topk_idx_in,
                        void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Backward pass with the optimiser step fused into the weight-gradient products (Sec. 3.3: the schedule trains
 * the adapters in stage 1 and adapters plus experts in stage 2; the paper's optimiser is not this one -- plain
 * SGD is what can be applied tile by tile without optimiser state, and it is enough to show the mechanism).
 * For every matrix named in sgd->mask the product that would have produced its fp32 gradient applies
 *     W <- W - lr * dL/dW
 * to the weight itself, tile by tile, in its epilogue, and the gradient is never written: at the benchmark
 * block shape that saves the 2.1 GB of fp32 expert gradients.  Without a master copy the step is taken on the
 * stored weight (bf16 weights: read, updated in fp32, rounded to nearest even; steps much smaller than the
 * weight's last bit are lost, as in any pure-bf16 update).  With a master copy (sgd->m_X, fp32, same shape) the
 * step is taken there and W receives the rounded master value.
 *   - `w` is modified: the matrices named in the mask are written through their (const) pointers.  Every product
 *     of this call that reads such a matrix runs before the product that updates it.
 *   - grads: as in revffn_moe_backward for everything NOT in the mask (the vectors norm_gamma, ws_sgate, w_router,
 *     b_router are never fused); a matrix may not be both in the mask and have a gradient pointer
 *     (REVFFN_ERR_UNSUPPORTED).  grads->accumulate applies to the written gradients only.
 *   - Stage masks: stage 1 = REVFFN_UPD_W_UP | REVFFN_UPD_W_DOWN, stage 2 = REVFFN_UPD_ALL.
 *   - A workspace that caches the folded router (REVFFN_FLAG_ROUTER_FOLDED) is stale once w_up has been updated.
 * revffn_moe_stack_backward_sgd: the reversible sweep of revffn_moe_stack_backward with one revffn_moe_sgd per
 * layer (HOST array of n_blocks structs, or NULL for none): layer l's weights are updated right after the last
 * use of layer l in the sweep, so the sweep is one training step of the whole stack with no gradient buffers
 * for the matrices in the masks.
 */
#define REVFFN_UPD_W_UP 1u
#define REVFFN_UPD_W_DOWN 2u
#define REVFFN_UPD_W_GATE 4u
#define REVFFN_UPD_W_UPX 8u
#define REVFFN_UPD_W_DOWNX 16u
#define REVFFN_UPD_WS_GATE 32u
#define REVFFN_UPD_WS_UP 64u
#define REVFFN_UPD_WS_DOWN 128u
#define REVFFN_UPD_ALL 255u
typedef struct {
  float lr;
  uint32_t mask;          /* REVFFN_UPD_* bits                                              */
  float *m_w_up, *m_w_down, *m_w_gate, *m_w_upx, *m_w_downx, *m_ws_gate, *m_ws_up, *m_ws_down;   /* fp32 master copies or NULL */
} revffn_moe_sgd;
int revffn_moe_backward_sgd(const revffn_moe_desc* desc, const revffn_moe_weights* w,
                            const float* y1, const float* dy2, float* dy1_inout,
                            const revffn_moe_grads* grads, const revffn_moe_sgd* sgd, const int32_t* topk_idx_in,
                            void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * The same fusion with Adam (decoupled weight decay) as the rule.  (The paper names no optimiser for its method;
 * this is the second reading of "the update applied where the gradient is produced", for callers that train
 * with moment estimates.)  Per element of every matrix in the mask, with g the gradient the product has just
 * accumulated, all in fp32:
 *     m <- beta1 m + (1 - beta1) g          v <- beta2 v + (1 - beta2) g^2
 *     W <- W - lr ( (m / (1 - beta1^step)) / (sqrt(v / (1 - beta2^step)) + eps) + weight_decay W )
 * mom[i] / var[i] (fp32, shape of matrix i, 16-byte aligned, caller-owned, zero before the first step) are read
 * and rewritten in the same epilogue; master[i] is the optional fp32 copy of the weight as in revffn_moe_sgd.
 * Index i is the position of the matrix's REVFFN_UPD_* bit (w_up 0, w_down 1, w_gate 2, w_upx 3, w_downx 4,
 * ws_gate 5, ws_up 6, ws_down 7).  step >= 1 is the caller's step counter.  Everything else (mask rules, which
 * gradients are still written, ordering of reads and updates) is as for revffn_moe_backward_sgd;
 * revffn_moe_stack_backward_adam is the reversible sweep with one such struct per layer.  The moments
 * add 16 bytes of traffic per element to the 4 of the weight: the fused form saves the gradient's 8 (write, then
 * read by a separate optimiser pass), not the moments'.
 */
typedef struct {
  float lr, beta1, beta2, eps, weight_decay;
  int32_t step;
  uint32_t mask;          /* REVFFN_UPD_* bits                                              */
  float* mom[8];          /* first moments, by bit position                                 */
  float* var[8];          /* second moments                                                 */
  float* master[8];       /* fp32 master copies or NULL                                     */
} revffn_moe_adam;
int revffn_moe_backward_adam(const revffn_moe_desc* desc, const revffn_moe_weights* w,
                             const float* y1, const float* dy2, float* dy1_inout,
                             const revffn_moe_grads* grads, const revffn_moe_adam* adam, const int32_t* topk_idx_in,
                             void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Quantise the bf16 expert weights for REVFFN_FLAG_FP8_EXPERTS: per output row r of w_gate / w_upx ([E*I] rows of
 * d) and of w_downx ([E*d] rows of I), scale[r] = max|row| / 448 (1 for an all-zero row) and
 * code = e4m3(w * (1 / scale[r])), every step a correctly rounded fp32 operation, round to nearest even,
 * saturating.  Writes the six q_* / s_* buffers named in `w`
 * (caller-owned device memory of the sizes given at revffn_moe_weights, 16-byte aligned); call again whenever
 * the bf16 weights change.  Needs d and I to be multiples of 128 and at most 2048.  Enqueued on the stream.
 */
int revffn_moe_quantize_experts(const revffn_moe_desc* desc, const revffn_moe_weights* w, void* cuda_stream);

/* Synchronise the stream and copy the workspace's device status word to
 * *device_status (host pointer): 0 or a negative revffn_error.  (No paper counterpart.) */
int revffn_moe_status(const void* ws, void* cuda_stream, int32_t* device_status);

/* Text for an error code; static storage. */
const char* revffn_strerror(int code);

/*
 * A stack of n_blocks coupling branches (Sec. 3.1: a layer's two output streams are the
 * next layer's input; Sec. 2: during back-propagation each layer's input is rebuilt from
 * its output, so no activation outlives its layer).  Only the MoE branch of each block is
 * in this library, so the streams swap roles between layers: layer l reads stream P_l and
 * updates stream R_l in place, (P_l, R_l) = (stream_a, stream_b) for even l and
 * (stream_b, stream_a) for odd l.
 *
 *   weights, grads   HOST arrays of n_blocks structs (device pointers inside); several
 *                    layers may name the same gradient buffers.
 *   stream_a/b       fp32 [T, h], stride ld_stream, updated in place.
 *   ws               one workspace of bwd_bytes shared by all layers.
 *   cache            NULL: reversible operation, nothing is kept between layers.
 *                    non-NULL: the activation-caching variant the reversible design is
 *                    measured against: n_blocks slots of revffn_moe_stack_cache_stride
 *                    bytes (256-byte aligned); forward keeps every layer's input stream
 *                    and intermediates there, backward reads them and runs no inverse.
 *
 * revffn_moe_stack_forward: for l = 0 .. n_blocks-1:  R_l += MLP_l(Norm(P_l))   (Eq. 2).
 *   topk_idx  optional int32 [n_blocks, T, k], the expert sets of every layer (with
 *             REVFFN_FLAG_ROUTING_RECORD: n_blocks routing records back to back).
 * revffn_moe_stack_backward: for l = n_blocks-1 .. 0:  R_l -= MLP_l(Norm(P_l)) (the inverse
 *   pass), then dP_l += J_l^T dR_l and layer l's weight gradients; the gradient pass reuses
 *   the branch evaluation of the inverse pass.  On entry stream_a/b hold the stack's
 *   outputs and grad_a/b the loss gradients w.r.t. them; on return stream_a/b hold the
 *   reconstructed inputs (reversible operation only) and grad_a/b the gradients w.r.t.
 *   the inputs.
 *   topk_idx  optional: reuse these expert sets instead of re-selecting them from the
 *             reconstructed streams (a reconstructed stream differs from the original by
 *             rounding, which can flip a near-tie).
 * Same ownership, stream and error conventions as the single-layer entry points.
 */
int revffn_moe_stack_cache_stride(const revffn_moe_desc* desc, size_t* bytes);
int revffn_moe_stack_forward(const revffn_moe_desc* desc, const revffn_moe_weights* weights, int32_t n_blocks,
                             float* stream_a, float* stream_b, int32_t* topk_idx, void* cache, size_t cache_bytes,
                             void* ws, size_t ws_bytes, void* cuda_stream);
int revffn_moe_stack_backward(const revffn_moe_desc* desc, const revffn_moe_weights* weights, int32_t n_blocks,
                              float* stream_a, float* stream_b, float* grad_a, float* grad_b,
                              const revffn_moe_grads* grads, const int32_t* topk_idx, void* cache,
                              size_t cache_bytes, void* ws, size_t ws_bytes, void* cuda_stream);

int revffn_moe_stack_backward_sgd(const revffn_moe_desc* desc, const revffn_moe_weights* weights, int32_t n_blocks,
                                  float* stream_a, float* stream_b, float* grad_a, float* grad_b,
                                  const revffn_moe_grads* grads, const revffn_moe_sgd* sgd, const int32_t* topk_idx,
                                  void* cache, size_t cache_bytes, void* ws, size_t ws_bytes, void* cuda_stream);

/* The reversible sweep with one revffn_moe_adam per layer (HOST array of n_blocks structs): as
 * revffn_moe_stack_backward_sgd, with the rule of revffn_moe_backward_adam. */
int revffn_moe_stack_backward_adam(const revffn_moe_desc* desc, const revffn_moe_weights* weights, int32_t n_blocks,
                                   float* stream_a, float* stream_b, float* grad_a, float* grad_b,
                                   const revffn_moe_grads* grads, const revffn_moe_adam* adam, const int32_t* topk_idx,
                                   void* cache, size_t cache_bytes, void* ws, size_t ws_bytes, void* cuda_stream);

/* Size of one routing record (REVFFN_FLAG_ROUTING_RECORD), a multiple of 16.  (Planner; no paper counterpart.) */
int revffn_moe_routing_record_bytes(const revffn_moe_desc* desc, size_t* bytes);

/* Bytes at the start of a workspace that hold what REVFFN_FLAG_SAVE_ACTIVATIONS keeps for
 * the gradient pass (the rest of bwd_bytes is scratch of the gradient pass itself).
 * (Planner; no paper counterpart.) */
int revffn_moe_saved_size(const revffn_moe_desc* desc, size_t* bytes);

/*
 * One whole step of the path with HOST-resident streams: copies y1, x2 and dy2
 * (host, [T, h] packed, ideally pinned) to the device, runs forward (Eq. 2),
 * inverse (Sec. 3.1) and backward (dy1 starting from zero; it reuses the branch
 * evaluation of the inverse pass, REVFFN_FLAG_SAVE/REUSE_ACTIVATIONS), and copies y2,
 * the reconstructed x2 and dy1 back to the host buffers.  `staging` is caller-owned
 * device memory of at least 6 * round_up(T*h*4, 256) bytes, 256-byte aligned;
 * requires ld_stream == h.  Asynchronous on the stream like the other entry
 * points: synchronise cuda_stream before reading the host outputs.
 * copy_stream: NULL, or a second stream of the caller's on which the transfers that a
 * pass does not need at once run beside the passes (the second half of y1 and x2 in while
 * the forward pass works on the first half of the tokens, dy2 in during forward and inverse,
 * y2 out during the inverse pass, the reconstructed x2 out during backward).  The call
 * orders the two streams with events (seven per device, created on its first use); when it
 * returns, work queued on cuda_stream afterwards follows everything of this step.
 *
 * REVFFN_FLAG_STEP_PIPELINED (needs copy_stream and staging of 12 slots, else REVFFN_ERR_UNSUPPORTED /
 * REVFFN_ERR_WORKSPACE): for a loop of steps.  Consecutive calls on a device use the two halves of `staging` in
 * turn; the inputs go up on a stream the library creates on first use, the results come down on copy_stream,
 * and cuda_stream does NOT wait for the downloads.  The uploads of a call therefore run while the passes of
 * the previous call are still computing, and its downloads while the next call computes: in a loop the
 * transfers disappear behind the passes.  The contract changes accordingly: the host outputs of a call are
 * complete when copy_stream has completed the work this call queued on it (record an event there after the
 * call); the host inputs may be overwritten from then on too; the results are the same bits as in the plain
 * form.  The workspace is shared by consecutive calls and is used in stream order.
 * (Convenience for end-to-end use; no paper counterpart.)
 */
int revffn_moe_step_host(const revffn_moe_desc* desc, const revffn_moe_weights* w, const revffn_moe_grads* grads,
                         const float* y1_host, const float* x2_host, const float* dy2_host, float* y2_host,
                         float* x2_rec_host, float* dy1_host, void* staging, size_t staging_bytes, void* ws,
                         size_t ws_bytes, void* cuda_stream, void* copy_stream);

/*
 * Routing only, for callers that must not allocate.  (The paper has no
 * counterpart: this is a packaging of the router step of MLP_pt.)
 *
 * Some callers cannot provide a workspace because they cannot call cudaMalloc
 * at the point where they need the routing decision: code running inside a
 * stream-ordered region that forbids allocation, a plug-in whose host gives it
 * only its input and output tensors, or a process that has handed all device
 * memory to another allocator.  For them this entry point computes
 *   topk_idx_out [T, k] int32   selected experts per token, descending logit
 *   gates_out    [T, k] fp32    softmax over the selected logits
 *   sgate_out    [T]    fp32    shared-expert sigmoid gate (0 without one)
 * from y1 ([T, h] fp32, stride ld_stream) with the selection rule of
 * revffn_moe_forward (fp64 logits from the folded router, ties to the lower
 * index, softmax over the k selected logits), but keeps its one piece of
 * scratch -- the router folded through P_up, (E + 1) * h doubles -- in a fixed
 * array inside the library's device image rather than in a workspace.  The fold
 * is summed in a different order than in revffn_moe_forward (which splits it
 * over partial sums that need scratch of their own), so the folded matrix
 * agrees to fp64 rounding, not bit for bit; the selected experts differ only
 * for tokens whose k-th and (k+1)-th logits tie to about 1e-13.  It calls no
 * cudaMalloc, cudaFree or other allocating routine.
 *
 * Limits and sharing
 *   - (E + 1) * h <= REVFFN_ROUTE_NOALLOC_MAX_ELEMS (512 KB of scratch, held by
 *     every device that loads the library until the process exits); otherwise
 *     REVFFN_ERR_NOALLOC_LIMIT and nothing is launched.  The router kernel keeps
 *     a 32-token tile of logits in shared memory, 8 * 32 * (E + 1) bytes plus
 *     27.3 KB of operand staging: above 48 KB in total (E >= 83) the first call on
 *     a device raises the kernel's dynamic shared-memory limit, which is a
 *     function attribute, not an allocation; E = 256 needs 92 KB.
 *   - REVFFN_FLAG_GATE_SOFTMAX_ALL is not supported here (its gates need the
 *     softmax over all E logits, which this entry point does not form):
 *     REVFFN_ERR_UNSUPPORTED, nothing is launched.  Other flags are ignored.
 *   - The first call on a device looks up the array's device address (and may
 *     raise the shared-memory limit, above); make that first call outside any
 *     stream capture.
 *   - All calls on a device share the one array.  Each call rewrites the part
 *     it uses before reading it, so nothing has to be cleared, but two calls
 *     that overlap on the GPU (different streams) race: order them.
 */
#define REVFFN_ROUTE_NOALLOC_MAX_ELEMS 65536
int revffn_moe_route_noalloc(const revffn_moe_desc* desc, const revffn_moe_weights* w, const float* y1,
                             int32_t* topk_idx_out, float* gates_out, float* sgate_out, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* REVFFN_MOE_H_ */
