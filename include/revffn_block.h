/*
 * revffn_block.h -- C ABI for a whole RevFFN block and a stack of blocks (sm_100a).
 *
 * The block of paper Sec. 3.1 with the adapters of Sec. 3.2, both coupling branches in order:
 *
 *   forward   Y1 = X1 + Attn(Norm(X1), Norm(X2), Norm(X2))            (Eq. 1)
 *             Y2 = X2 + MLP(Norm(Y1))                                  (Eq. 2)
 *   inverse   X2 = Y2 - MLP(Norm(Y1));  X1 by `inverse_iters` fixed-point iterations of
 *             X1 <- Y1 - Attn(Norm(X1), Norm(X2), Norm(X2)) started from Y1   (Sec. 3.1 inverse pass)
 *   backward  reversible back-propagation (Sec. 2): the block's inputs are rebuilt from its
 *             outputs, then (dY1, dY2) is pushed through Eq. 2 and Eq. 1 in reverse order; no
 *             activation of the forward pass is kept.
 *
 * These calls only sequence the entry points of revffn_attn.h and revffn_moe.h on one
 * workspace; shapes, dtypes, alignment, ownership, stream and error conventions are theirs.
 * The two descriptors must describe the same tokens: attn.batch * attn.seq_len == moe.tokens,
 * equal d_model, weight_dtype and ld_stream (else REVFFN_ERR_SHAPE).
 */
#ifndef REVFFN_BLOCK_H_
#define REVFFN_BLOCK_H_

#include "revffn_attn.h"
#include "revffn_moe.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
  revffn_attn_desc attn;
  revffn_moe_desc moe;
  int32_t inverse_iters;   /* fixed-point iterations of the attention inverse; the paper uses 1 */
} revffn_block_desc;

/* Workspace for forward/inverse (fwd_bytes) and backward (bwd_bytes): the larger of the two
 * branches' workspaces (they run one after the other) plus one stream-sized buffer.
 * (Planner; no paper counterpart.) */
int revffn_block_workspace_size(const revffn_block_desc* desc, size_t* fwd_bytes, size_t* bwd_bytes);

/* Eq. 1 then Eq. 2.  x1, x2 in, y1, y2 out, fp32 [T, h] with stride ld_stream; y1 may alias x1 and
 * y2 may alias x2.  topk_idx_out: optional, as in revffn_moe_forward. */
int revffn_block_forward(const revffn_block_desc* desc, const revffn_attn_weights* wa, const revffn_moe_weights* wm,
                         const float* x1, const float* x2, float* y1, float* y2, int32_t* topk_idx_out,
                         void* ws, size_t ws_bytes, void* cuda_stream);

/* Inverse pass of Sec. 3.1.  x1 may alias y1 and x2 may alias y2.  topk_idx_in: optional, as in
 * revffn_moe_inverse. */
int revffn_block_inverse(const revffn_block_desc* desc, const revffn_attn_weights* wa, const revffn_moe_weights* wm,
                         const float* y1, const float* y2, float* x1, float* x2, const int32_t* topk_idx_in,
                         void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Reversible back-propagation through one block, in place:
 *   s1, s2  on entry the block's outputs Y1, Y2; on return its rebuilt inputs X1, X2
 *   g1, g2  on entry dL/dY1, dL/dY2; on return dL/dX1, dL/dX2
 *   ga, gm  weight gradients of the two branches (members may be NULL; each struct's own
 *           accumulate flag applies)
 * The MoE branch is evaluated once for its inverse and its gradient pass together.  The
 * gradients are taken at the REBUILT inputs, as the method prescribes; they differ from the
 * gradients at the true inputs by the reconstruction error of the inverse pass.
 */
int revffn_block_backward(const revffn_block_desc* desc, const revffn_attn_weights* wa, const revffn_moe_weights* wm,
                          float* s1, float* s2, float* g1, float* g2, const revffn_attn_grads* ga,
                          const revffn_moe_grads* gm, const int32_t* topk_idx_in,
                          void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * A stack of n_blocks blocks: block l+1 reads block l's [Y1, Y2] as its [X1, X2] (Sec. 3.1).
 * wa, wm, ga, gm are HOST arrays of n_blocks structs.  s1, s2 (and g1, g2) are updated in place
 * as above, through all layers.  topk_idx: optional int32 [n_blocks, T, k] (with
 * REVFFN_FLAG_ROUTING_RECORD: n_blocks routing records), written by forward, read by backward.
 */
int revffn_block_stack_forward(const revffn_block_desc* desc, const revffn_attn_weights* wa, const revffn_moe_weights* wm,
                               int32_t n_blocks, float* s1, float* s2, int32_t* topk_idx,
                               void* ws, size_t ws_bytes, void* cuda_stream);
int revffn_block_stack_backward(const revffn_block_desc* desc, const revffn_attn_weights* wa, const revffn_moe_weights* wm,
                                int32_t n_blocks, float* s1, float* s2, float* g1, float* g2,
                                const revffn_attn_grads* ga, const revffn_moe_grads* gm, const int32_t* topk_idx,
                                void* ws, size_t ws_bytes, void* cuda_stream);

/* Synchronise the stream and report the first device-side error of the most recent block or stack
 * call on this workspace: 0 or a negative revffn_error.  (No paper counterpart.) */
int revffn_block_status(const void* ws, void* cuda_stream, int32_t* device_status);

#ifdef __cplusplus
}
#endif

#endif /* REVFFN_BLOCK_H_ */
