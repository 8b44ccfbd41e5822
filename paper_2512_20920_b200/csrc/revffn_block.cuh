// Whole RevFFN block and stack: sequences the two branches' entry points on one workspace.
// See include/revffn_block.h.  Included at the end of revffn_moe.cu.
#pragma once

#include "../../include/revffn_block.h"

namespace revffn {

struct BlockLayout {
  size_t sub_fwd, sub_bwd;   // the branches' shared workspace
  size_t tmp_bytes;          // one packed stream [T, h] fp32 (row stride ld_stream)
  size_t fwd_bytes, bwd_bytes;
};

static int plan_block(const revffn_block_desc* D, BlockLayout* L) {
  if (!D) return REVFFN_ERR_NULL;
  CKR(validate_attn_desc(&D->attn));
  CKR(validate_desc(&D->moe));
  if ((int64_t)D->attn.batch * D->attn.seq_len != D->moe.tokens || D->attn.d_model != D->moe.d_model ||
      D->attn.weight_dtype != D->moe.weight_dtype || D->attn.ld_stream != D->moe.ld_stream || D->inverse_iters < 0)
    return REVFFN_ERR_SHAPE;
  const AttnLayout A = plan_attn(D->attn);
  const WsLayout M = plan_workspace(D->moe);
  L->sub_fwd = (size_t)round_up((int64_t)(A.fwd_bytes > M.fwd_bytes ? A.fwd_bytes : M.fwd_bytes), 256);
  L->sub_bwd = (size_t)round_up((int64_t)(A.bwd_bytes > M.bwd_bytes ? A.bwd_bytes : M.bwd_bytes), 256);
  if (L->sub_bwd < L->sub_fwd) L->sub_bwd = L->sub_fwd;
  L->tmp_bytes = (size_t)round_up((int64_t)D->moe.tokens * D->moe.ld_stream * 4 + 256, 256);
  L->fwd_bytes = L->sub_fwd + L->tmp_bytes + 256;
  L->bwd_bytes = L->sub_bwd + L->tmp_bytes + 256;
  return REVFFN_OK;
}

// first error wins: keeps the status word of a branch call that a later branch call will clear
__global__ void status_merge_kernel(int* __restrict__ accum, const int* __restrict__ word) {
  if (*accum == 0 && *word != 0) *accum = *word;
}

// workspace: [status word 256 B | spare stream | the branches' shared workspace]
struct BlockWs {
  char* ws; size_t sub; float* tmp; int* accum;
};
static BlockWs block_ws(void* ws, const BlockLayout& L, size_t ws_bytes) {
  BlockWs b;
  char* base = reinterpret_cast<char*>(ws);
  b.accum = reinterpret_cast<int*>(base);
  b.tmp = reinterpret_cast<float*>(base + 256);
  b.ws = base + 256 + L.tmp_bytes;
  b.sub = ws_bytes - 256 - L.tmp_bytes;
  return b;
}
static int block_merge(const BlockWs& b, cudaStream_t st) {
  status_merge_kernel<<<1, 1, 0, st>>>(b.accum, reinterpret_cast<const int*>(b.ws));
  return cudaGetLastError() == cudaSuccess ? REVFFN_OK : REVFFN_ERR_CUDA;
}

static int block_forward_one(const revffn_block_desc& D, const revffn_attn_weights* wa, const revffn_moe_weights* wm,
                             const float* x1, const float* x2, float* y1, float* y2, int32_t* idx_out, const BlockWs& b,
                             void* stream) {
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  CKR(revffn_attn_forward(&D.attn, wa, x1, x2, y1, b.ws, b.sub, stream));
  CKR(block_merge(b, st));
  CKR(revffn_moe_forward(&D.moe, wm, y1, x2, y2, idx_out, b.ws, b.sub, stream));
  return block_merge(b, st);
}

static int block_backward_one(const revffn_block_desc& D, const revffn_attn_weights* wa, const revffn_moe_weights* wm,
                              float* s1, float* s2, float* g1, float* g2, const revffn_attn_grads* ga,
                              const revffn_moe_grads* gm, const int32_t* idx_in, const BlockWs& b, void* stream) {
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  revffn_moe_desc d_inv = D.moe, d_bwd = D.moe;
  d_inv.flags |= REVFFN_FLAG_SAVE_ACTIVATIONS;
  d_bwd.flags |= REVFFN_FLAG_REUSE_ACTIVATIONS;
  // Eq. 2 backwards: X2 = Y2 - MLP(Norm(Y1)), then dY1 += J^T dY2 (dX2 = dY2 so far)
  CKR(revffn_moe_inverse(&d_inv, wm, s1, s2, s2, idx_in, b.ws, b.sub, stream));
  CKR(block_merge(b, st));
  CKR(revffn_moe_backward(&d_bwd, wm, s1, g2, g1, gm, idx_in, b.ws, b.sub, stream));
  CKR(block_merge(b, st));
  // Eq. 1 backwards: X1 by fixed-point iteration, then both stream gradients through the attention branch
  CKR(revffn_attn_inverse(&D.attn, wa, s1, s2, b.tmp, D.inverse_iters, b.ws, b.sub, stream));
  CKR(block_merge(b, st));
  // the inverse pass has just evaluated the key/value side from the same X2 in this workspace
  revffn_attn_desc d_ab = D.attn;
  if (D.inverse_iters >= 1) d_ab.flags |= REVFFN_FLAG_REUSE_ACTIVATIONS;
  CKR(revffn_attn_backward(&d_ab, wa, b.tmp, s2, g1, g1, g2, ga, b.ws, b.sub, stream));
  CKR(block_merge(b, st));
  if (D.moe.tokens > 0)
    CK(cudaMemcpy2DAsync(s1, (size_t)D.moe.ld_stream * 4, b.tmp, (size_t)D.moe.ld_stream * 4,
                         (size_t)(D.moe.d_model / 2) * 4, (size_t)D.moe.tokens, cudaMemcpyDeviceToDevice, st));
  return REVFFN_OK;
}

static int block_check(const revffn_block_desc* desc, BlockLayout* L, void* ws, size_t ws_bytes, bool bwd) {
  CKR(plan_block(desc, L));
  if (!ws) return REVFFN_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(ws) & 255u) return REVFFN_ERR_ALIGN;
  if (ws_bytes < (bwd ? L->bwd_bytes : L->fwd_bytes)) return REVFFN_ERR_WORKSPACE;
  return REVFFN_OK;
}

}  // namespace revffn

extern "C" {

int revffn_block_workspace_size(const revffn_block_desc* desc, size_t* fwd_bytes, size_t* bwd_bytes) {
  BlockLayout L;
  int r = plan_block(desc, &L);
  if (r != REVFFN_OK) return r;
  if (fwd_bytes) *fwd_bytes = L.fwd_bytes;
  if (bwd_bytes) *bwd_bytes = L.bwd_bytes;
  return REVFFN_OK;
}

int revffn_block_forward(const revffn_block_desc* desc, const revffn_attn_weights* wa, const revffn_moe_weights* wm,
                         const float* x1, const float* x2, float* y1, float* y2, int32_t* topk_idx_out, void* ws,
                         size_t ws_bytes, void* cuda_stream) {
  BlockLayout L;
  int r = block_check(desc, &L, ws, ws_bytes, false);
  if (r != REVFFN_OK) return r;
  BlockWs b = block_ws(ws, L, ws_bytes);
  CK(cudaMemsetAsync(b.accum, 0, 256, reinterpret_cast<cudaStream_t>(cuda_stream)));
  return block_forward_one(*desc, wa, wm, x1, x2, y1, y2, topk_idx_out, b, cuda_stream);
}

int revffn_block_inverse(const revffn_block_desc* desc, const revffn_attn_weights* wa, const revffn_moe_weights* wm,
                         const float* y1, const float* y2, float* x1, float* x2, const int32_t* topk_idx_in, void* ws,
                         size_t ws_bytes, void* cuda_stream) {
  BlockLayout L;
  int r = block_check(desc, &L, ws, ws_bytes, false);
  if (r != REVFFN_OK) return r;
  BlockWs b = block_ws(ws, L, ws_bytes);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  CK(cudaMemsetAsync(b.accum, 0, 256, st));
  CKR(revffn_moe_inverse(&desc->moe, wm, y1, y2, x2, topk_idx_in, b.ws, b.sub, cuda_stream));
  CKR(block_merge(b, st));
  // more than one iteration reads y1 again after x1 has been written: go through the spare stream when they alias
  const bool via_tmp = x1 == y1 && desc->inverse_iters > 1;
  CKR(revffn_attn_inverse(&desc->attn, wa, y1, x2, via_tmp ? b.tmp : x1, desc->inverse_iters, b.ws, b.sub, cuda_stream));
  CKR(block_merge(b, st));
  if (via_tmp && desc->moe.tokens > 0)
    CK(cudaMemcpy2DAsync(x1, (size_t)desc->moe.ld_stream * 4, b.tmp, (size_t)desc->moe.ld_stream * 4,
                         (size_t)(desc->moe.d_model / 2) * 4, (size_t)desc->moe.tokens, cudaMemcpyDeviceToDevice, st));
  return REVFFN_OK;
}

int revffn_block_backward(const revffn_block_desc* desc, const revffn_attn_weights* wa, const revffn_moe_weights* wm,
                          float* s1, float* s2, float* g1, float* g2, const revffn_attn_grads* ga,
                          const revffn_moe_grads* gm, const int32_t* topk_idx_in, void* ws, size_t ws_bytes,
                          void* cuda_stream) {
  BlockLayout L;
  int r = block_check(desc, &L, ws, ws_bytes, true);
  if (r != REVFFN_OK) return r;
  BlockWs b = block_ws(ws, L, ws_bytes);
  CK(cudaMemsetAsync(b.accum, 0, 256, reinterpret_cast<cudaStream_t>(cuda_stream)));
  return block_backward_one(*desc, wa, wm, s1, s2, g1, g2, ga, gm, topk_idx_in, b, cuda_stream);
}

int revffn_block_stack_forward(const revffn_block_desc* desc, const revffn_attn_weights* wa, const revffn_moe_weights* wm,
                               int32_t n_blocks, float* s1, float* s2, int32_t* topk_idx, void* ws, size_t ws_bytes,
                               void* cuda_stream) {
  BlockLayout L;
  int r = block_check(desc, &L, ws, ws_bytes, false);
  if (r != REVFFN_OK) return r;
  if (n_blocks < 0) return REVFFN_ERR_SHAPE;
  if (n_blocks > 0 && (!wa || !wm)) return REVFFN_ERR_NULL;
  BlockWs b = block_ws(ws, L, ws_bytes);
  CK(cudaMemsetAsync(b.accum, 0, 256, reinterpret_cast<cudaStream_t>(cuda_stream)));
  const size_t idx_stride = routing_stride(desc->moe);
  for (int l = 0; l < n_blocks; ++l) {
    int32_t* idx = topk_idx ? reinterpret_cast<int32_t*>(reinterpret_cast<char*>(topk_idx) + (size_t)l * idx_stride) : nullptr;
    CKR(block_forward_one(*desc, &wa[l], &wm[l], s1, s2, s1, s2, idx, b, cuda_stream));
  }
  return REVFFN_OK;
}

int revffn_block_stack_backward(const revffn_block_desc* desc, const revffn_attn_weights* wa, const revffn_moe_weights* wm,
                                int32_t n_blocks, float* s1, float* s2, float* g1, float* g2,
                                const revffn_attn_grads* ga, const revffn_moe_grads* gm, const int32_t* topk_idx, void* ws,
                                size_t ws_bytes, void* cuda_stream) {
  BlockLayout L;
  int r = block_check(desc, &L, ws, ws_bytes, true);
  if (r != REVFFN_OK) return r;
  if (n_blocks < 0) return REVFFN_ERR_SHAPE;
  if (n_blocks > 0 && (!wa || !wm || !ga || !gm)) return REVFFN_ERR_NULL;
  BlockWs b = block_ws(ws, L, ws_bytes);
  CK(cudaMemsetAsync(b.accum, 0, 256, reinterpret_cast<cudaStream_t>(cuda_stream)));
  const size_t idx_stride = routing_stride(desc->moe);
  for (int l = n_blocks - 1; l >= 0; --l) {
    const int32_t* idx =
        topk_idx ? reinterpret_cast<const int32_t*>(reinterpret_cast<const char*>(topk_idx) + (size_t)l * idx_stride) : nullptr;
    CKR(block_backward_one(*desc, &wa[l], &wm[l], s1, s2, g1, g2, &ga[l], &gm[l], idx, b, cuda_stream));
  }
  return REVFFN_OK;
}

int revffn_block_status(const void* ws, void* cuda_stream, int32_t* device_status) {
  return revffn_moe_status(ws, cuda_stream, device_status);     // the block's word is the first of its workspace
}

}  // extern "C"
