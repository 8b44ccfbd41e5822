/*
 * revffn_debug.h -- instrumentation and test hooks of the RevFFN B200 library.
 *
 * Nothing here is part of the method (the paper has no counterpart for any of
 * it): launch accounting and per-kernel timing, a name -> offset lookup into
 * the workspace layout, and a single-product entry point that lets the tests
 * drive one matrix product through either GEMM back end.  The product entry
 * points are in revffn_moe.h, revffn_attn.h and revffn_block.h.
 */
#ifndef REVFFN_DEBUG_H_
#define REVFFN_DEBUG_H_

#include "revffn_moe.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Launch accounting and optional per-kernel timing.  (No paper counterpart.)
 * revffn_prof_enable(1) makes every later kernel launch of this library record
 * a CUDA event before and after itself on the caller's stream;
 * revffn_prof_collect waits for those events and returns, per slot, the summed
 * device milliseconds and the number of launches (host arrays of
 * revffn_prof_num_slots() entries), then forgets them.  Slots are named
 * "<pass>/<kernel>", pass in {fwd, inv, bwd}.  revffn_prof_launches counts
 * every kernel this library has launched since it was loaded, enabled or not.
 * Not thread-safe.
 */
int revffn_prof_enable(int on);
long long revffn_prof_launches(void);
int revffn_prof_num_slots(void);
const char* revffn_prof_slot_name(int slot);
int revffn_prof_collect(float* ms, int32_t* count, int n_slots);

/*
 * Introspection for tests: byte offset and size inside the backward workspace
 * layout of a named intermediate ("n", "u", "gates", "sgate", "tok_row",
 * "row_tok", "expert_off", "up", "hmid", "o", "hs", "s", "z", "ab", ...).
 * The forward layout is a prefix of the backward layout.  Returns
 * REVFFN_ERR_UNSUPPORTED for unknown names.  (No paper counterpart.)
 */
int revffn_moe_ws_lookup(const revffn_moe_desc* desc, const char* name, size_t* offset, size_t* bytes);

/*
 * Verify the guard zones of a workspace laid out for `desc` (REVFFN_FLAG_DEBUG_CHECKS must be set in it)
 * now, on the given stream: REVFFN_ERR_CANARY appears in the status word if one was overwritten since the
 * last pass filled it.  Every pass with the flag runs the same check when it ends; this entry point lets a
 * caller (or a test) check between passes.  Offsets of the zones: revffn_moe_ws_lookup with the names
 * "guard0", "guard1", ... (REVFFN_ERR_UNSUPPORTED past the last one).
 */
int revffn_dbg_check_guards(const revffn_moe_desc* desc, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * One C = A * B^T problem on either GEMM backend; used by the tests to check
 * the tcgen05 kernels against the CUDA-core kernels.  See revffn_gemm_problem
 * in the library source for field meanings.  (No paper counterpart.)
 */
typedef struct {
  int32_t M, N, K;
  int32_t a_mn_major, b_mn_major;  /* 0: [rows, K] K contiguous; 1: [K, rows] rows contiguous */
  int32_t concat;                  /* 0 none, 1 N-concat (SwiGLU pair), 2 K-concat            */
  int32_t epilogue;                /* 0 store, 1 swiglu, 2 rowscale, 3 couple, 4 dswiglu, 5 wgrad */
  int32_t out_f32;                 /* store epilogue: fp32 instead of bf16 output             */
  int32_t accumulate;
  int32_t use_simt;
  const void *A, *B0, *B1;         /* bf16                                                    */
  int64_t lda, ldb;
  void *C, *C1;
  int64_t ldc, ldc1;
  const float* rowscale;
  const float* resid; int64_t ld_resid; float resid_sign;
  void* ab; int64_t ld_ab;         /* dswiglu: [M, 2N] bf16 a|b in, da|db out                  */
  float* dg_part; int32_t dg_ld;
  /* grouping: 0 none, 1 rows grouped (group_off, tile_group, rows_total), 2 K grouped */
  int32_t group_mode, n_groups;
  const int32_t *group_off, *tile_group, *rows_total;
  int64_t b_group_stride, c_group_stride;
  int32_t a_col0, b_col0;
  /* rows grouped: optional table of (expert, first row, rows, 0) runs of real rows, rows a multiple of
   * 32 and at most 256, int32 x 4 each, 16-byte aligned; their number at rows_total[1].  With it the
   * tcgen05 back end works store / gate-scale products with the rows on the MMA N side. */
  const void* tok_chunks;
  int32_t no_pair;                 /* tcgen05 back end: one CTA per tile even where CTA pairs apply */
  /* Failure-path test (tcgen05 back end, one CTA per tile only).  wait_cycles > 0 replaces the bound on
   * every device-side wait (clock cycles; 0 = the default of about two seconds).  starve_operands != 0
   * makes the load warp issue nothing, so that the first wait for operands runs out: the kernel must then
   * raise REVFFN_ERR_DEVICE_WAIT in the status word, release its tensor memory and return, and the
   * context must stay usable.  Nothing is in flight when that wait expires. */
  int64_t wait_cycles;
  int32_t starve_operands;
  /* measurements: operand loads issued by two threads (1) or by one (2); 0 = the library's choice per epilogue */
  int32_t split_loads;
  /* tests: 1 = load MN-major operands as 64 x 64 boxes of 2-D tensor maps, the form the library falls back to when a
   * leading dimension or column offset is not a multiple of 64 (0 = 3-D maps, 128 columns per load, where possible) */
  int32_t mn_boxes;
} revffn_dbg_gemm_args;
int revffn_dbg_gemm(const revffn_dbg_gemm_args* args, int32_t* status_word_dev, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* REVFFN_DEBUG_H_ */
