// Causal attention core on tcgen05 / TMEM / TMA (Attn_pt of Eq. 1 between the projections):
//   O = softmax(scale * Q K^T, keys <= query position) V   per (sequence, head),
// without materialising the score matrix.
//
// One CTA per (sequence, head, block of 128 query positions); it walks the key/value blocks
// 0 .. its own diagonal block.  320 threads:
//   warp 0      TMA producer: Q once, then K and V blocks into two-stage rings
//   warp 1      MMA issuer and TMEM owner.  TMEM (512 columns): two score accumulators S0/S1 and two
//               output accumulators O0/O1 of 128 fp32 columns each.
//               S_j = Q K_j^T is issued one block ahead of O_j = P_j V_j, so the tensor pipe computes
//               the next scores while the softmax warps work on the current ones.  P_j is the A operand
//               of the second product straight from tensor memory.
//   warps 2..9  softmax: two threads per query row (= TMEM lane), 64 keys each.  Per block: the scores
//               into registers, row maximum (the halves exchange theirs through shared memory),
//               p = exp2((s - m) * scale * log2 e), P as bf16 pairs over the first 64 columns of the
//               score accumulator it came from (tcgen05.st; no shared-memory round trip, and the
//               tensor core reads 4 KB less per instruction), then the PREVIOUS block's O_j (this
//               thread's 64 columns) is added into a register accumulator,
//               acc = acc * exp2((m_old - m_new) ...) + O_j.  Every O_j is a fresh TMEM accumulator, so
//               no rescaling pass over TMEM is needed and P_j V_j never waits for a correction.
// Operands: q, k, v head-major [.., S_pad, hd] bf16 with hd = 128 (rows past the sequence are zero);
// output token-major [T, ld_o] bf16, plus the row log-sum-exp (natural log, of the scaled scores).
// Every wait is bounded; a wait that runs out sets the status word and all roles leave.
#pragma once

#include "gemm_tcgen05.cuh"

namespace revffn {

constexpr int FA_THREADS = 320;
constexpr int FA_BLK = 128;                       // query rows per CTA and keys per block
constexpr int FA_HD = 128;                        // head dimension
constexpr int FA_TILE = FA_BLK * 64 * 2;          // one 64-wide K block of an operand tile: 16 KB
constexpr int FA_Q_OFF = 0;                       // Q: 2 tiles
constexpr int FA_K_OFF = 2 * FA_TILE;             // K: 2 stages x 2 tiles
constexpr int FA_V_OFF = FA_K_OFF + 4 * FA_TILE;  // V: 2 stages x 2 k-blocks (each 2 chunks of 8 KB)
constexpr int FA_BAR_OFF = FA_V_OFF + 4 * FA_TILE;
constexpr int FA_XMAX_OFF = FA_BAR_OFF + 256;             // row maxima exchanged between the two halves: [2][2][128] floats
constexpr int FA_XSUM_OFF = FA_XMAX_OFF + 2048;           // row sums exchanged at the end: [2][128] floats
constexpr int FA_SMEM_BYTES = FA_XSUM_OFF + 1024 + 1024;  // + alignment slack

__device__ __forceinline__ float fa_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Row maximum over this thread's 64 scores.  DIAG: the diagonal block, where key c of the block is masked
// for query row `row` when c > row (col0 = first key of this thread's half).
template <bool DIAG>
__device__ __forceinline__ float fa_row_max(const uint32_t (&r0)[32], const uint32_t (&r1)[32], int col0, int row) {
  float mx = -INFINITY;
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    if (!DIAG || col0 + i <= row) mx = fmaxf(mx, __uint_as_float(r0[i]));
    if (!DIAG || col0 + 32 + i <= row) mx = fmaxf(mx, __uint_as_float(r1[i]));
  }
  return mx;
}

// p = exp2(s * cl - mc) for this thread's 64 scores, packed to bf16 (eight 16-byte pieces); returns their sum.
template <bool DIAG>
__device__ __forceinline__ float fa_probs(const uint32_t (&r0)[32], const uint32_t (&r1)[32], float cl, float mc, int col0,
                                          int row, uint4 (&pk)[8]) {
  float sum = 0.f;
#pragma unroll
  for (int g = 0; g < 8; ++g) {
    float pv[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int kk = 8 * g + i;
      float p = fa_exp2(__uint_as_float(kk < 32 ? r0[kk] : r1[kk - 32]) * cl - mc);
      if (DIAG && col0 + kk > row) p = 0.f;
      pv[i] = p;
      sum += p;
    }
    pk[g] = pack8(pv);
  }
  return sum;
}

// 32 consecutive 32-bit columns of this thread's TMEM lane, written from registers.
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]),
        "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]),
        "r"(r[30]), "r"(r[31]) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// D += A B with A in tensor memory (rows = lanes, two 16-bit K elements per 32-bit column), B from shared memory.
__device__ __forceinline__ void tc_mma_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}

struct FlashParams {
  int S, Sp, n_heads, rep;        // rep = query heads per key/value head
  bf16* o; int64_t ld_o;          // [T, ld_o]
  float* lse;                     // [B * n_heads * Sp] or NULL
  float* o32;                     // [B * n_heads * Sp, 128] or NULL: the output before rounding, head-major
  float scale_log2e, scale;
  int* status;
};

__global__ void __launch_bounds__(FA_THREADS, 1)
flash_fwd_kernel(const FlashParams P, const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v) {
  extern __shared__ uint8_t fa_smem_raw[];
  const uint32_t raw = smem_u32(fa_smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen_base = fa_smem_raw + (base - raw);
  const uint32_t bars = base + FA_BAR_OFF;
  // barrier slots (8 bytes each)
  auto bar = [&](int i) -> uint32_t { return bars + 8u * (uint32_t)i; };
  enum { B_QFULL = 0, B_KFULL = 1, B_KEMPTY = 3, B_VFULL = 5, B_VEMPTY = 7, B_SFULL = 9, B_SEMPTY = 11, B_PFULL = 13,
         B_OFULL = 15, B_OEMPTY = 17, B_COUNT = 19 };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_base + FA_BAR_OFF + 8 * B_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen_base + FA_BAR_OFF + 8 * B_COUNT + 8);
  int* issued = reinterpret_cast<int*>(gen_base + FA_BAR_OFF + 8 * B_COUNT + 16);   // [5]: q, k0, k1, v0, v1 -> phase + 1
  float* xmax = reinterpret_cast<float*>(gen_base + FA_XMAX_OFF);
  float* xsum = reinterpret_cast<float*>(gen_base + FA_XSUM_OFF);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_qblk = P.Sp / FA_BLK;
  // heavy work first: the last query block of every (sequence, head) has the most key blocks
  const int bh_count = (int)gridDim.x / n_qblk;
  const int qblk = n_qblk - 1 - (int)blockIdx.x / bh_count;
  const int bh = (int)blockIdx.x % bh_count;           // sequence * n_heads + head
  const int n_blk = qblk + 1;
  const int q_row0 = bh * P.Sp + qblk * FA_BLK;
  const int kv_row0 = (bh / P.rep) * P.Sp;             // (sequence * n_kv_heads + head / rep) * S_pad

  if (threadIdx.x == 0) {
    mbar_init(bar(B_QFULL), 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(bar(B_KFULL + s), 1); mbar_init(bar(B_KEMPTY + s), 1);
      mbar_init(bar(B_VFULL + s), 1); mbar_init(bar(B_VEMPTY + s), 1);
      mbar_init(bar(B_SFULL + s), 1); mbar_init(bar(B_SEMPTY + s), 1); mbar_init(bar(B_PFULL + s), 8);
      mbar_init(bar(B_OFULL + s), 1); mbar_init(bar(B_OEMPTY + s), 8);
    }
    for (int i = 0; i < 5; ++i) issued[i] = 0;
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // instruction descriptors: fp32 accumulate, bf16 operands, M = 128, N = 128; V is stored [key, hd] (N contiguous)
  const uint32_t idesc_qk = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(FA_BLK >> 3) << 17) | ((uint32_t)(FA_BLK >> 4) << 24);
  const uint32_t idesc_pv = idesc_qk | (1u << 16);

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      mbar_expect_tx(bar(B_QFULL), 2 * FA_TILE);
      issued[0] = 1;
      for (int kb = 0; kb < 2; ++kb) tma_load_2d(base + FA_Q_OFF + kb * FA_TILE, &map_q, 64 * kb, q_row0, bar(B_QFULL));
      for (int j = 0; j < n_blk; ++j) {
        const int s = j & 1;
        const uint32_t ph = (uint32_t)(j >> 1) & 1u;
        if (!mbar_wait(bar(B_KEMPTY + s), ph ^ 1u, abort_flag, P.status)) break;
        mbar_expect_tx(bar(B_KFULL + s), 2 * FA_TILE);
        issued[1 + s] = (int)ph + 1;
        for (int kb = 0; kb < 2; ++kb)
          tma_load_2d(base + FA_K_OFF + (2 * s + kb) * FA_TILE, &map_k, 64 * kb, kv_row0 + j * FA_BLK, bar(B_KFULL + s));
        if (!mbar_wait(bar(B_VEMPTY + s), ph ^ 1u, abort_flag, P.status)) break;
        mbar_expect_tx(bar(B_VFULL + s), 2 * FA_TILE);
        issued[3 + s] = (int)ph + 1;
        for (int kb = 0; kb < 2; ++kb)        // 64 keys per k-block, two 64-column chunks of hd each
          for (int nj = 0; nj < 2; ++nj)
            tma_load_2d(base + FA_V_OFF + (2 * s + kb) * FA_TILE + nj * 8192, &map_v, 64 * nj,
                        kv_row0 + j * FA_BLK + 64 * kb, bar(B_VFULL + s));
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      bool ok = mbar_wait(bar(B_QFULL), 0u, abort_flag, P.status);
      tc_fence_after();
      auto issue_qk = [&](int j) -> bool {
        const int b = j & 1;
        const uint32_t ph = (uint32_t)(j >> 1) & 1u;
        if (!mbar_wait(bar(B_KFULL + b), ph, abort_flag, P.status)) return false;
        if (!mbar_wait(bar(B_SEMPTY + b), ph ^ 1u, abort_flag, P.status)) return false;
        tc_fence_after();
        const uint32_t d = tmem_base + (uint32_t)(b * FA_BLK);
#pragma unroll
        for (int kb = 0; kb < 2; ++kb) {
          const uint64_t a_desc = make_smem_desc(base + FA_Q_OFF + kb * FA_TILE, 16, 1024);
          const uint64_t b_desc = make_smem_desc(base + FA_K_OFF + (2 * b + kb) * FA_TILE, 16, 1024);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            tc_mma(d, a_desc + (uint64_t)(2 * ks), b_desc + (uint64_t)(2 * ks), idesc_qk, (kb | ks) != 0 ? 1u : 0u);
        }
        tc_commit(bar(B_KEMPTY + b));
        tc_commit(bar(B_SFULL + b));
        return true;
      };
      if (ok) ok = issue_qk(0);
      for (int j = 0; ok && j < n_blk; ++j) {
        if (j + 1 < n_blk && !issue_qk(j + 1)) { ok = false; break; }
        const int b = j & 1;
        const uint32_t ph = (uint32_t)(j >> 1) & 1u;
        if (!mbar_wait(bar(B_VFULL + b), ph, abort_flag, P.status)) { ok = false; break; }
        if (!mbar_wait(bar(B_OEMPTY + b), ph ^ 1u, abort_flag, P.status)) { ok = false; break; }
        if (!mbar_wait(bar(B_PFULL + b), ph, abort_flag, P.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d = tmem_base + (uint32_t)(2 * FA_BLK + b * FA_BLK);
        const uint32_t a_tmem = tmem_base + (uint32_t)(b * FA_BLK);      // P over the first 64 columns of S
#pragma unroll
        for (int kb = 0; kb < 2; ++kb) {
          const uint64_t b_desc = make_smem_desc(base + FA_V_OFF + (2 * b + kb) * FA_TILE, 8192, 1024);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            tc_mma_ta(d, a_tmem + (uint32_t)(8 * (4 * kb + ks)), b_desc + (uint64_t)(128 * ks), idesc_pv, (kb | ks) != 0 ? 1u : 0u);
        }
        tc_commit(bar(B_VEMPTY + b));
        tc_commit(bar(B_OFULL + b));
        tc_commit(bar(B_SEMPTY + b));      // the scores' columns (now holding P) are free again
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax (warps 2..9)
    // Two threads per query row: warps 2..5 take keys (and output columns) 0..63 of a block, warps 6..9
    // take 64..127.  The two halves of a row exchange their maxima through shared memory once per block;
    // every thread passes the named barrier in every iteration, also after an abandoned wait, so that
    // nobody is left waiting at it.
    const int q = warp & 3;                      // TMEM lane quadrant this warp may access
    const int half = (warp - 2) >> 2;
    const int row = q * 32 + lane;               // query row within the block
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(64 * half);
    float acc[64];
#pragma unroll
    for (int i = 0; i < 64; ++i) acc[i] = 0.f;
    float m = -INFINITY, l = 0.f, alpha_pending = 0.f;
    const float cl = P.scale_log2e;
    bool ok = true;
    // acc = acc * alpha + O_j (this thread's 64 columns); the caller has seen O_j complete
    auto add_block = [&](int j, float alpha) {
      const int b = j & 1;
      uint32_t r0[32], r1[32];
      tmem_ld32(lane_addr + (uint32_t)(2 * FA_BLK + b * FA_BLK), r0);
      tmem_ld32(lane_addr + (uint32_t)(2 * FA_BLK + b * FA_BLK + 32), r1);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        acc[i] = acc[i] * alpha + __uint_as_float(r0[i]);
        acc[32 + i] = acc[32 + i] * alpha + __uint_as_float(r1[i]);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_OEMPTY + b));
    };
    auto wait_o = [&](int j) -> bool {           // O_j = P_j V_j complete (P's buffer is free again)
      if (!mbar_wait(bar(B_OFULL + (j & 1)), (uint32_t)(j >> 1) & 1u, abort_flag, P.status)) return false;
      tc_fence_after();
      return true;
    };
    for (int j = 0; j < n_blk; ++j) {
      const int b = j & 1;
      const uint32_t ph = (uint32_t)(j >> 1) & 1u;
      const bool diag = j == qblk;               // keys past the query position exist only in the diagonal block
      uint32_t r0[32], r1[32];
      float mx = -INFINITY;
      if (ok && !mbar_wait(bar(B_SFULL + b), ph, abort_flag, P.status)) ok = false;
      if (ok) {
        tc_fence_after();
        tmem_ld32(lane_addr + (uint32_t)(b * FA_BLK), r0);
        tmem_ld32(lane_addr + (uint32_t)(b * FA_BLK + 32), r1);
        tmem_ld_wait();
        mx = diag ? fa_row_max<true>(r0, r1, 64 * half, row) : fa_row_max<false>(r0, r1, 64 * half, row);
        xmax[(b * 2 + half) * FA_BLK + row] = mx;
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (ok) {
        const float m_new = fmaxf(m, fmaxf(mx, xmax[(b * 2 + (half ^ 1)) * FA_BLK + row]));
        const float alpha = fa_exp2((m - m_new) * cl);        // first block: exp2(-inf) = 0
        const float mc = m_new * cl;
        uint4 pk[8];                             // this thread's 64 probabilities as bf16
        const float sum = diag ? fa_probs<true>(r0, r1, cl, mc, 64 * half, row, pk)
                               : fa_probs<false>(r0, r1, cl, mc, 64 * half, row, pk);
        l = l * alpha + sum;
        m = m_new;
        {
          // P over the scores in tensor memory: this thread's 64 keys are 32 columns of packed pairs.  Both halves
          // of the row have their scores in registers (they met at the barrier above).
          uint32_t pw[32];
#pragma unroll
          for (int g = 0; g < 8; ++g) { pw[4 * g] = pk[g].x; pw[4 * g + 1] = pk[g].y; pw[4 * g + 2] = pk[g].z; pw[4 * g + 3] = pk[g].w; }
          tmem_st32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * FA_BLK + 32 * half), pw);
          tmem_st_wait();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(B_PFULL + b));
          if (j >= 1 && !wait_o(j - 1)) ok = false;
        }
        if (ok) {
          if (j >= 1) add_block(j - 1, alpha_pending);
          alpha_pending = alpha;
        }
      }
    }
    if (ok) ok = wait_o(n_blk - 1);
    if (ok) add_block(n_blk - 1, alpha_pending);
    // the row's denominator is the sum of the two halves' partial sums (both are relative to the same maximum)
    xsum[half * FA_BLK + row] = l;
    asm volatile("bar.sync 1, 256;" ::: "memory");
    l += xsum[(half ^ 1) * FA_BLK + row];
    const int s_pos = qblk * FA_BLK + row;
    if (ok && s_pos < P.S) {
      const float inv = 1.f / l;
      const int seq = bh / P.n_heads, head = bh % P.n_heads;
      bf16* dst = P.o + ((int64_t)seq * P.S + s_pos) * P.ld_o + (int64_t)head * FA_HD + 64 * half;
#pragma unroll
      for (int g = 0; g < 8; ++g) {
        float f[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) f[i] = acc[8 * g + i] * inv;
        *reinterpret_cast<uint4*>(dst + 8 * g) = pack8(f);
      }
      if (P.lse && half == 0) P.lse[(int64_t)bh * P.Sp + s_pos] = m * P.scale + logf(l);
      if (P.o32) {
        float* d32 = P.o32 + ((int64_t)bh * P.Sp + s_pos) * FA_HD + 64 * half;
#pragma unroll
        for (int g = 0; g < 16; ++g)
          *reinterpret_cast<float4*>(d32 + 4 * g) =
              make_float4(acc[4 * g] * inv, acc[4 * g + 1] * inv, acc[4 * g + 2] * inv, acc[4 * g + 3] * inv);
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag && threadIdx.x == 0) {
    // loads already issued into this CTA's shared memory must land before the CTA exits
    const int bidx[5] = {B_QFULL, B_KFULL, B_KFULL + 1, B_VFULL, B_VFULL + 1};
    for (int i = 0; i < 5; ++i) {
      if (issued[i] == 0) continue;
      long long t0 = clock64();
      while (!mbar_try_wait(bar(bidx[i]), (uint32_t)(issued[i] - 1)) && clock64() - t0 < TC_WAIT_CYCLES) {}
    }
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// q: [B * n_heads * Sp, 128], k, v: [B * n_kv_heads * Sp, 128] bf16 head-major; o: [B * S, ld_o] bf16.
inline int launch_flash_fwd(const bf16* q, const bf16* k, const bf16* v, int batch, int n_heads, int n_kv_heads, int S, int Sp,
                            bf16* o, int64_t ld_o, float* lse, float* o32, int* status, cudaStream_t st) {
  TcState& s = tc_state();
  if (!s.ready) return REVFFN_ERR_CUDA;
  if (batch <= 0) return REVFFN_OK;
  static bool attr_set[64] = {false};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return REVFFN_ERR_CUDA;
  if (!attr_set[dev]) {
    if (cudaFuncSetAttribute(flash_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FA_SMEM_BYTES) != cudaSuccess)
      return REVFFN_ERR_CUDA;
    attr_set[dev] = true;
  }
  CUtensorMap mq, mk, mv;
  int r = tc_make_map(&mq, q, FA_HD, (uint64_t)batch * n_heads * Sp, FA_HD, 64, 128);
  if (r) return r;
  r = tc_make_map(&mk, k, FA_HD, (uint64_t)batch * n_kv_heads * Sp, FA_HD, 64, 128);
  if (r) return r;
  r = tc_make_map(&mv, v, FA_HD, (uint64_t)batch * n_kv_heads * Sp, FA_HD, 64, 64);
  if (r) return r;
  FlashParams P;
  P.S = S; P.Sp = Sp; P.n_heads = n_heads; P.rep = n_heads / n_kv_heads;
  P.o = o; P.ld_o = ld_o; P.lse = lse; P.o32 = o32;
  P.scale = 1.f / sqrtf((float)FA_HD);
  P.scale_log2e = P.scale * 1.4426950408889634f;
  P.status = status;
  const int grid = batch * n_heads * (Sp / FA_BLK);
  flash_fwd_kernel<<<grid, FA_THREADS, FA_SMEM_BYTES, st>>>(P, mq, mk, mv);
  return cudaGetLastError() == cudaSuccess ? REVFFN_OK : REVFFN_ERR_CUDA;
}

// ---------------------------------------------------------------------------
// ---------------------------------------------------------------------------
// Backward of the attention core, also without a score matrix in HBM.  P is rebuilt from the row
// log-sum-exp the forward kernel stored:  P = exp(scale * S - lse),  dS = scale * P * (dP - D) with
// D = <dO_row, O_row>.  Two kernels, neither uses atomics:
//   flash_bwd_dkv_kernel  a CTA owns 128 keys of one key/value head and walks the 64-row query tiles at or
//                         below them (of every query head of the group):  dV += P^T dO,  dK += dS^T Q
//   flash_bwd_dq_kernel   a CTA owns 128 query rows of one head and walks the 128-key tiles up to its diagonal:
//                         dQ += dS K
// In both the "own" side is the MMA M side and the walked tile the N side.  dK/dV, per step:
//   S' = K_j Q_t^T,  dP' = V_j dO_t^T   (128 x 64, K = hd)
// into TMEM (double-buffered), eight warps (two threads per key row, 32 query columns each) turn them into P' and
// dS' as bf16 K-major operand tiles in shared memory, and the accumulators (fresh TMEM columns, summed over
// all steps by the tensor core itself) take  dV += P' dO_t  and  dK += dS' Q_t,  where the same shared-memory
// bytes of a walked tile that served as a K-major operand are read again as an MN-major one.
// No cross-thread reduction is needed: the row statistics come from memory.
// ---------------------------------------------------------------------------
// Shared memory of the dK/dV kernel: [K_j, V_j 64 KB | 3 stages of walked tiles 96 KB | P' tile 16 KB | dS' tile
// 16 KB | barriers | row statistics of the stages].  A stage: [Q_t 2 x 8 KB | dO_t 2 x 8 KB].  The walked tiles
// come from L2 with a latency of more than one step, hence the ring of three.
constexpr int FB_X_OFF = 0;
constexpr int FB_STAGE = 2 * FA_TILE;
constexpr int FB_NS = 3;
constexpr int FB_Y_OFF = 4 * FA_TILE;
constexpr int FB_P_OFF = FB_Y_OFF + FB_NS * FB_STAGE;
constexpr int FB_DS_OFF = FB_P_OFF + FA_TILE;
constexpr int FB_BAR_OFF = FB_DS_OFF + FA_TILE;
constexpr int FB_LD_OFF = FB_BAR_OFF + 256;        // (lse * log2 e, D * scale) of a stage's 64 query rows, 512 B per stage
constexpr int FB_SMEM_BYTES = FB_LD_OFF + 2048 + 1024;

struct FlashBwdParams {
  int S, Sp, n_heads, rep;
  const float2* lse_d;            // per query row (head-major index): (lse * log2 e, D * scale)
  const bf16* x0; const bf16* x1; // dQ kernel: its owned operands (q, d_o head-major), read by the CTA's threads themselves
  // Outputs, token-major bf16 [T, ld_out]: a row's head lands at column col + head * 128.  out0: dV (dK/dV kernel, as
  // it is); out1: dK or dQ, with the rotation of the forward pass undone (its transpose), pairs (i, i + 64).
  bf16* out0; bf16* out1;
  int64_t ld_out0, ld_out1;
  int col0, col1;
  int heads_own;                  // heads per sequence on the owned side (key/value heads for dK/dV, query heads for dQ)
  const float2* cs;               // [S, 64] (cos, sin)
  float scale_log2e, scale;
  int* status;
};

// Untiled bulk copy global -> shared (both addresses 16-byte aligned, size a multiple of 16), completing on an mbarrier.
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar) : "memory");
}

// This thread's 32 elements of a step: P' = exp2(s * cl - lse2), dS' = P' * (dP * scale - D * scale), packed to bf16.
// The row statistics belong to the query: the column's (DKV, read from shared memory) or this thread's own row's.
// MASK: the tile touches the causal diagonal or the end of the sequence and every element is tested.
template <bool DKV, bool MASK>
__device__ __forceinline__ void fb_tile(const uint32_t (&rs)[32], const uint32_t (&rd)[32], const float4* __restrict__ ld_cols,
                                        float2 own_ld, float cl, float scale, int col0, int own_pos, int S, uint4 (&pp)[4],
                                        uint4 (&pd)[4]) {
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    float pv[8], dv[8];
#pragma unroll
    for (int i = 0; i < 8; i += 2) {
      float4 ld = make_float4(own_ld.x, own_ld.y, own_ld.x, own_ld.y);
      if (DKV) ld = ld_cols[(8 * g + i) >> 1];          // two columns' (lse2, D * scale)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int c = 8 * g + i + e;
        const float l2 = e ? ld.z : ld.x, dsc = e ? ld.w : ld.y;
        float p = fa_exp2(__uint_as_float(rs[c]) * cl - l2);
        float ds = p * fmaf(__uint_as_float(rd[c]), scale, -dsc);
        if (MASK) {
          // DKV: own row = key, column = query (needs query >= key, query inside the sequence); else the roles swap
          const bool valid = DKV ? (col0 + c >= own_pos && col0 + c < S) : (col0 + c <= own_pos && own_pos < S);
          if (!valid) { p = 0.f; ds = 0.f; }
        }
        pv[i + e] = p;
        dv[i + e] = ds;
      }
    }
    if (DKV) pp[g] = pack8(pv);
    pd[g] = pack8(dv);
  }
}

__global__ void __launch_bounds__(FA_THREADS, 1)
flash_bwd_dkv_kernel(const FlashBwdParams P, const __grid_constant__ CUtensorMap map_x0, const __grid_constant__ CUtensorMap map_x1,
                 const __grid_constant__ CUtensorMap map_y0, const __grid_constant__ CUtensorMap map_y1) {
  extern __shared__ uint8_t fa_smem_raw[];
  const uint32_t raw = smem_u32(fa_smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen_base = fa_smem_raw + (base - raw);
  const uint32_t bars = base + FB_BAR_OFF;
  auto bar = [&](int i) -> uint32_t { return bars + 8u * (uint32_t)i; };
  constexpr int NS = FB_NS;
  constexpr int Y_OFF = FB_Y_OFF;
  constexpr bool DKV = true;      // the element routine is shared with the dQ kernel and takes the role as a parameter
  enum { B_XFULL = 0, B_YFULL = 1, B_YEMPTY = 1 + FB_NS, B_SDFULL = 1 + 2 * FB_NS, B_SDEMPTY = B_SDFULL + 2,
         B_PDFULL = B_SDEMPTY + 2, B_PDEMPTY = B_PDFULL + 1, B_ACCFULL = B_PDEMPTY + 1, B_COUNT = B_ACCFULL + 1 };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_base + FB_BAR_OFF + 8 * B_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen_base + FB_BAR_OFF + 8 * B_COUNT + 8);
  int* issued = reinterpret_cast<int*>(gen_base + FB_BAR_OFF + 8 * B_COUNT + 16);   // [1 + NS]: x, y stages -> phase + 1

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_blk = P.Sp / FA_BLK;                  // 128-row blocks per head
  const int n_t64 = P.Sp / 64;                      // 64-row tiles per head
  // heavy work first: low key blocks see the most query tiles
  const int per = (int)gridDim.x / n_blk;
  const int blk = (int)blockIdx.x / per;            // own 128-key block within the head
  const int grp = (int)blockIdx.x % per;            // sequence * n_kv_heads + kv head
  const int own_row0 = grp * P.Sp + blk * FA_BLK;
  const int t_begin = 2 * blk;
  const int n_inner = n_t64 - 2 * blk;
  const int n_steps = P.rep * n_inner;              // every query head of the group in turn
  const int y_base = grp * P.rep * P.Sp;            // first row of the group's first query head
  auto y_row_of = [&](int s) -> int { return y_base + (s / n_inner) * P.Sp + 64 * (t_begin + s % n_inner); };

  if (threadIdx.x == 0) {
    mbar_init(bar(B_XFULL), 1);
    mbar_init(bar(B_ACCFULL), 1);
    mbar_init(bar(B_PDFULL), 8);
    mbar_init(bar(B_PDEMPTY), 1);
    for (int s = 0; s < NS; ++s) { mbar_init(bar(B_YFULL + s), 1); mbar_init(bar(B_YEMPTY + s), 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(bar(B_SDFULL + s), 1); mbar_init(bar(B_SDEMPTY + s), 8); }
    for (int i = 0; i < 1 + NS; ++i) issued[i] = 0;
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // TMEM columns: step buffer b: S' at 128 b, dP' at 128 b + 64; acc0 at 256, acc1 at 384
  const uint32_t idesc_sd = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(64 >> 3) << 17) | ((uint32_t)(FA_BLK >> 4) << 24);
  const uint32_t idesc_acc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(FA_HD >> 3) << 17) |
                             ((uint32_t)(FA_BLK >> 4) << 24);

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      mbar_expect_tx(bar(B_XFULL), 4 * FA_TILE);
      issued[0] = 1;
      for (int kb = 0; kb < 2; ++kb) {
        tma_load_2d(base + FB_X_OFF + kb * FA_TILE, &map_x0, 64 * kb, own_row0, bar(B_XFULL));
        tma_load_2d(base + FB_X_OFF + (2 + kb) * FA_TILE, &map_x1, 64 * kb, own_row0, bar(B_XFULL));
      }
      for (int s = 0; s < n_steps; ++s) {
        const int st = s % NS;
        const uint32_t ph = (uint32_t)(s / NS) & 1u;
        if (!mbar_wait(bar(B_YEMPTY + st), ph ^ 1u, abort_flag, P.status)) break;
        mbar_expect_tx(bar(B_YFULL + st), FB_STAGE + 512);
        issued[1 + st] = (int)ph + 1;
        const int yr = y_row_of(s);
        bulk_load_1d(base + FB_LD_OFF + st * 512, P.lse_d + yr, 512, bar(B_YFULL + st));
        const uint32_t ys = base + Y_OFF + st * FB_STAGE;
        for (int kb = 0; kb < 2; ++kb) {
          tma_load_2d(ys + kb * 8192, &map_y0, 64 * kb, yr, bar(B_YFULL + st));
          tma_load_2d(ys + FA_TILE + kb * 8192, &map_y1, 64 * kb, yr, bar(B_YFULL + st));
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      bool ok = mbar_wait(bar(B_XFULL), 0u, abort_flag, P.status);
      tc_fence_after();
      auto issue_sd = [&](int s) -> bool {
        const int b = s & 1, st = s % NS;
        const uint32_t ph = (uint32_t)(s >> 1) & 1u;
        if (!mbar_wait(bar(B_YFULL + st), (uint32_t)(s / NS) & 1u, abort_flag, P.status)) return false;
        if (!mbar_wait(bar(B_SDEMPTY + b), ph ^ 1u, abort_flag, P.status)) return false;
        tc_fence_after();
        const uint32_t ys = base + Y_OFF + st * FB_STAGE;
#pragma unroll
        for (int w = 0; w < 2; ++w) {            // w = 0: S' = X0 Y0^T, w = 1: dP' = X1 Y1^T
          const uint32_t d = tmem_base + (uint32_t)(b * 128 + w * 64);
#pragma unroll
          for (int kb = 0; kb < 2; ++kb) {
            const uint64_t a_desc = make_smem_desc(base + FB_X_OFF + (2 * w + kb) * FA_TILE, 16, 1024);
            const uint64_t b_desc = make_smem_desc(ys + w * FA_TILE + kb * 8192, 16, 1024);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
              tc_mma(d, a_desc + (uint64_t)(2 * ks), b_desc + (uint64_t)(2 * ks), idesc_sd, (kb | ks) != 0 ? 1u : 0u);
          }
        }
        tc_commit(bar(B_SDFULL + b));
        return true;
      };
      if (ok) ok = issue_sd(0);
      for (int s = 0; ok && s < n_steps; ++s) {
        if (s + 1 < n_steps && !issue_sd(s + 1)) { ok = false; break; }
        const int st = s % NS;
        if (!mbar_wait(bar(B_PDFULL), (uint32_t)s & 1u, abort_flag, P.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t ys = base + Y_OFF + st * FB_STAGE;
        // the walked tiles again, now as [64 rows (K), 128 columns (N)] operands: the two 64-column halves are 8 KB apart
        {
          const uint64_t a_desc = make_smem_desc(base + FB_P_OFF, 16, 1024);
          const uint64_t b_desc = make_smem_desc(ys + FA_TILE, 8192, 1024);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            tc_mma(tmem_base + 256u, a_desc + (uint64_t)(2 * ks), b_desc + (uint64_t)(128 * ks), idesc_acc, (s | ks) != 0 ? 1u : 0u);
        }
        {
          const uint64_t a_desc = make_smem_desc(base + FB_DS_OFF, 16, 1024);
          const uint64_t b_desc = make_smem_desc(ys, 8192, 1024);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            tc_mma(tmem_base + 384u, a_desc + (uint64_t)(2 * ks), b_desc + (uint64_t)(128 * ks), idesc_acc, (s | ks) != 0 ? 1u : 0u);
        }
        tc_commit(bar(B_YEMPTY + st));
        tc_commit(bar(B_PDEMPTY));
      }
      if (ok) tc_commit(bar(B_ACCFULL));
    }
  } else {
    // ------------------------------------------------------------------ P' / dS' (warps 2..9)
    const int q = warp & 3;                      // TMEM lane quadrant this warp may access
    const int hh = (warp - 2) >> 2;              // which 32 of the step's 64 columns
    const int row = q * 32 + lane;               // own row within the block
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
    const float cl = P.scale_log2e, scale = P.scale;
    const int own_pos = blk * FA_BLK + row;      // position in the sequence of this thread's own row
    const float2 own_ld = make_float2(0.f, 0.f);      // unused by the key-row role
    bool ok = true;
    for (int s = 0; s < n_steps; ++s) {
      const int b = s & 1;
      const uint32_t ph = (uint32_t)(s >> 1) & 1u;
      if (!mbar_wait(bar(B_SDFULL + b), ph, abort_flag, P.status)) { ok = false; break; }
      // this thread reads the stage's row statistics itself, so it observes the stage's barrier itself
      if (!mbar_wait(bar(B_YFULL + s % NS), (uint32_t)(s / NS) & 1u, abort_flag, P.status)) { ok = false; break; }
      tc_fence_after();
      uint32_t rs[32], rd[32];
      tmem_ld32(lane_addr + (uint32_t)(b * 128 + 32 * hh), rs);
      tmem_ld32(lane_addr + (uint32_t)(b * 128 + 64 + 32 * hh), rd);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_SDEMPTY + b));
      const int t = t_begin + s % n_inner;
      const int col0 = 64 * t + 32 * hh;         // position in the sequence of this thread's first column
      // tiles that touch the diagonal or the end of the sequence need the element-wise test
      const bool mask = t < 2 * blk + 2 || 64 * t + 63 >= P.S;
      // the step's row statistics came with the walked tiles
      const float4* ld_cols = reinterpret_cast<const float4*>(gen_base + FB_LD_OFF + (s % NS) * 512) + 16 * hh;
      uint4 pp[4], pd[4];
      if (mask) fb_tile<DKV, true>(rs, rd, ld_cols, own_ld, cl, scale, col0, own_pos, P.S, pp, pd);
      else fb_tile<DKV, false>(rs, rd, ld_cols, own_ld, cl, scale, col0, own_pos, P.S, pp, pd);
      // the operand tiles have one buffer: the previous step's accumulating products must have read them
      if (!mbar_wait(bar(B_PDEMPTY), ((uint32_t)s & 1u) ^ 1u, abort_flag, P.status)) { ok = false; break; }
      uint8_t* prow = gen_base + FB_P_OFF + row * 128;
      uint8_t* drow = gen_base + FB_DS_OFF + row * 128;
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const int piece = ((4 * hh + g) ^ (row & 7)) << 4;
        *reinterpret_cast<uint4*>(prow + piece) = pp[g];
        *reinterpret_cast<uint4*>(drow + piece) = pd[g];
      }
      fence_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_PDFULL));
    }
    if (ok && !mbar_wait(bar(B_ACCFULL), 0u, abort_flag, P.status)) ok = false;
    if (ok) {
      tc_fence_after();
      // This thread takes columns [32 hh, +32) and their rotation partners [64 + 32 hh, +32) of its row.  The
      // tensor-memory loads are warp-wide instructions: every lane executes them, rows past the sequence only
      // skip the stores.
      const bool row_ok = own_pos < P.S;
      const int seq = grp / P.heads_own, head = grp % P.heads_own;
      const int64_t tok = (int64_t)seq * P.S + (row_ok ? own_pos : 0);
      {
#pragma unroll
        for (int a = 0; a < 2; ++a) {          // a = 0: dV as it is, a = 1: dK with the rotation undone
          uint32_t rl[32], rh[32];
          __syncwarp();               // lanes that skipped the previous output rejoin before the warp-wide loads
          tmem_ld32(lane_addr + (uint32_t)(256 + 128 * a + 32 * hh), rl);
          tmem_ld32(lane_addr + (uint32_t)(256 + 128 * a + 64 + 32 * hh), rh);
          tmem_ld_wait();
          if (!row_ok) continue;
          float y0[32], y1[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) { y0[i] = __uint_as_float(rl[i]); y1[i] = __uint_as_float(rh[i]); }
          if (a == 1) {
            const float4* cs2 = reinterpret_cast<const float4*>(P.cs + own_pos * 64 + 32 * hh);
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float4 cs = cs2[i];
              const float a0 = y0[2 * i], b0 = y1[2 * i], a1 = y0[2 * i + 1], b1 = y1[2 * i + 1];
              y0[2 * i] = a0 * cs.x + b0 * cs.y;         y1[2 * i] = b0 * cs.x - a0 * cs.y;
              y0[2 * i + 1] = a1 * cs.z + b1 * cs.w;     y1[2 * i + 1] = b1 * cs.z - a1 * cs.w;
            }
          }
          bf16* dst = (a == 0 ? P.out0 + tok * P.ld_out0 + P.col0 : P.out1 + tok * P.ld_out1 + P.col1) + head * FA_HD + 32 * hh;
          store32_bf16(dst, y0);
          store32_bf16(dst + 64, y1);
        }
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag && threadIdx.x == 0) {
    for (int i = 0; i < 1 + NS; ++i) {      // slot 0: the owned operands, slot 1 + st: stage st of the walked tiles
      if (issued[i] == 0) continue;
      long long t0 = clock64();
      while (!mbar_try_wait(bar(i == 0 ? B_XFULL : B_YFULL + i - 1), (uint32_t)(issued[i] - 1)) && clock64() - t0 < TC_WAIT_CYCLES) {}
    }
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ---------------------------------------------------------------------------
// dQ with 128-key walked tiles.  The 128 x 64 x 16 instructions of the kernel above run at 55 clk against 32 at
// full rate; the dQ launch has the tensor memory for the 128-wide shape: its owned operands (Q_i, dO_i) sit in
// tensor memory as A operands (128 columns), S' and dP' take 128 columns each (one buffer: the softmax warps free
// it once the scores are in registers) and dQ the last 128.  Shared memory: three 64 KB stages of [K_t | V_t] and
// the dS' operand tile.
// ---------------------------------------------------------------------------
constexpr int FQ_NS = 3;
constexpr int FQ_STAGE = 4 * FA_TILE;
constexpr int FQ_DS_OFF = FQ_NS * FQ_STAGE;
constexpr int FQ_BAR_OFF = FQ_DS_OFF + 2 * FA_TILE;
constexpr int FQ_SMEM_BYTES = FQ_BAR_OFF + 256 + 1024;

__global__ void __launch_bounds__(FA_THREADS, 1)
flash_bwd_dq_kernel(const FlashBwdParams P, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v) {
  extern __shared__ uint8_t fa_smem_raw[];
  const uint32_t raw = smem_u32(fa_smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen_base = fa_smem_raw + (base - raw);
  const uint32_t bars = base + FQ_BAR_OFF;
  auto bar = [&](int i) -> uint32_t { return bars + 8u * (uint32_t)i; };
  enum { B_XFULL = 0, B_YFULL = 1, B_YEMPTY = 1 + FQ_NS, B_SDFULL = 1 + 2 * FQ_NS, B_SDEMPTY, B_PDFULL, B_PDEMPTY, B_ACCFULL, B_COUNT };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_base + FQ_BAR_OFF + 8 * B_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen_base + FQ_BAR_OFF + 8 * B_COUNT + 8);
  int* issued = reinterpret_cast<int*>(gen_base + FQ_BAR_OFF + 8 * B_COUNT + 16);   // [FQ_NS]: stage -> phase + 1

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_blk = P.Sp / FA_BLK;
  const int per = (int)gridDim.x / n_blk;
  const int blk = n_blk - 1 - (int)blockIdx.x / per;     // heavy work first: high query blocks see the most key tiles
  const int grp = (int)blockIdx.x % per;                 // sequence * n_heads + head
  const int own_row0 = grp * P.Sp + blk * FA_BLK;
  const int n_steps = blk + 1;                           // key tiles 0 .. the diagonal one
  const int kv_row0 = (grp / P.rep) * P.Sp;

  if (threadIdx.x == 0) {
    mbar_init(bar(B_XFULL), 8);
    mbar_init(bar(B_SDFULL), 1); mbar_init(bar(B_SDEMPTY), 8);
    mbar_init(bar(B_PDFULL), 8); mbar_init(bar(B_PDEMPTY), 1);
    mbar_init(bar(B_ACCFULL), 1);
    for (int s = 0; s < FQ_NS; ++s) { mbar_init(bar(B_YFULL + s), 1); mbar_init(bar(B_YEMPTY + s), 1); issued[s] = 0; }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // TMEM columns: S' 0..127, dP' 128..255, Q_i 256..319, dO_i 320..383 (packed pairs), dQ 384..511
  const uint32_t idesc_sd = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(FA_BLK >> 3) << 17) | ((uint32_t)(FA_BLK >> 4) << 24);
  const uint32_t idesc_acc = idesc_sd | (1u << 16);

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      for (int s = 0; s < n_steps; ++s) {
        const int st = s % FQ_NS;
        const uint32_t ph = (uint32_t)(s / FQ_NS) & 1u;
        if (!mbar_wait(bar(B_YEMPTY + st), ph ^ 1u, abort_flag, P.status)) break;
        mbar_expect_tx(bar(B_YFULL + st), FQ_STAGE);
        issued[st] = (int)ph + 1;
        const int yr = kv_row0 + s * FA_BLK;
        const uint32_t ys = base + st * FQ_STAGE;
        for (int kb = 0; kb < 2; ++kb) {
          tma_load_2d(ys + kb * FA_TILE, &map_k, 64 * kb, yr, bar(B_YFULL + st));
          tma_load_2d(ys + (2 + kb) * FA_TILE, &map_v, 64 * kb, yr, bar(B_YFULL + st));
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      bool ok = mbar_wait(bar(B_XFULL), 0u, abort_flag, P.status);
      tc_fence_after();
      auto issue_sd = [&](int s) -> bool {
        const int st = s % FQ_NS;
        if (!mbar_wait(bar(B_YFULL + st), (uint32_t)(s / FQ_NS) & 1u, abort_flag, P.status)) return false;
        if (!mbar_wait(bar(B_SDEMPTY), ((uint32_t)s & 1u) ^ 1u, abort_flag, P.status)) return false;
        tc_fence_after();
        const uint32_t ys = base + st * FQ_STAGE;
#pragma unroll
        for (int w = 0; w < 2; ++w) {            // w = 0: S' = Q_i K_t^T, w = 1: dP' = dO_i V_t^T
#pragma unroll
          for (int kb = 0; kb < 2; ++kb) {
            const uint64_t b_desc = make_smem_desc(ys + (2 * w + kb) * FA_TILE, 16, 1024);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
              tc_mma_ta(tmem_base + (uint32_t)(128 * w), tmem_base + (uint32_t)(256 + 64 * w + 8 * (4 * kb + ks)),
                        b_desc + (uint64_t)(2 * ks), idesc_sd, (kb | ks) != 0 ? 1u : 0u);
          }
        }
        tc_commit(bar(B_SDFULL));
        return true;
      };
      if (ok) ok = issue_sd(0);
      for (int s = 0; ok && s < n_steps; ++s) {
        if (s + 1 < n_steps && !issue_sd(s + 1)) { ok = false; break; }
        const int st = s % FQ_NS;
        if (!mbar_wait(bar(B_PDFULL), (uint32_t)s & 1u, abort_flag, P.status)) { ok = false; break; }
        tc_fence_after();
        // dQ += dS' K_t: K_t's two 64-column tiles read as one [128 keys, 128 columns] operand, halves 16 KB apart
        const uint64_t b_desc = make_smem_desc(base + st * FQ_STAGE, 2 * 8192, 1024);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint64_t a_desc = make_smem_desc(base + FQ_DS_OFF + (kk >> 2) * FA_TILE, 16, 1024);
          tc_mma(tmem_base + 384u, a_desc + (uint64_t)(2 * (kk & 3)), b_desc + (uint64_t)(128 * kk), idesc_acc, (s | kk) != 0 ? 1u : 0u);
        }
        tc_commit(bar(B_YEMPTY + st));
        tc_commit(bar(B_PDEMPTY));
      }
      if (ok) tc_commit(bar(B_ACCFULL));
    }
  } else {
    // ------------------------------------------------------------------ dS' (warps 2..9)
    const int q = warp & 3;
    const int hh = (warp - 2) >> 2;              // which 64 of the tile's 128 keys
    const int row = q * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
    const float cl = P.scale_log2e, scale = P.scale;
    const int own_pos = blk * FA_BLK + row;
    float2 own_ld = make_float2(0.f, 0.f);
    if (own_pos < P.S) own_ld = P.lse_d[own_row0 + row];
    __syncwarp();
    // the owned operands into tensor memory: this thread's 64 columns of its row of Q_i and of dO_i
#pragma unroll
    for (int w = 0; w < 2; ++w) {
      const uint4* src = reinterpret_cast<const uint4*>((w ? P.x1 : P.x0) + (int64_t)(own_row0 + row) * FA_HD + 64 * hh);
      uint32_t xw[32];
#pragma unroll
      for (int g = 0; g < 8; ++g) {
        const uint4 v = __ldg(src + g);
        xw[4 * g] = v.x; xw[4 * g + 1] = v.y; xw[4 * g + 2] = v.z; xw[4 * g + 3] = v.w;
      }
      tmem_st32(lane_addr + (uint32_t)(256 + 64 * w + 32 * hh), xw);
    }
    tmem_st_wait();
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(bar(B_XFULL));
    bool ok = true;
    const bool edge = blk * FA_BLK + FA_BLK - 1 >= P.S;
    for (int s = 0; s < n_steps; ++s) {
      if (!mbar_wait(bar(B_SDFULL), (uint32_t)s & 1u, abort_flag, P.status)) { ok = false; break; }
      __syncwarp();
      tc_fence_after();
      const bool mask = s == blk || edge;
      const int col0 = FA_BLK * s + 64 * hh;     // position in the sequence of this thread's first key
      uint32_t rs[32], rd[32];
      uint4 pp[4], pa[4], pb[4];
      tmem_ld32(lane_addr + (uint32_t)(64 * hh), rs);
      tmem_ld32(lane_addr + (uint32_t)(128 + 64 * hh), rd);
      tmem_ld_wait();
      if (mask) fb_tile<false, true>(rs, rd, nullptr, own_ld, cl, scale, col0, own_pos, P.S, pp, pa);
      else fb_tile<false, false>(rs, rd, nullptr, own_ld, cl, scale, col0, own_pos, P.S, pp, pa);
      __syncwarp();
      tmem_ld32(lane_addr + (uint32_t)(64 * hh + 32), rs);
      tmem_ld32(lane_addr + (uint32_t)(128 + 64 * hh + 32), rd);
      tmem_ld_wait();
      // every score of the step is in registers: the buffer may take the next tile's
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_SDEMPTY));
      if (mask) fb_tile<false, true>(rs, rd, nullptr, own_ld, cl, scale, col0 + 32, own_pos, P.S, pp, pb);
      else fb_tile<false, false>(rs, rd, nullptr, own_ld, cl, scale, col0 + 32, own_pos, P.S, pp, pb);
      // the operand tile has one buffer: the previous step's accumulating product must have read it
      if (!mbar_wait(bar(B_PDEMPTY), ((uint32_t)s & 1u) ^ 1u, abort_flag, P.status)) { ok = false; break; }
      uint8_t* drow = gen_base + FQ_DS_OFF + hh * FA_TILE + row * 128;      // this thread's 64 keys are tile hh
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        *reinterpret_cast<uint4*>(drow + ((g ^ (row & 7)) << 4)) = pa[g];
        *reinterpret_cast<uint4*>(drow + (((4 + g) ^ (row & 7)) << 4)) = pb[g];
      }
      fence_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_PDFULL));
    }
    if (ok && !mbar_wait(bar(B_ACCFULL), 0u, abort_flag, P.status)) ok = false;
    if (ok) {
      tc_fence_after();
      // columns [32 hh, +32) and their rotation partners [64 + 32 hh, +32); every lane executes the warp-wide loads
      const bool row_ok = own_pos < P.S;
      const int seq = grp / P.heads_own, head = grp % P.heads_own;
      const int64_t tok = (int64_t)seq * P.S + (row_ok ? own_pos : 0);
      uint32_t rl[32], rh[32];
      __syncwarp();
      tmem_ld32(lane_addr + (uint32_t)(384 + 32 * hh), rl);
      tmem_ld32(lane_addr + (uint32_t)(384 + 64 + 32 * hh), rh);
      tmem_ld_wait();
      if (row_ok) {
        float y0[32], y1[32];
        const float4* cs2 = reinterpret_cast<const float4*>(P.cs + own_pos * 64 + 32 * hh);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const float4 cs = cs2[i];
          const float a0 = __uint_as_float(rl[2 * i]), b0 = __uint_as_float(rh[2 * i]);
          const float a1 = __uint_as_float(rl[2 * i + 1]), b1 = __uint_as_float(rh[2 * i + 1]);
          y0[2 * i] = a0 * cs.x + b0 * cs.y;         y1[2 * i] = b0 * cs.x - a0 * cs.y;
          y0[2 * i + 1] = a1 * cs.z + b1 * cs.w;     y1[2 * i + 1] = b1 * cs.z - a1 * cs.w;
        }
        bf16* dst = P.out1 + tok * P.ld_out1 + P.col1 + head * FA_HD + 32 * hh;
        store32_bf16(dst, y0);
        store32_bf16(dst + 64, y1);
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag && threadIdx.x == 0) {
    for (int i = 0; i < FQ_NS; ++i) {
      if (issued[i] == 0) continue;
      long long t0 = clock64();
      while (!mbar_try_wait(bar(B_YFULL + i), (uint32_t)(issued[i] - 1)) && clock64() - t0 < TC_WAIT_CYCLES) {}
    }
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// (lse * log2 e, scale * <dO_row, O_row>) per query row; one warp per head-major row.  O is taken before its rounding to
// bf16: D stands for sum_j P_j dP_j, and with a peaked row dP - D cancels, so an error in D would show in dS.
__global__ void attn_rowdot_kernel(const float* __restrict__ o32, const bf16* __restrict__ d_o, const float* __restrict__ lse,
                                   int S, int Sp, int64_t rows, float scale, float2* __restrict__ lse_d) {
  const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (row >= rows || (int)(row % Sp) >= S) return;
  const float4 a = *reinterpret_cast<const float4*>(o32 + row * FA_HD + 4 * lane);
  const uint2 b = *reinterpret_cast<const uint2*>(d_o + row * FA_HD + 4 * lane);
  const __nv_bfloat162* bh = reinterpret_cast<const __nv_bfloat162*>(&b);
  const float2 y0 = __bfloat1622float2(bh[0]), y1 = __bfloat1622float2(bh[1]);
  float dot = a.x * y0.x + a.y * y0.y + a.z * y1.x + a.w * y1.y;
  dot = warp_sum(dot);
  if (lane == 0) lse_d[row] = make_float2(lse[row] * 1.4426950408889634f, dot * scale);
}

// q, d_o: [B * n_heads * Sp, 128]; k, v: [B * n_kv_heads * Sp, 128] bf16 head-major (rows past the sequence zero).
// Outputs token-major bf16, rotation undone: dq [T, ld_dq]; dk at column 0 and dv at column dv_col of dkv [T, ld_dkv].
inline int launch_flash_bwd(const bf16* q, const bf16* k, const bf16* v, const bf16* d_o, const float2* lse_d, const float2* cs,
                            int batch, int n_heads, int n_kv_heads, int S, int Sp, bf16* dq, int64_t ld_dq, bf16* dkv,
                            int64_t ld_dkv, int dv_col, int* status, cudaStream_t st) {
  TcState& s = tc_state();
  if (!s.ready) return REVFFN_ERR_CUDA;
  if (batch <= 0) return REVFFN_OK;
  static bool attr_set[64] = {false};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return REVFFN_ERR_CUDA;
  if (!attr_set[dev]) {
    if (cudaFuncSetAttribute(flash_bwd_dkv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FB_SMEM_BYTES) != cudaSuccess ||
        cudaFuncSetAttribute(flash_bwd_dq_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FQ_SMEM_BYTES) != cudaSuccess)
      return REVFFN_ERR_CUDA;
    attr_set[dev] = true;
  }
  const uint64_t q_rows = (uint64_t)batch * n_heads * Sp, kv_rows = (uint64_t)batch * n_kv_heads * Sp;
  CUtensorMap q128, do128, k128, v128, q64, do64, k64, v64;
  int r = 0;
  if (!r) r = tc_make_map(&q128, q, FA_HD, q_rows, FA_HD, 64, 128);
  if (!r) r = tc_make_map(&do128, d_o, FA_HD, q_rows, FA_HD, 64, 128);
  if (!r) r = tc_make_map(&k128, k, FA_HD, kv_rows, FA_HD, 64, 128);
  if (!r) r = tc_make_map(&v128, v, FA_HD, kv_rows, FA_HD, 64, 128);
  if (!r) r = tc_make_map(&q64, q, FA_HD, q_rows, FA_HD, 64, 64);
  if (!r) r = tc_make_map(&do64, d_o, FA_HD, q_rows, FA_HD, 64, 64);
  if (!r) r = tc_make_map(&k64, k, FA_HD, kv_rows, FA_HD, 64, 64);
  if (!r) r = tc_make_map(&v64, v, FA_HD, kv_rows, FA_HD, 64, 64);
  if (r) return r;
  FlashBwdParams P;
  P.S = S; P.Sp = Sp; P.n_heads = n_heads; P.rep = n_heads / n_kv_heads;
  P.lse_d = lse_d;
  P.scale = 1.f / sqrtf((float)FA_HD);
  P.scale_log2e = P.scale * 1.4426950408889634f;
  P.status = status;
  P.cs = cs;
  P.out0 = dkv; P.ld_out0 = ld_dkv; P.col0 = dv_col;
  P.out1 = dkv; P.ld_out1 = ld_dkv; P.col1 = 0;
  P.heads_own = n_kv_heads;
  P.x0 = nullptr; P.x1 = nullptr;
  flash_bwd_dkv_kernel<<<batch * n_kv_heads * (Sp / FA_BLK), FA_THREADS, FB_SMEM_BYTES, st>>>(P, k128, v128, q64, do64);
  if (cudaGetLastError() != cudaSuccess) return REVFFN_ERR_CUDA;
  P.out0 = nullptr; P.ld_out0 = 0; P.col0 = 0;
  P.out1 = dq; P.ld_out1 = ld_dq; P.col1 = 0;
  P.heads_own = n_heads;
  P.x0 = q; P.x1 = d_o;
  flash_bwd_dq_kernel<<<batch * n_heads * (Sp / FA_BLK), FA_THREADS, FQ_SMEM_BYTES, st>>>(P, k128, v128);
  return cudaGetLastError() == cudaSuccess ? REVFFN_OK : REVFFN_ERR_CUDA;
}

}  // namespace revffn
