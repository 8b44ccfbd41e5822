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
//               the next scores while the softmax warps work on the current ones.
//   warps 2..9  softmax: two threads per query row (= TMEM lane), 64 keys each.  Per block: the scores
//               into registers, row maximum (the halves exchange theirs through shared memory),
//               p = exp2((s - m) * scale * log2 e), P as bf16 into shared memory in the K-major
//               128-byte-swizzled operand layout (one buffer: written once the previous block's
//               P V product has read it), then the PREVIOUS block's O_j (this thread's 64 columns) is
//               added into a register accumulator,
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
constexpr int FA_P_OFF = FA_V_OFF + 4 * FA_TILE;  // P: 2 tiles
constexpr int FA_BAR_OFF = FA_P_OFF + 2 * FA_TILE;
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

struct FlashParams {
  int S, Sp, n_heads, rep;        // rep = query heads per key/value head
  bf16* o; int64_t ld_o;          // [T, ld_o]
  float* lse;                     // [B * n_heads * Sp] or NULL
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
         B_OFULL = 14, B_OEMPTY = 16, B_COUNT = 18 };
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
    mbar_init(bar(B_PFULL), 8);
    for (int s = 0; s < 2; ++s) {
      mbar_init(bar(B_KFULL + s), 1); mbar_init(bar(B_KEMPTY + s), 1);
      mbar_init(bar(B_VFULL + s), 1); mbar_init(bar(B_VEMPTY + s), 1);
      mbar_init(bar(B_SFULL + s), 1); mbar_init(bar(B_SEMPTY + s), 8);
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
        if (!mbar_wait(bar(B_PFULL), (uint32_t)j & 1u, abort_flag, P.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d = tmem_base + (uint32_t)(2 * FA_BLK + b * FA_BLK);
#pragma unroll
        for (int kb = 0; kb < 2; ++kb) {
          const uint64_t a_desc = make_smem_desc(base + FA_P_OFF + kb * FA_TILE, 16, 1024);
          const uint64_t b_desc = make_smem_desc(base + FA_V_OFF + (2 * b + kb) * FA_TILE, 8192, 1024);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            tc_mma(d, a_desc + (uint64_t)(2 * ks), b_desc + (uint64_t)(128 * ks), idesc_pv, (kb | ks) != 0 ? 1u : 0u);
        }
        tc_commit(bar(B_VEMPTY + b));
        tc_commit(bar(B_OFULL + b));
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
        // scores are in registers: the accumulator may be overwritten by the block after next
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(B_SEMPTY + b));
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
        // P has one buffer: the previous block's P V product must have read it
        if (j >= 1 && !wait_o(j - 1)) ok = false;
        if (ok) {
          // this thread's 64 keys are exactly tile `half` of P (64 keys per tile): eight 16-byte pieces of its row
          uint8_t* tile_row = gen_base + FA_P_OFF + half * FA_TILE + row * 128;
#pragma unroll
          for (int g = 0; g < 8; ++g) *reinterpret_cast<uint4*>(tile_row + ((g ^ (row & 7)) << 4)) = pk[g];
          fence_async_smem();                    // P visible to the tensor core's reads
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(B_PFULL));
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
                            bf16* o, int64_t ld_o, float* lse, int* status, cudaStream_t st) {
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
  P.o = o; P.ld_o = ld_o; P.lse = lse;
  P.scale = 1.f / sqrtf((float)FA_HD);
  P.scale_log2e = P.scale * 1.4426950408889634f;
  P.status = status;
  const int grid = batch * n_heads * (Sp / FA_BLK);
  flash_fwd_kernel<<<grid, FA_THREADS, FA_SMEM_BYTES, st>>>(P, mq, mk, mv);
  return cudaGetLastError() == cudaSuccess ? REVFFN_OK : REVFFN_ERR_CUDA;
}

}  // namespace revffn
