// tcgen05 / TMEM / TMA back end for every bf16 matrix product on the path.
//
// One persistent, warp-specialised kernel (1 CTA per SM, 352 threads):
//   warps 0, 10 TMA producers: cp.async.bulk.tensor loads (128-byte swizzle) of
//               A and B tiles into a ring of shared-memory stages, completion on
//               mbarriers (no multicast LOADS anywhere: every CTA fetches its own operands; the only
//               cluster-wide instruction is the pair mode's tcgen05.commit, a barrier arrive).  One thread
//               of warp 0 announces a stage's bytes and loads the first operand's share, one thread of
//               warp 10 loads the second operand's: a single thread cannot issue a stage's loads as fast
//               as the tensor core consumes them.
//   warp 1      MMA issuer: owns the TMEM allocation (two accumulators, so the
//               epilogue of tile i overlaps the main loop of tile i+1); one
//               elected lane issues tcgen05.mma kind::f16 (bf16 x bf16 -> fp32),
//               M = 128 (256 across a CTA pair), N up to 256, K = 16 per instruction; tcgen05.commit
//               releases stages and publishes finished accumulators.
//   warps 2..9  epilogue (two warps per TMEM lane quadrant, alternating 32-column blocks):
//               tcgen05.ld the accumulator (lane = tile row), apply the fused epilogue
//               (SwiGLU, gate scale, coupling add/sub, SwiGLU backward, fp32 weight
//               gradient) and pass each 32 x 32 output block through a per-warp staging
//               area in shared memory: bf16 blocks leave by TMA bulk tensor stores
//               (64-byte swizzle), fp32 blocks are transposed there and written with plain
//               16-byte stores, four 128-byte rows per instruction.  Global writes are whole
//               lines whatever the row stride.
// Tile = 128 rows x 256 columns (the last column tile of a row may be 128 wide: N only has
// to be a multiple of 128), K step 64 (one 128-byte swizzle atom of bf16).
// Both operands may be K-major or MN-major; MN-major tiles are fetched 128 columns x 64 K rows at a time through a
// 3-D view of the matrix (64 x 64 boxes of a 2-D map as the fallback) and described to the tensor core with
// leading/stride offsets.
// Every wait is bounded; on expiry the kernel sets the status word and leaves.
//
// Pair mode (template flag PAIR; dense and K-grouped problems whose N is a multiple of 256, or of 128
// when B is stored [K, N]):
// the grid is launched as clusters of two CTAs that work one 256 x 256 tile together with
// tcgen05.mma.cta_group::2.  Each CTA loads its own 128 rows of A and ITS HALF of B's columns
// (the tensor core reads both halves across the pair), so a K step costs a CTA 32 KB of operand
// traffic instead of 48 KB and six stages fit.  The even CTA issues the MMAs; its commits
// arrive on the barriers of both CTAs, both CTAs' loads complete on its "full" barriers, and
// both CTAs' epilogue warps release its accumulator barriers.
//
// Transposed pair mode (expert-grouped products with bf16 store or gate-scale epilogue): the
// pair computes C^T.  The MMA M side holds 256 output features (rows of the expert's weight
// matrix, 128 per CTA), the N side a run of up to 256 of the expert's token rows, real rows
// only (rounded up to 32), taken from a chunk table built with the permutation.  Padding rows
// then cost no tensor-core time, and these products get the pair mode's operand savings, which
// row tiles that must not straddle experts cannot have.  The epilogue transposes each
// 32-feature x 32-token block on its way through the staging area.
#pragma once

#include <cuda.h>
#include <cstring>
#include <mutex>
#include <type_traits>

#include "common.cuh"
#include "gemm.cuh"

namespace revffn {

constexpr int TC_BM = 128;
constexpr int TC_BK = 64;
constexpr int TC_THREADS = 352;      // warp 0, 10: operand loads; warp 1: products; warps 2..9: epilogue
constexpr int TC_LOAD_WARP_B = 10;   // the second load warp
constexpr int TC_EPI_WARPS = 8;
constexpr int TC_A_BYTES = TC_BM * TC_BK * 2;            // 16 KB
constexpr long long TC_WAIT_CYCLES = 4000000000LL;       // ~2 s: bound on any single wait

template <int MMA_N, int EPI, bool PAIR> struct TcCfg {
  static constexpr int B_BYTES = (PAIR ? MMA_N / 2 : MMA_N) * TC_BK * 2;
  static constexpr int STAGE_BYTES = TC_A_BYTES + B_BYTES;
  static constexpr int STAGES = PAIR ? 6 : 4;
  static constexpr int EPI_WARP_BYTES = 4096;           // staging per epilogue warp: two 32 x 32 bf16 blocks or one fp32 block
  static constexpr int TMEM_COLS = 2 * MMA_N;           // two accumulators; a power of two >= 32
  // stage ring | epilogue staging | barriers; the ring starts 1024-byte aligned and
  // every stage is a multiple of 1024 bytes, so the staging area is aligned too
  static constexpr int EPI_OFF = STAGES * STAGE_BYTES;
  static constexpr int BAR_OFF = EPI_OFF + TC_EPI_WARPS * EPI_WARP_BYTES;
  static constexpr int SMEM_BYTES = BAR_OFF + 1024 /*align*/ + 512 /*barriers*/;
};

struct TcParams {
  GemmProblem p;
  int tiles_m, tiles_n;      // GROUP_M: tiles_m is an upper bound, the device value comes from rows_total
  int tile_n;                // logical output columns per tile
  int k_blocks;              // dense / GROUP_M
  int tr;                    // transposed pair mode: weights on the MMA M side, an expert's token rows on the N side
  int tiles_f;               // tr: 256-wide feature tiles per token chunk
  uint32_t idesc;
  long long wait_cycles;     // bound on every wait of the kernel (clock cycles)
  int starve;                // failure-path test: the load warp issues nothing, so the first wait for operands runs out
  int bk;                    // operand elements per K step: 64 (bf16) or 128 (e4m3); a K step is 128 bytes of a row either way
  int mn3d;                  // MN-major operands are loaded 128 columns at a time through 3-D tensor maps
  int split_loads;           // 1: the second load warp issues the second operand's loads; 0: one thread issues all of them
};

// ---------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the wait was abandoned (this or another
// role ran out of time); the caller then leaves its loop.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                          long long limit = TC_WAIT_CYCLES) {
  if (mbar_try_wait(bar, parity)) return true;
  long long t0 = clock64();
  int spins = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (((++spins) & 63) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > limit) {
        *abort_flag = 1;
        set_status(status, REVFFN_ERR_DEVICE_WAIT);
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar) : "memory");
}

// Shared -> global bulk tensor store of one box (the box and the swizzle come from the map).
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(src) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Wait until at most N of this thread's bulk groups still read their shared-memory source.
template <int N> __device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// Orders this thread's shared-memory writes before later async-proxy (TMA) reads of them.
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Pair mode: the same load, completing on a barrier that may live in the partner CTA (cluster address).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar_cluster) : "memory");
}
// 128 columns x 64 K rows of an MN-major operand ([K rows, ld columns] in memory) into two consecutive 8 KB
// blocks of 64 columns each, the layout the MMA descriptors expect.  mn3d: one load through a 3-D view of the
// matrix {64 columns, K rows, ld / 64 column groups} with a box of two groups; else two 2-D loads of 64 x 64.
// A tensor load costs its issuing thread a couple of hundred clocks whatever its size, so halving their number
// matters as much as spreading them over two threads.
__device__ __forceinline__ void tma_load_mn128(bool mn3d, uint32_t dst, const CUtensorMap* map, int col, int krow, uint32_t bar) {
  if (mn3d) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(0), "r"(krow), "r"(col >> 6), "r"(bar) : "memory");
  } else {
    tma_load_2d(dst, map, col, krow, bar);
    tma_load_2d(dst + 8192, map, col + 64, krow, bar);
  }
}
__device__ __forceinline__ void tma_load_mn128_pair(bool mn3d, uint32_t dst, const CUtensorMap* map, int col, int krow,
                                                    uint32_t bar_cluster, bool second_block = true) {
  if (mn3d) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(0), "r"(krow), "r"(col >> 6), "r"(bar_cluster) : "memory");
  } else {
    tma_load_2d_pair(dst, map, col, krow, bar_cluster);
    if (second_block) tma_load_2d_pair(dst + 8192, map, col + 64, krow, bar_cluster);
  }
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Cluster-wide address of the location `addr` (own shared window) in the CTA of rank `rank`.
__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}
// All threads of both CTAs of the pair.
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Pair mode: arrive on the barrier at this shared-memory offset in both CTAs once the MMAs issued so far are done.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}

// One product with the descriptors given as (low, high) words: the high words never change inside a kernel, and
// the low words move by small additions, so the issuing thread carries 32-bit values only.
// The same for e4m3 operands (kind::f8f6f4: 32 one-byte elements of K per instruction, the same 32 bytes).
template <bool PAIR>
__device__ __forceinline__ void tc_mma_lohi_f8(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                               uint32_t idesc, uint32_t acc) {
  if constexpr (PAIR)
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(acc) : "memory");
  else
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(acc) : "memory");
}

template <bool PAIR>
__device__ __forceinline__ void tc_mma_lohi(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                            uint32_t idesc, uint32_t acc) {
  if constexpr (PAIR)
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(acc) : "memory");
  else
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(acc) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}

// 32 consecutive accumulator columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle, tile base 1024-byte aligned.
//   K-major : rows of 128 bytes, 8-row groups 1024 bytes apart (SBO); LBO unused (1)
//   MN-major: 64-element chunks along M/N are lbo bytes apart, 8-k-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= 1ull << 46;      // descriptor version of this architecture
  d |= 2ull << 61;      // 128-byte swizzle
  return d;
}

__device__ __forceinline__ uint4 pack8(const float* f) {
  uint4 u;
  __nv_bfloat162 h;
  h = __floats2bfloat162_rn(f[0], f[1]); u.x = *reinterpret_cast<uint32_t*>(&h);
  h = __floats2bfloat162_rn(f[2], f[3]); u.y = *reinterpret_cast<uint32_t*>(&h);
  h = __floats2bfloat162_rn(f[4], f[5]); u.z = *reinterpret_cast<uint32_t*>(&h);
  h = __floats2bfloat162_rn(f[6], f[7]); u.w = *reinterpret_cast<uint32_t*>(&h);
  return u;
}
__device__ __forceinline__ void unpack8(uint4 u, float* f) {
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int i = 0; i < 4; ++i) { float2 t = __bfloat1622float2(h[i]); f[2 * i] = t.x; f[2 * i + 1] = t.y; }
}
// store 32 floats as 32 bf16 (64 contiguous bytes)
__device__ __forceinline__ void store32_bf16(bf16* dst, const float* f) {
  uint4* o = reinterpret_cast<uint4*>(dst);
#pragma unroll
  for (int i = 0; i < 4; ++i) o[i] = pack8(f + 8 * i);
}
__device__ __forceinline__ void load32_bf16(const bf16* src, float* f) {
  const uint4* s = reinterpret_cast<const uint4*>(src);
#pragma unroll
  for (int i = 0; i < 4; ++i) unpack8(s[i], f + 8 * i);
}

// Output staging.  A warp stages a 32-row x 32-column bf16 block, one row per lane, in the layout
// the store's tensor map expects: rows of 64 bytes under the 64-byte swizzle.  `buf` is aligned to
// the swizzle period, so the 16-byte piece j of row r lands at piece j ^ ((r >> 1) & 3); lanes of
// one store instruction then hit distinct banks.
__device__ __forceinline__ void stage32_bf16(uint8_t* buf, int r, const float* f) {
  uint8_t* row = buf + r * 64;
#pragma unroll
  for (int j = 0; j < 4; ++j) *reinterpret_cast<uint4*>(row + ((j ^ ((r >> 1) & 3)) << 4)) = pack8(f + 8 * j);
}

// A warp's 32-row x 32-column bf16 block (rows of 64 bytes, row stride ld elements) between global memory and
// the staging layout above, in "distributed" form: instruction i of four moves rows 8i .. 8i+7, lane l the
// 16-byte piece l & 3 of row 8i + (l >> 2).  Eight lanes cover four whole 64-byte row segments, so every
// 32-byte sector a request touches is used in full, and the 512 contiguous staging bytes an instruction
// touches spread over all banks.  rows_ok: rows of the block that exist (the rest read as zeros / are not stored).
__device__ __forceinline__ void blk_load_dist(const bf16* g, int64_t ld, int rows_ok, int lane, uint4 (&raw)[4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = 8 * i + (lane >> 2);
    raw[i] = (r < rows_ok) ? __ldcg(reinterpret_cast<const uint4*>(g + (int64_t)r * ld + (lane & 3) * 8))
                           : make_uint4(0u, 0u, 0u, 0u);
  }
}
__device__ __forceinline__ void blk_dist_to_stage(uint8_t* buf, int lane, const uint4 (&raw)[4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = 8 * i + (lane >> 2);
    *reinterpret_cast<uint4*>(buf + r * 64 + (((lane & 3) ^ ((r >> 1) & 3)) << 4)) = raw[i];
  }
}
__device__ __forceinline__ void blk_stage_to_global(const uint8_t* buf, int lane, bf16* g, int64_t ld, int rows_ok) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = 8 * i + (lane >> 2);
    const uint4 v = *reinterpret_cast<const uint4*>(buf + r * 64 + (((lane & 3) ^ ((r >> 1) & 3)) << 4));
    if (r < rows_ok) *reinterpret_cast<uint4*>(g + (int64_t)r * ld + (lane & 3) * 8) = v;
  }
}

// Logistic function from one ex2.approx and one rcp.approx (relative error about 2^-21, far inside what the
// bf16 results around it can show).
__device__ __forceinline__ float sigmoid_approx(float x) {
  float e, r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(x * -1.4426950408889634f));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.f + e));
  return r;
}

__device__ __forceinline__ float2 sigmoid_approx2(float2 x) {
  const float2 t = __fmul2_rn(x, make_float2(-1.4426950408889634f, -1.4426950408889634f));
  float e0, e1, r0, r1;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(t.x));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(t.y));
  const float2 den = __fadd2_rn(make_float2(e0, e1), make_float2(1.f, 1.f));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r0) : "f"(den.x));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r1) : "f"(den.y));
  return make_float2(r0, r1);
}

// Tile coordinates shared by the three roles.
struct TcTile {
  int m0, n0, group, k_blocks, krow0;
  int ncols;      // accumulator columns in use: 256, or 128 in the last column tile of an odd multiple of 128
  bool valid;
};

// pair_rank < 0: one CTA per 128-row tile.  pair_rank 0 / 1: w counts 256-row tiles worked by two CTAs,
// this CTA takes rows 128 * pair_rank .. + 127 of it (rows past M are loaded as zeros and never stored).
__device__ __forceinline__ TcTile tc_tile(const TcParams& P, int w, int tiles_m_dev, int pair_rank = -1) {
  TcTile t;
  const GemmProblem& p = P.p;
  if (P.tr) {
    // w = token chunk * tiles_f + feature tile; m0 = first token row, ncols = token rows (the MMA N),
    // n0 = first feature of this CTA's 128
    const int ci = w / P.tiles_f, ft = w - ci * P.tiles_f;
    t.group = 0; t.krow0 = 0; t.k_blocks = P.k_blocks; t.ncols = 0; t.m0 = t.n0 = 0;
    t.valid = ci < p.rows_total[1];
    if (!t.valid) return t;
    const int4 ch = p.tok_chunks[ci];
    t.group = ch.x; t.m0 = ch.y; t.ncols = ch.z;
    t.n0 = ft * 2 * TC_BM + pair_rank * TC_BM;
    return t;
  }
  if (pair_rank >= 0) tiles_m_dev = (tiles_m_dev + 1) / 2;
  int per_group = tiles_m_dev * P.tiles_n;
  t.group = 0;
  t.krow0 = 0;
  t.k_blocks = P.k_blocks;
  int total = (p.group_mode == GROUP_K) ? per_group * p.n_groups : per_group;
  t.valid = w < total;
  t.ncols = 0;
  if (!t.valid) { t.m0 = t.n0 = 0; return t; }
  int r = w;
  if (p.group_mode == GROUP_K) {
    t.group = w / per_group;
    r = w - t.group * per_group;
    if (p.group_off) {
      int k0 = p.group_off[t.group], k1 = p.group_off[t.group + 1];
      t.krow0 = k0;
      t.k_blocks = (k1 - k0) / TC_BK;
      if (p.group_cnt) t.k_blocks = min(t.k_blocks, (p.group_cnt[t.group] + TC_BK - 1) / TC_BK);   // skip all-zero K blocks
    } else {
      // equal slices of a dense K (split-K): rows past K in the last K step load as zeros
      const int slice = (int)split_k_rows(p.K, p.n_groups);
      const int k0 = min(t.group * slice, p.K), k1 = min(k0 + slice, p.K);
      t.krow0 = k0;
      t.k_blocks = (k1 - k0 + TC_BK - 1) / TC_BK;
    }
  }
  int tm = r / P.tiles_n, tn = r - tm * P.tiles_n;
  t.m0 = (pair_rank >= 0) ? tm * 2 * TC_BM + pair_rank * TC_BM : tm * TC_BM;
  t.n0 = tn * P.tile_n;
  t.ncols = (p.concat == CONCAT_N) ? 2 * P.tile_n : min(P.tile_n, p.N - t.n0);
  if (p.group_mode == GROUP_M) t.group = p.tile_group[tm];
  return t;
}

// ---------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------
template <int MMA_N, int EPI, bool PAIR>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ TcParams P, const __grid_constant__ CUtensorMap map_a,
               const __grid_constant__ CUtensorMap map_b0, const __grid_constant__ CUtensorMap map_b1,
               const __grid_constant__ CUtensorMap map_c, const __grid_constant__ CUtensorMap map_c1) {
  using Cfg = TcCfg<MMA_N, EPI, PAIR>;
  extern __shared__ uint8_t smem_raw[];
  const GemmProblem& p = P.p;
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;                 // stage ring, 1024-byte aligned
  uint8_t* gen_base = smem_raw + (base - raw);
  const uint32_t bars = base + Cfg::BAR_OFF;                    // barrier block
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (Cfg::STAGES + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * Cfg::STAGES + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * Cfg::STAGES + 2 + a); };
  const uint32_t drain_bar = bars + 320u;      // abort path of the MMA thread: "every product issued so far is done"
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_base + Cfg::BAR_OFF + 256);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* issued = reinterpret_cast<int*>(tmem_slot + 2);   // [STAGES] parity+1 of the last load issued per stage
  int* issued_b = issued + Cfg::STAGES;                  // the same for the second load warp: nonzero once it has issued

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int crank = PAIR ? (int)cluster_ctarank() : 0;     // rank in the pair; rank 0 issues the MMAs
  const int prank = PAIR ? crank : -1;
  const int w0 = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;       // first tile and tile stride of this CTA / pair
  const int wstride = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;

  if (threadIdx.x == 0) {
    for (int s = 0; s < Cfg::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); issued[s] = 0; issued_b[s] = 0; }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), PAIR ? 2 * TC_EPI_WARPS : TC_EPI_WARPS); }
    mbar_init(drain_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    if constexpr (PAIR) {      // the same warp of both CTAs, the same shared-memory offset
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                   ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)Cfg::TMEM_COLS) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                   ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)Cfg::TMEM_COLS) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if constexpr (PAIR) cluster_sync_all();      // the partner's barriers exist before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  int tiles_m_dev = P.tiles_m;
  if (p.group_mode == GROUP_M) tiles_m_dev = min(P.tiles_m, *p.rows_total / TC_BM);

  if (warp == 0 || warp == TC_LOAD_WARP_B) {
    // ------------------------------------------------------------------ operand loads
    // Two threads, one in each load warp, walk the same tiles and stages.  A tensor load takes the issuing thread
    // 150-250 clocks (more in the pair form, whose completion is signalled in the partner CTA), and a stage needs
    // two to six of them: issued by one thread they took 500-850 clocks per stage, more than the 512 clocks of
    // tensor work in a stage, and the MMA thread waited for operands in every product.  Thread A announces the
    // stage's bytes and loads the first operand's share of the stage, thread B loads the second operand's; the
    // bytes may arrive before they are announced (the barrier's phase cannot complete before the announcing
    // arrival).
    // (A version of this loop that kept per-tile "load slots" -- tensor-map pointer, destination, coordinates --
    // in registers and issued one load per slot measured 15-40 % slower: a load whose tensor map is named through
    // a pointer chosen at run time, rather than as the kernel parameter itself, is slow to issue.)
    // la: this thread loads the first operand's share (and announces the stage); lb: the second operand's.
    // Without split_loads the first warp's thread does both and the second warp has nothing to do.
    const bool la = warp == 0, lb = P.split_loads ? warp != 0 : warp == 0;
    if (lane == 0 && !P.starve && (la || lb)) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int w = w0; ok; w += wstride) {
        TcTile t = tc_tile(P, w, tiles_m_dev, prank);
        if (!t.valid) break;
        const int k_half = t.k_blocks / 2;
        for (int kb = 0; kb < t.k_blocks; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, P.wait_cycles)) { ok = false; break; }
          const uint32_t sa = base + stage * Cfg::STAGE_BYTES;
          const uint32_t sb = sa + TC_A_BYTES;
          if constexpr (PAIR) {
            // both CTAs' loads complete on the even CTA's barrier, which expects the bytes of both
            const uint32_t fbc = mapa_u32(full_bar(stage), 0);
            if (P.tr) {
              // M side: 128 rows of the expert's weights; N side: this CTA's half of the chunk's token rows
              // (a full 128-row box either way; rows past the half are loaded and not used)
              if (la) {
                if (crank == 0) mbar_expect_tx(full_bar(stage), 2 * Cfg::STAGE_BYTES);
                int kw = kb;
                const bool second = p.concat == CONCAT_K && kb >= k_half;
                if (second) kw = kb - k_half;
                if (!p.b_mn_major) {
                  if (second) tma_load_2d_pair(sa, &map_b1, kw * P.bk, t.group * p.N + t.n0, fbc);
                  else tma_load_2d_pair(sa, &map_b0, kw * P.bk, t.group * p.N + t.n0, fbc);
                } else {
                  const int kdim = (p.concat == CONCAT_K) ? k_half * TC_BK : t.k_blocks * TC_BK;
                  const int krow = t.group * kdim + kw * TC_BK;
                  if (second) tma_load_mn128_pair(P.mn3d, sa, &map_b1, p.b_col0 + t.n0, krow, fbc);
                  else tma_load_mn128_pair(P.mn3d, sa, &map_b0, p.b_col0 + t.n0, krow, fbc);
                }
              }
              if (lb) tma_load_2d_pair(sb, &map_a, kb * P.bk, t.m0 + crank * (t.ncols / 2), fbc);
              if (++stage == Cfg::STAGES) { stage = 0; phase ^= 1u; }
              continue;
            }
            const int nhalf = t.ncols / 2;       // this CTA's share of the tile's columns: 128, or 64 in a ragged last tile
            if (la) {
              // (a 3-D load of an MN-major B always brings 128 columns, also where this CTA's share is 64)
              const int b_cols = (p.b_mn_major && P.mn3d) ? 128 : nhalf;
              if (crank == 0) mbar_expect_tx(full_bar(stage), 2 * (TC_A_BYTES + b_cols * TC_BK * 2));
              if (!p.a_mn_major) {
                tma_load_2d_pair(sa, &map_a, kb * TC_BK, t.m0, fbc);
              } else {
                tma_load_mn128_pair(P.mn3d, sa, &map_a, p.a_col0 + t.m0, t.krow0 + kb * TC_BK, fbc);
              }
            }
            if (lb) {
              const bool second = p.concat == CONCAT_K && kb >= k_half;
              const int kbp = second ? kb - k_half : kb;
              if (!p.b_mn_major) {
                // this CTA's 128 of the 256 accumulator columns: gate rows (rank 0) or up rows (rank 1) of a
                // SwiGLU pair, else rows n0 + 128 rank .. + 127 of B
                // (the tensor map is named directly in each call: a map chosen through a pointer is slow to issue)
                if (p.concat == CONCAT_N) {
                  if (crank == 0) tma_load_2d_pair(sb, &map_b0, kbp * TC_BK, t.n0, fbc);
                  else tma_load_2d_pair(sb, &map_b1, kbp * TC_BK, t.n0, fbc);
                } else if (second) {
                  tma_load_2d_pair(sb, &map_b1, kbp * TC_BK, t.n0 + 128 * crank, fbc);
                } else {
                  tma_load_2d_pair(sb, &map_b0, kbp * TC_BK, t.n0 + 128 * crank, fbc);
                }
              } else {
                const int krow = t.krow0 + kbp * TC_BK;
                if (second) tma_load_mn128_pair(P.mn3d, sb, &map_b1, p.b_col0 + t.n0 + nhalf * crank, krow, fbc, nhalf > 64);
                else tma_load_mn128_pair(P.mn3d, sb, &map_b0, p.b_col0 + t.n0 + nhalf * crank, krow, fbc, nhalf > 64);
              }
            }
            if (++stage == Cfg::STAGES) { stage = 0; phase ^= 1u; }
            continue;
          }
          const uint32_t fb = full_bar(stage);
          const bool second = p.concat == CONCAT_K && kb >= k_half;
          const int kb_b = second ? kb - k_half : kb;
          // An MN-major B tile is four 64 x 64 boxes against one or two loads for A: with two load threads the
          // first takes B's last boxes too (3 + 2 loads, or 3 + 3 when A is MN-major as well).
          const int b_mn_split = !p.b_mn_major ? 0 : (!P.split_loads ? 0 : ((p.a_mn_major && !P.mn3d) ? 3 : 2));
          if (la) {
            mbar_expect_tx(fb, TC_A_BYTES + t.ncols * TC_BK * 2);
            issued[stage] = (int)phase + 1;
            // A tile
            if (!p.a_mn_major) {
              tma_load_2d(sa, &map_a, kb * P.bk, t.m0, fb);
            } else {
              tma_load_mn128(P.mn3d, sa, &map_a, p.a_col0 + t.m0, t.krow0 + kb * TC_BK, fb);
            }
            if (b_mn_split) {
              int kdim = (p.concat == CONCAT_K) ? k_half * TC_BK : t.k_blocks * TC_BK;
              int krow = (p.group_mode == GROUP_M ? t.group * kdim : t.krow0) + kb_b * TC_BK;
              if (P.mn3d) {          // the second 128 columns
                if (t.ncols > 128) {
                  if (second) tma_load_mn128(true, sb + 16384, &map_b1, p.b_col0 + t.n0 + 128, krow, fb);
                  else tma_load_mn128(true, sb + 16384, &map_b0, p.b_col0 + t.n0 + 128, krow, fb);
                }
              } else {
#pragma unroll
                for (int j = 2; j < MMA_N / 64; ++j) {
                  if (j < b_mn_split || 64 * j >= t.ncols) continue;
                  if (second) tma_load_2d(sb + j * 8192, &map_b1, p.b_col0 + t.n0 + 64 * j, krow, fb);
                  else tma_load_2d(sb + j * 8192, &map_b0, p.b_col0 + t.n0 + 64 * j, krow, fb);
                }
              }
            }
          }
          if (lb) {
            issued_b[stage] = (int)phase + 1;
            // B tile
            if (!p.b_mn_major) {
              // rows of the flattened [groups * N, K] weight tensor
              int row0 = (p.group_mode == GROUP_M ? t.group * p.N : 0) + t.n0;
              if (p.concat == CONCAT_N) {
                tma_load_2d(sb, &map_b0, kb_b * P.bk, row0, fb);
                tma_load_2d(sb + 16384, &map_b1, kb_b * P.bk, row0, fb);
              } else {
#pragma unroll
                for (int j = 0; j < MMA_N / 128; ++j) {
                  if (128 * j >= t.ncols) continue;
                  if (second) tma_load_2d(sb + j * 16384, &map_b1, kb_b * P.bk, row0 + 128 * j, fb);
                  else tma_load_2d(sb + j * 16384, &map_b0, kb_b * P.bk, row0 + 128 * j, fb);
                }
              }
            } else {
              // rows of the flattened [groups * Kdim, N] weight tensor, or token rows (GROUP_K / dense wgrad)
              int kdim = (p.concat == CONCAT_K) ? k_half * TC_BK : t.k_blocks * TC_BK;
              int krow = (p.group_mode == GROUP_M ? t.group * kdim : t.krow0) + kb_b * TC_BK;
              if (P.mn3d) {
                if (second) tma_load_mn128(true, sb, &map_b1, p.b_col0 + t.n0, krow, fb);
                else tma_load_mn128(true, sb, &map_b0, p.b_col0 + t.n0, krow, fb);
                if (!b_mn_split && t.ncols > 128) {
                  if (second) tma_load_mn128(true, sb + 16384, &map_b1, p.b_col0 + t.n0 + 128, krow, fb);
                  else tma_load_mn128(true, sb + 16384, &map_b0, p.b_col0 + t.n0 + 128, krow, fb);
                }
              } else {
#pragma unroll
                for (int j = 0; j < MMA_N / 64; ++j) {
                  if ((b_mn_split && j >= b_mn_split) || 64 * j >= t.ncols) continue;
                  if (second) tma_load_2d(sb + j * 8192, &map_b1, p.b_col0 + t.n0 + 64 * j, krow, fb);
                  else tma_load_2d(sb + j * 8192, &map_b0, p.b_col0 + t.n0 + 64 * j, krow, fb);
                }
              }
            }
          }
          if (++stage == Cfg::STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // One thread issues every product of the CTA (pair), so the cycles this loop spends per K step bound the
    // kernel as surely as the tensor pipe does: four products take about 300 clocks to issue and the commit
    // 60, against 512 clocks of tensor work in a 128 x 256 x 64 step.  Everything that does not change inside a
    // tile (descriptor high words, layout steps, barrier addresses) is therefore set up outside the loop, and a
    // K step costs the wait, two additions, the four products and the commit.
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int it = 0;
      // the M-side slot holds A (or, transposed, the weights B); the N-side slot the other operand
      const int m_mn = P.tr ? p.b_mn_major : p.a_mn_major, n_mn = P.tr ? p.a_mn_major : p.b_mn_major;
      const uint64_t a_desc0 = m_mn ? make_smem_desc(base, 8192, 1024) : make_smem_desc(base, 16, 1024);
      const uint64_t b_desc0 = n_mn ? make_smem_desc(base + TC_A_BYTES, 8192, 1024) : make_smem_desc(base + TC_A_BYTES, 16, 1024);
      const uint32_t a_hi = (uint32_t)(a_desc0 >> 32), b_hi = (uint32_t)(b_desc0 >> 32);
      const uint32_t a_lo0 = (uint32_t)a_desc0, b_lo0 = (uint32_t)b_desc0;    // address field (bits 0..13, 16-byte units) + leading offset
      const uint32_t a_step = m_mn ? (2048u >> 4) : (32u >> 4);   // 16 k-elements per instruction
      const uint32_t b_step = n_mn ? (2048u >> 4) : (32u >> 4);
      constexpr uint32_t SB16 = (uint32_t)Cfg::STAGE_BYTES >> 4;  // the whole ring stays below 256 KB: no carry out of the field
      uint32_t a_lo = a_lo0, b_lo = b_lo0, fbar = full_bar(0), ebar = empty_bar(0);
      for (int w = w0; ok && crank == 0; w += wstride, ++it) {
        TcTile t = tc_tile(P, w, tiles_m_dev, prank);
        if (!t.valid) break;
        const int acc = it & 1;
        const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.status, P.wait_cycles)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * MMA_N);
        const uint32_t idesc = (P.idesc & ~(0x3Fu << 17)) | ((uint32_t)(t.ncols >> 3) << 17);   // N of this tile
        const int nk = t.k_blocks;
        for (int kb = 0; kb < nk; ++kb) {
          if (!mbar_wait(fbar, phase, abort_flag, p.status, P.wait_cycles)) { ok = false; break; }
          tc_fence_after();
          if (p.fp8) {
            tc_mma_lohi_f8<PAIR>(d_tmem, a_lo, a_hi, b_lo, b_hi, idesc, kb != 0 ? 1u : 0u);
            tc_mma_lohi_f8<PAIR>(d_tmem, a_lo + a_step, a_hi, b_lo + b_step, b_hi, idesc, 1u);
            tc_mma_lohi_f8<PAIR>(d_tmem, a_lo + 2 * a_step, a_hi, b_lo + 2 * b_step, b_hi, idesc, 1u);
            tc_mma_lohi_f8<PAIR>(d_tmem, a_lo + 3 * a_step, a_hi, b_lo + 3 * b_step, b_hi, idesc, 1u);
          } else {
            tc_mma_lohi<PAIR>(d_tmem, a_lo, a_hi, b_lo, b_hi, idesc, kb != 0 ? 1u : 0u);
            tc_mma_lohi<PAIR>(d_tmem, a_lo + a_step, a_hi, b_lo + b_step, b_hi, idesc, 1u);
            tc_mma_lohi<PAIR>(d_tmem, a_lo + 2 * a_step, a_hi, b_lo + 2 * b_step, b_hi, idesc, 1u);
            tc_mma_lohi<PAIR>(d_tmem, a_lo + 3 * a_step, a_hi, b_lo + 3 * b_step, b_hi, idesc, 1u);
          }
          // stage reusable once these MMAs have read it (in both CTAs of a pair)
          if constexpr (PAIR) tc_commit_pair(ebar); else tc_commit(ebar);
          a_lo += SB16; b_lo += SB16; fbar += 8u; ebar += 8u;
          if (++stage == Cfg::STAGES) { stage = 0; phase ^= 1u; a_lo = a_lo0; b_lo = b_lo0; fbar = full_bar(0); ebar = empty_bar(0); }
        }
        if (!ok) break;
        if constexpr (PAIR) tc_commit_pair(tfull_bar(acc)); else tc_commit(tfull_bar(acc));   // accumulator complete
      }
      if (!ok && !PAIR) {
        // A wait was abandoned.  Products issued before it may still be running: they read the stage ring and
        // write tensor memory, so they must have finished before the teardown below releases either.  A commit
        // on a barrier of its own completes once every product issued so far is done (products wait for
        // nothing themselves, so this ends; the wait is bounded all the same).
        tc_commit(drain_bar);
        const long long t0 = clock64();
        while (!mbar_try_wait(drain_bar, 0u) && clock64() - t0 < P.wait_cycles) {}
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9)
    const int q = warp & 3;                      // TMEM lane quadrant this warp may access
    const int ew = warp - 2;                     // epilogue warp index
    const int half = ew >> 2;                    // this warp takes the 32-column blocks half, half+2, ...
    const int row_in_tile = q * 32 + lane;
    uint8_t* stg = gen_base + Cfg::EPI_OFF + ew * Cfg::EPI_WARP_BYTES;   // this warp's staging area
    const uint32_t stg_u32 = base + Cfg::EPI_OFF + ew * Cfg::EPI_WARP_BYTES;
    bool ok = true;
    int it = 0;
    uint32_t n_grp = 0;                          // bulk groups committed so far (same in every lane)
    for (int w = w0; ok; w += wstride, ++it) {
      TcTile t = tc_tile(P, w, tiles_m_dev, prank);
      if (!t.valid) break;
      const int acc = it & 1;
      const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
      const int m = t.m0 + row_in_tile;
      const int m_lim = (p.group_mode == GROUP_M) ? tiles_m_dev * TC_BM : p.M;
      const bool m_ok = m < m_lim;
      const bool slab_ok = t.m0 + q * 32 < m_lim;             // this warp's 32 rows hold at least one real row
      const int rows_ok = min(32, m_lim - (t.m0 + q * 32));   // real rows among them (<= 0: none)
      // SwiGLU backward: the a|b operands of the warp's first block do not depend on the accumulator, so
      // their loads go out before the wait for it (ds_a / ds_b: one block in distributed form)
      uint4 ds_a[4], ds_b[4];
      bf16* ds_blk = nullptr;
      if constexpr (EPI == EPI_DSWIGLU) {
        ds_blk = reinterpret_cast<bf16*>(p.ab) + (int64_t)(t.m0 + q * 32) * p.ld_ab + t.n0;
        if (slab_ok && half * 32 < t.ncols) {
          blk_load_dist(ds_blk + half * 32, p.ld_ab, rows_ok, lane, ds_a);
          blk_load_dist(ds_blk + p.N + half * 32, p.ld_ab, rows_ok, lane, ds_b);
        }
      }
      if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.status, P.wait_cycles)) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * MMA_N);
      // row coordinate of the slab in the output tensor map (rows past its extent are clipped by the store)
      const int y0 = (p.group_mode == GROUP_K ? t.group * p.M : 0) + t.m0 + q * 32;
      const bool have_acc = t.k_blocks > 0;      // an empty K range leaves the accumulator undefined: use zeros
      uint32_t r0[32];
      float f[32];

      if (PAIR && P.tr) {
        if constexpr (PAIR && (EPI == EPI_STORE || EPI == EPI_ROWSCALE)) {
          // Transposed tile: this lane holds output feature t.n0 + 32 q + lane for 32 token rows per block.
          // Lanes 2i and 2i+1 trade halves so that each ends up with feature PAIRS of single tokens (the even
          // lane of the even tokens, the odd lane of the odd ones), which it writes as 4-byte pieces into
          // the [32 tokens][32 features] staging block; a TMA store then writes 32 rows of 64 bytes.
          const bool odd = lane & 1;
#pragma unroll 1
          for (int c = half * 32; c < t.ncols; c += 64) {
            tmem_ld32(taddr + c, r0);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) f[i] = __uint_as_float(r0[i]);
            if (p.fp8) {
              // e4m3 operands: this lane's feature scale times the 32 tokens' row scales
              const float sw = p.b_scale0[(int64_t)t.group * p.N + t.n0 + q * 32 + lane];
              const float4* a4 = reinterpret_cast<const float4*>(p.a_scale + t.m0 + c);    // the same for every lane
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const float4 a = a4[i];
                f[4 * i] *= sw * a.x; f[4 * i + 1] *= sw * a.y; f[4 * i + 2] *= sw * a.z; f[4 * i + 3] *= sw * a.w;
              }
            }
            if constexpr (EPI == EPI_ROWSCALE) {
              const float4* g4 = reinterpret_cast<const float4*>(p.rowscale + t.m0 + c);   // the same for every lane
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const float4 g = g4[i];
                f[4 * i] *= g.x; f[4 * i + 1] *= g.y; f[4 * i + 2] *= g.z; f[4 * i + 3] *= g.w;
              }
            }
            const uint32_t off = (n_grp & 1u) * 2048u;
            if (lane == 0) bulk_wait_read<1>();
            __syncwarp();
            uint8_t* blk = stg + off;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float send = odd ? f[2 * j] : f[2 * j + 1];
              const float recv = __shfl_xor_sync(0xffffffffu, send, 1);
              const int tok = 2 * j + (odd ? 1 : 0);
              const __nv_bfloat162 v = odd ? __floats2bfloat162_rn(recv, f[2 * j + 1]) : __floats2bfloat162_rn(f[2 * j], recv);
              const int piece = lane >> 3, within = ((lane >> 1) & 3) * 4;
              *reinterpret_cast<__nv_bfloat162*>(blk + tok * 64 + ((piece ^ ((tok >> 1) & 3)) << 4) + within) = v;
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
              tma_store_2d(&map_c, stg_u32 + off, t.n0 + q * 32, t.m0 + c);
              bulk_commit();
            }
            ++n_grp;
          }
        }
      } else if constexpr (EPI == EPI_STORE || EPI == EPI_ROWSCALE || EPI == EPI_COUPLE || EPI == EPI_WGRAD) {
        float rs = 1.f;
        if (EPI == EPI_ROWSCALE && m_ok) rs = p.rowscale[m];
        const bool f32_out = (EPI == EPI_COUPLE) || (EPI == EPI_WGRAD) || (EPI == EPI_STORE && p.out_f32);
        // where this warp's slab of an fp32 result goes
        const int piece = lane & 7;
        int64_t y_lim, yb;                                 // row limit and first output row of this warp's slab
        float* cptr;
        bf16* wptr;
        float *mptr, *momptr, *varptr;
        auto slab_target = [&](const TcTile& tt, int64_t y0_tt) {
          y_lim = (p.group_mode == GROUP_K) ? (int64_t)(tt.group + 1) * p.M
                                            : (p.group_mode == GROUP_M ? (int64_t)m_lim : (int64_t)p.M);
          yb = y0_tt;
          cptr = reinterpret_cast<float*>(p.C);
          wptr = reinterpret_cast<bf16*>(p.upd_w);
          mptr = p.upd_m; momptr = p.upd_mom; varptr = p.upd_var;
          if (EPI == EPI_WGRAD && p.split_m > 0) {
            // two outputs: the slab lies wholly in the first or in the second (split_m is a multiple of 128)
            int local = tt.m0 + q * 32;
            if (local >= p.split_m) {
              local -= p.split_m;
              cptr = reinterpret_cast<float*>(p.C2); wptr = reinterpret_cast<bf16*>(p.upd_w2); mptr = p.upd_m2;
              momptr = p.upd_mom2; varptr = p.upd_var2;
            }
            yb = (int64_t)tt.group * p.split_m + local;
            y_lim = (int64_t)(tt.group + 1) * p.split_m;
          }
        };
        slab_target(t, y0);
        // Read-modify-write forms of the weight-gradient epilogue (fused update, accumulation): what the eight
        // pieces of a block need is requested before the block's accumulator is fetched and staged, and used
        // after.  Taken piece by piece, each piece's loads waited behind the previous piece's stores (the compiler
        // cannot tell that they do not overlap) and a 32 x 32 block cost eight memory round trips: the fused SGD
        // pass measured 2.4 ms slower than writing the gradients.  (Asking the next tile's lines into the L2 a
        // tile ahead, prefetch.global.L2 per row, changed nothing measurable on top of this.)
        const bool rmw = EPI == EPI_WGRAD && (wptr != nullptr || p.accumulate);
        auto as_f4 = [](const uint4& u) {
          return make_float4(__uint_as_float(u.x), __uint_as_float(u.y), __uint_as_float(u.z), __uint_as_float(u.w));
        };
        auto bf_f4 = [](const uint4& u) {
          const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.x));
          const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.y));
          return make_float4(lo.x, lo.y, hi.x, hi.y);
        };
#pragma unroll 1
        for (int c = half * 32; c < t.ncols; c += 64) {
          const int n = t.n0 + c;
          if (!slab_ok) continue;      // warp-uniform
          const int64_t col = n + piece * 4;
          uint4 ld[8];          // four floats (stored gradient or master copy), or four bf16 weights in .x, .y
          if (rmw) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int r = i * 4 + (lane >> 3);
              const int64_t at = (yb + r) * p.ldc + col;
              if (yb + r < y_lim) {
                if (!wptr) ld[i] = *reinterpret_cast<const uint4*>(cptr + at);
                else if (mptr) ld[i] = *reinterpret_cast<const uint4*>(mptr + at);
                else { const uint2 w2 = *reinterpret_cast<const uint2*>(wptr + at); ld[i].x = w2.x; ld[i].y = w2.y; }
              }
            }
          }
          if (have_acc) { tmem_ld32(taddr + c, r0); tmem_ld_wait(); }
#pragma unroll
          for (int i = 0; i < 32; ++i) f[i] = have_acc ? __uint_as_float(r0[i]) : 0.f;
          if constexpr (EPI == EPI_ROWSCALE) {
#pragma unroll
            for (int i = 0; i < 32; ++i) f[i] *= rs;
          } else if constexpr (EPI == EPI_COUPLE) {
            if (m_ok) {
              const float4* x = reinterpret_cast<const float4*>(p.resid + (int64_t)m * p.ld_resid + n);
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                float4 xv = x[i];
                f[4 * i] = xv.x + p.resid_sign * f[4 * i];
                f[4 * i + 1] = xv.y + p.resid_sign * f[4 * i + 1];
                f[4 * i + 2] = xv.z + p.resid_sign * f[4 * i + 2];
                f[4 * i + 3] = xv.w + p.resid_sign * f[4 * i + 3];
              }
            }
          }
          // bf16 blocks (32 x 32, 2 KB) leave through two alternating staging buffers and TMA stores.
          // fp32 blocks (32 x 32, 4 KB) are transposed through the staging area and written with plain
          // 16-byte stores, 4 rows x 128 bytes per instruction: whole lines, and nothing to wait for
          // before the area is reused.  (A TMA store of such a block sat behind the producer's operand
          // loads in the copy engine; with the short K of a weight gradient that wait set the pace.)
          if (f32_out) {
            if (lane == 0) bulk_wait_read<0>();     // no bulk store of this warp reads the area any more
            __syncwarp();
            {
              uint8_t* row = stg + lane * 128;
#pragma unroll
              for (int j = 0; j < 8; ++j)
                *reinterpret_cast<float4*>(row + ((j ^ (lane & 7)) << 4)) =
                    make_float4(f[4 * j], f[4 * j + 1], f[4 * j + 2], f[4 * j + 3]);
            }
            __syncwarp();
            if (rmw) {
              if (wptr && p.upd.kind != 0) {
                // Adam: the element's two moments live beside the weight (fp32, same layout), 16 bytes each per lane;
                // two passes of four pieces keep the registers in bounds
#pragma unroll
                for (int h4 = 0; h4 < 8; h4 += 4) {
                  float4 mo[4], va[4];
#pragma unroll
                  for (int i = 0; i < 4; ++i) {
                    const int r = (h4 + i) * 4 + (lane >> 3);
                    const int64_t at = (yb + r) * p.ldc + col;
                    if (yb + r < y_lim) {
                      mo[i] = *reinterpret_cast<const float4*>(momptr + at);
                      va[i] = *reinterpret_cast<const float4*>(varptr + at);
                    }
                  }
#pragma unroll
                  for (int i = 0; i < 4; ++i) {
                    const int r = (h4 + i) * 4 + (lane >> 3);
                    const int64_t at = (yb + r) * p.ldc + col;
                    if (yb + r >= y_lim) continue;
                    const float4 v = *reinterpret_cast<const float4*>(stg + r * 128 + ((piece ^ (r & 7)) << 4));
                    float4 w4 = mptr ? as_f4(ld[h4 + i]) : bf_f4(ld[h4 + i]);
                    w4.x = upd_step(p.upd, w4.x, v.x, &mo[i].x, &va[i].x);
                    w4.y = upd_step(p.upd, w4.y, v.y, &mo[i].y, &va[i].y);
                    w4.z = upd_step(p.upd, w4.z, v.z, &mo[i].z, &va[i].z);
                    w4.w = upd_step(p.upd, w4.w, v.w, &mo[i].w, &va[i].w);
                    *reinterpret_cast<float4*>(momptr + at) = mo[i];
                    *reinterpret_cast<float4*>(varptr + at) = va[i];
                    if (mptr) *reinterpret_cast<float4*>(mptr + at) = w4;
                    uint2 out;
                    __nv_bfloat162 h2 = __floats2bfloat162_rn(w4.x, w4.y);
                    out.x = *reinterpret_cast<uint32_t*>(&h2);
                    h2 = __floats2bfloat162_rn(w4.z, w4.w);
                    out.y = *reinterpret_cast<uint32_t*>(&h2);
                    *reinterpret_cast<uint2*>(wptr + at) = out;
                  }
                }
              } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                  const int r = i * 4 + (lane >> 3);
                  const int64_t at = (yb + r) * p.ldc + col;
                  if (yb + r >= y_lim) continue;
                  const float4 v = *reinterpret_cast<const float4*>(stg + r * 128 + ((piece ^ (r & 7)) << 4));
                  if (!wptr) {          // accumulate into the stored gradient
                    const float4 o = as_f4(ld[i]);
                    *reinterpret_cast<float4*>(cptr + at) = make_float4(o.x + v.x, o.y + v.y, o.z + v.z, o.w + v.w);
                    continue;
                  }
                  // fused SGD step on the weight tile this gradient tile belongs to; the gradient is not stored
                  float4 w4 = mptr ? as_f4(ld[i]) : bf_f4(ld[i]);
                  w4.x -= p.upd.lr * v.x; w4.y -= p.upd.lr * v.y; w4.z -= p.upd.lr * v.z; w4.w -= p.upd.lr * v.w;
                  if (mptr) *reinterpret_cast<float4*>(mptr + at) = w4;
                  uint2 out;
                  __nv_bfloat162 h2 = __floats2bfloat162_rn(w4.x, w4.y);
                  out.x = *reinterpret_cast<uint32_t*>(&h2);
                  h2 = __floats2bfloat162_rn(w4.z, w4.w);
                  out.y = *reinterpret_cast<uint32_t*>(&h2);
                  *reinterpret_cast<uint2*>(wptr + at) = out;
                }
              }
            } else {
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const int r = i * 4 + (lane >> 3);
                const float4 v = *reinterpret_cast<const float4*>(stg + r * 128 + ((piece ^ (r & 7)) << 4));
                if (yb + r < y_lim) *reinterpret_cast<float4*>(cptr + (yb + r) * p.ldc + col) = v;
              }
            }
            __syncwarp();
          } else {
            const uint32_t off = (n_grp & 1u) * 2048u;
            if (lane == 0) bulk_wait_read<1>();
            __syncwarp();
            stage32_bf16(stg + off, lane, f);
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
              tma_store_2d(&map_c, stg_u32 + off, n, y0);
              bulk_commit();
            }
            ++n_grp;
          }
        }
      } else if constexpr (EPI == EPI_HEADS) {
        // Columns are heads of 128: the tile holds two (or, ragged, one).  This warp's 32-column blocks c and c + 64
        // are the two halves of a rotated pair range: bias, rotation by the position's angles, bf16, and out as
        // 64-byte pieces of the row's place in the head-major tensor.
        uint32_t r1[32];
        const int seq = m_ok ? m / p.hm_S : 0, pos = m_ok ? m % p.hm_S : 0;
        const int n_heads = p.N / 128;
#pragma unroll 1
        for (int c = half * 32; c < t.ncols; c += 128) {
          if (!slab_ok) continue;      // warp-uniform
          const int n = t.n0 + c;      // first column of the lower half-range; n + 64 is its partner
          __syncwarp();                // lanes past the last row skipped the previous block's stores: rejoin before the warp-wide loads
          tmem_ld32(taddr + c, r0);
          tmem_ld32(taddr + c + 64, r1);
          tmem_ld_wait();
          if (!m_ok) continue;
          const int head = n / 128, i0 = n % 128;            // i0 is 0 or 32
          bf16* dst = reinterpret_cast<bf16*>(p.C) + (((int64_t)seq * n_heads + head) * p.hm_Sp + pos) * 128 + i0;
          float y0[32], y1[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) { y0[i] = __uint_as_float(r0[i]); y1[i] = __uint_as_float(r1[i]); }
          if (p.hm_bias) {
            const float4* b0 = reinterpret_cast<const float4*>(p.hm_bias + n);        // the same for every lane
            const float4* b1 = reinterpret_cast<const float4*>(p.hm_bias + n + 64);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float4 u = b0[i], v = b1[i];
              y0[4 * i] += u.x; y0[4 * i + 1] += u.y; y0[4 * i + 2] += u.z; y0[4 * i + 3] += u.w;
              y1[4 * i] += v.x; y1[4 * i + 1] += v.y; y1[4 * i + 2] += v.z; y1[4 * i + 3] += v.w;
            }
          }
          if (p.hm_cs) {
            const float4* cs2 = reinterpret_cast<const float4*>(p.hm_cs + pos * 64 + i0);   // two (cos, sin) pairs per load
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float4 cs = cs2[i];
              const float a0 = y0[2 * i], b0v = y1[2 * i], a1 = y0[2 * i + 1], b1v = y1[2 * i + 1];
              y0[2 * i] = a0 * cs.x - b0v * cs.y;         y1[2 * i] = b0v * cs.x + a0 * cs.y;
              y0[2 * i + 1] = a1 * cs.z - b1v * cs.w;     y1[2 * i + 1] = b1v * cs.z + a1 * cs.w;
            }
          }
          store32_bf16(dst, y0);
          store32_bf16(dst + 64, y1);
        }
      } else if constexpr (EPI == EPI_SWIGLU) {
        // columns [0, MMA_N/2) hold the gate projection, [MMA_N/2, MMA_N) the up projection.
        // H (times the row's scale, when one is given: the routed experts' gate weight) goes out through two
        // alternating 2 KB staging buffers and TMA stores; when the a|b copy is wanted too, a|b and H take turns
        // in the staging area.  (Plain line-wide stores for the a|b copy measured 0.01 ms slower per launch.)
        uint32_t r1[32];
        float g[32];
        const float rs = (p.rowscale && m_ok) ? p.rowscale[m] : 1.f;
#pragma unroll 1
        for (int c = half * 32; c < MMA_N / 2; c += 64) {
          const int n = t.n0 + c;
          if (!slab_ok) continue;      // warp-uniform
          tmem_ld32(taddr + c, r0);
          tmem_ld32(taddr + MMA_N / 2 + c, r1);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            f[i] = __uint_as_float(r0[i]);
            g[i] = __uint_as_float(r1[i]);
          }
          if (p.fp8) {
            // e4m3 operands: the sums of code products times the row's and the columns' scales
            const float sa = m_ok ? p.a_scale[m] : 0.f;
            const int64_t col0 = (p.group_mode == GROUP_M ? (int64_t)t.group * p.N : 0) + n;
            const float4* s0 = reinterpret_cast<const float4*>(p.b_scale0 + col0);      // the same for every lane
            const float4* s1 = reinterpret_cast<const float4*>(p.b_scale1 + col0);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float4 u0 = s0[i], u1 = s1[i];
              f[4 * i] *= sa * u0.x; f[4 * i + 1] *= sa * u0.y; f[4 * i + 2] *= sa * u0.z; f[4 * i + 3] *= sa * u0.w;
              g[4 * i] *= sa * u1.x; g[4 * i + 1] *= sa * u1.y; g[4 * i + 2] *= sa * u1.z; g[4 * i + 3] *= sa * u1.w;
            }
          }
          if (p.C1) {
            // the a|b copy goes first, through the whole staging area; H follows once that store has read it
            if (lane == 0) bulk_wait_read<0>();
            __syncwarp();
            stage32_bf16(stg, lane, f);
            stage32_bf16(stg + 2048, lane, g);
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
              tma_store_2d(&map_c1, stg_u32, n, y0);
              tma_store_2d(&map_c1, stg_u32 + 2048, p.N + n, y0);
              bulk_commit();
            }
          }
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const float2 A = make_float2(f[i], f[i + 1]);
            const float2 Hh = __fmul2_rn(__fmul2_rn(__fmul2_rn(A, sigmoid_approx2(A)), make_float2(g[i], g[i + 1])), make_float2(rs, rs));
            f[i] = Hh.x; f[i + 1] = Hh.y;
          }
          const uint32_t off = p.C1 ? 0u : (n_grp & 1u) * 2048u;
          if (lane == 0) { if (p.C1) bulk_wait_read<0>(); else bulk_wait_read<1>(); }
          __syncwarp();
          stage32_bf16(stg + off, lane, f);
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_store_2d(&map_c, stg_u32 + off, n, y0);
            bulk_commit();
          }
          ++n_grp;
        }
      } else {   // EPI_DSWIGLU
        // Per 32-column block: a|b arrive in distributed form by plain 16-byte loads (the next block's are in
        // flight during this block's arithmetic), pass through the staging area into row-per-lane form, da|db are
        // written over them there and leave by plain line-wide stores.  Nothing in this path queues behind the
        // load warp's operand traffic in the copy engine or waits for a bulk store to drain, which is what
        // bounded the first version of this epilogue (a|b by TMA, two sets, three bulk stores per block).
        const float rs = (p.rowscale && m_ok) ? p.rowscale[m] : 1.f;
        float2 dg2 = make_float2(0.f, 0.f);
#pragma unroll 1
        for (int c = half * 32; c < t.ncols; c += 64) {
          if (!slab_ok) continue;      // warp-uniform
          blk_dist_to_stage(stg, lane, ds_a);
          blk_dist_to_stage(stg + 2048, lane, ds_b);
          __syncwarp();
          if (c + 64 < t.ncols) {
            blk_load_dist(ds_blk + c + 64, p.ld_ab, rows_ok, lane, ds_a);
            blk_load_dist(ds_blk + p.N + c + 64, p.ld_ab, rows_ok, lane, ds_b);
          }
          tmem_ld32(taddr + c, r0);
          tmem_ld_wait();
          uint8_t* row_a = stg + lane * 64;
          uint8_t* row_b = stg + 2048 + lane * 64;
          const int sw = (lane >> 1) & 3;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            float a[8], b[8];
            unpack8(*reinterpret_cast<const uint4*>(row_a + ((j ^ sw) << 4)), a);
            unpack8(*reinterpret_cast<const uint4*>(row_b + ((j ^ sw) << 4)), b);
            // two elements at a time on the packed fp32 pipe (half the instructions of the scalar form)
#pragma unroll
            for (int i = 0; i < 8; i += 2) {
              const float2 A = make_float2(a[i], a[i + 1]), B = make_float2(b[i], b[i + 1]);
              const float2 V = make_float2(__uint_as_float(r0[8 * j + i]), __uint_as_float(r0[8 * j + i + 1]));
              const float2 S = sigmoid_approx2(A);
              const float2 SI = __fmul2_rn(A, S);                         // silu(a)
              const float2 DH = __fmul2_rn(make_float2(rs, rs), V);       // dL/dH of this row
              dg2 = __ffma2_rn(V, __fmul2_rn(SI, B), dg2);                // <dH', H>: gradient of the row's gate weight
              // da = dh b silu'(a), silu'(a) = s (1 + a (1 - s)) = s (1 + a - silu(a));  db = dh silu(a)
              const float2 T1 = __fadd2_rn(__fadd2_rn(A, make_float2(1.f, 1.f)), make_float2(-SI.x, -SI.y));
              const float2 DA = __fmul2_rn(__fmul2_rn(DH, B), __fmul2_rn(S, T1));
              const float2 DB = __fmul2_rn(DH, SI);
              a[i] = DA.x; a[i + 1] = DA.y; b[i] = DB.x; b[i + 1] = DB.y;
            }
            *reinterpret_cast<uint4*>(row_a + ((j ^ sw) << 4)) = pack8(a);
            *reinterpret_cast<uint4*>(row_b + ((j ^ sw) << 4)) = pack8(b);
          }
          __syncwarp();
          blk_stage_to_global(stg, lane, ds_blk + c, p.ld_ab, rows_ok);
          blk_stage_to_global(stg + 2048, lane, ds_blk + p.N + c, p.ld_ab, rows_ok);
          __syncwarp();
        }
        if (p.dg_part && m_ok) p.dg_part[(int64_t)m * p.dg_ld + 2 * (t.n0 / P.tile_n) + half] = dg2.x + dg2.y;
      }
      // accumulator may be overwritten by the MMA warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if constexpr (PAIR) mbar_arrive_cluster(mapa_u32(tempty_bar(acc), 0));   // the even CTA's MMA warp waits for both
        else mbar_arrive(tempty_bar(acc));
      }
    }
    // this lane's stores must be complete (shared memory read, global memory written) before the CTA exits
    if (lane == 0) bulk_wait_all();
  }

  // ------------------------------------------------------------------ teardown
  __syncthreads();
  if (*abort_flag && threadIdx.x == 0) {
    // loads already issued into this CTA's shared memory must land before the CTA exits
    bool unannounced = false;     // the second load warp issued into a stage whose bytes the first never announced
    for (int s = 0; s < Cfg::STAGES; ++s) {
      if (issued_b[s] != 0 && issued_b[s] != issued[s]) unannounced = true;
      if (issued[s] == 0) continue;
      long long t0 = clock64();
      while (!mbar_try_wait(full_bar(s), (uint32_t)(issued[s] - 1)) && clock64() - t0 < P.wait_cycles) {}
    }
    if (unannounced) {            // that stage's barrier cannot complete: give its loads a bounded time to land
      const long long t0 = clock64();
      while (clock64() - t0 < 4000000LL) {}
    }
  }
  __syncthreads();
  if constexpr (PAIR) {
    // After an abandoned wait, loads of this CTA may still be in flight (their completion is counted on the
    // even CTA's barriers, so the per-stage drain above does not see them): give them a bounded time to land.
    if (*abort_flag) {
      const long long t0 = clock64();
      while (clock64() - t0 < 4000000LL) {}
    }
    // neither CTA frees tensor memory or leaves while the other may still signal its barriers or
    // have MMAs in flight that write its accumulators
    tc_fence_before();
    cluster_sync_all();
  }
  if (warp == 1) {
    tc_fence_after();
    if constexpr (PAIR)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)Cfg::TMEM_COLS)
                   : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)Cfg::TMEM_COLS)
                   : "memory");
  }
}

// ---------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Per-device set-up state (kernel attributes and the SM count belong to a device, not to the process).
struct TcState {
  EncodeTiledFn encode = nullptr;
  int n_sms = 0;
  bool ready = false;
};
constexpr int TC_MAX_DEVICES = 64;
// State of the current device; devices beyond the table share the last slot and are refused by tc_prepare.
inline TcState& tc_state() {
  static TcState s[TC_MAX_DEVICES + 1];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= TC_MAX_DEVICES) dev = TC_MAX_DEVICES;
  return s[dev];
}

template <int MMA_N, int EPI>
inline cudaError_t tc_set_attr() {
  cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<MMA_N, EPI, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       TcCfg<MMA_N, EPI, false>::SMEM_BYTES);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(gemm_tc_kernel<MMA_N, EPI, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              TcCfg<MMA_N, EPI, true>::SMEM_BYTES);
}

// Once per device (under a lock: two host threads may arrive together): driver entry point for tensor-map
// encoding, SM count, shared-memory opt-in of every kernel instance.
inline int tc_prepare() {
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  TcState& s = tc_state();
  if (s.ready) return REVFFN_OK;
  {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return REVFFN_ERR_CUDA;
    if (dev < 0 || dev >= TC_MAX_DEVICES) return REVFFN_ERR_UNSUPPORTED;
  }
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn)
    return REVFFN_ERR_CUDA;
  s.encode = reinterpret_cast<EncodeTiledFn>(fn);
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return REVFFN_ERR_CUDA;
  if (cudaDeviceGetAttribute(&s.n_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return REVFFN_ERR_CUDA;
  cudaError_t e = cudaSuccess;
  if (e == cudaSuccess) e = tc_set_attr<256, EPI_STORE>();
  if (e == cudaSuccess) e = tc_set_attr<256, EPI_SWIGLU>();
  if (e == cudaSuccess) e = tc_set_attr<256, EPI_ROWSCALE>();
  if (e == cudaSuccess) e = tc_set_attr<256, EPI_COUPLE>();
  if (e == cudaSuccess) e = tc_set_attr<256, EPI_DSWIGLU>();
  if (e == cudaSuccess) e = tc_set_attr<256, EPI_WGRAD>();
  if (e == cudaSuccess) e = tc_set_attr<256, EPI_HEADS>();
  if (e != cudaSuccess) return REVFFN_ERR_CUDA;
  s.ready = true;
  return REVFFN_OK;
}

// 2D bf16 tensor map: `inner` contiguous elements per row, `outer` rows of stride ld elements.
// u8 = true: one-byte elements (e4m3 codes), box_inner counts bytes.
inline int tc_make_map(CUtensorMap* map, const void* ptr, uint64_t inner, uint64_t outer, uint64_t ld,
                       uint32_t box_inner, uint32_t box_outer, bool u8 = false) {
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {ld * (u8 ? 1u : 2u)};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = tc_state().encode(map, u8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box,
                                 estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? REVFFN_OK : REVFFN_ERR_CUDA;
}

// Tensor map of an MN-major bf16 operand ([rows, ld] in memory, rows = K) seen as {64 columns, rows, ld / 64
// column groups}: a box of 64 x 64 x 2 is 128 columns of 64 K rows, delivered as two 8 KB blocks of 64 columns.
inline int tc_make_map_mn3d(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t ld) {
  cuuint64_t dims[3] = {64, rows, ld / 64};
  cuuint64_t strides[2] = {ld * 2u, 128u};
  cuuint32_t box[3] = {64, 64, 2};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = tc_state().encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? REVFFN_OK : REVFFN_ERR_CUDA;
}

// Tensor map of an epilogue output: boxes of 32 rows x 64 bytes (32 bf16 or 16 fp32 columns),
// 64-byte swizzle.
inline int tc_make_out_map(CUtensorMap* map, const void* ptr, bool f32, uint64_t inner, uint64_t outer, uint64_t ld) {
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {ld * (f32 ? 4u : 2u)};
  cuuint32_t box[2] = {f32 ? 16u : 32u, 32};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = tc_state().encode(map, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                                 const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                 CU_TENSOR_MAP_SWIZZLE_64B,
                                 CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? REVFFN_OK : REVFFN_ERR_CUDA;
}

inline int tc_dg_parts(int N) { return 2 * (int)ceil_div(N, 256); }   // two epilogue warps per row and column tile

template <int MMA_N, int EPI>
inline int tc_launch(const TcParams& P, const CUtensorMap& ma, const CUtensorMap& mb0, const CUtensorMap& mb1,
                     const CUtensorMap& mc, const CUtensorMap& mc1, int grid, bool pair, cudaStream_t st) {
  if (!pair) {
    gemm_tc_kernel<MMA_N, EPI, false><<<grid, TC_THREADS, TcCfg<MMA_N, EPI, false>::SMEM_BYTES, st>>>(P, ma, mb0, mb1, mc, mc1);
    return cudaGetLastError() == cudaSuccess ? REVFFN_OK : REVFFN_ERR_CUDA;
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(TC_THREADS);
  cfg.dynamicSmemBytes = TcCfg<MMA_N, EPI, true>::SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = 2;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<MMA_N, EPI, true>, P, ma, mb0, mb1, mc, mc1) == cudaSuccess
             ? REVFFN_OK : REVFFN_ERR_CUDA;
}

inline int launch_gemm_tc(const GemmProblem& p, cudaStream_t st) {
  TcState& s = tc_state();
  if (!s.ready) return REVFFN_ERR_CUDA;
  if (p.M <= 0 || p.N <= 0) return REVFFN_OK;
  const int mma_n = 256;
  TcParams P;
  P.p = p;
  P.tile_n = (p.concat == CONCAT_N) ? mma_n / 2 : mma_n;
  P.tiles_m = (int)ceil_div(p.M, TC_BM);
  P.tiles_n = (int)ceil_div(p.N, P.tile_n);
  const bool f8 = p.fp8 != 0;
  P.bk = f8 ? 2 * TC_BK : TC_BK;
  P.k_blocks = (int)ceil_div(p.K, P.bk);
  if (f8) {
    // e4m3 operands: K-major on both sides, the SwiGLU pair (one CTA per tile) or the transposed store
    if (p.a_mn_major || p.b_mn_major || p.concat == CONCAT_K || !p.a_scale || !p.b_scale0 ||
        (p.concat == CONCAT_N && !p.b_scale1) || p.lda % 16 != 0 || p.ldb % 16 != 0 || p.K % 16 != 0)
      return REVFFN_ERR_UNSUPPORTED;
    if (!((p.epilogue == EPI_SWIGLU && p.group_mode == GROUP_M && !p.C1) ||
          (p.epilogue == EPI_STORE && !p.out_f32 && p.group_mode == GROUP_M && p.tok_chunks)))
      return REVFFN_ERR_UNSUPPORTED;
  }
  P.wait_cycles = p.dbg_wait_cycles > 0 ? p.dbg_wait_cycles : TC_WAIT_CYCLES;
  P.starve = p.dbg_starve;
  // Two load threads in every mode: measured against one thread in the same process, alternating, the whole step
  // is 4-5 % faster and no product is slower (the one-thread form stays selectable for such measurements).
  P.split_loads = p.dbg_split_loads != 2;
  if (p.dbg_starve && !p.no_pair) return REVFFN_ERR_UNSUPPORTED;      // the starved-wait test runs one CTA per tile
  if (p.N % 128 != 0) return REVFFN_ERR_SHAPE;
  // K need not be a multiple of the 64-wide K step: the tensor maps end at K, so the rest of the last
  // step is loaded as zeros (K-major rows must still start on 16-byte boundaries: lda, ldb)
  if (p.concat == CONCAT_K && (P.k_blocks & 1)) return REVFFN_ERR_SHAPE;
  // fp32 accumulator; operand formats bf16 (1) for kind::f16, e4m3 (0) for kind::f8f6f4
  const uint32_t fmt = f8 ? 0u : ((1u << 7) | (1u << 10));
  P.idesc = (1u << 4) | fmt | ((uint32_t)(p.a_mn_major ? 1 : 0) << 15) |
            ((uint32_t)(p.b_mn_major ? 1 : 0) << 16) | ((uint32_t)(mma_n >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);

  // 3-D views of the MN-major operands need whole 64-column groups everywhere
  P.mn3d = !p.dbg_mn_boxes && (!p.a_mn_major || (p.lda % 64 == 0 && p.a_col0 % 64 == 0)) && (!p.b_mn_major || (p.ldb % 64 == 0 && p.b_col0 % 64 == 0));
  const int groups = p.n_groups > 0 ? p.n_groups : 1;
  CUtensorMap ma, mb0, mb1;
  const int k_half = (p.concat == CONCAT_K) ? p.K / 2 : p.K;
  auto operand_maps = [&](bool mn3d) -> int {
    // A
    if (!p.a_mn_major) {
      // [rows, K]: dense M rows, or the padded row space for GROUP_M
      int r = tc_make_map(&ma, p.A, (uint64_t)p.K, (uint64_t)p.M, (uint64_t)p.lda, f8 ? 128 : 64, 128, f8);
      if (r) return r;
    } else {
      // [K rows, lda columns]; K rows = tokens (dense) or the bound on padded rows (GROUP_K)
      int r = mn3d ? tc_make_map_mn3d(&ma, p.A, (uint64_t)p.K, (uint64_t)p.lda)
                   : tc_make_map(&ma, p.A, (uint64_t)p.lda, (uint64_t)p.K, (uint64_t)p.lda, 64, 64);
      if (r) return r;
    }
    // B
    if (!p.b_mn_major) {
      uint64_t rows = (p.group_mode == GROUP_M) ? (uint64_t)groups * p.N : (uint64_t)p.N;
      int r = tc_make_map(&mb0, p.B0, (uint64_t)k_half, rows, (uint64_t)p.ldb, f8 ? 128 : 64, 128, f8);
      if (r) return r;
      r = tc_make_map(&mb1, p.B1 ? p.B1 : p.B0, (uint64_t)k_half, rows, (uint64_t)p.ldb, f8 ? 128 : 64, 128, f8);
      if (r) return r;
    } else {
      uint64_t rows = (p.group_mode == GROUP_M) ? (uint64_t)groups * k_half : (uint64_t)p.K;
      int r = mn3d ? tc_make_map_mn3d(&mb0, p.B0, rows, (uint64_t)p.ldb)
                   : tc_make_map(&mb0, p.B0, (uint64_t)p.ldb, rows, (uint64_t)p.ldb, 64, 64);
      if (r) return r;
      r = mn3d ? tc_make_map_mn3d(&mb1, p.B1 ? p.B1 : p.B0, rows, (uint64_t)p.ldb)
               : tc_make_map(&mb1, p.B1 ? p.B1 : p.B0, (uint64_t)p.ldb, rows, (uint64_t)p.ldb, 64, 64);
      if (r) return r;
    }
    return REVFFN_OK;
  };
  // should the driver not take the 3-D view (its column-group stride is smaller than its row stride), the 64 x 64
  // boxes of the plain 2-D maps do the same work with twice the loads
  if (P.mn3d && operand_maps(true) != REVFFN_OK) P.mn3d = 0;
  if (!P.mn3d) {
    int r = operand_maps(false);
    if (r) return r;
  }
  // epilogue outputs written through TMA stores
  CUtensorMap mc, mc1;
  memset(&mc, 0, sizeof(mc));
  memset(&mc1, 0, sizeof(mc1));
  if (p.epilogue == EPI_HEADS) {
    // plain stores into the head-major tensor, no output map
    if (p.group_mode != 0 || p.N % 128 != 0 || p.hm_S <= 0 || p.hm_Sp < p.hm_S || (reinterpret_cast<uintptr_t>(p.C) & 15u))
      return REVFFN_ERR_SHAPE;
  } else if (p.epilogue == EPI_DSWIGLU) {
    // a|b are read and rewritten in place with plain 16-byte accesses, no tensor map
    if ((reinterpret_cast<uintptr_t>(p.ab) & 15u) || (p.ld_ab * 2) % 16 != 0) return REVFFN_ERR_ALIGN;
    if (p.C1) return REVFFN_ERR_UNSUPPORTED;
  } else {
    const bool f32_out = p.epilogue == EPI_COUPLE || p.epilogue == EPI_WGRAD || (p.epilogue == EPI_STORE && p.out_f32);
    uint64_t rows = (uint64_t)p.M;
    if (p.group_mode == GROUP_K) {
      // group g's block must start g * M rows further down one 2D tensor (g * split_m rows with two outputs)
      const int64_t m_out = p.split_m > 0 ? p.split_m : p.M;
      if (p.M % TC_BM != 0 || p.c_group_stride != m_out * p.ldc) return REVFFN_ERR_SHAPE;
      rows = (uint64_t)groups * p.M;
    }
    if (p.split_m > 0 && (p.epilogue != EPI_WGRAD || p.M != 2 * p.split_m || p.split_m % TC_BM != 0)) return REVFFN_ERR_SHAPE;
    if (p.epilogue == EPI_WGRAD && p.upd_w) {
      // fused update: the weights (and master copies) are read and rewritten 8 / 16 bytes at a time
      if ((reinterpret_cast<uintptr_t>(p.upd_w) & 15u) || (reinterpret_cast<uintptr_t>(p.upd_w2) & 15u) ||
          (reinterpret_cast<uintptr_t>(p.upd_m) & 15u) || (reinterpret_cast<uintptr_t>(p.upd_m2) & 15u) ||
          (reinterpret_cast<uintptr_t>(p.upd_mom) & 15u) || (reinterpret_cast<uintptr_t>(p.upd_mom2) & 15u) ||
          (reinterpret_cast<uintptr_t>(p.upd_var) & 15u) || (reinterpret_cast<uintptr_t>(p.upd_var2) & 15u) || p.ldc % 4 != 0)
        return REVFFN_ERR_ALIGN;
      if (p.split_m > 0 && !p.upd_w2) return REVFFN_ERR_NULL;
      if (p.upd.kind == 1 && (!p.upd_mom || !p.upd_var || (p.split_m > 0 && (!p.upd_mom2 || !p.upd_var2)))) return REVFFN_ERR_NULL;
    } else {
      if (!p.C || (p.split_m > 0 && !p.C2)) return REVFFN_ERR_NULL;
      if ((reinterpret_cast<uintptr_t>(p.C) & 15u) || (reinterpret_cast<uintptr_t>(p.C2) & 15u) || (p.ldc * (f32_out ? 4 : 2)) % 16 != 0)
        return REVFFN_ERR_ALIGN;
    }
    if (!f32_out) {      // fp32 outputs leave through plain stores and need no map
      int r = tc_make_out_map(&mc, p.C, false, (uint64_t)p.N, rows, (uint64_t)p.ldc);
      if (r) return r;
    }
    int r = 0;
    if (p.epilogue == EPI_SWIGLU && p.C1) {
      if ((reinterpret_cast<uintptr_t>(p.C1) & 15u) || (p.ldc1 * 2) % 16 != 0) return REVFFN_ERR_ALIGN;
      r = tc_make_out_map(&mc1, p.C1, false, (uint64_t)2 * p.N, (uint64_t)p.M, (uint64_t)p.ldc1);
      if (r) return r;
    }
  }
  // Pair mode wherever a 256-row tile cannot straddle two experts and every column tile is 256 wide.
  // (a ragged 128-wide last tile splits into 64-column halves, which only the [K, N] storage of B can load)
  const bool tr = p.group_mode == GROUP_M && p.tok_chunks != nullptr && p.N % 256 == 0 && !p.a_mn_major &&
                  p.concat != CONCAT_N && !p.no_pair && s.n_sms % 2 == 0 &&
                  (p.epilogue == EPI_ROWSCALE || (p.epilogue == EPI_STORE && !p.out_f32));
  const bool pair = tr || (p.group_mode != GROUP_M && (p.N % 256 == 0 || p.b_mn_major) && !p.no_pair);
  if (f8 && p.epilogue == EPI_STORE && !tr) return REVFFN_ERR_UNSUPPORTED;      // only the transposed store scales its accumulator
  P.tr = tr ? 1 : 0;
  P.tiles_f = p.N / 256;
  int64_t total = (int64_t)P.tiles_m * P.tiles_n * (p.group_mode == GROUP_K ? groups : 1);
  int grid = (int)(total < s.n_sms ? total : s.n_sms);
  if (tr) {
    // the number of token chunks is only known on the device: a full persistent grid
    grid = s.n_sms;
    P.idesc = (1u << 4) | fmt | ((uint32_t)(p.b_mn_major ? 1 : 0) << 15) |
              ((uint32_t)(p.a_mn_major ? 1 : 0) << 16) | ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(2 * TC_BM >> 4) << 24);
  } else if (pair) {
    total = (int64_t)((P.tiles_m + 1) / 2) * P.tiles_n * (p.group_mode == GROUP_K ? groups : 1);
    const int64_t pairs = total < s.n_sms / 2 ? total : s.n_sms / 2;
    grid = (int)(2 * pairs);
    P.idesc = (P.idesc & ~(0x1Fu << 24)) | ((uint32_t)(2 * TC_BM >> 4) << 24);   // M = 256 across the pair
  }
  if (grid <= 0) return REVFFN_OK;

#define TC_CASE(N_, E_) \
  if (mma_n == N_ && p.epilogue == E_) return tc_launch<N_, E_>(P, ma, mb0, mb1, mc, mc1, grid, pair, st);
  TC_CASE(256, EPI_STORE) TC_CASE(256, EPI_SWIGLU) TC_CASE(256, EPI_ROWSCALE) TC_CASE(256, EPI_COUPLE)
  TC_CASE(256, EPI_DSWIGLU) TC_CASE(256, EPI_WGRAD) TC_CASE(256, EPI_HEADS)
#undef TC_CASE
  return REVFFN_ERR_UNSUPPORTED;
}

}  // namespace revffn
