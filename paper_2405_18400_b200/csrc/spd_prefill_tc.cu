// Long-prefix prefill (the dense pass over the prefix that precedes Eq. 1): blocks of 128..512 prefix tokens at a
// time, their matrix products on the fifth-generation tensor cores (tcgen05.mma, operands staged in shared
// memory by tiled TMA copies, float32 accumulators in tensor memory), everything between the products in small
// row-wise kernels.  Only the cache is produced here: the prefix's last tokens, the LM head and the first
// timestep stay with spd_prefill_kernel, which finds these positions in the cache like any earlier launch's.
//
// Product: Y[token][row] = sum_c X[token][c] W[row][c], W bf16 [rows][cols] as stored, X float32 activations
// split exactly into three bf16 terms (x = hi + mid + lo, 8 + 8 + 8 significant bits), so that the tensor
// cores see exact operands and the float32 accumulator receives what a float32 product would.  One block
// computes a tile of 128 tokens x 128 rows: a producer thread fills a ring of stages (three term tiles of
// 128 tokens x 64 columns and one weight tile of 128 rows x 64 columns, all in the 128-byte-swizzled K-major
// layout the tensor cores read), one thread issues the 12 instructions of a stage (3 terms x 4 k-steps of 16
// columns) and hands the stage back with tcgen05.commit; four accumulators take turns, each the sum of 8 stages,
// and four warps add those sums in registers (round-to-nearest) and write the tile to global memory.  Every wait is bounded; a wait that runs out records SPD_ETIMEOUT in the
// context's state, the block waits for its copies in flight, frees its tensor memory and returns.
#include <cuda_runtime.h>
#include <math_constants.h>

#include "spd_params.h"
#include "spd_prefill_tc.h"
#include "spd_ptx.cuh"

namespace spd {

constexpr int kTcM = 128;                      // tokens of a tile = lanes of tensor memory
constexpr int kTcN = 128;                      // weight rows of a tile = float32 columns of tensor memory
constexpr int kTcKB = 64;                      // columns per stage: one 128-byte swizzle row of bf16
constexpr int kTcTermBytes = kTcM * kTcKB * 2; // one term tile
constexpr int kTcWBytes = kTcN * kTcKB * 2;
constexpr int kTcStageBytes = 3 * kTcTermBytes + kTcWBytes;  // 64 KB
constexpr int kTcStages = 3;
constexpr int kTcThreads = 192;                // producer warp, issuing warp, four warps for the accumulator
constexpr int kTcWBoxRows = 32;                // the weights' tensor maps describe boxes of 32 rows x 64 columns
constexpr int kTcSegSteps = 8;                 // stages summed inside tensor memory before the sum moves to registers
constexpr int kTcAccs = 4;                     // accumulators in rotation: 4 x 128 columns = all of tensor memory
constexpr unsigned long long kTcWaitNs = 1500ull * 1000ull * 1000ull;

// ---------------------------------------------------------------- PTX: tensor memory and tcgen05
__device__ __forceinline__ void tc_box_load(uint32_t dst, const void *tmap, int x, int y, uint64_t *bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
               "l"(tmap), "r"(x), "r"(y), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// Whole warp: allocates `cols` columns (a power of two >= 32) of tensor memory, base address into *slot (shared).
__device__ __forceinline__ void tc_alloc(uint32_t *slot, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_dealloc(uint32_t base, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(cols) : "memory");
}
// Shared-memory operand descriptor: K-major tile whose rows are 128 bytes (64 bf16) in the 128-byte swizzle,
// groups of 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t tc_desc(uint32_t saddr) {
  uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);  // start address / 16
  d |= (uint64_t)1 << 16;                             // leading byte offset: unused for a swizzled K-major tile
  d |= (uint64_t)(1024 >> 4) << 32;                   // stride byte offset: one group of 8 rows
  d |= (uint64_t)1 << 46;                             // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                             // 128-byte swizzle
  return d;
}
// Instruction descriptor of kind::f16: float32 accumulator, bf16 x bf16, both operands K-major, M x N tile.
__device__ __forceinline__ constexpr uint32_t tc_idesc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The mbarrier receives one arrival once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void tc_commit(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 32 consecutive float32 columns of this thread's lane of tensor memory.
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// 16 consecutive float32 columns of this thread's lane of tensor memory.
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

struct TcShared {
  uint64_t full[kTcStages], empty[kTcStages], acc_full[kTcAccs], acc_empty[kTcAccs];
  uint32_t tmem_base;
  int dead;
};

// The same for the small-batch product, whose ring has up to kBgMaxStages stages.
constexpr int kBgMaxStages = 8;
struct BgShared {
  uint64_t full[kBgMaxStages], empty[kBgMaxStages], acc_full[kTcAccs], acc_empty[kTcAccs];
  uint32_t tmem_base;
  int dead;
};

// Bounded wait on an mbarrier phase; false when the block gave up (here or elsewhere).
template <typename Shared>
__device__ __forceinline__ bool tc_wait(Shared &sh, State *st, uint64_t *bar, uint32_t parity, int info) {
  if (mbar_try_wait(bar, parity)) return true;
  volatile int *dead = &sh.dead;
  unsigned long long t0 = globaltimer();
  uint32_t n = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++n & 63u) == 0) {
      if (*dead) return false;
      if (globaltimer() - t0 > kTcWaitNs) {
        if (atomicCAS(&st->err, 0, -7) == 0) st->err_info = info;
        *dead = 1;
        return false;
      }
    }
  }
  return true;
}

// Y[m0 .. m0+127][n0 .. n0+127] of Y = X W^T.  tmap_x: the term tiles, a [3 * x_term_rows][C] bf16 matrix in boxes
// of 128 rows x 64 columns (term j's tokens start at row j * x_term_rows); tmap_w: W [N][C] in boxes of 32 rows x
// 64 columns.  Rows and columns past either matrix arrive as zeros.  grid = (ceil(tokens / 128), ceil(N / 128)).
// stall (test hook): the producer announces its first stage but issues no copies for it, so the wait for that
// stage runs out.
__global__ void __launch_bounds__(kTcThreads, 1)
    spd_tc_gemm_kernel(const void *tmap_x, const void *tmap_w, float *Y, int N, int C, int x_term_rows, State *st, int stall) {
  extern __shared__ __align__(16) uint8_t tc_smem_raw[];
  uint8_t *smem = tc_smem_raw + ((1024u - (smem_u32(tc_smem_raw) & 1023u)) & 1023u);
  __shared__ TcShared sh;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nk = (C + kTcKB - 1) / kTcKB;
  const int m0 = blockIdx.x * kTcM, n0 = blockIdx.y * kTcN;  // token tiles vary fastest: blocks that share weight rows run together
  if (threadIdx.x == 0) {
    sh.dead = 0;
    for (int s = 0; s < kTcStages; ++s) {
      mbar_init(&sh.full[s], 1);
      mbar_init(&sh.empty[s], 1);
    }
    for (int a = 0; a < kTcAccs; ++a) {
      mbar_init(&sh.acc_full[a], 1);
      mbar_init(&sh.acc_empty[a], 4);  // one arrival per warp that reads the accumulator
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tc_alloc(&sh.tmem_base, kTcAccs * kTcN);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh.tmem_base;
  const uint32_t ring = smem_u32(smem);

  if (warp == 0) {
    if (lane == 0) {
      // producer: the activations were written by ordinary stores of earlier kernels on the stream
      uint32_t stage = 0, phase = 0, issued = 0;
      bool ok = true;
      for (int ks = 0; ks < nk; ++ks) {
        if (!tc_wait(sh, st, &sh.empty[stage], phase ^ 1u, 400)) { ok = false; break; }
        mbar_expect_tx(&sh.full[stage], (uint32_t)kTcStageBytes);
        const uint32_t base = ring + stage * (uint32_t)kTcStageBytes;
        if (stall && ks == 0) {
          if (++stage == (uint32_t)kTcStages) { stage = 0; phase ^= 1u; }
          continue;  // nothing in flight for this stage
        }
#pragma unroll
        for (int j = 0; j < 3; ++j) tc_box_load(base + j * kTcTermBytes, tmap_x, ks * kTcKB, j * x_term_rows + m0, &sh.full[stage]);
#pragma unroll
        for (int j = 0; j < kTcN / kTcWBoxRows; ++j)
          tc_box_load(base + 3 * kTcTermBytes + j * (kTcWBoxRows * kTcKB * 2), tmap_w, ks * kTcKB, n0 + j * kTcWBoxRows, &sh.full[stage]);
        if (issued < (uint32_t)kTcStages) ++issued;
        if (++stage == (uint32_t)kTcStages) { stage = 0; phase ^= 1u; }
      }
      if (!ok) {
        // giving up: wait (bounded) for the copies already issued, so that none lands after the block has gone
        uint32_t s = stage, ph = phase;
        for (uint32_t i = 0; i < issued; ++i) {
          if (s == 0) { s = (uint32_t)kTcStages; ph ^= 1u; }
          --s;
          unsigned long long t0 = globaltimer();
          while (!mbar_try_wait(&sh.full[s], ph) && globaltimer() - t0 < kTcWaitNs) {}
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = tc_idesc(kTcM, kTcN);
      uint32_t stage = 0, phase = 0;
      for (int ks = 0; ks < nk; ++ks) {
        const int seg = ks / kTcSegSteps, in_seg = ks - seg * kTcSegSteps, a = seg % kTcAccs;
        if (in_seg == 0 && !tc_wait(sh, st, &sh.acc_empty[a], (uint32_t)((seg / kTcAccs) & 1) ^ 1u, 430)) break;  // its last sum has been read
        if (!tc_wait(sh, st, &sh.full[stage], phase, 410)) break;
        tc_fence_after();
        const uint32_t base = ring + stage * (uint32_t)kTcStageBytes;
#pragma unroll
        for (int j = 0; j < 3; ++j)
#pragma unroll
          for (int kk = 0; kk < kTcKB / 16; ++kk)  // 16 columns = 32 bytes further into the swizzled rows
            tc_mma(tmem + (uint32_t)(a * kTcN), tc_desc(base + j * kTcTermBytes + kk * 32), tc_desc(base + 3 * kTcTermBytes + kk * 32),
                   idesc, (uint32_t)((in_seg | j | kk) != 0));
        tc_commit(&sh.empty[stage]);  // the stage is free once these have read it
        if (in_seg == kTcSegSteps - 1 || ks == nk - 1) tc_commit(&sh.acc_full[a]);  // the segment's sum is complete
        if (++stage == (uint32_t)kTcStages) { stage = 0; phase ^= 1u; }
      }
    }
    __syncwarp();
  } else {
    // The sums of kTcSegSteps stages each move from tensor memory to registers, where they are added with
    // round-to-nearest: the tensor cores add into their accumulator with truncation, whose error grows with the
    // length of the chain.  Warp w may read lanes 32 (w % 4) .. 32 (w % 4) + 31, a token per thread.
    const int quarter = warp & 3;
    float sum[kTcN];
#pragma unroll
    for (int j = 0; j < kTcN; ++j) sum[j] = 0.f;
    const int nseg = (nk + kTcSegSteps - 1) / kTcSegSteps;
    bool ok = true;
    for (int seg = 0; seg < nseg; ++seg) {
      const int a = seg % kTcAccs;
      if (!tc_wait(sh, st, &sh.acc_full[a], (uint32_t)((seg / kTcAccs) & 1), 420)) { ok = false; break; }
      tc_fence_after();
#pragma unroll
      for (int c0 = 0; c0 < kTcN; c0 += 32) {
        uint32_t r[32];
        tc_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(a * kTcN + c0), r);
#pragma unroll
        for (int j = 0; j < 32; ++j) sum[c0 + j] += __uint_as_float(r[j]);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.acc_empty[a]);
    }
    if (ok) {
      float *row = Y + (size_t)(m0 + quarter * 32 + lane) * N + n0;
#pragma unroll
      for (int j = 0; j < kTcN; j += 4)
        if (n0 + j < N) *reinterpret_cast<float4 *>(row + j) = make_float4(sum[j], sum[j + 1], sum[j + 2], sum[j + 3]);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tc_dealloc(tmem, kTcAccs * kTcN);
  }
}

// ---------------------------------------------------------------- products of a small batch
// Y[token][row] = sum_c X[token][c] W[row][c] for up to NP <= 64 token rows (the requests of a batched timestep).
// With so few tokens the product is bound by the weight stream, so the tile is turned round: the 128 weight rows
// are the wide operand of tcgen05.mma (M = 128) and the requests' terms the narrow one (N = NP), a stage holds
// 16 KB of weights and only 3 x NP x 128 bytes of terms (spd_tc_gemm_kernel, built for 128 tokens per tile, brings
// 48 KB of terms per 16 KB of weights), and the columns are split among blockIdx.y so that every product fills
// the GPU: block (x, y) adds columns [64 kb_lo, 64 kb_hi) of rows 128 x .. 128 x + 127 into its own copy of Y
// (Y + y * split_stride), which the kernels that read Y add up in a fixed order.  Accumulators as in
// spd_tc_gemm_kernel: sets of tensor-memory columns in rotation, each the sum of a segment of stages (96 additions),
// fetched by the epilogue warps and added in registers with round-to-nearest (BgShape says how many sets and
// stages for each box).  Every wait is bounded.
// Launched as a programmatic dependent (a batched timestep), a block is set up and copies the weights of its first
// stages while the kernel before it still runs; the terms, which that kernel writes, are asked for after dep_wait.
template <int NP>
struct BgShape {
  static constexpr int kTermBytes = NP * kTcKB * 2;                 // one term tile: NP token rows x 64 columns
  static constexpr int kStageBytes = kTcWBytes + 3 * kTermBytes;    // 128 weight rows x 64 columns, then the three term tiles
  // Two blocks per SM wherever they fit (91, 87 and 83 KB for NP = 16, 32, 64; NP = 128: one block of 197 KB): one
  // block's set-up and epilogue run beside the other's stages.  64 token rows with one block of five stages took
  // 6.9 ms per 7B timestep, with two blocks of two stages 5.5 ms; three blocks of fewer stages for NP <= 32 were
  // slower than two (4.4 against 4.0 ms for 8 requests).
  static constexpr int kStages = NP <= 16 ? 4 : (NP <= 32 ? 3 : (NP <= 64 ? 2 : 3));
  // Boxes of 16 and 32 rows: the three term tiles lie behind one another in a stage, 3 NP rows of one K-major operand,
  // so one instruction of N = 3 NP per 16 columns multiplies all three (a third of the instructions; an instruction
  // of N = 16 costs about as much as one of N = 48: 8 requests 3.63 -> 3.35 ms per 7B timestep).  Each term then has
  // its own NP accumulator columns, added up in the epilogue's registers, and an accumulator may take three times
  // as many stages for the same number of additions (96) before it is fetched.  Two blocks per SM share the 512
  // columns of tensor memory, so a block has 256: four accumulator sets of 48 columns, two of 96, or one of 192
  // (the product then waits while its sum is fetched, once or twice per block; the SM's other block does not).
  // Boxes of 128 rows keep one instruction per term.
  static constexpr bool kFused = NP <= 64;
  static constexpr int kAccCols = kFused ? 3 * NP : NP;  // columns of one accumulator set
  static constexpr int kAccs = NP == 32 ? 2 : (NP == 64 ? 1 : kTcAccs);  // accumulator sets in rotation
  static constexpr int kSegSteps = kFused ? 3 * kTcSegSteps : kTcSegSteps;  // stages summed in one accumulator
  static constexpr int kTmemCols = kFused ? 256 : 4 * NP;  // a power of two
  static_assert(kAccs * kAccCols <= kTmemCols && kAccs <= kTcAccs, "the accumulator sets fit the allocation and the barrier arrays");
};

template <int NP>
__global__ void __launch_bounds__(kTcThreads)
    spd_batch_gemm_kernel(const void *tmap_x, const void *tmap_w, float *Y, size_t split_stride, int n_tok, int N, int C, int x_term_rows,
                          State *st) {
  using S = BgShape<NP>;
  static_assert(S::kStages <= kBgMaxStages, "the block's mbarrier arrays hold kBgMaxStages stages");
  extern __shared__ __align__(16) uint8_t tc_smem_raw[];
  uint8_t *smem = tc_smem_raw + ((1024u - (smem_u32(tc_smem_raw) & 1023u)) & 1023u);
  __shared__ BgShared sh;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nk_all = (C + kTcKB - 1) / kTcKB;
  const int kb_lo = (int)((long long)nk_all * blockIdx.y / gridDim.y), kb_hi = (int)((long long)nk_all * (blockIdx.y + 1) / gridDim.y);
  const int nk = kb_hi - kb_lo;
  const int n0 = blockIdx.x * kTcN;
  dep_launch();
  if (threadIdx.x == 0) {
    // the two descriptors on their way before the first copies ask for them
    asm volatile("prefetch.tensormap [%0];" ::"l"(tmap_w) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(tmap_x) : "memory");
    sh.dead = 0;
    for (int s = 0; s < S::kStages; ++s) {
      mbar_init(&sh.full[s], 1);
      mbar_init(&sh.empty[s], 1);
    }
    for (int a = 0; a < kTcAccs; ++a) {
      mbar_init(&sh.acc_full[a], 1);
      mbar_init(&sh.acc_empty[a], 4);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tc_alloc(&sh.tmem_base, S::kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh.tmem_base;
  const uint32_t ring = smem_u32(smem);

  if (warp == 0) {
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, issued = 0;
      bool ok = true;
      // the first round of the ring: every stage is free; the weights go first, the terms once they are written
      const int first = nk < S::kStages ? nk : S::kStages;
      for (int ks = 0; ks < first; ++ks) {
        mbar_expect_tx(&sh.full[ks], (uint32_t)S::kStageBytes);
        const uint32_t base = ring + (uint32_t)ks * (uint32_t)S::kStageBytes;
#pragma unroll
        for (int j = 0; j < kTcN / kTcWBoxRows; ++j)
          tc_box_load(base + j * (kTcWBoxRows * kTcKB * 2), tmap_w, (kb_lo + ks) * kTcKB, n0 + j * kTcWBoxRows, &sh.full[ks]);
      }
      dep_wait();
      asm volatile("fence.proxy.async;" ::: "memory");  // the terms were written with ordinary stores
      for (int ks = 0; ks < first; ++ks) {
        const uint32_t base = ring + (uint32_t)ks * (uint32_t)S::kStageBytes;
#pragma unroll
        for (int j = 0; j < 3; ++j) tc_box_load(base + kTcWBytes + j * S::kTermBytes, tmap_x, (kb_lo + ks) * kTcKB, j * x_term_rows, &sh.full[ks]);
      }
      issued = (uint32_t)first;
      if (first == S::kStages) phase = 1u;
      else stage = (uint32_t)first;
      for (int ks = first; ks < nk; ++ks) {
        if (!tc_wait(sh, st, &sh.empty[stage], phase ^ 1u, 500)) { ok = false; break; }
        mbar_expect_tx(&sh.full[stage], (uint32_t)S::kStageBytes);
        const uint32_t base = ring + stage * (uint32_t)S::kStageBytes;
        const int col = (kb_lo + ks) * kTcKB;
#pragma unroll
        for (int j = 0; j < kTcN / kTcWBoxRows; ++j)
          tc_box_load(base + j * (kTcWBoxRows * kTcKB * 2), tmap_w, col, n0 + j * kTcWBoxRows, &sh.full[stage]);
#pragma unroll
        for (int j = 0; j < 3; ++j) tc_box_load(base + kTcWBytes + j * S::kTermBytes, tmap_x, col, j * x_term_rows, &sh.full[stage]);
        if (++stage == (uint32_t)S::kStages) { stage = 0; phase ^= 1u; }
      }
      if (!ok) {
        uint32_t s = stage, ph = phase;
        for (uint32_t i = 0; i < issued; ++i) {
          if (s == 0) { s = (uint32_t)S::kStages; ph ^= 1u; }
          --s;
          unsigned long long t0 = globaltimer();
          while (!mbar_try_wait(&sh.full[s], ph) && globaltimer() - t0 < kTcWaitNs) {}
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = tc_idesc(kTcN, S::kAccCols);  // M = 128 weight rows, N = NP token rows (x 3 terms when fused)
      uint32_t stage = 0, phase = 0;
      for (int ks = 0; ks < nk; ++ks) {
        const int seg = ks / S::kSegSteps, in_seg = ks - seg * S::kSegSteps, a = seg % S::kAccs;
        if (in_seg == 0 && !tc_wait(sh, st, &sh.acc_empty[a], (uint32_t)((seg / S::kAccs) & 1) ^ 1u, 530)) break;
        if (!tc_wait(sh, st, &sh.full[stage], phase, 510)) break;
        tc_fence_after();
        const uint32_t base = ring + stage * (uint32_t)S::kStageBytes;
        if constexpr (S::kFused) {
#pragma unroll
          for (int kk = 0; kk < kTcKB / 16; ++kk)
            tc_mma(tmem + (uint32_t)(a * S::kAccCols), tc_desc(base + kk * 32), tc_desc(base + kTcWBytes + kk * 32), idesc,
                   (uint32_t)((in_seg | kk) != 0));
        } else {
#pragma unroll
          for (int j = 0; j < 3; ++j)
#pragma unroll
            for (int kk = 0; kk < kTcKB / 16; ++kk)
              tc_mma(tmem + (uint32_t)(a * S::kAccCols), tc_desc(base + kk * 32), tc_desc(base + kTcWBytes + j * S::kTermBytes + kk * 32), idesc,
                     (uint32_t)((in_seg | j | kk) != 0));
        }
        tc_commit(&sh.empty[stage]);
        if (in_seg == S::kSegSteps - 1 || ks == nk - 1) tc_commit(&sh.acc_full[a]);
        if (++stage == (uint32_t)S::kStages) { stage = 0; phase ^= 1u; }
      }
    }
    __syncwarp();
  } else {
    // lane l of warp w reads tensor-memory lane 32 (w % 4) + l: weight row n0 + that, a token per column
    const int quarter = warp & 3;
    float sum[NP];
#pragma unroll
    for (int j = 0; j < NP; ++j) sum[j] = 0.f;
    const int nseg = (nk + S::kSegSteps - 1) / S::kSegSteps;
    bool ok = true;
    for (int seg = 0; seg < nseg; ++seg) {
      const int a = seg % S::kAccs;
      if (!tc_wait(sh, st, &sh.acc_full[a], (uint32_t)((seg / S::kAccs) & 1), 520)) { ok = false; break; }
      tc_fence_after();
#pragma unroll
      for (int c0 = 0; c0 < S::kAccCols; c0 += 16) {  // (fused: the columns of term c0 / NP, added to the same tokens' sums)
        uint32_t r[16];
        tc_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(a * S::kAccCols + c0), r);
#pragma unroll
        for (int j = 0; j < 16; ++j) sum[c0 % NP + j] += __uint_as_float(r[j]);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.acc_empty[a]);
    }
    const int row = n0 + quarter * 32 + lane;
    dep_wait();  // (long since true: the sums came from terms copied after the producer's dep_wait)
    if (ok && row < N) {
      float *out = Y + (size_t)blockIdx.y * split_stride + row;
#pragma unroll
      for (int j = 0; j < NP; ++j)
        if (j < n_tok) out[(size_t)j * N] = sum[j];  // the lanes of a warp write 32 consecutive floats of token j's row
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tc_dealloc(tmem, S::kTmemCols);
  }
}

// ---------------------------------------------------------------- row-wise kernels between the products
// v = hi + mid + lo exactly: each term takes the leading 8 significant bits of what is left, by truncation.
__device__ __forceinline__ void tc_put3(uint16_t *X, size_t term_stride, size_t at, float v) {
  const uint32_t hi = __float_as_uint(v) & 0xffff0000u;
  const float r1 = v - __uint_as_float(hi);
  const uint32_t mid = __float_as_uint(r1) & 0xffff0000u;
  const float r2 = r1 - __uint_as_float(mid);
  X[at] = (uint16_t)(hi >> 16);
  X[at + term_stride] = (uint16_t)(mid >> 16);
  X[at + 2 * term_stride] = (uint16_t)(__float_as_uint(r2) >> 16);
}

// Block sum in a fixed order (256 threads).
__device__ __forceinline__ float tc_block_sum(float v, float *scratch) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
  __syncthreads();
  float s = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) s += scratch[w];
  __syncthreads();
  return s;
}

// One token per block: the residual row (the embedding of ids[t] when `ids`, else h + y when `y`; y, like every
// product's output read below, is the sum of nz partial products zs floats apart), stored, and
// when `gain`: its RMSNorm (x * rsqrt(mean x^2 + eps) * gain) as three bf16 terms for the next product.
__global__ void __launch_bounds__(256) spd_tc_resid_norm_kernel(float *h, const float *y, const int32_t *ids, const __nv_bfloat16 *emb,
                                                                const __nv_bfloat16 *gain, uint16_t *X, size_t term_stride, int d, float eps,
                                                                int nz, size_t zs) {
  dep_wait();    // the kernel before this one in the stream wrote what this one reads
  dep_launch();  // the next one may set itself up meanwhile
  __shared__ float scratch[8];
  const int t = blockIdx.x;
  float *hr = h + (size_t)t * d;
  float ss = 0.f;
  for (int c = threadIdx.x; c < d; c += 256) {
    float v;
    if (ids) v = __bfloat162float(emb[(size_t)ids[t] * d + c]);
    else {
      v = hr[c];
      for (int z = 0; z < nz; ++z) v += y[z * zs + (size_t)t * d + c];
    }
    hr[c] = v;
    ss = fmaf(v, v, ss);
  }
  if (!gain) return;
  const float rs = rsqrtf(tc_block_sum(ss, scratch) / (float)d + eps);
  for (int c = threadIdx.x; c < d; c += 256) tc_put3(X, term_stride, (size_t)t * d + c, hr[c] * rs * __bfloat162float(gain[c]));
}

// One token per block: rotary embedding of q and k (adjacent pairs), q to Q, k and v into the cache at the
// token's position.  Y row = [q | k | v].
__global__ void __launch_bounds__(256) spd_tc_rope_cache_kernel(const float *Y, float *Q, void *kcache, void *vcache, const float2 *rope,
                                                                int d, int hd, int max_pos, int layer, int pos0, int kv_bf16, int nz, size_t zs) {
  dep_wait();    // the kernel before this one in the stream wrote what this one reads
  dep_launch();  // the next one may set itself up meanwhile
  const int t = blockIdx.x, pos = pos0 + t;
  const float *yr = Y + (size_t)t * 3 * d;
  const size_t crow = ((size_t)layer * max_pos + pos) * d;
  for (int i = threadIdx.x; i < d / 2; i += 256) {
    const float2 cs = rope[(size_t)pos * (hd / 2) + (i % (hd / 2))];
    float qe = 0.f, qo = 0.f, ke = 0.f, ko = 0.f, v0 = 0.f, v1 = 0.f;
    for (int z = 0; z < nz; ++z) {
      const float *yz = yr + z * zs;
      qe += yz[2 * i]; qo += yz[2 * i + 1];
      ke += yz[d + 2 * i]; ko += yz[d + 2 * i + 1];
      v0 += yz[2 * d + 2 * i]; v1 += yz[2 * d + 2 * i + 1];
    }
    Q[(size_t)t * d + 2 * i] = qe * cs.x - qo * cs.y;
    Q[(size_t)t * d + 2 * i + 1] = qe * cs.y + qo * cs.x;
    const float k0 = ke * cs.x - ko * cs.y, k1 = ke * cs.y + ko * cs.x;
    if (kv_bf16) {
      reinterpret_cast<__nv_bfloat162 *>(kcache)[(crow >> 1) + i] = __halves2bfloat162(__float2bfloat16_rn(k0), __float2bfloat16_rn(k1));
      reinterpret_cast<__nv_bfloat162 *>(vcache)[(crow >> 1) + i] = __halves2bfloat162(__float2bfloat16_rn(v0), __float2bfloat16_rn(v1));
    } else {
      reinterpret_cast<float2 *>(kcache)[(crow >> 1) + i] = make_float2(k0, k1);
      reinterpret_cast<float2 *>(vcache)[(crow >> 1) + i] = make_float2(v0, v1);
    }
  }
}

// One token per block: u = SiLU(gate) * up from Y row = [gate_0, up_0, gate_1, up_1, ...], as three bf16 terms.
__global__ void __launch_bounds__(256) spd_tc_swiglu_kernel(const float *Y, uint16_t *X, size_t term_stride, int f, int nz, size_t zs) {
  dep_wait();    // the kernel before this one in the stream wrote what this one reads
  dep_launch();  // the next one may set itself up meanwhile
  const int t = blockIdx.x;
  const float2 *yr = reinterpret_cast<const float2 *>(Y + (size_t)t * 2 * f);
  for (int j = threadIdx.x; j < f; j += 256) {
    float2 gu = yr[j];
    for (int z = 1; z < nz; ++z) {
      const float2 more = yr[z * (zs / 2) + j];
      gu.x += more.x;
      gu.y += more.y;
    }
    tc_put3(X, term_stride, (size_t)t * f + j, gu.x / (1.f + __expf(-gu.x)) * gu.y);
  }
}

// Causal attention over a float32 cache (a bf16 cache takes spd_tc_attn_mma_kernel below): 16 consecutive tokens
// of one head.  The block brings 32 cached positions at
// a time into shared memory as float32 (keys with padded rows, so that a lane per position reads its row without
// bank conflicts); a warp owns two tokens: scores with a lane per position, the tile's softmax weights by warp
// reductions (online softmax across tiles), weighted value sums with HD / 32 dimensions per lane and the weights
// passed round by shuffles.  Every cache row is read once per 16 tokens.  Output as three bf16 terms.
template <int HD>
__global__ void __launch_bounds__(256) spd_tc_attn_kernel(const float *Q, const float *kcache, const float *vcache, uint16_t *X,
                                                          size_t term_stride, int d, int max_pos, int layer, int pos0, int n_tok) {
  dep_wait();    // the kernel before this one in the stream wrote what this one reads
  dep_launch();  // the next one may set itself up meanwhile
  constexpr int kTok = 16, kPos = 32;
  constexpr int KS = HD + 4;    // key row stride in floats: 16-byte aligned, rows 4 banks apart
  constexpr int DPL = HD / 32;  // value dimensions per lane
  __shared__ __align__(16) float sq[kTok * HD];
  __shared__ __align__(16) float sk[kPos * KS];
  __shared__ __align__(16) float sv[kPos * HD];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
  const int head = blockIdx.y, t0 = blockIdx.x * kTok;
  const float scale = 1.f / sqrtf((float)HD);
  for (int i = tid; i < kTok * HD; i += 256) {
    const int tt = i / HD, c = i - tt * HD;
    sq[i] = t0 + tt < n_tok ? Q[(size_t)(t0 + tt) * d + head * HD + c] * scale : 0.f;
  }
  const int last_pos = pos0 + min(t0 + kTok - 1, n_tok - 1);  // the last position a token of this block sees
  const int ta = t0 + 2 * warp, tb = ta + 1;
  const int pa = pos0 + ta, pb = pos0 + tb;
  float ma = -CUDART_INF_F, mb = -CUDART_INF_F, la = 0.f, lb = 0.f;
  float acca[DPL], accb[DPL];
#pragma unroll
  for (int e = 0; e < DPL; ++e) acca[e] = accb[e] = 0.f;
  for (int tile0 = 0; tile0 <= last_pos; tile0 += kPos) {
    __syncthreads();  // the previous tile has been used (first round: nothing)
    for (int i = tid; i < kPos * HD / 8; i += 256) {
      const int r = i / (HD / 8), c8 = (i - r * (HD / 8)) * 8;
      const int pos = tile0 + r;
      float kf[8], vf[8];
      if (pos <= last_pos) {
        const size_t at = ((size_t)layer * max_pos + pos) * d + head * HD + c8;
        const float4 *kp = reinterpret_cast<const float4 *>(kcache + at), *vp = reinterpret_cast<const float4 *>(vcache + at);
        const float4 k0 = kp[0], k1 = kp[1], v0 = vp[0], v1 = vp[1];
        kf[0] = k0.x; kf[1] = k0.y; kf[2] = k0.z; kf[3] = k0.w; kf[4] = k1.x; kf[5] = k1.y; kf[6] = k1.z; kf[7] = k1.w;
        vf[0] = v0.x; vf[1] = v0.y; vf[2] = v0.z; vf[3] = v0.w; vf[4] = v1.x; vf[5] = v1.y; vf[6] = v1.z; vf[7] = v1.w;
      } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) kf[j] = vf[j] = 0.f;
      }
      float4 *kd = reinterpret_cast<float4 *>(sk + r * KS + c8), *vd = reinterpret_cast<float4 *>(sv + r * HD + c8);
      kd[0] = make_float4(kf[0], kf[1], kf[2], kf[3]);
      kd[1] = make_float4(kf[4], kf[5], kf[6], kf[7]);
      vd[0] = make_float4(vf[0], vf[1], vf[2], vf[3]);
      vd[1] = make_float4(vf[4], vf[5], vf[6], vf[7]);
    }
    __syncthreads();
    // scores of position tile0 + lane for the warp's two tokens
    float sa = 0.f, sb = 0.f;
    {
      const float4 *kr = reinterpret_cast<const float4 *>(sk + lane * KS);
      const float4 *qa = reinterpret_cast<const float4 *>(sq + (2 * warp) * HD), *qb = qa + HD / 4;
#pragma unroll 8
      for (int c = 0; c < HD / 4; ++c) {
        const float4 k4 = kr[c], a4 = qa[c], b4 = qb[c];
        sa = fmaf(a4.x, k4.x, sa); sa = fmaf(a4.y, k4.y, sa); sa = fmaf(a4.z, k4.z, sa); sa = fmaf(a4.w, k4.w, sa);
        sb = fmaf(b4.x, k4.x, sb); sb = fmaf(b4.y, k4.y, sb); sb = fmaf(b4.z, k4.z, sb); sb = fmaf(b4.w, k4.w, sb);
      }
    }
    const int pos = tile0 + lane;
    sa = pos <= pa ? sa : -CUDART_INF_F;
    sb = pos <= pb ? sb : -CUDART_INF_F;
    float xa = sa, xb = sb;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      xa = fmaxf(xa, __shfl_xor_sync(0xffffffffu, xa, o));
      xb = fmaxf(xb, __shfl_xor_sync(0xffffffffu, xb, o));
    }
    // position 0 is visible to every token, so the running maxima are finite from the first tile on
    const float mna = fmaxf(ma, xa), mnb = fmaxf(mb, xb);
    const float ca = __expf(ma - mna), cb = __expf(mb - mnb);
    const float wa = __expf(sa - mna), wb = __expf(sb - mnb);
    float ua = wa, ub = wb;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      ua += __shfl_xor_sync(0xffffffffu, ua, o);
      ub += __shfl_xor_sync(0xffffffffu, ub, o);
    }
    la = fmaf(la, ca, ua);
    lb = fmaf(lb, cb, ub);
    ma = mna;
    mb = mnb;
#pragma unroll
    for (int e = 0; e < DPL; ++e) {
      acca[e] *= ca;
      accb[e] *= cb;
    }
#pragma unroll
    for (int j = 0; j < kPos; ++j) {
      const float ja = __shfl_sync(0xffffffffu, wa, j), jb = __shfl_sync(0xffffffffu, wb, j);
      const float *vr = sv + j * HD + lane * DPL;
      float v[DPL];
      if (DPL == 4) {
        const float4 v4 = *reinterpret_cast<const float4 *>(vr);
        v[0] = v4.x; v[1] = v4.y; v[DPL - 2] = v4.z; v[DPL - 1] = v4.w;
      } else {
        const float2 v2 = *reinterpret_cast<const float2 *>(vr);
        v[0] = v2.x; v[1] = v2.y;
      }
#pragma unroll
      for (int e = 0; e < DPL; ++e) {
        acca[e] = fmaf(ja, v[e], acca[e]);
        accb[e] = fmaf(jb, v[e], accb[e]);
      }
    }
  }
  const float ia = 1.f / la, ib = 1.f / lb;
#pragma unroll
  for (int e = 0; e < DPL; ++e) {
    if (ta < n_tok) tc_put3(X, term_stride, (size_t)ta * d + head * HD + lane * DPL + e, acca[e] * ia);
    if (tb < n_tok) tc_put3(X, term_stride, (size_t)tb * d + head * HD + lane * DPL + e, accb[e] * ib);
  }
}

// ---------------------------------------------------------------- attention over a bf16 cache on tensor cores
__device__ __forceinline__ void tc_mma_sync(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void tc_ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void tc_ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
// The three bf16 terms of v (v = hi + mid + lo exactly), each in the upper half of a word.
__device__ __forceinline__ void tc_split3(float v, uint32_t &hi, uint32_t &mid, uint32_t &lo) {
  hi = __float_as_uint(v) & 0xffff0000u;
  const float r1 = v - __uint_as_float(hi);
  mid = __float_as_uint(r1) & 0xffff0000u;
  lo = __float_as_uint(r1 - __uint_as_float(mid)) & 0xffff0000u;
}

// Causal attention of 64 consecutive tokens of one head over a bf16 cache, on tensor cores (mma.sync m16n8k16:
// the attention's share of the arithmetic is small, so the warp-level instructions serve).  Keys and values
// are bf16 already and therefore exact operands; the scaled queries and the softmax weights are float32 and go
// in as three bf16 terms each, as the activations of the products do.  A warp owns 16 tokens: scores of a tile of
// 64 cached positions (tokens x positions, keys read from padded shared-memory rows), online softmax on the
// accumulator fragments, the weights' terms repacked in registers as the next product's left operand, values
// through transposing matrix loads.  Rows of every shared-memory tile are 16 bytes longer than their data: eight
// consecutive rows then start in different bank groups.
template <int HD>
__global__ void __launch_bounds__(128) spd_tc_attn_mma_kernel(const float *Q, const uint16_t *kcache, const uint16_t *vcache, uint16_t *X,
                                                              size_t term_stride, int d, int max_pos, int layer, int pos0, int n_tok) {
  dep_wait();    // the kernel before this one in the stream wrote what this one reads
  dep_launch();  // the next one may set itself up meanwhile
  constexpr int kTok = 64, kPos = 64;
  constexpr int RS = HD * 2 + 16;  // bytes per tile row
  constexpr int KS = HD / 16;      // k-steps over the head's dimensions
  constexpr int DT = HD / 8;       // output tiles of 8 dimensions
  extern __shared__ __align__(16) uint8_t at_smem[];
  uint8_t *sq = at_smem;                // [3 terms][64 tokens][RS]
  uint8_t *sk = sq + 3 * kTok * RS;     // [64 positions][RS]
  uint8_t *sv = sk + kPos * RS;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, q = lane & 3;
  const int head = blockIdx.y, t0 = blockIdx.x * kTok;
  const float scale = 1.f / sqrtf((float)HD);
  for (int i = tid; i < kTok * HD; i += 128) {
    const int tt = i / HD, c = i - tt * HD;
    const float v = t0 + tt < n_tok ? Q[(size_t)(t0 + tt) * d + head * HD + c] * scale : 0.f;
    uint32_t hi, mid, lo;
    tc_split3(v, hi, mid, lo);
    uint16_t *dst = reinterpret_cast<uint16_t *>(sq + tt * RS) + c;
    dst[0] = (uint16_t)(hi >> 16);
    dst[kTok * RS / 2] = (uint16_t)(mid >> 16);
    dst[2 * kTok * RS / 2] = (uint16_t)(lo >> 16);
  }
  const int last_pos = pos0 + min(t0 + kTok - 1, n_tok - 1);  // the last position a token of this block sees
  const int tw = t0 + warp * 16;
  const int p_lo = pos0 + tw + g, p_hi = p_lo + 8, warp_last = pos0 + tw + 15;
  float m[2] = {-CUDART_INF_F, -CUDART_INF_F}, l[2] = {0.f, 0.f};
  float o[DT][4];
#pragma unroll
  for (int i = 0; i < DT; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  const uint32_t sq_u = smem_u32(sq), sk_u = smem_u32(sk), sv_u = smem_u32(sv);
  // per-lane offsets: left operand (tokens x dimensions), keys (32-bit words), values (transposed matrices)
  const uint32_t a_off = (uint32_t)((warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * RS + (lane >> 4) * 16);
  const uint32_t k_off = (uint32_t)(g * RS + q * 4);
  const uint32_t v_off = (uint32_t)((((lane >> 3) & 1) * 8 + (lane & 7)) * RS + (lane >> 4) * 16);
  for (int tile0 = 0; tile0 <= last_pos; tile0 += kPos) {
    __syncthreads();  // the previous tile has been used; first round: the queries are in place after the next barrier
    for (int i = tid; i < kPos * HD / 8; i += 128) {
      const int r = i / (HD / 8), c8 = i - r * (HD / 8);
      const int pos = tile0 + r;
      uint4 a = make_uint4(0u, 0u, 0u, 0u), b = a;
      if (pos <= last_pos) {
        const size_t at = ((size_t)layer * max_pos + pos) * d + head * HD + c8 * 8;
        a = *reinterpret_cast<const uint4 *>(kcache + at);
        b = *reinterpret_cast<const uint4 *>(vcache + at);
      }
      *reinterpret_cast<uint4 *>(sk + r * RS + c8 * 16) = a;
      *reinterpret_cast<uint4 *>(sv + r * RS + c8 * 16) = b;
    }
    __syncthreads();
    if (tile0 > warp_last) continue;  // nothing of this tile is visible to the warp's tokens (the barriers are above)
    float s[kPos / 8][4];
#pragma unroll
    for (int i = 0; i < kPos / 8; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      uint32_t a[3][4];
#pragma unroll
      for (int j = 0; j < 3; ++j) tc_ldsm_x4(sq_u + (uint32_t)(j * kTok * RS) + a_off + (uint32_t)(ks * 32), a[j]);
#pragma unroll
      for (int nt = 0; nt < kPos / 8; ++nt) {
        uint32_t b0, b1;
        const uint32_t addr = sk_u + k_off + (uint32_t)(nt * 8 * RS + ks * 32);
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(b0) : "r"(addr));
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(b1) : "r"(addr + 16));
#pragma unroll
        for (int j = 0; j < 3; ++j) tc_mma_sync(s[nt], a[j], b0, b1);
      }
    }
    // causal mask, row maxima (rows g and g + 8 of the warp's 16 tokens; a row lives in the four lanes of a quad)
    float mx[2] = {-CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
    for (int nt = 0; nt < kPos / 8; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int pos = tile0 + nt * 8 + 2 * q + (e & 1);
        if (pos > (e < 2 ? p_lo : p_hi)) s[nt][e] = -CUDART_INF_F;
        mx[e >> 1] = fmaxf(mx[e >> 1], s[nt][e]);
      }
    float c[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      const float mn = fmaxf(m[r], mx[r]);  // finite: position 0 is visible to every token in the first tile
      c[r] = __expf(m[r] - mn);
      m[r] = mn;
      l[r] *= c[r];
    }
#pragma unroll
    for (int i = 0; i < DT; ++i) {
      o[i][0] *= c[0]; o[i][1] *= c[0]; o[i][2] *= c[1]; o[i][3] *= c[1];
    }
    // the weights and their terms, repacked as left operands: positions 16 kk .. 16 kk + 15 are score tiles 2 kk, 2 kk + 1
    uint32_t pt[kPos / 16][3][4];
#pragma unroll
    for (int nt = 0; nt < kPos / 8; ++nt) {
      float pw[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) pw[e] = __expf(s[nt][e] - m[e >> 1]);
      l[0] += pw[0] + pw[1];
      l[1] += pw[2] + pw[3];
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        uint32_t h0, m0, l0, h1, m1, l1;
        tc_split3(pw[2 * r], h0, m0, l0);
        tc_split3(pw[2 * r + 1], h1, m1, l1);
        const int reg = (nt & 1) * 2 + r;
        pt[nt >> 1][0][reg] = h1 | (h0 >> 16);
        pt[nt >> 1][1][reg] = m1 | (m0 >> 16);
        pt[nt >> 1][2][reg] = l1 | (l0 >> 16);
      }
    }
#pragma unroll
    for (int kk = 0; kk < kPos / 16; ++kk)
#pragma unroll
      for (int dp = 0; dp < DT / 2; ++dp) {
        uint32_t b[4];
        tc_ldsm_x4_trans(sv_u + v_off + (uint32_t)(kk * 16 * RS + dp * 32), b);
#pragma unroll
        for (int j = 0; j < 3; ++j) {
          tc_mma_sync(o[2 * dp], pt[kk][j], b[0], b[1]);
          tc_mma_sync(o[2 * dp + 1], pt[kk][j], b[2], b[3]);
        }
      }
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l[r] += __shfl_xor_sync(0xffffffffu, l[r], 1);
    l[r] += __shfl_xor_sync(0xffffffffu, l[r], 2);
  }
  const float inv[2] = {1.f / l[0], 1.f / l[1]};
#pragma unroll
  for (int i = 0; i < DT; ++i)
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int t = tw + g + (e >> 1) * 8;
      if (t < n_tok) tc_put3(X, term_stride, (size_t)t * d + head * HD + i * 8 + 2 * q + (e & 1), o[i][e] * inv[e >> 1]);
    }
}

}  // namespace spd

namespace {

template <int HD>
constexpr size_t attn_mma_smem() { return (size_t)5 * 64 * (HD * 2 + 16); }  // three query terms, keys, values: 64 padded rows each

template <int HD>
cudaError_t launch_attn(const spd::TcJob &j, int layer, int n_tok, cudaStream_t s) {
  const size_t ts = (size_t)j.x_term_rows * j.d;
  if (j.kv_bf16)
    return spd::launch_dep(spd::spd_tc_attn_mma_kernel<HD>, dim3((n_tok + 63) / 64, j.H), dim3(128), attn_mma_smem<HD>(), s, j.q,
                           static_cast<const uint16_t *>(j.kcache), static_cast<const uint16_t *>(j.vcache), j.x, ts, j.d, j.max_pos, layer, j.pos0,
                           n_tok);
  return spd::launch_dep(spd::spd_tc_attn_kernel<HD>, dim3((n_tok + 15) / 16, j.H), dim3(256), 0, s, j.q, static_cast<const float *>(j.kcache),
                         static_cast<const float *>(j.vcache), j.x, ts, j.d, j.max_pos, layer, j.pos0, n_tok);
}

size_t tc_gemm_smem() { return (size_t)spd::kTcStages * spd::kTcStageBytes + 1024; }

}  // namespace

extern "C" cudaError_t spd_internal_tc_prepare(void) {
  cudaError_t e = cudaFuncSetAttribute(reinterpret_cast<const void *>(&spd::spd_tc_gemm_kernel), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)tc_gemm_smem());
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(reinterpret_cast<const void *>(&spd::spd_tc_attn_mma_kernel<64>), cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)attn_mma_smem<64>());
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(reinterpret_cast<const void *>(&spd::spd_tc_attn_mma_kernel<128>), cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)attn_mma_smem<128>());
  return e;
}

namespace {
template <int NP>
cudaError_t launch_batch_gemm(const void *xmap, const void *wmap, float *Y, size_t zs, int nz, int n_tok, int N, int C, int x_term_rows,
                              spd::State *st, cudaStream_t s, int dep) {
  using S = spd::BgShape<NP>;
  const size_t smem = (size_t)S::kStages * S::kStageBytes + 1024;
  // the shared-memory attribute is per device: set on a device's first launch of this instance
  static bool ready[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !ready[dev]) {
    e = cudaFuncSetAttribute(reinterpret_cast<const void *>(&spd::spd_batch_gemm_kernel<NP>), cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) ready[dev] = true;
  }
  const dim3 grid((N + spd::kTcN - 1) / spd::kTcN, nz);
  if (dep) return spd::launch_dep(spd::spd_batch_gemm_kernel<NP>, grid, dim3(spd::kTcThreads), smem, s, xmap, wmap, Y, zs, n_tok, N, C, x_term_rows, st);
  spd::spd_batch_gemm_kernel<NP><<<grid, spd::kTcThreads, smem, s>>>(xmap, wmap, Y, zs, n_tok, N, C, x_term_rows, st);
  return cudaGetLastError();
}
}  // namespace

// Product of a batch (n_tok <= 128 token rows): xmaps = the term buffer's tensor maps with boxes of 128, 16, 32 and 64
// rows (two each: d_model and d_ffn columns; `wide` picks the second).  The columns are split nz ways (chosen here
// for the fewest waves of blocks, within y_floats of room for the partial sums); *out_nz and
// *out_zs tell the reader of Y how many partial sums there are and how far apart.
extern "C" cudaError_t spd_internal_batch_gemm(const uint8_t *xmaps, int wide, const void *wmap, float *Y, size_t y_floats, int n_tok, int N, int C,
                                               int x_term_rows, spd::State *st, int sm_count, cudaStream_t s, int dep, int *out_nz, size_t *out_zs) {
  const int np = n_tok <= 16 ? 16 : (n_tok <= 32 ? 32 : (n_tok <= 64 ? 64 : 128));
  // the term buffer's tensor maps: boxes of 128 rows first, then 16, 32 and 64 (two each: d_model and d_ffn columns)
  const int slot = (np == 128 ? 0 : (np == 16 ? 1 : (np == 32 ? 2 : 3))) * 2 + (wide ? 1 : 0);
  const void *xmap = xmaps + (size_t)slot * spd::kTensorMapBytes;
  const int tiles = (N + spd::kTcN - 1) / spd::kTcN, nk = (C + spd::kTcKB - 1) / spd::kTcKB;
  const size_t zs = (size_t)n_tok * N;
  // The split that needs the fewest stage times: the blocks run in waves of as many as fit the GPU (two per SM, one
  // with boxes of 128 rows), a block costs its stages plus about eight stages' worth of set-up, ring fill and epilogue,
  // and a last wave that is nearly empty costs as much as a full one (the 7B gate / up product, 172 row tiles: two
  // ways = 344 blocks = two waves of 32 stages, three ways = 516 blocks = two waves of 22).  At least 8 stages of
  // work per block, and room for the partial sums.
  const int slots = (np == 128 ? 1 : 2) * (sm_count > 0 ? sm_count : 1);
  int nz_max = nk / 8;
  if ((size_t)nz_max * zs > y_floats) nz_max = (int)(y_floats / zs);
  if (nz_max < 1) nz_max = 1;
  int nz = 1;
  long best = -1;
  for (int z = 1; z <= nz_max; ++z) {
    const long waves = ((long)tiles * z + slots - 1) / slots;
    const long cost = waves * ((nk + z - 1) / z + 8);
    if (best < 0 || cost < best) { best = cost; nz = z; }
  }
  *out_nz = nz;
  *out_zs = zs;
  if (np == 16) return launch_batch_gemm<16>(xmap, wmap, Y, zs, nz, n_tok, N, C, x_term_rows, st, s, dep);
  if (np == 32) return launch_batch_gemm<32>(xmap, wmap, Y, zs, nz, n_tok, N, C, x_term_rows, st, s, dep);
  if (np == 64) return launch_batch_gemm<64>(xmap, wmap, Y, zs, nz, n_tok, N, C, x_term_rows, st, s, dep);
  return launch_batch_gemm<128>(xmap, wmap, Y, zs, nz, n_tok, N, C, x_term_rows, st, s, dep);
}

// Test hook: one tile of the first layer's QKV product whose first stage never arrives (see the kernel's `stall`).
extern "C" cudaError_t spd_internal_tc_stall(const spd::TcJob *job, cudaStream_t s) {
  const spd::TcJob &j = *job;
  spd::spd_tc_gemm_kernel<<<dim3(1, 1), spd::kTcThreads, tc_gemm_smem(), s>>>(j.x_tmaps, j.w_tmaps, j.y, 3 * j.d, j.d, j.x_term_rows, j.st, 1);
  return cudaGetLastError();
}

// Enqueues the decoder over j.n_tok tokens (at most j.x_term_rows) at positions j.pos0 ..: their keys and values
// enter the cache.  The products run over whole tiles of 128 tokens: the rows past n_tok of the last tile hold
// whatever an earlier job left, give rows of Y that nothing reads (a row of Y depends on its own token only).
// *launches receives the number of kernels enqueued.
extern "C" cudaError_t spd_internal_tc_prefill(const spd::TcJob *job, cudaStream_t s, int *launches) {
  const spd::TcJob &j = *job;
  const int n = j.n_tok, d = j.d, f = j.f;
  const size_t ts_d = (size_t)j.x_term_rows * d, ts_f = (size_t)j.x_term_rows * f;
  const uint8_t *xmap_d = j.x_tmaps, *xmap_f = j.x_tmaps + spd::kTensorMapBytes;
  int count = 0;
  cudaError_t e = cudaSuccess;
  // A job of up to 128 tokens is one token tile: its products are bound by the weight stream and take the product
  // made for few token rows (weights as the wide operand, columns split among blocks; its output is nz partial sums
  // zs floats apart, which the row-wise kernels add up).
  int nz = 1;
  size_t zs = 0;
  auto gemm = [&](const uint8_t *xmap, int which, int N, int C) {
    if (e != cudaSuccess) return;
    const uint8_t *wmap = j.w_tmaps + (size_t)which * spd::kTensorMapBytes;
    if (n <= spd::kTcM) {
      e = spd_internal_batch_gemm(j.x_tmaps, xmap != xmap_d, wmap, j.y, j.y_floats, n, N, C, j.x_term_rows, j.st, j.sm_count, s, 1, &nz, &zs);
    } else {
      const dim3 grid((n + spd::kTcM - 1) / spd::kTcM, (N + spd::kTcN - 1) / spd::kTcN);
      spd::spd_tc_gemm_kernel<<<grid, spd::kTcThreads, tc_gemm_smem(), s>>>(xmap, wmap, j.y, N, C, j.x_term_rows, j.st, 0);
      e = cudaGetLastError();
    }
    ++count;
  };
  if (n <= spd::kTcM) {
    // ... and the column-parallel row-wise kernels of a batched timestep (a block per 512 columns of a token row
    // instead of one per row; RMSNorm's 1 / rms applied behind the product from per-chunk sums of squares).
    e = spd_internal_job_input(job, j.ss, s);
    ++count;
    for (int l = 0; l < j.L && e == cudaSuccess; ++l) {
      gemm(xmap_d, 4 * l, 3 * d, d);
      if (e != cudaSuccess) break;
      e = spd_internal_job_rope_cache(job, j.ss, nz, zs, l, s);
      if (e != cudaSuccess) break;
      e = j.hd == 128 ? launch_attn<128>(j, l, n, s) : launch_attn<64>(j, l, n, s);
      count += 2;
      gemm(xmap_d, 4 * l + 1, d, d);
      if (e != cudaSuccess) break;
      e = spd_internal_job_resid(job, j.ss, nz, zs, j.layers[l].ffn_norm, s);
      ++count;
      gemm(xmap_d, 4 * l + 2, 2 * f, d);
      if (e != cudaSuccess) break;
      e = spd_internal_job_swiglu(job, j.ss, nz, zs, s);
      ++count;
      gemm(xmap_f, 4 * l + 3, d, f);
      if (e != cudaSuccess) break;
      if (l + 1 < j.L) {  // the last layer's output feeds nothing here
        e = spd_internal_job_resid(job, j.ss, nz, zs, j.layers[l + 1].attn_norm, s);
        ++count;
      }
    }
    if (launches) *launches = count;
    return e;
  }
  auto resid = [&](const float *y, const int32_t *ids, const __nv_bfloat16 *gain) {
    if (e != cudaSuccess) return;
    e = spd::launch_dep(spd::spd_tc_resid_norm_kernel, dim3(n), dim3(256), 0, s, j.h, y, ids, j.tok_emb, gain, j.x, ts_d, d, j.eps, nz, zs);
    ++count;
  };
  resid(nullptr, j.ids, j.layers[0].attn_norm);
  for (int l = 0; l < j.L && e == cudaSuccess; ++l) {
    gemm(xmap_d, 4 * l, 3 * d, d);
    if (e != cudaSuccess) break;
    e = spd::launch_dep(spd::spd_tc_rope_cache_kernel, dim3(n), dim3(256), 0, s, j.y, j.q, j.kcache, j.vcache, j.rope, d, j.hd, j.max_pos, l, j.pos0,
                        j.kv_bf16, nz, zs);
    if (e != cudaSuccess) break;
    e = j.hd == 128 ? launch_attn<128>(j, l, n, s) : launch_attn<64>(j, l, n, s);  // other head sizes never get here
    count += 2;
    gemm(xmap_d, 4 * l + 1, d, d);
    resid(j.y, nullptr, j.layers[l].ffn_norm);
    gemm(xmap_d, 4 * l + 2, 2 * f, d);
    if (e != cudaSuccess) break;
    e = spd::launch_dep(spd::spd_tc_swiglu_kernel, dim3(n), dim3(256), 0, s, j.y, j.x, ts_f, f, nz, zs);
    ++count;
    gemm(xmap_f, 4 * l + 3, d, f);
    if (l + 1 < j.L) resid(j.y, nullptr, j.layers[l + 1].attn_norm);  // the last layer's output feeds nothing here
  }
  if (launches) *launches = count;
  return e;
}
