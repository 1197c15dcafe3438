// Prefill kernel: the decoder over up to 16 prefix tokens at once, and, in the launch that holds the prefix's
// last token, the LM head on that token and the first timestep (Eq. 1).  With several tokens per weight the
// products are real matrix-matrix contractions, so they run on tensor cores: mma.sync m16n8k16 with A = 16
// weight rows x 16 columns straight from the bf16 rows, B = the tokens' activations split exactly into three
// bf16 terms (x = hi + mid + lo to float32 precision), float32 accumulation.
//
// One persistent cooperative launch per chunk of tokens.  Per block: a producer warp streams the block's
// weight rows (chunks of 32 rows x 512 columns = 8 tiled TMA copies in the 128-byte-swizzled layout that
// ldmatrix reads without bank conflicts) through a shared-memory ring; eight consumer warps share every chunk
// by k-steps and keep the accumulators of up to 10 row tiles in registers, so that a block's rows of a matrix
// are streamed once; per-warp partial sums meet in shared memory once per 16 rows.  Activations travel
// between phases already split and laid out as mma B fragments: the epilogue that produces a value writes its
// three bf16 terms into a fragment buffer in global memory, and in the next phase a second producer warp pulls
// 512 columns of all 16 tokens (48 KB) at a time into shared memory with one bulk copy; each consumer warp
// takes its k-steps' fragments into registers at once, which frees the buffer for the next K block while the
// current one is multiplied.  No block repeats the conversion.  RMSNorm's gain is applied before the split,
// its per-token 1/rms (from per-block partial sums of squares) after the product: it is a scalar per token.
// The five phases per layer are separated by grid barriers as in decoding; every wait is bounded.
#include <cuda_runtime.h>
#include <math_constants.h>

#include "spd_params.h"
#include "spd_ptx.cuh"
#include "spd_tail.cuh"

namespace spd {

constexpr int kPfWarps = 8;
constexpr int kPfThreads = kPfWarps * 32;  // consumer threads
constexpr int kPfBlock = kPfThreads + 64;  // plus the weight producer warp and the fragment producer warp
constexpr int kPfKB = 512;                 // columns per K block
constexpr int kPfKSteps = kPfKB / 16;
constexpr int kPfTileRows = 16;            // rows of one mma tile
constexpr int kPfChunkRows = 32;           // rows of one ring stage: two tiles
constexpr int kPfMaxTiles = 10;            // row tiles whose accumulators a warp keeps at a time
constexpr int kPfMaxChunks = kPfMaxTiles / 2;
static_assert(kPfMaxTiles % 2 == 0, "a full group must end on the second partial-sum buffer");
constexpr int kPfBoxCols = 64;             // one tensor-copy box: 32 rows x 64 columns = 32 x 128 bytes, 128-byte swizzle
constexpr int kPfBoxBytes = kPfChunkRows * kPfBoxCols * 2;
constexpr int kPfBoxes = kPfKB / kPfBoxCols;
constexpr int kPfStageBytes = kPfBoxes * kPfBoxBytes;
constexpr int kPfStages = 5;
constexpr int kPfXBufs = 1;                // shared-memory fragment buffers (the consumers empty one into registers at once)
constexpr int kPfKStepBytes = 2 * 3 * 32 * 8;             // fragments of one k-step: [token tile][term][lane] x 8 bytes
constexpr int kPfXBytes = kPfKSteps * kPfKStepBytes;      // one K block of fragments
constexpr int kPfRedBytes = kPfWarps * kPfTileRows * kPfTokens * 4;  // one buffer of partial sums; there are two
constexpr int kPfMaxSplit = 8;              // attention: position ranges a head is split into
constexpr int kPfAmFloats = 3 * kPfWarps * 8 + 2 * 8;  // attention item of 8 tokens: (max, sum, factor) per warp and token, merged (max, sum)
constexpr unsigned long long kPfWaitNs = 1500ull * 1000ull * 1000ull;

struct PfBlk {
  const KParams *p;
  uint8_t *ring;
  uint8_t *xblk;  // kPfXBufs fragment buffers of kPfXBytes
  float *red;
  float *rs;      // [16] per-token 1/rms
  float *am;      // attention merge scratch: kPfAmFloats floats
  uint64_t *full, *empty, *xfull, *xempty, *xgo;
  volatile int *dead, *quit;
  int *last;      // attention: whether this block merges a head's splits
  unsigned int bar_target;
  uint32_t c_stage, c_phase;
  uint32_t x_n;  // fragment copies consumed so far: copy n sits in buffer n % kPfXBufs and is that buffer's use n / kPfXBufs
};

__device__ __forceinline__ void pf_give_up(PfBlk &b, int code, int info) {
  State *st = b.p->st;
  if (atomicCAS(&st->err, 0, code) == 0) st->err_info = info;
  atomicExch(&st->abort_flag, 1u);
  *b.dead = 1;
}

// Bounded wait on an mbarrier phase; false when the block gave up instead.
__device__ __forceinline__ bool pf_wait(PfBlk &b, uint64_t *bar, uint32_t parity, int info) {
  if (mbar_try_wait(bar, parity)) return true;
  if (*b.dead) return false;
  unsigned long long t0 = globaltimer();
  uint32_t n = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++n & 31u) == 0) {
      if (*b.dead) return false;
      if (ld_relaxed(&b.p->st->abort_flag)) { *b.dead = 1; return false; }
      if (globaltimer() - t0 > kPfWaitNs) { pf_give_up(b, -7, info); return false; }
    }
  }
  return true;
}

__device__ __forceinline__ bool pf_grid_barrier(PfBlk &b) {
  named_sync(1, kPfThreads);
  if (threadIdx.x == 0) {
    b.bar_target += gridDim.x;
    if (!*b.dead) {
      unsigned int *bar = &b.p->st->bar;
      __threadfence();
      if (!(b.p->pf_stall && blockIdx.x == 0)) atomicAdd(bar, 1u);  // the test hook's missing arrival: every wait runs out
      unsigned long long t0 = globaltimer();
      uint32_t n = 0;
      while ((int)(ld_acquire(bar) - b.bar_target) < 0) {
        if ((++n & 63u) == 0) {
          if (ld_relaxed(&b.p->st->abort_flag)) { *b.dead = 1; break; }
          if (globaltimer() - t0 > kPfWaitNs) { pf_give_up(b, -7, 101); break; }
        }
      }
    }
    *b.quit = *b.dead;
  }
  named_sync(1, kPfThreads);
  return *b.quit != 0;
}

__device__ __forceinline__ void pf_rows(int R, int gran, int &r0, int &r1) {
  long long U = R / gran;
  r0 = (int)(U * blockIdx.x / gridDim.x) * gran;
  r1 = (int)(U * (blockIdx.x + 1) / gridDim.x) * gran;
}

struct PfPhase {
  const __nv_bfloat16 *W;
  int R, C, gran;
};
__device__ __forceinline__ int pf_phases(const KParams &p) { return 4 * p.L + (p.pf_head ? 1 : 0); }
__device__ __forceinline__ PfPhase pf_phase(const KParams &p, int ph) {
  PfPhase d;
  if (ph == 4 * p.L) {  // the LM head, after the last layer
    d.W = p.lm_head; d.R = p.V; d.C = p.d; d.gran = 1;
    return d;
  }
  const LayerW &lw = p.layers[ph >> 2];
  switch (ph & 3) {
    case 0: d.W = lw.wqkv; d.R = 3 * p.d; d.C = p.d; d.gran = 2; break;
    case 1: d.W = lw.wo; d.R = p.d; d.C = p.d; d.gran = 1; break;
    case 2: d.W = lw.wgate_up; d.R = 2 * p.f; d.C = p.d; d.gran = 2; break;
    default: d.W = lw.wdown; d.R = p.d; d.C = p.f; d.gran = 1; break;
  }
  return d;
}

// ---------------------------------------------------------------- producer
// Tiled bulk copy of one box (64 columns x 32 rows at column x, row y of the matrix the tensor map describes)
// into shared memory; rows and columns past the matrix arrive as zeros; completion is counted on `bar` in bytes.
__device__ __forceinline__ void pf_box_load(void *dst, const void *tmap, int x, int y, uint64_t *bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
                   smem_u32(dst)),
               "l"(tmap), "r"(x), "r"(y), "r"(smem_u32(bar))
               : "memory");
}

// Chunk order of a phase: per group of up to kPfMaxTiles row tiles, K block by K block, chunk (32 rows) by chunk.
// A chunk is 8 boxes, one per lane 0..7, in the 128-byte-swizzled layout that ldmatrix reads without bank
// conflicts: box j of a stage holds columns 64 j .. 64 j + 63, row r of it lies at r * 128, and its 16-byte
// unit u sits at unit u ^ (r % 8).
__device__ void pf_producer(PfBlk &b) {
  const KParams &p = *b.p;
  const int lane = threadIdx.x & 31;
  uint32_t stage = 0, phase = 0, issued = 0;
  bool ok = true;
  for (int ph = 0; ph < pf_phases(p) && ok; ++ph) {
    const PfPhase pd = pf_phase(p, ph);
    int r0, r1;
    pf_rows(pd.R, pd.gran, r0, r1);
    const uint8_t *tmap = reinterpret_cast<const uint8_t *>(p.pf_tmaps) + (size_t)ph * kTensorMapBytes;
    const int nkb = (pd.C + kPfKB - 1) / kPfKB;
    for (int g0 = r0; g0 < r1 && ok; g0 += kPfMaxTiles * kPfTileRows) {
      const int g1 = min(g0 + kPfMaxTiles * kPfTileRows, r1);
      for (int kb = 0; kb < nkb && ok; ++kb) {
        const int nbox = min(kPfBoxes, (pd.C - kb * kPfKB + kPfBoxCols - 1) / kPfBoxCols);  // boxes that touch the matrix
        for (int c0 = g0; c0 < g1 && ok; c0 += kPfChunkRows) {
          int dead = 0;
          if (lane == 0) {
            pf_wait(b, &b.empty[stage], phase ^ 1u, 200);
            dead = *b.dead;
            if (!dead) mbar_expect_tx(&b.full[stage], (uint32_t)(nbox * kPfBoxBytes));
          }
          dead = __shfl_sync(0xffffffffu, dead, 0);
          if (dead) { ok = false; break; }
          if (lane < nbox)
            pf_box_load(b.ring + (size_t)stage * kPfStageBytes + (size_t)lane * kPfBoxBytes, tmap, kb * kPfKB + lane * kPfBoxCols, c0,
                        &b.full[stage]);
          if (issued < (uint32_t)kPfStages) ++issued;
          if (++stage == (uint32_t)kPfStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  }
  if (!ok && lane == 0) {
    // giving up: wait (bounded) for the copies already issued, so that none lands after the block has gone
    uint32_t s = stage, ph = phase;
    for (uint32_t i = 0; i < issued; ++i) {
      if (s == 0) { s = (uint32_t)kPfStages; ph ^= 1u; }
      --s;
      unsigned long long t0 = globaltimer();
      while (!mbar_try_wait(&b.full[s], ph) && globaltimer() - t0 < kPfWaitNs) {}
    }
  }
  __syncwarp();
}

// ---------------------------------------------------------------- fragments
__device__ __forceinline__ void pf_mma(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void pf_ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}

// Writes activation v of (token t, column c) into a fragment buffer as three bf16 terms with
// hi + mid + lo = v exactly: each term takes the leading 8 significant bits of what is left, by truncation,
// and a float32 has 24.  Layout: [k-step c / 16][token tile t / 8][term][lane (t % 8) * 4 + (c % 8) / 2]
// x {columns (2q, 2q+1), columns (8 + 2q, 9 + 2q)} bf16, which is what one lane of the mma wants as B.
__device__ __forceinline__ void pf_put(uint16_t *F, int t, int c, float v) {
  const uint32_t hi = __float_as_uint(v) & 0xffff0000u;
  const float r1 = v - __uint_as_float(hi);
  const uint32_t mid = __float_as_uint(r1) & 0xffff0000u;
  const float r2 = r1 - __uint_as_float(mid);
  const uint32_t lo = __float_as_uint(r2);
  const size_t unit = (size_t)(c >> 4) * 2 + (t >> 3);
  const size_t e = ((unit * 3) * 32 + (size_t)((t & 7) * 4 + ((c & 7) >> 1))) * 4 + ((c >> 3) & 1) * 2 + (c & 1);
  F[e] = (uint16_t)(hi >> 16);
  F[e + 128] = (uint16_t)(mid >> 16);
  F[e + 256] = (uint16_t)(lo >> 16);
}

// Fragment producer (one thread): copies the K blocks of each phase's fragment buffer into shared memory, in the order the consumers take them.  A phase's fragments are complete once the consumers have
// passed the grid barrier before it (they say so on `xgo`); a buffer is free again once all consumer warps
// have taken their fragments of it into registers (`xempty`).
__device__ void pf_xproducer(PfBlk &b) {
  const KParams &p = *b.p;
  uint32_t n = 0;
  bool ok = true;
  for (int ph = 0; ph < pf_phases(p) && ok; ++ph) {
    const PfPhase pd = pf_phase(p, ph);
    int r0, r1;
    pf_rows(pd.R, pd.gran, r0, r1);
    const uint8_t *F = reinterpret_cast<const uint8_t *>((ph & 1) == 0 ? p.pf_xh : (ph & 3) == 1 ? p.pf_xo : p.pf_xu);
    const int nks_total = (pd.C + 15) / 16;
    const int nkb = (pd.C + kPfKB - 1) / kPfKB;
    if (!pf_wait(b, b.xgo, (uint32_t)ph & 1u, 320)) break;
    asm volatile("fence.proxy.async;" ::: "memory");  // the fragments were written with ordinary stores by other blocks
    for (int g0 = r0; g0 < r1 && ok; g0 += kPfMaxTiles * kPfTileRows)
      for (int kb = 0; kb < nkb; ++kb) {
        const int buf = n % kPfXBufs;
        if (!pf_wait(b, &b.xempty[buf], ((n / kPfXBufs) & 1u) ^ 1u, 330)) { ok = false; break; }
        const uint32_t bytes = (uint32_t)min(kPfKSteps, nks_total - kb * kPfKSteps) * (uint32_t)kPfKStepBytes;
        mbar_expect_tx(&b.xfull[buf], bytes);
        bulk_load(b.xblk + (size_t)buf * kPfXBytes, F + (size_t)kb * kPfXBytes, bytes, &b.xfull[buf]);
        ++n;
      }
  }
  if (*b.dead) {
    // giving up: wait (bounded) for the last copy into each buffer, the only ones that can still be in flight
    for (uint32_t i = 0; i < (uint32_t)kPfXBufs && i < n; ++i) {
      const uint32_t m = n - 1 - i;
      unsigned long long t0 = globaltimer();
      while (!mbar_try_wait(&b.xfull[m % kPfXBufs], (m / kPfXBufs) & 1u) && globaltimer() - t0 < kPfWaitNs) {}
    }
  }
}

// Per-token 1/rms of the residual rows from the blocks' partial sums of squares (each block publishes the sums
// over the rows or columns it produced; added here in a fixed order).
__device__ void pf_token_rms(PfBlk &b, int d) {
  const KParams &p = *b.p;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int t = warp; t < kPfTokens; t += kPfWarps) {
    float ss = 0.f;
    for (int blk = lane; blk < (int)gridDim.x; blk += 32) ss += __ldcg(p.pf_ss + (size_t)blk * kPfTokens + t);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if (lane == 0) b.rs[t] = rsqrtf(ss / (float)d + p.eps);
  }
  named_sync(1, kPfThreads);
}

// Publishes this block's sums of squares: thread (slot = tid / 16, token = tid % 16) brings the sum over the
// residual values of its token that it produced.
__device__ void pf_publish_ss(PfBlk &b, float ssq) {
  named_sync(1, kPfThreads);  // the scratch is no longer read
  b.red[threadIdx.x] = ssq;
  named_sync(1, kPfThreads);
  if (threadIdx.x < kPfTokens) {
    float s = 0.f;
#pragma unroll
    for (int r = 0; r < kPfThreads / kPfTokens; ++r) s += b.red[r * kPfTokens + threadIdx.x];
    b.p->pf_ss[(size_t)blockIdx.x * kPfTokens + threadIdx.x] = s;
  }
}

constexpr int kPfOwnSteps = kPfKSteps / kPfWarps;  // k-steps of a K block that one warp multiplies

// One tile against this warp's k-steps of the K block: 16 rows x 16 columns of weights per k-step times the
// three terms of both token tiles (fragments already in registers).  The two token tiles' accumulators
// alternate so that consecutive mma do not depend on each other.
__device__ __forceinline__ void pf_tile(float (&acc)[2][4], uint32_t base, const uint2 (&bb)[kPfOwnSteps][6]) {
#pragma unroll
  for (int s = 0; s < kPfOwnSteps; ++s) {
    uint32_t a0, a1, a2, a3;
    pf_ldsm_x4(base + (uint32_t)s * (uint32_t)(kPfWarps / 4 * kPfBoxBytes), a0, a1, a2, a3);  // k-step warp + 8 s: two boxes on
#pragma unroll
    for (int k = 0; k < 3; ++k)
#pragma unroll
      for (int n = 0; n < 2; ++n) pf_mma(acc[n], a0, a1, a2, a3, bb[s][n * 3 + k].x, bb[s][n * 3 + k].y);
  }
}

enum PfEpi { kPfQKV = 0, kPfAddH = 1, kPfSwiGLU = 2, kPfLogits = 3 };

// One matrix for the 16 tokens: out[t][r] = scale_t * sum_c W[r][c] x[t][c] for this block's rows (x from the
// phase's fragment buffer; scale_t = 1/rms of token t when `norm`, else 1), then the phase's epilogue.  `gain_next`
// (kPfAddH): gain of the RMSNorm that reads the new residual next, or null when nothing does.
__device__ void pf_gemm(PfBlk &b, const PfPhase &pd, bool norm, int kind, const __nv_bfloat16 *gain_next,
                        int layer, int which, int pos0, int n_tok) {
  const KParams &p = *b.p;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
  int r0, r1;
  pf_rows(pd.R, pd.gran, r0, r1);
  const int nks_total = (pd.C + 15) / 16;
  const int nkb = (pd.C + kPfKB - 1) / kPfKB;
  if (tid == 0) mbar_arrive(b.xgo);  // the grid barrier before this phase is behind us: its fragments are complete
  if (norm) pf_token_rms(b, pd.C);
  float ssq = 0.f;  // kPfAddH: sum of squares of the residual values this thread produces (its token = tid % 16)
  // ldmatrix address of this lane for the warp's first k-step (k-step = warp) of a chunk's first tile: row
  // (lane % 8) + 8 for the lower half of the tile, 16-byte unit 2 (k-step % 4) + (columns 8-15 ? 1 : 0), swizzled
  const uint32_t l_row = (uint32_t)((lane & 7) + ((lane >> 3) & 1) * 8);
  const uint32_t lane_off = (uint32_t)(warp >> 2) * kPfBoxBytes + l_row * 128u + (((uint32_t)((warp & 3) * 2 + (lane >> 4)) ^ (l_row & 7u)) << 4);
  for (int g0 = r0; g0 < r1; g0 += kPfMaxTiles * kPfTileRows) {
    const int g1 = min(g0 + kPfMaxTiles * kPfTileRows, r1);
    float acc[kPfMaxTiles][2][4];
#pragma unroll
    for (int i = 0; i < kPfMaxTiles; ++i)
#pragma unroll
      for (int n = 0; n < 2; ++n) acc[i][n][0] = acc[i][n][1] = acc[i][n][2] = acc[i][n][3] = 0.f;
    for (int kb = 0; kb < nkb; ++kb) {
      const int buf = b.x_n % kPfXBufs;
      pf_wait(b, &b.xfull[buf], (b.x_n / kPfXBufs) & 1u, 310);
      b.x_n += 1;
      // this warp's k-steps of the block: fragments to registers (zeros past the row's end, so that whatever
      // the ring holds there does not count), then the buffer is free for the K block after the next
      const uint2 *xb = reinterpret_cast<const uint2 *>(b.xblk + (size_t)buf * kPfXBytes) + lane;
      const int nks = min(kPfKSteps, nks_total - kb * kPfKSteps);
      uint2 bb[kPfOwnSteps][6];
#pragma unroll
      for (int s = 0; s < kPfOwnSteps; ++s) {
        const int ks = warp + s * kPfWarps;
#pragma unroll
        for (int e = 0; e < 6; ++e) bb[s][e] = ks < nks ? xb[(ks * 6 + e) * 32] : make_uint2(0u, 0u);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&b.xempty[buf]);
#pragma unroll
      for (int j = 0; j < kPfMaxChunks; ++j) {
        if (g0 + j * kPfChunkRows < g1) {
          pf_wait(b, &b.full[b.c_stage], b.c_phase, 300);
          const uint32_t cbase = smem_u32(b.ring + (size_t)b.c_stage * kPfStageBytes) + lane_off;
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const int i = 2 * j + h;
            if (g0 + i * kPfTileRows < g1) pf_tile(acc[i], cbase + (uint32_t)(h * kPfTileRows * 128), bb);
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(&b.empty[b.c_stage]);
          if (++b.c_stage == (uint32_t)kPfStages) { b.c_stage = 0; b.c_phase ^= 1u; }
        }
      }
    }
    // per tile: the warps' partial sums meet in shared memory, then the epilogue
#pragma unroll
    for (int i = 0; i < kPfMaxTiles; ++i) {
      if (g0 + i * kPfTileRows < g1) {
        const int t0 = g0 + i * kPfTileRows;
        // two buffers alternate: the barrier of the tile in between separates a buffer's readers from its next writers
        float *red = b.red + (i & 1) * (kPfRedBytes / 4);
        float *mine = red + warp * (kPfTileRows * kPfTokens);
        const int gr = lane >> 2, q = lane & 3;
#pragma unroll
        for (int n = 0; n < 2; ++n) {
          mine[gr * kPfTokens + n * 8 + 2 * q] = acc[i][n][0];
          mine[gr * kPfTokens + n * 8 + 2 * q + 1] = acc[i][n][1];
          mine[(gr + 8) * kPfTokens + n * 8 + 2 * q] = acc[i][n][2];
          mine[(gr + 8) * kPfTokens + n * 8 + 2 * q + 1] = acc[i][n][3];
        }
        named_sync(1, kPfThreads);
        const int row = tid >> 4, t = tid & 15;  // one thread per (row, token); rows r and r^1 sit 16 lanes apart
        float y = 0.f;
#pragma unroll
        for (int w = 0; w < kPfWarps; ++w) y += red[w * (kPfTileRows * kPfTokens) + row * kPfTokens + t];
        if (norm) y *= b.rs[t];
        const float other = __shfl_xor_sync(0xffffffffu, y, 16);
        const int r = t0 + row;
        if (r < g1) {
          // tokens past n_tok carry zeros through every phase; only the cache is not touched for them
          const int pos = pos0 + t;
          if (kind == kPfQKV) {
            if (t < n_tok) {
              const int sec = r / p.d, col = r - sec * p.d;
              float v = y;
              if (sec < 2) {
                const float2 cs = p.rope[(size_t)pos * (p.hd / 2) + (col % p.hd) / 2];
                v = (row & 1) ? other * cs.y + y * cs.x : y * cs.x - other * cs.y;
              }
              const size_t kv = ((size_t)layer * p.max_pos + pos) * p.d + col;
              if (sec == 0) {
                p.pf_q[(size_t)t * p.d + col] = v;
              } else {
                void *cache = sec == 1 ? p.kcache : p.vcache;
                if (p.kv_bf16) reinterpret_cast<__nv_bfloat16 *>(cache)[kv] = __float2bfloat16_rn(v);
                else reinterpret_cast<float *>(cache)[kv] = v;
              }
            }
          } else if (kind == kPfAddH) {
            float *h = p.pf_h + (size_t)t * p.d + r;
            const float hn = __ldcg(h) + y;
            *h = hn;
            ssq = fmaf(hn, hn, ssq);
            if (gain_next) pf_put(p.pf_xh, t, r, hn * __bfloat162float(gain_next[r]));
            if (p.pf_head && t == n_tok - 1) {  // the prefix's last token: what the decode kernel would leave behind
              if (p.trace) p.trace[((size_t)layer * 2 + which) * p.d + r] = hn;
              if (layer == p.L - 1 && which == 1) p.h[r] = hn;
            }
          } else if (kind == kPfLogits) {
            if (t == n_tok - 1) p.logits[r] = y;
          } else {
            if (!(row & 1)) pf_put(p.pf_xu, t, r >> 1, y / (1.f + __expf(-y)) * other);
          }
        }
      }
    }
  }
  if (kind == kPfAddH) pf_publish_ss(b, ssq);
}

// Causal attention of the chunk's tokens over the cache: one (token, head) item per block at a time, a warp
// per position with an online softmax, the warps merged through shared memory.  Items of tokens past n_tok
// only write zeros.
__device__ void pf_attention(PfBlk &b, int layer, int pos0, int n_tok) {
  const KParams &p = *b.p;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int epl = p.hd / 32;
  const float scale = 1.f / sqrtf((float)p.hd);
  float *s_acc = b.red;  // [warps][256]
  float *s_m = b.am, *s_l = b.am + kPfWarps;  // generic path: one (max, sum) per warp
  const int items = kPfTokens * p.H;
  for (int item = blockIdx.x; item < items; item += gridDim.x) {
    const int t = item / p.H, head = item - t * p.H;
    if (t >= n_tok) {
      for (int dim = threadIdx.x; dim < p.hd; dim += kPfThreads) pf_put(p.pf_xo, t, head * p.hd + dim, 0.f);
      continue;
    }
    const int T = pos0 + t + 1;
    float q[8], acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      q[e] = e < epl ? __ldcg(p.pf_q + (size_t)t * p.d + head * p.hd + lane * epl + e) : 0.f;
      acc[e] = 0.f;
    }
    float m = -CUDART_INF_F, l = 0.f;
    for (int tp = warp; tp < T; tp += kPfWarps) {
      const size_t base = ((size_t)layer * p.max_pos + tp) * p.d + head * p.hd + lane * epl;
      float dot = 0.f, vv[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        float kx = 0.f;
        vv[e] = 0.f;
        if (e < epl) {
          if (p.kv_bf16) {
            kx = __uint_as_float((uint32_t)__ldcg(reinterpret_cast<const unsigned short *>(p.kcache) + base + e) << 16);
            vv[e] = __uint_as_float((uint32_t)__ldcg(reinterpret_cast<const unsigned short *>(p.vcache) + base + e) << 16);
          } else {
            kx = __ldcg(reinterpret_cast<const float *>(p.kcache) + base + e);
            vv[e] = __ldcg(reinterpret_cast<const float *>(p.vcache) + base + e);
          }
        }
        dot = fmaf(q[e], kx, dot);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
      const float s = dot * scale;
      const float mn = fmaxf(m, s);
      const float c = __expf(m - mn), pw = __expf(s - mn);
      l = l * c + pw;
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] = acc[e] * c + pw * vv[e];
      m = mn;
    }
    named_sync(1, kPfThreads);  // scratch free again
#pragma unroll
    for (int e = 0; e < 8; ++e)
      if (e < epl) s_acc[warp * 256 + lane * epl + e] = acc[e];
    if (lane == 0) {
      s_m[warp] = m;
      s_l[warp] = l;
    }
    named_sync(1, kPfThreads);
    for (int dim = threadIdx.x; dim < p.hd; dim += kPfThreads) {
      float M = -CUDART_INF_F;
#pragma unroll
      for (int w = 0; w < kPfWarps; ++w) M = fmaxf(M, s_m[w]);
      float L = 0.f, A = 0.f;
#pragma unroll
      for (int w = 0; w < kPfWarps; ++w) {
        const float wgt = s_m[w] == -CUDART_INF_F ? 0.f : __expf(s_m[w] - M);
        L = fmaf(s_l[w], wgt, L);
        A = fmaf(s_acc[w * 256 + dim], wgt, A);
      }
      pf_put(p.pf_xo, t, head * p.hd + dim, A / L);
    }
  }
  named_sync(1, kPfThreads);
}

// ---------------------------------------------------------------- attention, bf16 cache, head_dim <= 128
// Item = (head, range of cached positions); all tokens of the chunk share every key / value row that is loaded.
// A warp takes one position at a time: lane = EPL dims of the row; the 8 tokens of a sweep have their partial
// dot products folded across the lanes so that lanes 4j..4j+3 end up with token j's score, keep its online
// softmax state there, and hand the weights back to every lane for the weighted sum of values.
template <int EPL>
__device__ __forceinline__ void pf_load_row(const __nv_bfloat16 *src, float (&x)[EPL]) {
  if (EPL == 4) {
    const uint2 v = __ldcg(reinterpret_cast<const uint2 *>(src));
    x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xffff0000u);
    x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xffff0000u);
  } else if (EPL == 2) {
    const unsigned int v = __ldcg(reinterpret_cast<const unsigned int *>(src));
    x[0] = __uint_as_float(v << 16); x[1] = __uint_as_float(v & 0xffff0000u);
  } else {
#pragma unroll
    for (int e = 0; e < EPL; ++e)
      x[e] = __uint_as_float((uint32_t)__ldcg(reinterpret_cast<const unsigned short *>(src) + e) << 16);
  }
}

// One warp, tokens t0..t0+7, positions lo + warp, lo + warp + 8, ... < hi.  Leaves (max, sum) of this lane's
// token (lanes 4j..4j+3: token t0 + j) and the unnormalised weighted value sums of all 8 tokens for this lane's
// dims.
template <int EPL>
__device__ __forceinline__ void pf_attn_sweep(const KParams &p, const __nv_bfloat16 *kbase, const __nv_bfloat16 *vbase, int lo,
                                              int hi, int t0, int pos0, int n_tok, int head, float &m, float &l,
                                              float (&acc)[8][EPL]) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const float scale = 1.f / sqrtf((float)p.hd);
  float q[8][EPL];
#pragma unroll
  for (int j = 0; j < 8; ++j)
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      q[j][e] = t0 + j < n_tok ? __ldcg(p.pf_q + (size_t)(t0 + j) * p.d + head * p.hd + lane * EPL + e) * scale : 0.f;
      acc[j][e] = 0.f;
    }
  const int mine = t0 + ((lane >> 2) & 7);
  const int limit = mine < n_tok ? pos0 + mine : -1;  // last position this lane's token may look at
  m = -CUDART_INF_F;
  l = 0.f;
  int tp = lo + warp;
  float kn[EPL], vn[EPL];
  if (tp < hi) {
    pf_load_row<EPL>(kbase + (size_t)tp * p.d, kn);
    pf_load_row<EPL>(vbase + (size_t)tp * p.d, vn);
  }
  for (; tp < hi; tp += kPfWarps) {
    float kx[EPL], vx[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      kx[e] = kn[e];
      vx[e] = vn[e];
    }
    if (tp + kPfWarps < hi) {  // next row's loads fly while this one is used
      pf_load_row<EPL>(kbase + (size_t)(tp + kPfWarps) * p.d, kn);
      pf_load_row<EPL>(vbase + (size_t)(tp + kPfWarps) * p.d, vn);
    }
    float d8[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      d8[j] = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) d8[j] = fmaf(q[j][e], kx[e], d8[j]);
    }
    // fold: 8 partial sums over 32 lanes -> lane holds the full sum of token (lane / 4) % 8
    float d4[4], d2[2], sc;
    {
      const bool up = lane & 16;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float send = up ? d8[j] : d8[j + 4], keep = up ? d8[j + 4] : d8[j];
        d4[j] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
      }
    }
    {
      const bool up = lane & 8;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const float send = up ? d4[j] : d4[j + 2], keep = up ? d4[j + 2] : d4[j];
        d2[j] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
      }
    }
    {
      const bool up = lane & 4;
      const float send = up ? d2[0] : d2[1], keep = up ? d2[1] : d2[0];
      sc = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    }
    sc += __shfl_xor_sync(0xffffffffu, sc, 2);
    sc += __shfl_xor_sync(0xffffffffu, sc, 1);
    const bool visible = tp <= limit;
    const float mn = visible ? fmaxf(m, sc) : m;
    const float c = mn == m ? 1.f : __expf(m - mn);
    const float pw = visible ? __expf(sc - mn) : 0.f;
    l = fmaf(l, c, pw);
    m = mn;
    if (__any_sync(0xffffffffu, c != 1.f)) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float cj = __shfl_sync(0xffffffffu, c, 4 * j);
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[j][e] *= cj;
      }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float pj = __shfl_sync(0xffffffffu, pw, 4 * j);
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[j][e] = fmaf(pj, vx[e], acc[j][e]);
    }
  }
}

// Item = (head, 8 of the chunk's 16 tokens, range of positions).  Short contexts are not split by position
// (the ranges' merge is not worth it); long ones are split as far as the grid has blocks for.
template <int EPL>
__device__ __forceinline__ void pf_attention_rows(const KParams *pp, float *am, float *red, int *last, int layer, int pos0,
                                                  int n_tok) {
  const KParams &p = *pp;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
  const int T = pos0 + n_tok;  // positions in the cache after this chunk
  int S = 1;
  if (T >= 256) S = max(1, min(kPfMaxSplit, (int)gridDim.x / (2 * p.H)));
  float *s_m = am, *s_l = am + kPfWarps * 8, *s_f = am + 2 * kPfWarps * 8;  // [warp][token]
  float *s_M = am + 3 * kPfWarps * 8, *s_L = s_M + 8;                      // [token]
  float *sum = red;                                                        // [8 tokens][hd] merged value sums
  const int items = p.H * 2 * S;
  for (int item = blockIdx.x; item < items; item += gridDim.x) {
    const int head = item / (2 * S), half = (item / S) & 1, sp = item % S;
    const int t0 = half * 8;
    if (t0 >= n_tok) {  // no such tokens in this chunk: their attention output is zero
      if (sp == 0)
        for (int i = tid; i < 8 * p.hd; i += kPfThreads) pf_put(p.pf_xo, t0 + i / p.hd, head * p.hd + i % p.hd, 0.f);
      continue;
    }
    const int lo = (int)((long long)T * sp / S), hi = (int)((long long)T * (sp + 1) / S);
    const __nv_bfloat16 *kbase = reinterpret_cast<const __nv_bfloat16 *>(p.kcache) + (size_t)layer * p.max_pos * p.d + head * p.hd + lane * EPL;
    const __nv_bfloat16 *vbase = reinterpret_cast<const __nv_bfloat16 *>(p.vcache) + (size_t)layer * p.max_pos * p.d + head * p.hd + lane * EPL;
    float m, l, acc[8][EPL];
    pf_attn_sweep<EPL>(p, kbase, vbase, lo, hi, t0, pos0, n_tok, head, m, l, acc);
    named_sync(1, kPfThreads);  // scratch of the item before is no longer read
    if ((lane & 3) == 0) {
      s_m[warp * 8 + (lane >> 2)] = m;
      s_l[warp * 8 + (lane >> 2)] = l;
    }
    named_sync(1, kPfThreads);
    if (tid < kPfWarps * 8) {  // (warp w, token j): this warp's factor towards the block's maximum
      const int j = tid & 7;
      float M = -CUDART_INF_F;
#pragma unroll
      for (int w = 0; w < kPfWarps; ++w) M = fmaxf(M, s_m[w * 8 + j]);
      s_f[tid] = s_m[tid] == -CUDART_INF_F ? 0.f : __expf(s_m[tid] - M);
      if (tid < 8) {
        float L = 0.f;
#pragma unroll
        for (int w = 0; w < kPfWarps; ++w) L = fmaf(s_l[w * 8 + j], s_m[w * 8 + j] == -CUDART_INF_F ? 0.f : __expf(s_m[w * 8 + j] - M), L);
        s_M[j] = M;
        s_L[j] = L;
      }
    }
    named_sync(1, kPfThreads);
    // the warps add their value sums one after the other: a fixed order
    for (int w = 0; w < kPfWarps; ++w) {
      if (warp == w) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float f = s_f[w * 8 + j];
#pragma unroll
          for (int e = 0; e < EPL; ++e) {
            float *dst = sum + (size_t)j * p.hd + lane * EPL + e;
            *dst = (w == 0 ? 0.f : *dst) + acc[j][e] * f;
          }
        }
      }
      named_sync(1, kPfThreads);
    }
    if (S == 1) {
      for (int i = tid; i < 8 * p.hd; i += kPfThreads) {
        const int j = i / p.hd;
        const float L = s_L[j];
        pf_put(p.pf_xo, t0 + j, head * p.hd + i - j * p.hd, L > 0.f ? sum[i] / L : 0.f);
      }
    } else {
      // partial result of this range to global memory; the block that completes the group merges its ranges
      const int group = item / S;  // (head, half)
      float *part = p.pf_part + (size_t)item * 8 * p.hd;
      float2 *ml = p.pf_ml + (size_t)item * 8;
      for (int i = tid; i < 8 * p.hd; i += kPfThreads) part[i] = sum[i];
      if (tid < 8) ml[tid] = make_float2(s_M[tid], s_L[tid]);
      __threadfence();
      named_sync(1, kPfThreads);
      if (tid == 0) {
        const unsigned int seen = atomicAdd(p.pf_cnt + group, 1u);
        *last = seen == (unsigned int)(S - 1);
        if (*last) {
          p.pf_cnt[group] = 0u;  // all ranges of this group have arrived: ready for the next layer
          __threadfence();
        }
      }
      named_sync(1, kPfThreads);
      if (*last) {
        const float *part0 = p.pf_part + (size_t)group * S * 8 * p.hd;
        const float2 *ml0 = p.pf_ml + (size_t)group * S * 8;
        for (int i = tid; i < 8 * p.hd; i += kPfThreads) {
          const int j = i / p.hd;
          float M = -CUDART_INF_F;
          for (int r = 0; r < S; ++r) M = fmaxf(M, __ldcg(&ml0[(size_t)r * 8 + j]).x);
          float L = 0.f, A = 0.f;
          for (int r = 0; r < S; ++r) {
            const float2 v = __ldcg(&ml0[(size_t)r * 8 + j]);
            const float f = v.x == -CUDART_INF_F ? 0.f : __expf(v.x - M);
            L = fmaf(v.y, f, L);
            A = fmaf(__ldcg(&part0[(size_t)r * 8 * p.hd + i]), f, A);
          }
          pf_put(p.pf_xo, t0 + j, head * p.hd + i - j * p.hd, L > 0.f ? A / L : 0.f);
        }
      }
    }
    named_sync(1, kPfThreads);
  }
}

// One dispatch on the head dimension.
__device__ __forceinline__ void pf_attention_bf16(const KParams *pp, float *am, float *red, int *last, int layer, int pos0,
                                               int n_tok) {
  switch (pp->hd / 32) {
    case 1: pf_attention_rows<1>(pp, am, red, last, layer, pos0, n_tok); break;
    case 2: pf_attention_rows<2>(pp, am, red, last, layer, pos0, n_tok); break;
    case 3: pf_attention_rows<3>(pp, am, red, last, layer, pos0, n_tok); break;
    default: pf_attention_rows<4>(pp, am, red, last, layer, pos0, n_tok); break;
  }
}

__device__ void pf_consumer(PfBlk &b) {
  const KParams &p = *b.p;
  const int n_tok = p.n_iters, pos0 = p.pos0;
  // residual rows start as the tokens' embeddings (zeros past n_tok); a block takes a range of columns
  {
    const __nv_bfloat16 *gain0 = p.layers[0].attn_norm;
    const int c0 = (int)((long long)p.d * blockIdx.x / gridDim.x), c1 = (int)((long long)p.d * (blockIdx.x + 1) / gridDim.x);
    const int t = threadIdx.x & 15;
    float ssq = 0.f;
    for (int c = c0 + (threadIdx.x >> 4); c < c1; c += kPfThreads / kPfTokens) {
      const float v = t < n_tok ? __bfloat162float(p.tok_emb[(size_t)p.prefix[t] * p.d + c]) : 0.f;
      p.pf_h[(size_t)t * p.d + c] = v;
      pf_put(p.pf_xh, t, c, v * __bfloat162float(gain0[c]));
      ssq = fmaf(v, v, ssq);
    }
    pf_publish_ss(b, ssq);
  }
  if (pf_grid_barrier(b)) return;
  for (int l = 0; l < p.L; ++l) {
    const LayerW &lw = p.layers[l];
    pf_gemm(b, pf_phase(p, 4 * l), true, kPfQKV, nullptr, l, 0, pos0, n_tok);
    if (pf_grid_barrier(b)) return;
    if (p.kv_bf16 && p.hd <= 128) {
      pf_attention_bf16(b.p, b.am, b.red, b.last, l, pos0, n_tok);
    } else {
      pf_attention(b, l, pos0, n_tok);
    }
    if (pf_grid_barrier(b)) return;
    pf_gemm(b, pf_phase(p, 4 * l + 1), false, kPfAddH, lw.ffn_norm, l, 0, pos0, n_tok);
    if (pf_grid_barrier(b)) return;
    pf_gemm(b, pf_phase(p, 4 * l + 2), true, kPfSwiGLU, nullptr, l, 0, pos0, n_tok);
    if (pf_grid_barrier(b)) return;
    pf_gemm(b, pf_phase(p, 4 * l + 3), false, kPfAddH,
            l + 1 < p.L ? p.layers[l + 1].attn_norm : (p.pf_head ? p.final_norm : nullptr), l, 1, pos0, n_tok);
    if (pf_grid_barrier(b)) return;
  }
  if (p.pf_head) {
    // the prefix ends here: logits of its last token, then the first timestep (Eq. 1) as in the decode kernel
    pf_gemm(b, pf_phase(p, 4 * p.L), true, kPfLogits, nullptr, 0, 0, pos0, n_tok);
    named_sync(1, kPfThreads);
    int r0, r1;
    pf_rows(p.V, 1, r0, r1);
    if (threadIdx.x < 32) block_topk(p, r0, r1, blockIdx.x);
    if (pf_grid_barrier(b)) return;
    if (blockIdx.x == 0 && threadIdx.x < 32) {
      tail_keep_topk(p, gridDim.x);
      tail_first(p, threadIdx.x, 0);
      __syncwarp();
      tail_gamma(p, threadIdx.x);
    }
  }
}

// Nine warps leave one scheduler with three of them: 16384 registers / (3 x 32) caps a thread at 168, which
// is what the compiler derives for a block of 384.
__global__ void __launch_bounds__(384, 1) spd_prefill_kernel(const __grid_constant__ KParams p) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  // the swizzle pattern of the tiled copies repeats every 1024 bytes of shared-memory address
  uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  __shared__ uint64_t s_full[kPfStages], s_empty[kPfStages], s_xfull[kPfXBufs], s_xempty[kPfXBufs], s_xgo;
  __shared__ float s_rs[kPfTokens], s_am[kPfAmFloats];
  __shared__ int s_last;
  __shared__ int s_dead, s_quit;
  PfBlk b;
  b.p = &p;
  b.ring = smem;
  b.xblk = smem + (size_t)kPfStages * kPfStageBytes;
  b.red = reinterpret_cast<float *>(smem + (size_t)kPfStages * kPfStageBytes + (size_t)kPfXBufs * kPfXBytes);
  b.rs = s_rs;
  b.am = s_am;
  b.last = &s_last;
  b.full = s_full;
  b.empty = s_empty;
  b.xfull = s_xfull;
  b.xempty = s_xempty;
  b.xgo = &s_xgo;
  b.dead = &s_dead;
  b.quit = &s_quit;
  b.bar_target = 0;
  b.c_stage = 0;
  b.c_phase = 0;
  b.x_n = 0;
  if (threadIdx.x == 0) {
    s_dead = 0;
    s_quit = 0;
    for (int s = 0; s < kPfStages; ++s) {
      mbar_init(&s_full[s], 1);
      mbar_init(&s_empty[s], kPfWarps);
    }
    for (int i = 0; i < kPfXBufs; ++i) {
      mbar_init(&s_xfull[i], 1);
      mbar_init(&s_xempty[i], kPfWarps);
    }
    mbar_init(&s_xgo, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // boxes wholly past a matrix's last column are never copied, yet every warp multiplies all its k-steps
  // (against zero fragments there): the ring starts zeroed so that such boxes hold finite values
  for (size_t i = threadIdx.x; i < (size_t)kPfStages * kPfStageBytes / 16; i += blockDim.x)
    reinterpret_cast<uint4 *>(smem)[i] = make_uint4(0u, 0u, 0u, 0u);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();
  if (threadIdx.x >= kPfThreads + 32) {
    if (threadIdx.x == kPfThreads + 32) pf_xproducer(b);
    __syncwarp();
  } else if (threadIdx.x >= kPfThreads) {
    pf_producer(b);
  } else {
    pf_consumer(b);
  }
  __syncthreads();
}

}  // namespace spd

extern "C" size_t spd_internal_prefill_smem(void) {
  return (size_t)spd::kPfStages * spd::kPfStageBytes + (size_t)spd::kPfXBufs * spd::kPfXBytes + 2 * spd::kPfRedBytes + 1024;  // + alignment slack
}

extern "C" cudaError_t spd_internal_prefill_prepare(int *blocks_per_sm) {
  const size_t dyn = spd_internal_prefill_smem();
  cudaError_t e = cudaFuncSetAttribute(reinterpret_cast<const void *>(&spd::spd_prefill_kernel),
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
  if (e != cudaSuccess) return e;
  return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, reinterpret_cast<const void *>(&spd::spd_prefill_kernel),
                                                       spd::kPfBlock, dyn);
}

extern "C" cudaError_t spd_internal_prefill_launch(const spd::KParams *p, int grid, cudaStream_t stream) {
  void *args[] = {const_cast<spd::KParams *>(p)};
  return cudaLaunchCooperativeKernel(reinterpret_cast<const void *>(&spd::spd_prefill_kernel), dim3(grid), dim3(spd::kPfBlock), args,
                                     spd_internal_prefill_smem(), stream);
}
