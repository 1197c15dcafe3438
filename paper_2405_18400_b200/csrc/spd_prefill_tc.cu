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
// columns) and hands the stage back with tcgen05.commit, four warps move the finished accumulator from
// tensor memory to global memory.  Every wait is bounded; a wait that runs out records SPD_ETIMEOUT in the
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

struct TcShared {
  uint64_t full[kTcStages], empty[kTcStages], accum;
  uint32_t tmem_base;
  int dead;
};

// Bounded wait on an mbarrier phase; false when the block gave up (here or elsewhere).
__device__ __forceinline__ bool tc_wait(TcShared &sh, State *st, uint64_t *bar, uint32_t parity, int info) {
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
// 64 columns.  Rows and columns past either matrix arrive as zeros.  grid = (ceil(N / 128), tokens / 128).
__global__ void __launch_bounds__(kTcThreads, 1)
    spd_tc_gemm_kernel(const void *tmap_x, const void *tmap_w, float *Y, int N, int C, int x_term_rows, State *st) {
  extern __shared__ __align__(16) uint8_t tc_smem_raw[];
  uint8_t *smem = tc_smem_raw + ((1024u - (smem_u32(tc_smem_raw) & 1023u)) & 1023u);
  __shared__ TcShared sh;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nk = (C + kTcKB - 1) / kTcKB;
  const int n0 = blockIdx.x * kTcN, m0 = blockIdx.y * kTcM;
  if (threadIdx.x == 0) {
    sh.dead = 0;
    for (int s = 0; s < kTcStages; ++s) {
      mbar_init(&sh.full[s], 1);
      mbar_init(&sh.empty[s], 1);
    }
    mbar_init(&sh.accum, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tc_alloc(&sh.tmem_base, kTcN);
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
      bool ok = true;
      for (int ks = 0; ks < nk; ++ks) {
        if (!tc_wait(sh, st, &sh.full[stage], phase, 410)) { ok = false; break; }
        tc_fence_after();
        const uint32_t base = ring + stage * (uint32_t)kTcStageBytes;
#pragma unroll
        for (int j = 0; j < 3; ++j)
#pragma unroll
          for (int kk = 0; kk < kTcKB / 16; ++kk)  // 16 columns = 32 bytes further into the swizzled rows
            tc_mma(tmem, tc_desc(base + j * kTcTermBytes + kk * 32), tc_desc(base + 3 * kTcTermBytes + kk * 32), idesc,
                   (uint32_t)((ks | j | kk) != 0));
        tc_commit(&sh.empty[stage]);  // the stage is free once these have read it
        if (++stage == (uint32_t)kTcStages) { stage = 0; phase ^= 1u; }
      }
      if (ok) tc_commit(&sh.accum);
    }
    __syncwarp();
  } else {
    // accumulator to global memory: warp w may read lanes 32 (w % 4) .. 32 (w % 4) + 31, a token per thread
    const int quarter = warp & 3;
    const bool ok = tc_wait(sh, st, &sh.accum, 0u, 420);
    tc_fence_after();
    if (ok) {
      float *row = Y + (size_t)(m0 + quarter * 32 + lane) * N;
#pragma unroll 1
      for (int c0 = 0; c0 < kTcN; c0 += 32) {
        uint32_t r[32];
        tc_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0, r);
#pragma unroll
        for (int j = 0; j < 32; j += 4)
          if (n0 + c0 + j < N)
            *reinterpret_cast<float4 *>(row + n0 + c0 + j) =
                make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]), __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tc_dealloc(tmem, kTcN);
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

// One token per block: the residual row (the embedding of ids[t] when `ids`, else h + y when `y`), stored, and
// when `gain`: its RMSNorm (x * rsqrt(mean x^2 + eps) * gain) as three bf16 terms for the next product.
__global__ void __launch_bounds__(256) spd_tc_resid_norm_kernel(float *h, const float *y, const int32_t *ids, const __nv_bfloat16 *emb,
                                                                const __nv_bfloat16 *gain, uint16_t *X, size_t term_stride, int d, float eps) {
  __shared__ float scratch[8];
  const int t = blockIdx.x;
  float *hr = h + (size_t)t * d;
  float ss = 0.f;
  for (int c = threadIdx.x; c < d; c += 256) {
    float v;
    if (ids) v = __bfloat162float(emb[(size_t)ids[t] * d + c]);
    else v = hr[c] + y[(size_t)t * d + c];
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
                                                                int d, int hd, int max_pos, int layer, int pos0, int kv_bf16) {
  const int t = blockIdx.x, pos = pos0 + t;
  const float *yr = Y + (size_t)t * 3 * d;
  const size_t crow = ((size_t)layer * max_pos + pos) * d;
  for (int i = threadIdx.x; i < d / 2; i += 256) {
    const float2 cs = rope[(size_t)pos * (hd / 2) + (i % (hd / 2))];
    const float qe = yr[2 * i], qo = yr[2 * i + 1], ke = yr[d + 2 * i], ko = yr[d + 2 * i + 1];
    Q[(size_t)t * d + 2 * i] = qe * cs.x - qo * cs.y;
    Q[(size_t)t * d + 2 * i + 1] = qe * cs.y + qo * cs.x;
    const float k0 = ke * cs.x - ko * cs.y, k1 = ke * cs.y + ko * cs.x;
    const float v0 = yr[2 * d + 2 * i], v1 = yr[2 * d + 2 * i + 1];
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
__global__ void __launch_bounds__(256) spd_tc_swiglu_kernel(const float *Y, uint16_t *X, size_t term_stride, int f) {
  const int t = blockIdx.x;
  const float2 *yr = reinterpret_cast<const float2 *>(Y + (size_t)t * 2 * f);
  for (int j = threadIdx.x; j < f; j += 256) {
    const float2 gu = yr[j];
    tc_put3(X, term_stride, (size_t)t * f + j, gu.x / (1.f + __expf(-gu.x)) * gu.y);
  }
}

// Causal attention of the block's tokens over the cache.  Block = (8 consecutive tokens, one head), a warp per
// token; the warp's lanes form 4 groups of 8: a group takes every fourth cached position, each of its lanes
// PER = head_dim / 8 dimensions of it; online softmax per group, the groups merged by shuffles at the end.
// The eight warps read the same cache rows at about the same time.  Output as three bf16 terms.
template <int PER, bool BF16>
__global__ void __launch_bounds__(256) spd_tc_attn_kernel(const float *Q, const void *kcache, const void *vcache, uint16_t *X,
                                                          size_t term_stride, int d, int hd, int max_pos, int layer, int pos0) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = blockIdx.x * 8 + warp, head = blockIdx.y;
  const int g = lane >> 3, s = lane & 7;
  const int per = PER > 0 ? PER : hd / 8;
  constexpr int kMax = PER > 0 ? PER : 32;
  const int T = pos0 + t + 1;
  const float scale = 1.f / sqrtf((float)hd);
  const int col = head * hd + s * per;
  float q[kMax], acc[kMax];
#pragma unroll
  for (int e = 0; e < kMax; ++e) {
    q[e] = e < per ? Q[(size_t)t * d + col + e] * scale : 0.f;
    acc[e] = 0.f;
  }
  float m = -CUDART_INF_F, l = 0.f;
  for (int tp0 = 0; tp0 < T; tp0 += 4) {
    const int tp = tp0 + g;
    const bool visible = tp < T;
    const size_t base = ((size_t)layer * max_pos + (visible ? tp : 0)) * d + col;
    float kv[kMax], vv[kMax];
    if (BF16) {
      const uint4 *kp = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(kcache) + base);
      const uint4 *vp = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(vcache) + base);
#pragma unroll
      for (int e = 0; e < kMax; e += 8) {
        if (e < per) {
          const uint4 a = kp[e >> 3], b = vp[e >> 3];
          const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            kv[e + 2 * j] = __uint_as_float(aw[j] << 16);
            kv[e + 2 * j + 1] = __uint_as_float(aw[j] & 0xffff0000u);
            vv[e + 2 * j] = __uint_as_float(bw[j] << 16);
            vv[e + 2 * j + 1] = __uint_as_float(bw[j] & 0xffff0000u);
          }
        }
      }
    } else {
      const float4 *kp = reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(kcache) + base);
      const float4 *vp = reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(vcache) + base);
#pragma unroll
      for (int e = 0; e < kMax; e += 4) {
        if (e < per) {
          const float4 a = kp[e >> 2], b = vp[e >> 2];
          kv[e] = a.x; kv[e + 1] = a.y; kv[e + 2] = a.z; kv[e + 3] = a.w;
          vv[e] = b.x; vv[e + 1] = b.y; vv[e + 2] = b.z; vv[e + 3] = b.w;
        }
      }
    }
    float dot = 0.f;
#pragma unroll
    for (int e = 0; e < kMax; ++e)
      if (e < per) dot = fmaf(q[e], kv[e], dot);
    dot += __shfl_xor_sync(0xffffffffu, dot, 1);
    dot += __shfl_xor_sync(0xffffffffu, dot, 2);
    dot += __shfl_xor_sync(0xffffffffu, dot, 4);
    if (visible) {
      const float mn = fmaxf(m, dot);
      const float c = __expf(m - mn), pw = __expf(dot - mn);  // m = -inf at first: c = 0
      l = fmaf(l, c, pw);
#pragma unroll
      for (int e = 0; e < kMax; ++e)
        if (e < per) acc[e] = fmaf(acc[e], c, pw * vv[e]);
      m = mn;
    }
  }
  // the four groups' states
#pragma unroll
  for (int off = 8; off <= 16; off <<= 1) {
    const float mo = __shfl_xor_sync(0xffffffffu, m, off), lo = __shfl_xor_sync(0xffffffffu, l, off);
    const float M = fmaxf(m, mo);
    const float cs = m == -CUDART_INF_F ? 0.f : __expf(m - M), co = mo == -CUDART_INF_F ? 0.f : __expf(mo - M);
    l = l * cs + lo * co;
#pragma unroll
    for (int e = 0; e < kMax; ++e) {
      const float ao = __shfl_xor_sync(0xffffffffu, acc[e], off);
      if (e < per) acc[e] = (g & (off >> 3)) ? ao * co + acc[e] * cs : acc[e] * cs + ao * co;
    }
    m = M;
  }
  if (g == 0) {
    const float inv = 1.f / l;
#pragma unroll
    for (int e = 0; e < kMax; ++e)
      if (e < per) tc_put3(X, term_stride, (size_t)t * d + col + e, acc[e] * inv);
  }
}

}  // namespace spd

namespace {

template <int PER>
cudaError_t launch_attn(const spd::TcJob &j, int layer, int n_tok, cudaStream_t s) {
  const dim3 grid(n_tok / 8, j.H);
  const size_t ts = (size_t)j.x_term_rows * j.d;
  if (j.kv_bf16)
    spd::spd_tc_attn_kernel<PER, true><<<grid, 256, 0, s>>>(j.q, j.kcache, j.vcache, j.x, ts, j.d, j.hd, j.max_pos, layer, j.pos0);
  else
    spd::spd_tc_attn_kernel<PER, false><<<grid, 256, 0, s>>>(j.q, j.kcache, j.vcache, j.x, ts, j.d, j.hd, j.max_pos, layer, j.pos0);
  return cudaGetLastError();
}

size_t tc_gemm_smem() { return (size_t)spd::kTcStages * spd::kTcStageBytes + 1024; }

}  // namespace

extern "C" cudaError_t spd_internal_tc_prepare(void) {
  return cudaFuncSetAttribute(reinterpret_cast<const void *>(&spd::spd_tc_gemm_kernel), cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)tc_gemm_smem());
}

// Enqueues the decoder over j.n_tok tokens (a multiple of 128, at most j.x_term_rows) at positions j.pos0 ..:
// their keys and values enter the cache.  *launches receives the number of kernels enqueued.
extern "C" cudaError_t spd_internal_tc_prefill(const spd::TcJob *job, cudaStream_t s, int *launches) {
  const spd::TcJob &j = *job;
  const int n = j.n_tok, d = j.d, f = j.f;
  const size_t ts_d = (size_t)j.x_term_rows * d, ts_f = (size_t)j.x_term_rows * f;
  const uint8_t *xmap_d = j.x_tmaps, *xmap_f = j.x_tmaps + spd::kTensorMapBytes;
  int count = 0;
  cudaError_t e = cudaSuccess;
  auto gemm = [&](const uint8_t *xmap, int which, int N, int C) {
    if (e != cudaSuccess) return;
    const dim3 grid((N + spd::kTcN - 1) / spd::kTcN, n / spd::kTcM);
    spd::spd_tc_gemm_kernel<<<grid, spd::kTcThreads, tc_gemm_smem(), s>>>(xmap, j.w_tmaps + (size_t)which * spd::kTensorMapBytes, j.y, N, C,
                                                                         j.x_term_rows, j.st);
    e = cudaGetLastError();
    ++count;
  };
  auto resid = [&](const float *y, const int32_t *ids, const __nv_bfloat16 *gain) {
    if (e != cudaSuccess) return;
    spd::spd_tc_resid_norm_kernel<<<n, 256, 0, s>>>(j.h, y, ids, j.tok_emb, gain, j.x, ts_d, d, j.eps);
    e = cudaGetLastError();
    ++count;
  };
  resid(nullptr, j.ids, j.layers[0].attn_norm);
  for (int l = 0; l < j.L && e == cudaSuccess; ++l) {
    gemm(xmap_d, 4 * l, 3 * d, d);
    if (e != cudaSuccess) break;
    spd::spd_tc_rope_cache_kernel<<<n, 256, 0, s>>>(j.y, j.q, j.kcache, j.vcache, j.rope, d, j.hd, j.max_pos, l, j.pos0, j.kv_bf16);
    if ((e = cudaGetLastError()) != cudaSuccess) break;
    e = j.hd == 128 ? launch_attn<16>(j, l, n, s) : j.hd == 64 ? launch_attn<8>(j, l, n, s) : launch_attn<0>(j, l, n, s);
    count += 2;
    gemm(xmap_d, 4 * l + 1, d, d);
    resid(j.y, nullptr, j.layers[l].ffn_norm);
    gemm(xmap_d, 4 * l + 2, 2 * f, d);
    if (e != cudaSuccess) break;
    spd::spd_tc_swiglu_kernel<<<n, 256, 0, s>>>(j.y, j.x, ts_f, f);
    e = cudaGetLastError();
    ++count;
    gemm(xmap_f, 4 * l + 3, d, f);
    if (l + 1 < j.L) resid(j.y, nullptr, j.layers[l + 1].attn_norm);  // the last layer's output feeds nothing here
  }
  if (launches) *launches = count;
  return e;
}
