// Persistent decode kernel for Superposed Decoding on sm_100a.
//
// One cooperative launch runs n_iters timesteps.  Every block keeps one producer warp and sixteen
// consumer warps.  The producer thread walks the static list of weight chunks that its block owns
// (contiguous row ranges of every matrix, in the order the decoder uses them) and streams them
// into a shared-memory ring with bulk asynchronous copies that signal mbarriers; because weights do
// not depend on activations it runs ahead across phase boundaries and across timesteps, so HBM
// stays busy while the consumers exchange activation vectors through L2 at grid barriers.  Matrices
// that also come in fragment order (spd_pack_image) are multiplied on the tensor cores: mma.sync over
// 8-row units whose 16-byte vectors are the instruction's weight registers, x as three exact bf16 terms
// kept as fragments in shared memory.  For the others the consumers split the columns of each row among
// all threads (the activation slice of a thread stays in registers for a whole phase) and reduce with
// shuffles.  Rows are finished in per-phase epilogues
// (rotary embedding + cache append, residual add, SwiGLU, logits + block-level top-k).  Block 0 then
// runs the method's tail: KeepTopK over the whole vocabulary, the k*k expansion with n-gram hash
// probes (Eq. 5), the interpolation (Eq. 6/7), the selection of the k best options (Eq. 2) and the
// new weights gamma (Eq. 4), and forms the next superposed input (Eq. 3).
//
// Every wait (mbarrier, grid barrier, table probe) is bounded; a wait that gives up records an
// error, raises an abort flag that turns all later waits into no-ops, and the kernel runs to its end.
#include <cuda_runtime.h>
#include <math_constants.h>

#include "spd_params.h"
#include "spd_ptx.cuh"
#include "spd_nucleus.cuh"
#include "spd_tail.cuh"
#include "spd_score.cuh"

namespace spd {

// The block's shared memory.  The kernels' loops name these variables directly (their addresses are constants)
// instead of carrying pointers to them in registers.
extern __shared__ __align__(128) uint8_t smem[];  // the ring's stages, then the scratch area (row partials / attention merge / tail)
__shared__ uint64_t s_full[kMaxStages], s_empty[kMaxStages];
__shared__ __align__(16) float s_red[64];
__shared__ float2 s_rope[128];  // the current position's row of the rotary table (head sizes up to 256)
constexpr int kGainSlots = 256;  // gain pointers kept in shared memory: models of up to 127 layers (deeper ones read them late)
__shared__ const __nv_bfloat16 *s_gain_ptrs[kGainSlots];
__shared__ int s_dead, s_quit;

__device__ __forceinline__ float *scratch_base(const KParams &p) { return reinterpret_cast<float *>(smem + (size_t)p.n_stages * p.stage_bytes); }

// Bounded wait on an mbarrier phase.  Returns at once when the block is already giving up.
__device__ __forceinline__ void wait_mbar(Blk &b, uint64_t *bar, uint32_t parity, int info) {
  if (mbar_try_wait(bar, parity)) return;
  if (s_dead) return;
  unsigned long long t0 = globaltimer();
  uint32_t n = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++n & 31u) == 0) {
      if (s_dead) return;
      if (ld_relaxed(&b.p->st->abort_flag)) { s_dead = 1; return; }
      if (globaltimer() - t0 > kWaitNs) { give_up(b, kErrTimeout, info); return; }
    }
  }
}

// Grid-wide barrier for the consumer threads of all blocks (all blocks are co-resident: cooperative launch).
// Returns true, to every consumer thread of the block alike, once the block is giving up.
__device__ __forceinline__ bool grid_barrier(Blk &b) {
  named_sync(1, kConsumerThreads);
  if (threadIdx.x == 0) {
    b.bar_target += gridDim.x;
    if (!s_dead) {
      unsigned int *bar = &b.p->st->bar;
      __threadfence();
      atomicAdd(bar, 1u);
      unsigned long long t0 = globaltimer();
      uint32_t n = 0;
      while ((int)(ld_acquire(bar) - b.bar_target) < 0) {
        if ((++n & 63u) == 0) {
          if (ld_relaxed(&b.p->st->abort_flag)) { s_dead = 1; break; }
          if (globaltimer() - t0 > kWaitNs) { give_up(b, kErrTimeout, 100); break; }
        }
      }
    }
    s_quit = s_dead;
  }
  named_sync(1, kConsumerThreads);
  return s_quit != 0;
}

__device__ __forceinline__ void cta_rows(int R, int gran, int &r0, int &r1) {
  long long U = R / gran;
  r0 = (int)(U * blockIdx.x / gridDim.x) * gran;
  r1 = (int)(U * (blockIdx.x + 1) / gridDim.x) * gran;
}

__device__ __forceinline__ int rows_per_chunk(const KParams &p, int C) {
  int rpc = p.stage_bytes / (C * 2);
  return rpc > kMaxRowsPerChunk ? kMaxRowsPerChunk : rpc;
}

// ---------------------------------------------------------------- producer
struct Producer {
  uint32_t stage, phase;
  uint32_t issued;  // chunks issued so far (saturating at n_stages for the drain)
};

__device__ __forceinline__ void produce_matrix(Blk &b, Producer &pr, const __nv_bfloat16 *W, int R, int C, int gran) {
  const KParams &p = *b.p;
  int r0, r1;
  cta_rows(R, gran, r0, r1);
  const int rpc = rows_per_chunk(p, C);
  const uint32_t rowbytes = (uint32_t)C * 2u;
  for (int t0 = r0; t0 < r1; t0 += kTile) {
    const int t1 = min(t0 + kTile, r1);
    for (int r = t0; r < t1; r += rpc) {
      const int n = min(rpc, t1 - r);
      wait_mbar(b, &s_empty[pr.stage], pr.phase ^ 1u, 200);
      if (s_dead) return;
      const uint32_t bytes = (uint32_t)n * rowbytes;
      mbar_expect_tx(&s_full[pr.stage], bytes);
      bulk_load(smem + (size_t)pr.stage * p.stage_bytes, (const uint8_t *)W + (size_t)r * rowbytes, bytes,
                &s_full[pr.stage]);
      if (pr.issued < (uint32_t)p.n_stages) ++pr.issued;
      if (++pr.stage == (uint32_t)p.n_stages) { pr.stage = 0; pr.phase ^= 1u; }
    }
  }
}

constexpr int kPairBytes = kUnitRows * 64;  // a unit's share of a pair of 16-column blocks: 4 lanes of 16 bytes per row
// Bytes of a fragment-order unit of C columns that one ring stage takes: the unit in the fewest equal parts that fit
// a stage, in whole pairs of 16-column blocks (the last part may be shorter).
__device__ __forceinline__ uint32_t img_chunk(const KParams &p, int C) {
  const uint32_t unit = (uint32_t)C * 2u * kUnitRows, cap = (uint32_t)p.stage_bytes / kPairBytes * kPairBytes;
  const uint32_t parts = (unit + cap - 1) / cap;
  const uint32_t pairs = ((uint32_t)C / 32 + parts - 1) / parts;
  return pairs * kPairBytes;
}

// A matrix in fragment order (spd_pack_image): the units of this block, each unit in stages of img_chunk bytes and a
// shorter last one.
__device__ __forceinline__ void produce_image(Blk &b, Producer &pr, const __nv_bfloat16 *img, int R, int C) {
  const KParams &p = *b.p;
  int r0, r1;
  cta_rows(R, kUnitRows, r0, r1);
  const uint32_t unit_bytes = (uint32_t)C * 2u * kUnitRows;
  for (int r = r0; r < r1; r += kUnitRows) {
    const uint8_t *src = reinterpret_cast<const uint8_t *>(img) + (size_t)(r / kUnitRows) * unit_bytes;
    const uint32_t chunk = img_chunk(p, C);
    for (uint32_t off = 0; off < unit_bytes; off += chunk) {
      const uint32_t bytes = unit_bytes - off < chunk ? unit_bytes - off : chunk;
      wait_mbar(b, &s_empty[pr.stage], pr.phase ^ 1u, 200);
      if (s_dead) return;
      mbar_expect_tx(&s_full[pr.stage], bytes);
      bulk_load(smem + (size_t)pr.stage * p.stage_bytes, src + off, bytes, &s_full[pr.stage]);
      if (pr.issued < (uint32_t)p.n_stages) ++pr.issued;
      if (++pr.stage == (uint32_t)p.n_stages) { pr.stage = 0; pr.phase ^= 1u; }
    }
  }
}

template <bool kSampler, bool kImg>
__device__ void producer_main(Blk &b) {
  const KParams &p = *b.p;
  Producer pr{0u, 0u, 0u};
  // The layers' pointers sit in device memory that the weight stream has long pushed out of L2 when their turn
  // comes: each layer's are fetched while the layer before is streamed.
  LayerW lw = p.layers[0];
  for (int it = 0; it < p.n_iters && !s_dead; ++it) {
    for (int l = 0; l < p.L && !s_dead; ++l) {
      const LayerW nxt = p.layers[l + 1 < p.L ? l + 1 : 0];
      if constexpr (kImg) {
        produce_image(b, pr, lw.wqkv_img, 3 * p.d, p.d);
        produce_image(b, pr, lw.wo_img, p.d, p.d);
        produce_image(b, pr, lw.wgate_up_img, 2 * p.f, p.d);
      } else {
        produce_matrix(b, pr, lw.wqkv, 3 * p.d, p.d, 2);
        produce_matrix(b, pr, lw.wo, p.d, p.d, 1);
        produce_matrix(b, pr, lw.wgate_up, 2 * p.f, p.d, 2);
      }
      produce_matrix(b, pr, lw.wdown, p.d, p.f, 1);
      lw = nxt;
    }
    const bool head = kSampler ? p.mode != kModePrefill : p.mode == kModeDecode;
    if (head || it == p.n_iters - 1) {
      if constexpr (kImg) produce_image(b, pr, p.lm_head_img, p.V, p.d);
      else produce_matrix(b, pr, p.lm_head, p.V, p.d, 1);
    }
  }
  if (s_dead) {
    // Giving up: nothing more is issued; wait (bounded) until every copy already issued has landed,
    // so that no copy writes into shared memory after the block has gone.
    uint32_t s = pr.stage, ph = pr.phase;
    for (uint32_t i = 0; i < pr.issued; ++i) {
      if (s == 0) { s = (uint32_t)p.n_stages; ph ^= 1u; }
      --s;
      unsigned long long t0 = globaltimer();
      while (!mbar_try_wait(&s_full[s], ph) && globaltimer() - t0 < kWaitNs) {}
    }
  }
}

// ---------------------------------------------------------------- consumer: row dot products
__device__ __forceinline__ float dot8(const uint4 w, const float (&x)[8], float acc) {
  acc = fmaf(__uint_as_float(w.x << 16), x[0], acc);
  acc = fmaf(__uint_as_float(w.x & 0xffff0000u), x[1], acc);
  acc = fmaf(__uint_as_float(w.y << 16), x[2], acc);
  acc = fmaf(__uint_as_float(w.y & 0xffff0000u), x[3], acc);
  acc = fmaf(__uint_as_float(w.z << 16), x[4], acc);
  acc = fmaf(__uint_as_float(w.z & 0xffff0000u), x[5], acc);
  acc = fmaf(__uint_as_float(w.w << 16), x[6], acc);
  acc = fmaf(__uint_as_float(w.w & 0xffff0000u), x[7], acc);
  return acc;
}

// Sums NR per-lane accumulators over the warp with a folding butterfly.  Afterwards lane
// r * (32 / NR) holds the total of accumulator r.
template <int NR>
__device__ __forceinline__ float warp_fold(float (&a)[NR], int lane) {
  if constexpr (NR == 8) {
    float b4[4];
    const bool up = lane & 16;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float send = up ? a[i] : a[i + 4];
      const float keep = up ? a[i + 4] : a[i];
      b4[i] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
    }
    float b2[2];
    const bool up2 = lane & 8;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const float send = up2 ? b4[i] : b4[i + 2];
      const float keep = up2 ? b4[i + 2] : b4[i];
      b2[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
    }
    const bool up3 = lane & 4;
    float v = (up3 ? b2[1] : b2[0]) + __shfl_xor_sync(0xffffffffu, up3 ? b2[0] : b2[1], 4);
    v += __shfl_xor_sync(0xffffffffu, v, 2);
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    return v;
  } else if constexpr (NR == 4) {
    float b2[2];
    const bool up = lane & 16;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const float send = up ? a[i] : a[i + 2];
      const float keep = up ? a[i + 2] : a[i];
      b2[i] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
    }
    const bool up2 = lane & 8;
    float v = (up2 ? b2[1] : b2[0]) + __shfl_xor_sync(0xffffffffu, up2 ? b2[0] : b2[1], 8);
    v += __shfl_xor_sync(0xffffffffu, v, 4);
    v += __shfl_xor_sync(0xffffffffu, v, 2);
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    return v;
  } else if constexpr (NR == 2) {
    const bool up = lane & 16;
    float v = (up ? a[1] : a[0]) + __shfl_xor_sync(0xffffffffu, up ? a[0] : a[1], 16);
    v += __shfl_xor_sync(0xffffffffu, v, 8);
    v += __shfl_xor_sync(0xffffffffu, v, 4);
    v += __shfl_xor_sync(0xffffffffu, v, 2);
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    return v;
  } else {
    float v = a[0];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
  }
}

// One chunk of n (<= NR) rows in a ring stage: every thread multiplies its column vectors, the warp
// folds, and the warp's partial of row j goes to part[(trow + j) * warps + warp].
template <int NR>
__device__ __forceinline__ void consume_chunk(const uint8_t *stage, int n, int rowbytes, int nv,
                                              const float (&xr)[kMaxVec][8], float *part_rows, int warp, int lane) {
  float acc[NR];
#pragma unroll
  for (int r = 0; r < NR; ++r) acc[r] = 0.f;
#pragma unroll
  for (int i = 0; i < kMaxVec; ++i) {
    const int v = (int)threadIdx.x + i * kConsumerThreads;
    if (v < nv) {
#pragma unroll
      for (int r = 0; r < NR; ++r) {
        if (r < n) {
          const uint4 w = lds128(stage + (size_t)r * rowbytes + (size_t)v * 16);
          acc[r] = dot8(w, xr[i], acc[r]);
        }
      }
    }
  }
  const float v = warp_fold<NR>(acc, lane);
  constexpr int kStride = 32 / NR;
  const int j = lane / kStride;
  if ((lane % kStride) == 0 && j < n) part_rows[j * kConsumerWarps + warp] = v;
}

enum Epi { kEpiQKV = 0, kEpiAddH = 1, kEpiSwiGLU = 2, kEpiLogits = 3 };

struct EpiArgs {
  int layer, pos, which;  // which: 0 = after attention, 1 = after FFN (trace slot)
};

__device__ __forceinline__ float part_sum(const float *row) {
  const float4 *q = reinterpret_cast<const float4 *>(row);
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < kConsumerWarps / 4; ++i) {
    const float4 a = q[i];
    s += a.x;
    s += a.y;
    s += a.z;
    s += a.w;
  }
  return s;
}

__device__ __forceinline__ void store_kv(const KParams &p, void *cache, size_t idx, float v) {
  if (p.kv_bf16) reinterpret_cast<__nv_bfloat16 *>(cache)[idx] = __float2bfloat16_rn(v);
  else reinterpret_cast<float *>(cache)[idx] = v;
}

// Finishes rows [t0, t1) of the current matrix from the warps' partial sums.
// rs: the factor of the phase's RMSNorm, 1 / rms(h), which the prologue left out of x (1 for a phase without one).
__device__ __forceinline__ void epilogue(Blk &b, int kind, const EpiArgs &ea, const float *part, int t0, int t1, bool have_h,
                                         float h_pre, float rs) {
  const KParams &p = *b.p;
  const int tid = threadIdx.x;
  const int rows = t1 - t0;
  if (kind == kEpiQKV) {
    // rows come in pairs (2i, 2i+1) of one head: rotate q and k, append k and v to the cache
    if (tid * 2 < rows) {
      const int r = t0 + tid * 2;
      float a = part_sum(part + (size_t)(tid * 2) * kConsumerWarps) * rs;
      float c = part_sum(part + (size_t)(tid * 2 + 1) * kConsumerWarps) * rs;
      const int sec = r / p.d, col = r - sec * p.d;
      if (sec < 2) {
        const float2 cs = s_rope[(col % p.hd) / 2];  // the position's row of the rotary table
        const float ra = a * cs.x - c * cs.y, rc = a * cs.y + c * cs.x;
        a = ra;
        c = rc;
      }
      const size_t kv = ((size_t)ea.layer * p.max_pos + ea.pos) * p.d + col;
      if (sec == 0) {
        p.q[col] = a;
        p.q[col + 1] = c;
      } else if (sec == 1) {
        store_kv(p, p.kcache, kv, a);
        store_kv(p, p.kcache, kv + 1, c);
      } else {
        store_kv(p, p.vcache, kv, a);
        store_kv(p, p.vcache, kv + 1, c);
      }
    }
  } else if (kind == kEpiAddH) {
    if (tid < rows) {
      const int r = t0 + tid;
      const float y = (have_h ? h_pre : __ldcg(p.h + r)) + part_sum(part + (size_t)tid * kConsumerWarps);
      p.h[r] = y;
      if (p.trace) p.trace[((size_t)ea.layer * 2 + ea.which) * p.d + r] = y;
    }
  } else if (kind == kEpiSwiGLU) {
    if (tid * 2 < rows) {
      const float g = part_sum(part + (size_t)(tid * 2) * kConsumerWarps) * rs;
      const float up = part_sum(part + (size_t)(tid * 2 + 1) * kConsumerWarps) * rs;
      p.u[(t0 >> 1) + tid] = g / (1.f + __expf(-g)) * up;
    }
  } else {
    if (tid < rows) p.logits[t0 + tid] = part_sum(part + (size_t)tid * kConsumerWarps) * rs;
  }
}

// Streams this block's rows of one matrix through the ring against the register-resident x.
__device__ __forceinline__ void consume_matrix(Blk &b, int R, int C, int gran, const float (&xr)[kMaxVec][8], int kind,
                                               const EpiArgs &ea) {
  const KParams &p = *b.p;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int r0, r1;
  cta_rows(R, gran, r0, r1);
  const int rpc = rows_per_chunk(p, C);
  const int rowbytes = C * 2, nv = C / 8;
  // the residual rows this thread will update in the first tile are fetched now, off the critical path
  float h_pre = 0.f;
  if (kind == kEpiAddH && r0 + (int)threadIdx.x < min(r0 + kTile, r1)) h_pre = __ldcg(p.h + r0 + threadIdx.x);
  float rs = 1.f;
  int buf = 0;
  for (int t0 = r0; t0 < r1; t0 += kTile) {
    const int t1 = min(t0 + kTile, r1);
    float *part = scratch_base(p) + (size_t)buf * kTile * kConsumerWarps;
    for (int r = t0; r < t1; r += rpc) {
      const int n = min(rpc, t1 - r);
      wait_mbar(b, &s_full[b.c_stage], b.c_phase, 300);
      const uint8_t *stage = smem + (size_t)b.c_stage * p.stage_bytes;
      float *prow = part + (size_t)(r - t0) * kConsumerWarps;
      if (n > 4) consume_chunk<8>(stage, n, rowbytes, nv, xr, prow, warp, lane);
      else if (n > 2) consume_chunk<4>(stage, n, rowbytes, nv, xr, prow, warp, lane);
      else if (n > 1) consume_chunk<2>(stage, n, rowbytes, nv, xr, prow, warp, lane);
      else consume_chunk<1>(stage, n, rowbytes, nv, xr, prow, warp, lane);
      __syncwarp();
      if (lane == 0) mbar_arrive(&s_empty[b.c_stage]);
      if (++b.c_stage == (uint32_t)p.n_stages) { b.c_stage = 0; b.c_phase ^= 1u; }
    }
    named_sync(1, kConsumerThreads);
    if (kind != kEpiAddH && t0 == r0) {
      // x came from prologue_norm without the factor 1 / rms(h): the warps' sums of squares are in red[] by now
      const float4 *q = reinterpret_cast<const float4 *>(s_red);
      float ss = 0.f;
#pragma unroll
      for (int i = 0; i < kConsumerWarps / 4; ++i) {
        const float4 a = q[i];
        ss += a.x;
        ss += a.y;
        ss += a.z;
        ss += a.w;
      }
      rs = rsqrtf(ss / (float)C + p.eps);
    }
    epilogue(b, kind, ea, part, t0, t1, t0 == r0, h_pre, rs);
    buf ^= 1;
  }
}

// ---------------------------------------------------------------- consumer: matrices in fragment order on the tensor cores
// D (16 x 8) += A (16 x 16) * B (16 x 8): mma.sync m16n8k16, bf16 in, float32 accumulate.  A = a unit's weight rows x 16
// columns in its first rows (the others are zero: a1 = a3 = 0), B = the three terms of 16 values of x in columns 0..2, so
// that a lane's B registers are all in use and stay in registers for a whole phase.  d[0], d[1] of lane 4 g + t: weight
// row g times terms 2t and 2t + 1; d[2], d[3] stay zero.
__device__ __forceinline__ void mma_terms(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}

// Term g (0, 1, 2) of v = hi + mid + lo, each the leading 8 significant bits of what is left (by truncation), so that
// the three bf16 terms add up to v exactly and the tensor cores multiply exact operands.
__device__ __forceinline__ uint32_t term_of(float v, int g) {
  const uint32_t hi = __float_as_uint(v) & 0xffff0000u;
  const float r1 = v - __uint_as_float(hi);
  const uint32_t mid = __float_as_uint(r1) & 0xffff0000u;
  const float r2 = r1 - __uint_as_float(mid);
  const uint32_t pick = g == 0 ? hi : (g == 1 ? mid : __float_as_uint(r2));
  return pick >> 16;
}

// The activation vector as B fragments in shared memory, behind the scratch area: per pair of 16-column blocks 12
// vectors of 16 bytes, vector 4 g + t = term g of columns 2t, 2t+1 | 2t+8, 2t+9 of the first block and the same of
// the second (what lane 4 g + t feeds to the two instructions of the pair; lanes 12..31 feed zeros).
__device__ __forceinline__ uint32_t *xfrag_base(const KParams &p) {
  return reinterpret_cast<uint32_t *>(smem + (size_t)p.n_stages * p.stage_bytes + kScratchBytes);
}

// Stores the thread's column vectors (8 consecutive columns each, as the prologues leave them in xr) as fragments.
__device__ __forceinline__ void store_frags(const KParams &p, int C, const float (&xr)[kMaxVec][8]) {
  uint32_t *xf = xfrag_base(p);
  const int nv = C / 8;
#pragma unroll
  for (int i = 0; i < kMaxVec; ++i) {
    const int v = (int)threadIdx.x + i * kConsumerThreads;
    if (v < nv) {
      // columns 8 v .. 8 v + 7: pair v / 4, word (v & 3) of each vector = block (v / 2) & 1, half v & 1
      uint32_t *dst = xf + (size_t)(v >> 2) * 48 + (v & 3);
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const float x0 = xr[i][2 * t], x1 = xr[i][2 * t + 1];
#pragma unroll
        for (int g = 0; g < 3; ++g) dst[g * 16 + t * 4] = term_of(x0, g) | (term_of(x1, g) << 16);
      }
    }
  }
}

// Streams this block's units of one matrix in fragment order through the ring: per unit and pair of column blocks one
// 16-byte load of weights (lanes of the unit's rows; the others feed zero rows) and one of x (the fragments of two
// instructions) and two instructions, the pairs of a stage dealt to the warps in turn; a row's sum is the sum of its
// three terms' columns of the accumulator.
__device__ __forceinline__ void consume_image(Blk &b, int R, int C, int kind, const EpiArgs &ea) {
  const KParams &p = *b.p;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int r0, r1;
  cta_rows(R, kUnitRows, r0, r1);
  const int n_pairs = C / 32;
  const uint4 *xf = reinterpret_cast<const uint4 *>(xfrag_base(p)) + lane;  // lanes < 12 only
  float h_pre = 0.f;
  if (kind == kEpiAddH && r0 + (int)threadIdx.x < min(r0 + kTile, r1)) h_pre = __ldcg(p.h + r0 + threadIdx.x);
  float rs = 1.f;
  int buf = 0;
  for (int t0 = r0; t0 < r1; t0 += kTile) {
    const int t1 = min(t0 + kTile, r1);
    float *part = scratch_base(p) + (size_t)buf * kTile * kConsumerWarps;
    for (int r = t0; r < t1; r += kUnitRows) {
      float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
      const int per_stage = (int)(img_chunk(p, C) / kPairBytes);
      for (int pr0 = 0; pr0 < n_pairs; pr0 += per_stage) {  // one stage
        wait_mbar(b, &s_full[b.c_stage], b.c_phase, 300);
        const uint8_t *stage = smem + (size_t)b.c_stage * p.stage_bytes;
        const int n = min(per_stage, n_pairs - pr0);
#pragma unroll 1  // unrolled, the loop costs more registers than the kernel has
        for (int j = warp; j < n; j += kConsumerWarps) {
          uint4 w = make_uint4(0u, 0u, 0u, 0u);
          if (lane < 4 * kUnitRows) w = lds128(stage + ((size_t)j * (4 * kUnitRows) + lane) * 16);
          uint4 x = make_uint4(0u, 0u, 0u, 0u);
          if (lane < 12) x = xf[(size_t)(pr0 + j) * 12];
          mma_terms(c0, w.x, w.y, x.x, x.y);
          mma_terms(c1, w.z, w.w, x.z, x.w);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&s_empty[b.c_stage]);
        if (++b.c_stage == (uint32_t)p.n_stages) { b.c_stage = 0; b.c_phase ^= 1u; }
      }
      // row g: terms 0 and 1 in lane 4 g, term 2 in lane 4 g + 1 (whose d[1] is a sum of zeros)
      const float s01 = (c0[0] + c1[0]) + (c0[1] + c1[1]);
      const float s2 = __shfl_down_sync(0xffffffffu, s01, 1);
      if ((lane & 3) == 0 && lane < 4 * kUnitRows) part[(size_t)(r - t0 + (lane >> 2)) * kConsumerWarps + warp] = s01 + s2;
    }
    named_sync(1, kConsumerThreads);
    if (kind != kEpiAddH && t0 == r0) {
      const float4 *q = reinterpret_cast<const float4 *>(s_red);
      float ss = 0.f;
#pragma unroll
      for (int i = 0; i < kConsumerWarps / 4; ++i) {
        const float4 a = q[i];
        ss += a.x;
        ss += a.y;
        ss += a.z;
        ss += a.w;
      }
      rs = rsqrtf(ss / (float)C + p.eps);
    }
    epilogue(b, kind, ea, part, t0, t1, t0 == r0, h_pre, rs);
    buf ^= 1;
  }
}

// ---------------------------------------------------------------- consumer: activation prologues
// Gain vector of an RMSNorm to come.  Its turn comes once per timestep, by when the weight stream has pushed it out
// of L2; a load issued after the grid barrier would add a trip to device memory to every phase boundary, so the
// thread's first two 16-byte vectors are asked for a phase ahead and wait in registers (columns beyond
// 2 * 512 * 8 are fetched late).
struct Gain {
  uint4 g[2];
};

// Pointer of the j-th RMSNorm gain of a timestep: attention norm of layer j / 2 (j even), FFN norm of layer j / 2
// (j odd), final norm (j = 2 L).
__device__ __forceinline__ const __nv_bfloat16 *gain_ptr(const Blk &b, int j) {
  const KParams &p = *b.p;
  if (2 * p.L + 1 <= kGainSlots) return s_gain_ptrs[j];
  return j == 2 * p.L ? p.final_norm : ((j & 1) ? p.layers[j >> 1].ffn_norm : p.layers[j >> 1].attn_norm);
}

__device__ __forceinline__ void fetch_gain(const __nv_bfloat16 *gain, int C, Gain &gq) {
  const int nv = C / 8;
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int v = (int)threadIdx.x + i * kConsumerThreads;
    if (v < nv) gq.g[i] = __ldg(reinterpret_cast<const uint4 *>(gain + (size_t)v * 8));
  }
}

__device__ __forceinline__ void prefetch_l2(const void *ptr) { asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr)); }

__device__ __forceinline__ void load8(const float *src, float (&x)[8]) {
  const float4 a = __ldcg(reinterpret_cast<const float4 *>(src));
  const float4 c = __ldcg(reinterpret_cast<const float4 *>(src) + 1);
  x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
  x[4] = c.x; x[5] = c.y; x[6] = c.z; x[7] = c.w;
}

// x = h * gain, each thread keeping its own column vectors; the factor 1 / rms(h) that completes RMSNorm(h) * gain
// is common to all columns and is applied to the row sums (epilogue): the warps' sums of squares go to red[], which
// the phase's first tile-end barrier makes visible, so no block-wide reduction stands between the grid barrier and
// the first multiply.  red[] is next written a grid barrier later at the earliest.
__device__ __forceinline__ void prologue_norm(Blk &b, const float *h, const Gain &gq, int j, int C, float (&xr)[kMaxVec][8]) {
  const int nv = C / 8;
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < kMaxVec; ++i) {
    const int v = (int)threadIdx.x + i * kConsumerThreads;
    if (v < nv) {
      load8(h + (size_t)v * 8, xr[i]);
#pragma unroll
      for (int e = 0; e < 8; ++e) ss = fmaf(xr[i][e], xr[i][e], ss);
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) xr[i][e] = 0.f;  // every vector is written: none outlives a phase
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = ss;
#pragma unroll
  for (int i = 0; i < kMaxVec; ++i) {
    const int v = (int)threadIdx.x + i * kConsumerThreads;
    if (v < nv) {
      const uint4 g = i < 2 ? gq.g[i] : __ldg(reinterpret_cast<const uint4 *>(gain_ptr(b, j) + (size_t)v * 8));
      const uint32_t gw[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        xr[i][2 * e] = xr[i][2 * e] * __uint_as_float(gw[e] << 16);
        xr[i][2 * e + 1] = xr[i][2 * e + 1] * __uint_as_float(gw[e] & 0xffff0000u);
      }
    }
  }
}

__device__ __forceinline__ void prologue_plain(const float *src, int C, float (&xr)[kMaxVec][8]) {
  const int nv = C / 8;
#pragma unroll
  for (int i = 0; i < kMaxVec; ++i) {
    const int v = (int)threadIdx.x + i * kConsumerThreads;
    if (v < nv) {
      load8(src + (size_t)v * 8, xr[i]);
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) xr[i][e] = 0.f;  // every vector is written: none outlives a phase
    }
  }
}

__device__ __forceinline__ int attn_splits(const KParams &p, int T) {
  int ms = (int)gridDim.x / p.H;
  ms = ms < 1 ? 1 : (ms > kMaxSplit ? kMaxSplit : ms);
  int ns = (T + 63) / 64;
  return ns < 1 ? 1 : (ns > ms ? ms : ns);
}

// x = attention output: merges the per-split partial sums of each head
__device__ __forceinline__ void prologue_attn(const KParams &p, int T, float (&xr)[kMaxVec][8]) {
  const int nv = p.d / 8, ns = attn_splits(p, T);
#pragma unroll
  for (int i = 0; i < kMaxVec; ++i) {
    const int v = (int)threadIdx.x + i * kConsumerThreads;
    if (v < nv) {
      const int col = v * 8, head = col / p.hd, c = col - head * p.hd;
      // one pass with a running maximum, so that a split's (max, sum) and its partial output are asked for
      // together: one trip to L2 after the grid barrier instead of two
      float M = -CUDART_INF_F, den = 0.f, acc[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] = 0.f;
#pragma unroll 2
      for (int s = 0; s < ns; ++s) {
        const float2 ml = __ldcg(&p.oml[head * ns + s]);
        float o[8];
        load8(p.opart + (size_t)(head * ns + s) * p.hd + c, o);
        const float Mn = fmaxf(M, ml.x);
        const float keep = M == -CUDART_INF_F ? 0.f : __expf(M - Mn), w = ml.x == -CUDART_INF_F ? 0.f : __expf(ml.x - Mn);
        den = fmaf(den, keep, ml.y * w);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = fmaf(acc[e], keep, o[e] * w);
        M = Mn;
      }
      const float inv = 1.f / den;
#pragma unroll
      for (int e = 0; e < 8; ++e) xr[i][e] = acc[e] * inv;
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) xr[i][e] = 0.f;
    }
  }
}

// ---------------------------------------------------------------- attention over the shared cache
__device__ __forceinline__ float load_kv(const KParams &p, const void *cache, size_t idx) {
  if (p.kv_bf16) {
    const unsigned short raw = __ldcg(reinterpret_cast<const unsigned short *>(cache) + idx);
    return __uint_as_float((uint32_t)raw << 16);
  }
  return __ldcg(reinterpret_cast<const float *>(cache) + idx);
}

// Asks the cache rows that this block's attention items will read into L2 (all but the new position's, which this
// phase writes).  They were last touched a timestep ago and the weight stream has pushed them out since: issued
// at the start of the QKV phase, the requests travel with the weight stream, and the attention phase, which
// stands between two grid barriers with the ring full, finds its rows in L2.
__device__ __forceinline__ void prefetch_kv(const KParams &p, int layer, int pos) {
  const int T = pos + 1, ns = attn_splits(p, T), items = p.H * ns;
  const int esz = p.kv_bf16 ? 2 : 4;
  const int lpr = (p.hd * esz + 127) >> 7;  // 128-byte lines per cache row of a head
  for (int item = blockIdx.x; item < items; item += gridDim.x) {
    const int head = item / ns, sp = item - head * ns;
    const int t0 = (int)((long long)T * sp / ns), t1 = min((int)((long long)T * (sp + 1) / ns), pos);
    const int n = (t1 - t0) * lpr;
    for (int i = threadIdx.x; i < n; i += kConsumerThreads) {
      const int t = t0 + i / lpr, c = i - (i / lpr) * lpr;
      const size_t off = (((size_t)layer * p.max_pos + t) * p.d + (size_t)head * p.hd) * esz + (size_t)c * 128;
      prefetch_l2(reinterpret_cast<const uint8_t *>(p.kcache) + off);
      prefetch_l2(reinterpret_cast<const uint8_t *>(p.vcache) + off);
    }
  }
}

// Fast path of the attention phase for a bf16 cache and head_dim 128 (a cache row of a head is 256 bytes):
// half a warp takes one position with 16-byte loads, and each warp keeps eight positions in flight, so a
// long context costs a few dependent memory round trips instead of one per position.  Each half-warp runs
// its own online softmax; halves, then warps, are merged at the end exactly like the general path.
__device__ void attention_phase_bf16_hd128(Blk &b, int layer, int pos) {
  const KParams &p = *b.p;
  const int T = pos + 1, ns = attn_splits(p, T), items = p.H * ns;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, half = lane >> 4, l16 = lane & 15;
  const float scale = 1.f / sqrtf(128.f);
  float *s_acc = scratch_base(p);                           // [warps][128]
  float *s_m = scratch_base(p) + kConsumerWarps * 256;      // [warps]
  float *s_l = s_m + kConsumerWarps;               // [warps]
  const __nv_bfloat16 *kc = reinterpret_cast<const __nv_bfloat16 *>(p.kcache);
  const __nv_bfloat16 *vc = reinterpret_cast<const __nv_bfloat16 *>(p.vcache);
  for (int item = blockIdx.x; item < items; item += gridDim.x) {
    const int head = item / ns, sp = item - head * ns;
    const int t0 = (int)((long long)T * sp / ns), t1 = (int)((long long)T * (sp + 1) / ns);
    float q[8], acc[8];
    load8(p.q + head * 128 + l16 * 8, q);
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;
    float m = -CUDART_INF_F, l = 0.f;
    const size_t col = (size_t)head * 128 + l16 * 8;
    // A round = four positions per half-warp; they enter the running softmax together (one rescale per round instead
    // of four dependent ones).
    constexpr int kStep = kConsumerWarps * 8;
    uint4 kq[4], vq[4];
    auto fetch = [&](int tb, const __nv_bfloat16 *cache, uint4 (&dst)[4]) {
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int t = max(min(tb + 2 * u + half, t1 - 1), 0);  // clamped: the extra loads are discarded below
        dst[u] = __ldcg(reinterpret_cast<const uint4 *>(cache + ((size_t)layer * p.max_pos + t) * p.d + col));
      }
    };
    for (int tb = t0 + warp * 8; tb < t1; tb += kStep) {
      fetch(tb, kc, kq);
      fetch(tb, vc, vq);
      float sc[4];
      float mn = m;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const uint32_t kw[4] = {kq[u].x, kq[u].y, kq[u].z, kq[u].w};
        float dot = 0.f;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          dot = fmaf(q[2 * e], __uint_as_float(kw[e] << 16), dot);
          dot = fmaf(q[2 * e + 1], __uint_as_float(kw[e] & 0xffff0000u), dot);
        }
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
        sc[u] = tb + 2 * u + half < t1 ? dot * scale : -CUDART_INF_F;  // uniform within the half-warp
        mn = fmaxf(mn, sc[u]);
      }
      if (mn > -CUDART_INF_F) {  // else nothing of this round (nor of an earlier one) belongs to the half-warp
        const float c = __expf(m - mn);
        l *= c;
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] *= c;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const float pw = __expf(sc[u] - mn);  // 0 for a position past the range
          l += pw;
          const uint32_t vw[4] = {vq[u].x, vq[u].y, vq[u].z, vq[u].w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            acc[2 * e] = fmaf(pw, __uint_as_float(vw[e] << 16), acc[2 * e]);
            acc[2 * e + 1] = fmaf(pw, __uint_as_float(vw[e] & 0xffff0000u), acc[2 * e + 1]);
          }
        }
        m = mn;
      }
    }
    // merge the two half-warps
    {
      const float mo = __shfl_xor_sync(0xffffffffu, m, 16), lo = __shfl_xor_sync(0xffffffffu, l, 16);
      const float M = fmaxf(m, mo);
      const float w_self = m == -CUDART_INF_F ? 0.f : __expf(m - M), w_oth = mo == -CUDART_INF_F ? 0.f : __expf(mo - M);
      l = l * w_self + lo * w_oth;
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] = acc[e] * w_self + __shfl_xor_sync(0xffffffffu, acc[e], 16) * w_oth;
      m = M;
    }
    if (half == 0) {
#pragma unroll
      for (int e = 0; e < 8; ++e) s_acc[warp * 256 + l16 * 8 + e] = acc[e];
    }
    if (lane == 0) {
      s_m[warp] = m;
      s_l[warp] = l;
    }
    named_sync(1, kConsumerThreads);
    if (threadIdx.x < 128) {
      float M = -CUDART_INF_F;
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) M = fmaxf(M, s_m[w]);
      float L = 0.f, A = 0.f;
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) {
        const float wgt = s_m[w] == -CUDART_INF_F ? 0.f : __expf(s_m[w] - M);
        L = fmaf(s_l[w], wgt, L);
        A = fmaf(s_acc[w * 256 + threadIdx.x], wgt, A);
      }
      p.opart[(size_t)item * 128 + threadIdx.x] = A;
      if (threadIdx.x == 0) p.oml[item] = make_float2(M, L);
    }
    named_sync(1, kConsumerThreads);
  }
}

__device__ void attention_phase(Blk &b, int layer, int pos) {
  const KParams &p = *b.p;
  if (p.kv_bf16 && p.hd == 128) {
    attention_phase_bf16_hd128(b, layer, pos);
    return;
  }
  const int T = pos + 1, ns = attn_splits(p, T), items = p.H * ns;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int epl = p.hd / 32;  // elements per lane, <= 8
  const float scale = 1.f / sqrtf((float)p.hd);
  float *s_acc = scratch_base(p);                           // [warps][hd]
  float *s_m = scratch_base(p) + kConsumerWarps * 256;      // [warps]
  float *s_l = s_m + kConsumerWarps;               // [warps]
  for (int item = blockIdx.x; item < items; item += gridDim.x) {
    const int head = item / ns, sp = item - head * ns;
    const int t0 = (int)((long long)T * sp / ns), t1 = (int)((long long)T * (sp + 1) / ns);
    float q[8], acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      q[e] = e < epl ? __ldcg(p.q + head * p.hd + lane * epl + e) : 0.f;
      acc[e] = 0.f;
    }
    float m = -CUDART_INF_F, l = 0.f;
    for (int t = t0 + warp; t < t1; t += kConsumerWarps) {
      const size_t base = ((size_t)layer * p.max_pos + t) * p.d + head * p.hd + lane * epl;
      float dot = 0.f, vv[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        if (e < epl) {
          dot = fmaf(q[e], load_kv(p, p.kcache, base + e), dot);
          vv[e] = load_kv(p, p.vcache, base + e);
        } else {
          vv[e] = 0.f;
        }
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
#pragma unroll
    for (int e = 0; e < 8; ++e)
      if (e < epl) s_acc[warp * 256 + lane * epl + e] = acc[e];
    if (lane == 0) {
      s_m[warp] = m;
      s_l[warp] = l;
    }
    named_sync(1, kConsumerThreads);
    if ((int)threadIdx.x < p.hd) {
      float M = -CUDART_INF_F;
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) M = fmaxf(M, s_m[w]);
      float L = 0.f, A = 0.f;
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) {
        const float wgt = s_m[w] == -CUDART_INF_F ? 0.f : __expf(s_m[w] - M);
        L = fmaf(s_l[w], wgt, L);
        A = fmaf(s_acc[w * 256 + threadIdx.x], wgt, A);
      }
      p.opart[(size_t)item * p.hd + threadIdx.x] = A;
      if (threadIdx.x == 0) p.oml[item] = make_float2(M, L);
    }
    named_sync(1, kConsumerThreads);
  }
}

// Next LM input (block 0): the token embedding in prefill and sampling, the superposed embedding of Eq. 3 in
// decode.
template <bool kSampler>
__device__ void embed_input(const KParams &p, int it) {
  const State *st = p.st;
  if (p.mode == kModePrefill || (kSampler && p.mode == kModeSample)) {
    const int tok = p.prefix[it];
    for (int c = threadIdx.x; c < p.d; c += kConsumerThreads) p.h[c] = __bfloat162float(p.tok_emb[(size_t)tok * p.d + c]);
  } else {
    for (int c = threadIdx.x; c < p.d; c += kConsumerThreads) {
      float acc = 0.f;
      for (int i = 0; i < p.k; ++i)
        acc = fmaf(st->gamma[i], __bfloat162float(p.tok_emb[(size_t)st->win[i][kWin - 1] * p.d + c]), acc);
      p.h[c] = acc;
    }
  }
}

// After the last sampled token's pass: every draft's history window is the end of the lengthened prefix
// (p.prefix[it] is its last token, at position pos0 + it), as the host sets it up before a prefill.
__device__ void sample_windows(const KParams &p, int it) {
  State *st = p.st;
  const int len = min(p.pos0 + it + 1, kWin);
  if ((int)threadIdx.x < p.k)
    for (int j = 0; j < len; ++j) st->win[threadIdx.x][kWin - len + j] = p.prefix[it - len + 1 + j];
  if (threadIdx.x == 0) {
    st->win_len = len;
    st->n_gen = 0;
  }
}

// ---------------------------------------------------------------- consumer main loop
// kImg: QKV, attention output, gate / up and LM head also come in fragment order: a prologue leaves x
// in shared memory as fragments (store_frags; the barrier after it orders the stores before the first instruction
// that reads them) and consume_image multiplies.
template <bool kSampler, bool kImg>
__device__ void consumer_main(Blk &b) {
  const KParams &p = *b.p;
  float xr[kMaxVec][8];
  // Everything a phase needs besides the activations is asked for at least a phase ahead (the gains of the RMSNorms,
  // the position's row of the rotary table, the cache rows of the attention items): after a grid barrier only the
  // activation vector itself is fetched, one trip to L2.
  Gain gq;
  fetch_gain(gain_ptr(b, 0), p.d, gq);
  for (int it = 0; it < p.n_iters; ++it) {
    const int pos = p.pos0 + it;
    const bool last = it == p.n_iters - 1;
    const bool head = (kSampler ? p.mode != kModePrefill : p.mode == kModeDecode) || last;
    if ((int)threadIdx.x < p.hd / 2) s_rope[threadIdx.x] = p.rope[(size_t)pos * (p.hd / 2) + threadIdx.x];
    if (blockIdx.x == 0) {
      if (kSampler && p.mode == kModeSample) {
        // the next token is drawn from the logits of the pass before (Section 4.5: a nucleus-sampled prefix)
        const int tok = ns_sample(p.logits, p.V, p.ns_inv_temp, p.ns_p, p.ns_u[it], reinterpret_cast<uint8_t *>(scratch_base(p)));
        if (threadIdx.x == 0) p.prefix[it] = tok;
        named_sync(1, kConsumerThreads);
      }
      embed_input<kSampler>(p, it);
    }
    if (grid_barrier(b)) return;
    if (p.eos_id >= 0 && p.mode == kModeDecode && it > 0) {
      // Stop token (Algorithm 1: "until max generation length or stop token"): block 0 raised the flag before the
      // barrier if the step before made the most probable draft end with it; every block then leaves, its producer
      // draining the copies in flight as when giving up, but without an error.
      if (threadIdx.x == 0) {
        if (ld_relaxed(&p.st->stop)) s_dead = 1;
        s_quit = s_dead;
      }
      named_sync(1, kConsumerThreads);
      if (s_quit) return;
    }
    for (int l = 0; l < p.L; ++l) {
      EpiArgs ea{l, pos, 0};
      prologue_norm(b, p.h, gq, 2 * l, p.d, xr);
      prefetch_kv(p, l, pos);
      if constexpr (kImg) {
        store_frags(p, p.d, xr);
        named_sync(1, kConsumerThreads);
        consume_image(b, 3 * p.d, p.d, kEpiQKV, ea);
      } else {
        consume_matrix(b, 3 * p.d, p.d, 2, xr, kEpiQKV, ea);
      }
      if (grid_barrier(b)) return;
      attention_phase(b, l, pos);
      if (grid_barrier(b)) return;
      prologue_attn(p, pos + 1, xr);
      fetch_gain(gain_ptr(b, 2 * l + 1), p.d, gq);
      if constexpr (kImg) {
        store_frags(p, p.d, xr);
        named_sync(1, kConsumerThreads);
        consume_image(b, p.d, p.d, kEpiAddH, ea);
      } else {
        consume_matrix(b, p.d, p.d, 1, xr, kEpiAddH, ea);
      }
      if (grid_barrier(b)) return;
      prologue_norm(b, p.h, gq, 2 * l + 1, p.d, xr);
      if constexpr (kImg) {
        store_frags(p, p.d, xr);
        named_sync(1, kConsumerThreads);
        consume_image(b, 2 * p.f, p.d, kEpiSwiGLU, ea);
      } else {
        consume_matrix(b, 2 * p.f, p.d, 2, xr, kEpiSwiGLU, ea);
      }
      if (grid_barrier(b)) return;
      prologue_plain(p.u, p.f, xr);
      fetch_gain(gain_ptr(b, l + 1 < p.L || head ? 2 * l + 2 : 0), p.d, gq);
      ea.which = 1;
      consume_matrix(b, p.d, p.f, 1, xr, kEpiAddH, ea);
      if (grid_barrier(b)) return;
    }
    if (head) {
      EpiArgs ea{0, pos, 0};
      prologue_norm(b, p.h, gq, 2 * p.L, p.d, xr);
      if (!last) fetch_gain(gain_ptr(b, 0), p.d, gq);
      if constexpr (kImg) {
        store_frags(p, p.d, xr);
        named_sync(1, kConsumerThreads);
        consume_image(b, p.V, p.d, kEpiLogits, ea);
      } else {
        consume_matrix(b, p.V, p.d, 1, xr, kEpiLogits, ea);
      }
      named_sync(1, kConsumerThreads);
      int r0, r1;
      cta_rows(p.V, kImg ? kUnitRows : 1, r0, r1);
      if (threadIdx.x < 32) block_topk(p, r0, r1, blockIdx.x);
      if (grid_barrier(b)) return;
      if (blockIdx.x == 0 && (!kSampler || p.mode != kModeSample || last)) {
        if (threadIdx.x < 32) tail_keep_topk(p, gridDim.x);
        const bool first = p.mode != kModeDecode;
        if (kSampler && p.mode == kModeSample) sample_windows(p, it);
        tail_score_select(b, first, first ? 0 : p.step0 + it);
        if (!first && p.eos_id >= 0 && threadIdx.x == 0 && p.hist_tok[(size_t)(p.step0 + it) * p.k] == p.eos_id) p.st->stop = 1u;
      }
    }
  }
}

template <bool kSampler, bool kImg>
__device__ __forceinline__ void kernel_body(const KParams &p) {
  Blk b;
  b.p = &p;
  b.part = reinterpret_cast<float *>(smem + (size_t)p.n_stages * p.stage_bytes);
  if (p.mode != kModeScoreOnly && p.mode != kModeNucleusOnly && 2 * p.L + 1 <= kGainSlots)
    for (int j = threadIdx.x; j <= 2 * p.L; j += kThreads)
      s_gain_ptrs[j] = j == 2 * p.L ? p.final_norm : ((j & 1) ? p.layers[j >> 1].ffn_norm : p.layers[j >> 1].attn_norm);
  b.dead = &s_dead;
  b.quit = &s_quit;
  b.bar_target = 0;
  b.c_stage = 0;
  b.c_phase = 0;
  if (threadIdx.x == 0) {
    s_dead = 0;
    s_quit = 0;
    for (int s = 0; s < p.n_stages; ++s) {
      mbar_init(&s_full[s], 1);
      mbar_init(&s_empty[s], kConsumerWarps);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (p.mode == kModeScoreOnly) {
    if (blockIdx.x == 0 && threadIdx.x < kConsumerThreads) tail_score_select(b, false, p.step0);
    return;
  }
  if (kSampler && p.mode == kModeNucleusOnly) {
    if (blockIdx.x == 0 && threadIdx.x < kConsumerThreads) {
      const int tok = ns_sample(p.logits, p.V, p.ns_inv_temp, p.ns_p, p.ns_u[0], reinterpret_cast<uint8_t *>(scratch_base(p)));
      if (threadIdx.x == 0) p.st->cand_tok[0] = tok;
    }
    return;
  }
  if (threadIdx.x >= kConsumerThreads) {
    if (threadIdx.x == kConsumerThreads) producer_main<kSampler, kImg>(b);
  } else {
    consumer_main<kSampler, kImg>(b);
  }
  __syncthreads();
}

// The decoding kernel, and its twin that also carries the nucleus sampler (kModeSample, kModeNucleusOnly): two
// entry points so that the sampler's code does not weigh on the register allocation of the decode loop.
__global__ void __launch_bounds__(kThreads, 1) spd_decode_kernel(const __grid_constant__ KParams p) { kernel_body<false, false>(p); }
__global__ void __launch_bounds__(kThreads, 1) spd_sample_kernel(const __grid_constant__ KParams p) { kernel_body<true, false>(p); }
// The decoding kernel for weights that also come in fragment order: QKV, attention output, gate / up and LM head
// products on the tensor cores.  The down projection stays with the float32 multiply loop: its rows are long, so whole
// units of them divide unevenly among the blocks and their fragments of x would take a third of the ring's memory
// (measured: 2.96 ms per 7B timestep with it on the tensor cores too, against 2.64 ms).
__global__ void __launch_bounds__(kThreads, 1) spd_decode_img_kernel(const __grid_constant__ KParams p) { kernel_body<false, true>(p); }

}  // namespace spd

// Host-side launcher used by the API file.
static const void *kernel_for(int mode, bool img) {
  if (mode == spd::kModeSample || mode == spd::kModeNucleusOnly) return reinterpret_cast<const void *>(&spd::spd_sample_kernel);
  return img ? reinterpret_cast<const void *>(&spd::spd_decode_img_kernel) : reinterpret_cast<const void *>(&spd::spd_decode_kernel);
}

extern "C" cudaError_t spd_internal_launch(const spd::KParams *p, int grid, size_t dyn_smem, cudaStream_t stream) {
  void *args[] = {const_cast<spd::KParams *>(p)};
  return cudaLaunchCooperativeKernel(kernel_for(p->mode, p->lm_head_img != nullptr), dim3(grid), dim3(spd::kThreads), args, dyn_smem, stream);
}

extern "C" cudaError_t spd_internal_prepare(size_t dyn_smem, int *blocks_per_sm) {
  int least = 1 << 30;
  const void *kernels[3] = {kernel_for(spd::kModeDecode, false), kernel_for(spd::kModeDecode, true), kernel_for(spd::kModeSample, false)};
  for (const void *kernel : kernels) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn_smem);
    if (e != cudaSuccess) return e;
    int n = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, spd::kThreads, dyn_smem);
    if (e != cudaSuccess) return e;
    if (n < least) least = n;
  }
  *blocks_per_sm = least;
  return cudaSuccess;
}

// ---------------------------------------------------------------- scoring stage without any allocation
// spd_score_static (see include/spd.h): the scoring stage of one timestep for callers that cannot
// allocate device memory.  The draft state the kernel normally keeps in the caller's workspace lives
// here in a fixed array that is part of the loaded library image on every GPU.
#include <cstring>
#include <mutex>

#include "spd.h"

namespace {

constexpr size_t kStaticStateBytes = (sizeof(spd::State) + 255) / 256 * 256;
constexpr size_t kStaticScratchBytes = kStaticStateBytes + 2 * SPD_MAX_K * sizeof(int32_t);
static_assert(kStaticScratchBytes <= 16384, "static scratch is documented as 16 KB");

static __device__ __align__(256) unsigned char g_static_scratch[16384];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void *g_static_ptr[kMaxDevices] = {};  // device address of g_static_scratch, per device, filled on first use

}  // namespace

extern "C" int spd_score_static(const spd_config *cfg, const spd_ngram_table *tables, int32_t n_tables,
                                const int32_t *hist, int32_t hist_len, const float *logp, const int32_t *cand_tok,
                                const float *cand_lp, int32_t *out_sel, float *out_logp, float *out_gamma,
                                float *out_score) {
  if (!cfg || !hist || !logp || !cand_tok || !cand_lp || (n_tables > 0 && !tables)) return SPD_EINVAL;
  // sizes beyond what the fixed scratch was laid out for are refused, never truncated
  if (cfg->k < 1 || cfg->k > SPD_MAX_K || n_tables < 0 || n_tables > spd::kMaxTables || hist_len < 0 || hist_len > spd::kWin)
    return SPD_ERANGE;
  if (cfg->n_min < 2 || cfg->n_max > SPD_MAX_N || cfg->vocab < 1 || cfg->vocab > 65535) return SPD_EINVAL;
  if (!(cfg->delta > 0.f) || cfg->delta > 1.f || !(cfg->alpha >= 0.f) || cfg->alpha > 1.f) return SPD_EINVAL;
  const int k = cfg->k;
  for (int t = 0; t < n_tables; ++t) {
    const spd_ngram_table &tb = tables[t];
    if (tb.n < 2 || tb.n > SPD_MAX_N || !tb.ngram || !tb.ctx || ((uintptr_t)tb.ngram % 16) || ((uintptr_t)tb.ctx % 16)) return SPD_EINVAL;
    if (!tb.ngram_slots || (tb.ngram_slots & (tb.ngram_slots - 1)) || !tb.ctx_slots || (tb.ctx_slots & (tb.ctx_slots - 1)))
      return SPD_EINVAL;
    if (t > 0 && tables[t - 1].n >= tb.n) return SPD_EINVAL;
  }
  for (int i = 0; i < k; ++i) {
    if (cand_tok[i] < 0 || cand_tok[i] >= cfg->vocab) return SPD_ERANGE;
    for (int j = 0; j < hist_len; ++j)
      if (hist[i * hist_len + j] < 0 || hist[i * hist_len + j] >= cfg->vocab) return SPD_ERANGE;
  }

  // Set-up, once per device, with that device current: in host code the array's name is only a
  // stand-in for the symbol, so its device address is asked for and that address is what the kernel gets.
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SPD_ECUDA;
  unsigned char *scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
      void *ptr = nullptr;
      if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
        cudaGetLastError();
        return SPD_ECUDA;
      }
      g_static_ptr[dev] = ptr;
    }
    scratch = static_cast<unsigned char *>(g_static_ptr[dev]);
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cfg->stream);

  // The array keeps whatever the previous call left: the whole state is overwritten with this call's
  // inputs (everything else zero, including the error word), and so are the two history rows.
  spd::State st;
  std::memset(&st, 0, sizeof st);
  st.win_len = hist_len;
  for (int i = 0; i < k; ++i) {
    for (int j = 0; j < hist_len; ++j) st.win[i][spd::kWin - hist_len + j] = hist[i * hist_len + j];
    st.logP[i] = logp[i];
    st.cand_tok[i] = cand_tok[i];
    st.cand_lp[i] = cand_lp[i];
  }
  if (cudaMemcpyAsync(scratch, &st, sizeof st, cudaMemcpyHostToDevice, stream) != cudaSuccess) return SPD_ECUDA;
  if (cudaMemsetAsync(scratch + kStaticStateBytes, 0, 2 * SPD_MAX_K * sizeof(int32_t), stream) != cudaSuccess) return SPD_ECUDA;

  spd::KParams kp;
  std::memset(&kp, 0, sizeof kp);
  kp.k = k; kp.n_min = cfg->n_min; kp.n_max = cfg->n_max; kp.n_tables = n_tables;
  for (int i = 0; i < 8; ++i) kp.lambda[i] = cfg->lambda[i];
  kp.alpha = cfg->alpha;
  kp.log_delta = logf(cfg->delta);
  for (int t = 0; t < n_tables; ++t) {
    kp.tab[t].n = tables[t].n;
    kp.tab[t].ngram = static_cast<const SpdSlot *>(tables[t].ngram);
    kp.tab[t].ctx = static_cast<const SpdSlot *>(tables[t].ctx);
    kp.tab[t].ngram_mask = tables[t].ngram_slots - 1;
    kp.tab[t].ctx_mask = tables[t].ctx_slots - 1;
  }
  kp.st = reinterpret_cast<spd::State *>(scratch);
  kp.hist_tok = reinterpret_cast<int32_t *>(scratch + kStaticStateBytes);
  kp.hist_par = kp.hist_tok + SPD_MAX_K;
  kp.mode = spd::kModeScoreOnly;
  kp.stage_bytes = 0;
  kp.n_stages = 1;
  spd::spd_decode_kernel<<<1, spd::kThreads, 20480, stream>>>(kp);
  if (cudaGetLastError() != cudaSuccess) return SPD_ECUDA;

  spd::State back;
  if (cudaMemcpyAsync(&back, scratch, sizeof back, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return SPD_ECUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return SPD_ECUDA;
  if (back.err) return back.err;
  for (int i = 0; i < k; ++i) {
    if (out_sel) out_sel[i] = back.sel[i];
    if (out_logp) out_logp[i] = back.logP[i];
    if (out_gamma) out_gamma[i] = back.gamma[i];
  }
  if (out_score)
    for (int q = 0; q < k * k; ++q) out_score[q] = back.score[q];
  return SPD_OK;
}

// ---------------------------------------------------------------- fragment order
// spd_pack_image (see include/spd.h): every block of 8 rows x 32 columns of a row-major bf16 matrix becomes 32
// vectors of 16 bytes, vector (g, t) = row g's column pairs 2t | 2t+8 | 2t+16 | 2t+24 of the block: the weight
// fragments of two m16n8k16 instructions for lane 4 g + t.  Units of 8 rows follow one another, each with its column
// blocks in order, so a unit is one contiguous run of cols * 16 bytes.
namespace spd {
__global__ void spd_pack_image_kernel(const uint32_t *w, uint4 *out, int rows, int cols) {
  const size_t n = (size_t)rows * cols / 8;  // 16-byte vectors
  const int pairs = cols / 32;
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < n; idx += (size_t)gridDim.x * blockDim.x) {
    const int lane = (int)(idx % (4 * kUnitRows));
    const size_t blk = idx / (4 * kUnitRows);
    const int pr = (int)(blk % pairs);
    const size_t unit = blk / pairs;
    const int g = lane >> 2, t = lane & 3;
    const uint32_t *src = w + ((unit * kUnitRows + g) * (size_t)cols + (size_t)pr * 32) / 2 + t;
    out[idx] = make_uint4(src[0], src[4], src[8], src[12]);
  }
}
}  // namespace spd

extern "C" cudaError_t spd_internal_pack_image(const void *w, void *out, int rows, int cols, cudaStream_t stream) {
  spd::spd_pack_image_kernel<<<1184, 256, 0, stream>>>(static_cast<const uint32_t *>(w), static_cast<uint4 *>(out), rows, cols);
  return cudaGetLastError();
}
