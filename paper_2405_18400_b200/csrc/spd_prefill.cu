// Prefill kernel: the decoder over up to 16 prefix tokens at once (first timestep, Eq. 1, all but the last
// prefix token; the last one goes through the decode kernel, which also takes the first-timestep
// decision).  With several tokens per weight the products are real matrix-matrix contractions, so they run
// on tensor cores: mma.sync m16n8k16 with A = 16 weight rows x 16 columns straight from the bf16 rows,
// B = the tokens' activations split exactly into three bf16 terms (x = hi + mid + lo to float32
// precision), float32 accumulation.  One persistent cooperative launch per chunk of tokens: a producer
// warp streams weight tiles (16 rows x 1024 columns) through a shared-memory ring with bulk copies, eight
// consumer warps share every tile by k-steps, per-warp partial sums are reduced through shared memory once
// per 16 rows, and the same five phases per layer as in decoding are separated by grid barriers.
#include <cuda_runtime.h>
#include <math_constants.h>

#include "spd_params.h"
#include "spd_ptx.cuh"

namespace spd {

constexpr int kPfWarps = 8;
constexpr int kPfThreads = kPfWarps * 32;  // consumer threads
constexpr int kPfBlock = kPfThreads + 32;  // plus the producer warp
constexpr int kPfKB = 1024;                // columns per K block
constexpr int kPfKSteps = kPfKB / 16;
constexpr int kPfTileRows = 16;
constexpr int kPfMaxTiles = 12;            // row tiles whose accumulators a warp keeps at a time
constexpr int kPfPitch = kPfKB * 2 + 16;   // bytes between the rows of a tile in a stage (padding: no bank conflicts)
constexpr int kPfStageBytes = kPfTileRows * kPfPitch;
constexpr int kPfStages = 3;
constexpr int kPfXblkBytes = kPfKSteps * 2 * 3 * 32 * 8;  // [k-step][token tile][term][lane] x 8 bytes
constexpr int kPfRedBytes = kPfWarps * kPfTileRows * kPfTokens * 4;
constexpr unsigned long long kPfWaitNs = 1500ull * 1000ull * 1000ull;

struct PfBlk {
  const KParams *p;
  uint8_t *ring;
  uint2 *xblk;
  float *red;
  float *rs;  // [16] per-token 1/rms
  uint64_t *full, *empty;
  volatile int *dead, *quit;
  unsigned int bar_target;
  uint32_t c_stage, c_phase;
};

__device__ __forceinline__ void pf_give_up(PfBlk &b, int code, int info) {
  State *st = b.p->st;
  if (atomicCAS(&st->err, 0, code) == 0) st->err_info = info;
  atomicExch(&st->abort_flag, 1u);
  *b.dead = 1;
}

__device__ __forceinline__ void pf_wait(PfBlk &b, uint64_t *bar, uint32_t parity, int info) {
  if (mbar_try_wait(bar, parity)) return;
  if (*b.dead) return;
  unsigned long long t0 = globaltimer();
  uint32_t n = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++n & 31u) == 0) {
      if (*b.dead) return;
      if (ld_relaxed(&b.p->st->abort_flag)) { *b.dead = 1; return; }
      if (globaltimer() - t0 > kPfWaitNs) { pf_give_up(b, -7, info); return; }
    }
  }
}

__device__ __forceinline__ bool pf_grid_barrier(PfBlk &b) {
  named_sync(1, kPfThreads);
  if (threadIdx.x == 0) {
    b.bar_target += gridDim.x;
    if (!*b.dead) {
      unsigned int *bar = &b.p->st->bar;
      __threadfence();
      atomicAdd(bar, 1u);
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
__device__ __forceinline__ PfPhase pf_phase(const KParams &p, int ph) {
  const LayerW &lw = p.layers[ph >> 2];
  PfPhase d;
  switch (ph & 3) {
    case 0: d.W = lw.wqkv; d.R = 3 * p.d; d.C = p.d; d.gran = 2; break;
    case 1: d.W = lw.wo; d.R = p.d; d.C = p.d; d.gran = 1; break;
    case 2: d.W = lw.wgate_up; d.R = 2 * p.f; d.C = p.d; d.gran = 2; break;
    default: d.W = lw.wdown; d.R = p.d; d.C = p.f; d.gran = 1; break;
  }
  return d;
}

// ---------------------------------------------------------------- producer
// Chunk order of a phase: per group of up to 12 row tiles, K block by K block, tile by tile.
__device__ void pf_producer(PfBlk &b) {
  const KParams &p = *b.p;
  const int lane = threadIdx.x & 31;
  uint32_t stage = 0, phase = 0, issued = 0;
  bool ok = true;
  for (int ph = 0; ph < 4 * p.L && ok; ++ph) {
    const PfPhase pd = pf_phase(p, ph);
    int r0, r1;
    pf_rows(pd.R, pd.gran, r0, r1);
    const uint8_t *W = reinterpret_cast<const uint8_t *>(pd.W);
    const size_t rowbytes = (size_t)pd.C * 2;
    const int nkb = (pd.C + kPfKB - 1) / kPfKB;
    for (int g0 = r0; g0 < r1 && ok; g0 += kPfMaxTiles * kPfTileRows) {
      const int g1 = min(g0 + kPfMaxTiles * kPfTileRows, r1);
      for (int kb = 0; kb < nkb && ok; ++kb) {
        const uint32_t piece = (uint32_t)min(kPfKB, pd.C - kb * kPfKB) * 2u;
        for (int t0 = g0; t0 < g1 && ok; t0 += kPfTileRows) {
          const int nrows = min(kPfTileRows, g1 - t0);
          int dead = 0;
          if (lane == 0) {
            pf_wait(b, &b.empty[stage], phase ^ 1u, 200);
            dead = *b.dead;
            if (!dead) mbar_expect_tx(&b.full[stage], piece * (uint32_t)nrows);
          }
          dead = __shfl_sync(0xffffffffu, dead, 0);
          if (dead) { ok = false; break; }
          if (lane < nrows)
            bulk_load(b.ring + (size_t)stage * kPfStageBytes + (size_t)lane * kPfPitch,
                      W + (size_t)(t0 + lane) * rowbytes + (size_t)kb * kPfKB * 2, piece, &b.full[stage]);
          if (issued < (uint32_t)kPfStages) ++issued;
          if (++stage == (uint32_t)kPfStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  }
  if (!ok && lane == 0) {
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

// ---------------------------------------------------------------- consumer helpers
__device__ __forceinline__ void pf_mma(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void pf_ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ uint32_t pf_bf16(float v) { return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v)); }

enum PfSrc { kPfNorm = 0, kPfPlain = 1 };

// Per-token 1/rms of the residual rows (every block computes all 16; rows past n_tok count as zero).
__device__ void pf_token_rms(PfBlk &b, const float *H, int d, int n_tok) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int t = warp; t < kPfTokens; t += kPfWarps) {
    float ss = 0.f;
    if (t < n_tok)
      for (int c = lane * 4; c < d; c += 128) {
        const float4 v = __ldcg(reinterpret_cast<const float4 *>(H + (size_t)t * d + c));
        ss = fmaf(v.x, v.x, ss); ss = fmaf(v.y, v.y, ss); ss = fmaf(v.z, v.z, ss); ss = fmaf(v.w, v.w, ss);
      }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if (lane == 0) b.rs[t] = rsqrtf(ss / (float)d + b.p->eps);
  }
  named_sync(1, kPfThreads);
}

// Stages K block kb of the 16 tokens' activations as B fragments: thread (token t = tid / 16, piece j =
// tid % 16) handles the 64 columns [kb*1024 + 64 j, +64) of token t = k-steps 4j..4j+3 of the block.
// Fragment store: xblk[((ks * 2 + token tile) * 3 + term) * 32 + (t % 8) * 4 + q] = {cols (2q, 2q+1), cols (8+2q, 9+2q)}.
__device__ void pf_stage_x(PfBlk &b, int src, const float *X, const __nv_bfloat16 *gain, int C, int kb, int n_tok) {
  const int t = threadIdx.x >> 4, j = threadIdx.x & 15;
  const int nt = t >> 3, g = t & 7;
  const float rs = src == kPfNorm ? b.rs[t] : 1.f;
#pragma unroll
  for (int kk = 0; kk < 4; ++kk) {
    const int ks = 4 * j + kk;
    const int c0 = kb * kPfKB + ks * 16;
    float x[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) x[e] = 0.f;
    if (t < n_tok) {
      // columns come in multiples of 8: the last k-step of a row may be half full
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const int c = c0 + 8 * half;
        if (c < C) {
          const float4 v0 = __ldcg(reinterpret_cast<const float4 *>(X + (size_t)t * C + c));
          const float4 v1 = __ldcg(reinterpret_cast<const float4 *>(X + (size_t)t * C + c) + 1);
          float *xh = x + 8 * half;
          xh[0] = v0.x; xh[1] = v0.y; xh[2] = v0.z; xh[3] = v0.w;
          xh[4] = v1.x; xh[5] = v1.y; xh[6] = v1.z; xh[7] = v1.w;
          if (src == kPfNorm) {
            const uint4 gv = *reinterpret_cast<const uint4 *>(gain + c);
            const uint32_t gw[4] = {gv.x, gv.y, gv.z, gv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              xh[2 * e] = xh[2 * e] * rs * __uint_as_float(gw[e] << 16);
              xh[2 * e + 1] = xh[2 * e + 1] * rs * __uint_as_float(gw[e] & 0xffff0000u);
            }
          }
        }
      }
    }
    uint32_t term[3][16];
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      term[0][e] = pf_bf16(x[e]);
      float r = x[e] - __uint_as_float(term[0][e] << 16);
      term[1][e] = pf_bf16(r);
      r -= __uint_as_float(term[1][e] << 16);
      term[2][e] = pf_bf16(r);
    }
#pragma unroll
    for (int k = 0; k < 3; ++k)
#pragma unroll
      for (int q = 0; q < 4; ++q)
        b.xblk[(size_t)((ks * 2 + nt) * 3 + k) * 32 + g * 4 + q] =
            make_uint2(term[k][2 * q] | (term[k][2 * q + 1] << 16), term[k][8 + 2 * q] | (term[k][9 + 2 * q] << 16));
  }
}

enum PfEpi { kPfQKV = 0, kPfAddH = 1, kPfSwiGLU = 2 };

// One matrix for the 16 tokens: out[t][r] = sum_c W[r][c] x[t][c] for this block's rows, then the
// phase's epilogue.
__device__ void pf_gemm(PfBlk &b, const PfPhase &pd, int src, const float *X, const __nv_bfloat16 *gain, int kind, int layer,
                        int pos0, int n_tok) {
  const KParams &p = *b.p;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
  int r0, r1;
  pf_rows(pd.R, pd.gran, r0, r1);
  const int nkb = (pd.C + kPfKB - 1) / kPfKB;
  if (src == kPfNorm) pf_token_rms(b, X, pd.C, n_tok);
  // ldmatrix addresses of this lane inside a tile: rows 0-7 / 8-15, columns k0 / k0+8
  const uint32_t lane_off = (uint32_t)((lane & 7) + ((lane >> 3) & 1) * 8) * kPfPitch + (uint32_t)(lane >> 4) * 16u;
  for (int g0 = r0; g0 < r1; g0 += kPfMaxTiles * kPfTileRows) {
    const int g1 = min(g0 + kPfMaxTiles * kPfTileRows, r1);
    float acc[kPfMaxTiles][2][4];
#pragma unroll
    for (int i = 0; i < kPfMaxTiles; ++i)
#pragma unroll
      for (int n = 0; n < 2; ++n) acc[i][n][0] = acc[i][n][1] = acc[i][n][2] = acc[i][n][3] = 0.f;
    for (int kb = 0; kb < nkb; ++kb) {
      named_sync(1, kPfThreads);  // everyone is done with the previous K block's fragments
      pf_stage_x(b, src, X, gain, pd.C, kb, n_tok);
      named_sync(1, kPfThreads);
      const int nks = min(kPfKSteps, (pd.C - kb * kPfKB + 15) / 16);
#pragma unroll
      for (int i = 0; i < kPfMaxTiles; ++i) {
        if (g0 + i * kPfTileRows < g1) {
          pf_wait(b, &b.full[b.c_stage], b.c_phase, 300);
          const uint32_t base = smem_u32(b.ring + (size_t)b.c_stage * kPfStageBytes) + lane_off;
          for (int ks = warp; ks < nks; ks += kPfWarps) {
            uint32_t a0, a1, a2, a3;
            pf_ldsm_x4(base + (uint32_t)ks * 32u, a0, a1, a2, a3);
            const uint2 *xb = b.xblk + (size_t)(ks * 6) * 32 + lane;
#pragma unroll
            for (int n = 0; n < 2; ++n)
#pragma unroll
              for (int k = 0; k < 3; ++k) {
                const uint2 bb = xb[(n * 3 + k) * 32];
                pf_mma(acc[i][n], a0, a1, a2, a3, bb.x, bb.y);
              }
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
        named_sync(1, kPfThreads);  // red[] free again
        float *mine = b.red + warp * (kPfTileRows * kPfTokens);
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
        for (int w = 0; w < kPfWarps; ++w) y += b.red[w * (kPfTileRows * kPfTokens) + row * kPfTokens + t];
        const float other = __shfl_xor_sync(0xffffffffu, y, 16);
        const int r = t0 + row;
        if (r < g1 && t < n_tok) {
          const int pos = pos0 + t;
          if (kind == kPfQKV) {
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
          } else if (kind == kPfAddH) {
            float *h = p.pf_h + (size_t)t * p.d + r;
            *h = __ldcg(h) + y;
          } else {
            if (!(row & 1)) p.pf_u[(size_t)t * p.f + (r >> 1)] = y / (1.f + __expf(-y)) * other;
          }
        }
      }
    }
  }
}

// Causal attention of the chunk's tokens over the cache: one (token, head) item per block at a time, a warp
// per position with an online softmax, the warps merged through shared memory.
__device__ void pf_attention(PfBlk &b, int layer, int pos0, int n_tok) {
  const KParams &p = *b.p;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int epl = p.hd / 32;
  const float scale = 1.f / sqrtf((float)p.hd);
  float *s_acc = b.red;                            // [warps][256] (red holds 8 x 256 floats)
  float *s_m = reinterpret_cast<float *>(b.xblk);  // the fragment area is idle during this phase
  float *s_l = s_m + kPfWarps;
  const int items = n_tok * p.H;
  for (int item = blockIdx.x; item < items; item += gridDim.x) {
    const int t = item / p.H, head = item - t * p.H;
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
      p.pf_o[(size_t)t * p.d + head * p.hd + dim] = A / L;
    }
  }
  named_sync(1, kPfThreads);
}

__device__ void pf_consumer(PfBlk &b) {
  const KParams &p = *b.p;
  const int n_tok = p.n_iters, pos0 = p.pos0;
  // residual rows start as the tokens' embeddings
  for (int i = blockIdx.x * kPfThreads + threadIdx.x; i < n_tok * p.d; i += gridDim.x * kPfThreads) {
    const int t = i / p.d, c = i - t * p.d;
    p.pf_h[i] = __bfloat162float(p.tok_emb[(size_t)p.prefix[t] * p.d + c]);
  }
  if (pf_grid_barrier(b)) return;
  for (int l = 0; l < p.L; ++l) {
    const LayerW &lw = p.layers[l];
    pf_gemm(b, pf_phase(p, 4 * l), kPfNorm, p.pf_h, lw.attn_norm, kPfQKV, l, pos0, n_tok);
    if (pf_grid_barrier(b)) return;
    pf_attention(b, l, pos0, n_tok);
    if (pf_grid_barrier(b)) return;
    pf_gemm(b, pf_phase(p, 4 * l + 1), kPfPlain, p.pf_o, nullptr, kPfAddH, l, pos0, n_tok);
    if (pf_grid_barrier(b)) return;
    pf_gemm(b, pf_phase(p, 4 * l + 2), kPfNorm, p.pf_h, lw.ffn_norm, kPfSwiGLU, l, pos0, n_tok);
    if (pf_grid_barrier(b)) return;
    pf_gemm(b, pf_phase(p, 4 * l + 3), kPfPlain, p.pf_u, nullptr, kPfAddH, l, pos0, n_tok);
    if (pf_grid_barrier(b)) return;
  }
}

// Nine warps leave one scheduler with three of them: 16384 registers / (3 x 32) caps a thread at 168, which
// is what the compiler derives for a block of 384.
__global__ void __launch_bounds__(384, 1) spd_prefill_kernel(const __grid_constant__ KParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ uint64_t s_full[kPfStages], s_empty[kPfStages];
  __shared__ float s_rs[kPfTokens];
  __shared__ int s_dead, s_quit;
  PfBlk b;
  b.p = &p;
  b.ring = smem;
  b.xblk = reinterpret_cast<uint2 *>(smem + (size_t)kPfStages * kPfStageBytes);
  b.red = reinterpret_cast<float *>(smem + (size_t)kPfStages * kPfStageBytes + kPfXblkBytes);
  b.rs = s_rs;
  b.full = s_full;
  b.empty = s_empty;
  b.dead = &s_dead;
  b.quit = &s_quit;
  b.bar_target = 0;
  b.c_stage = 0;
  b.c_phase = 0;
  if (threadIdx.x == 0) {
    s_dead = 0;
    s_quit = 0;
    for (int s = 0; s < kPfStages; ++s) {
      mbar_init(&s_full[s], 1);
      mbar_init(&s_empty[s], kPfWarps);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // rows of a last, short tile that no copy writes are still multiplied (into rows nobody reads): the ring
  // starts zeroed so that they hold finite values
  for (size_t i = threadIdx.x; i < (size_t)kPfStages * kPfStageBytes / 16; i += blockDim.x)
    reinterpret_cast<uint4 *>(smem)[i] = make_uint4(0u, 0u, 0u, 0u);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();
  if (threadIdx.x >= kPfThreads) pf_producer(b);
  else pf_consumer(b);
  __syncthreads();
}

}  // namespace spd

extern "C" size_t spd_internal_prefill_smem(void) {
  return (size_t)spd::kPfStages * spd::kPfStageBytes + spd::kPfXblkBytes + spd::kPfRedBytes;
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
