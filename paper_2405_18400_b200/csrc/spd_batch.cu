// Batched Superposed Decoding: one timestep of up to 128 requests per pass over the weights (the paper's closing
// remark: batching is complementary to the method, since each request still needs one pass for its k drafts).
//
// A request is a context of its own (prefix, KV cache, draft state); the requests of a batch share the weights and
// the n-gram tables.  Their superposed inputs (Eq. 3) are the token rows of one tile of the tensor-core products that
// the long-prefix path already has (spd_tc_gemm_kernel: tcgen05.mma with TMEM accumulators, activations as three
// exact bf16 terms), so the weights are streamed once per timestep whatever the number of requests.  Between the
// products run row-wise kernels, one block per request (and head): the superposed embedding, the rotary embedding
// and the append to the request's own cache at its own position, attention over that cache, residual + RMSNorm
// and SwiGLU (the long-prefix path's kernels).  After the LM head (one more product, a row of logits per request)
// a block per request runs the method's tail on the request's own draft state: KeepTopK, Eq. 5-7 with the n-gram
// probes, Eq. 2, Eq. 4.
#include <cuda_runtime.h>
#include <math_constants.h>

#include "spd_params.h"
#include "spd_prefill_tc.h"
#include "spd_ptx.cuh"
#include "spd_tail.cuh"
#include "spd_score.cuh"

namespace spd {

// v = hi + mid + lo exactly: each term takes the leading 8 significant bits of what is left, by truncation.
__device__ __forceinline__ void bt_put3(uint16_t *X, size_t term_stride, size_t at, float v) {
  const uint32_t hi = __float_as_uint(v) & 0xffff0000u;
  const float r1 = v - __uint_as_float(hi);
  const uint32_t mid = __float_as_uint(r1) & 0xffff0000u;
  const float r2 = r1 - __uint_as_float(mid);
  X[at] = (uint16_t)(hi >> 16);
  X[at + term_stride] = (uint16_t)(mid >> 16);
  X[at + 2 * term_stride] = (uint16_t)(__float_as_uint(r2) >> 16);
}

__device__ __forceinline__ float bt_block_sum(float v, float *scratch) {
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

// Position of the request's next input: the prefix's m positions, then one per superposed input so far.  The
// device copy of a request's parameters keeps m - 1 in pos0; n_gen counts the tokens generated per draft.
__device__ __forceinline__ int bt_pos(const KParams &p) { return p.pos0 + p.st->n_gen; }

// One request per block: the superposed input of Eq. 3, h = sum_i gamma_i E[last token of draft i], stored as the
// request's residual row, and its RMSNorm with the first layer's gain as three bf16 terms for the first product.
__global__ void __launch_bounds__(256) spd_batch_input_kernel(const KParams *kps, float *h, const __nv_bfloat16 *gain, uint16_t *X,
                                                              size_t term_stride, int d, float eps) {
  __shared__ float scratch[8];
  const KParams &p = kps[blockIdx.x];
  const State *st = p.st;
  float *hr = h + (size_t)blockIdx.x * d;
  float ss = 0.f;
  for (int c = threadIdx.x; c < d; c += 256) {
    float acc = 0.f;
    for (int i = 0; i < p.k; ++i) acc = fmaf(st->gamma[i], __bfloat162float(p.tok_emb[(size_t)st->win[i][kWin - 1] * d + c]), acc);
    hr[c] = acc;
    ss = fmaf(acc, acc, ss);
  }
  const float rs = rsqrtf(bt_block_sum(ss, scratch) / (float)d + eps);
  for (int c = threadIdx.x; c < d; c += 256) bt_put3(X, term_stride, (size_t)blockIdx.x * d + c, hr[c] * rs * __bfloat162float(gain[c]));
}

// One request per block: rotary embedding of q and k (adjacent pairs) at the request's own position, q to Q, k and
// v into the request's own cache.  Y row = [q | k | v].
__global__ void __launch_bounds__(256) spd_batch_rope_cache_kernel(const float *Y, float *Q, const KParams *kps, int d, int hd, int layer) {
  const KParams &p = kps[blockIdx.x];
  const int t = blockIdx.x, pos = bt_pos(p);
  const float *yr = Y + (size_t)t * 3 * d;
  const size_t crow = ((size_t)layer * p.max_pos + pos) * d;
  for (int i = threadIdx.x; i < d / 2; i += 256) {
    const float2 cs = p.rope[(size_t)pos * (hd / 2) + (i % (hd / 2))];
    const float qe = yr[2 * i], qo = yr[2 * i + 1], ke = yr[d + 2 * i], ko = yr[d + 2 * i + 1];
    Q[(size_t)t * d + 2 * i] = qe * cs.x - qo * cs.y;
    Q[(size_t)t * d + 2 * i + 1] = qe * cs.y + qo * cs.x;
    const float k0 = ke * cs.x - ko * cs.y, k1 = ke * cs.y + ko * cs.x;
    const float v0 = yr[2 * d + 2 * i], v1 = yr[2 * d + 2 * i + 1];
    if (p.kv_bf16) {
      reinterpret_cast<__nv_bfloat162 *>(p.kcache)[(crow >> 1) + i] = __halves2bfloat162(__float2bfloat16_rn(k0), __float2bfloat16_rn(k1));
      reinterpret_cast<__nv_bfloat162 *>(p.vcache)[(crow >> 1) + i] = __halves2bfloat162(__float2bfloat16_rn(v0), __float2bfloat16_rn(v1));
    } else {
      reinterpret_cast<float2 *>(p.kcache)[(crow >> 1) + i] = make_float2(k0, k1);
      reinterpret_cast<float2 *>(p.vcache)[(crow >> 1) + i] = make_float2(v0, v1);
    }
  }
}

// One (request, head) per block of four warps: softmax attention of the request's query over its own cache, a warp
// per position with an online softmax, the warps' states merged in shared memory; output as three bf16 terms.
__global__ void __launch_bounds__(128) spd_batch_attn_kernel(const float *Q, const KParams *kps, uint16_t *X, size_t term_stride, int d,
                                                             int hd, int layer) {
  __shared__ float s_acc[4][256];
  __shared__ float s_m[4], s_l[4];
  const KParams &p = kps[blockIdx.x];
  const int head = blockIdx.y, T = bt_pos(p) + 1;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int epl = hd / 32;  // elements per lane, <= 8
  const float scale = 1.f / sqrtf((float)hd);
  float q[8], acc[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    q[e] = e < epl ? Q[(size_t)blockIdx.x * d + head * hd + lane * epl + e] : 0.f;
    acc[e] = 0.f;
  }
  float m = -CUDART_INF_F, l = 0.f;
  for (int t = warp; t < T; t += 4) {
    const size_t base = ((size_t)layer * p.max_pos + t) * d + head * hd + lane * epl;
    float dot = 0.f, vv[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      vv[e] = 0.f;
      if (e < epl) {
        float kx;
        if (p.kv_bf16) {
          kx = __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(p.kcache)[base + e]);
          vv[e] = __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(p.vcache)[base + e]);
        } else {
          kx = reinterpret_cast<const float *>(p.kcache)[base + e];
          vv[e] = reinterpret_cast<const float *>(p.vcache)[base + e];
        }
        dot = fmaf(q[e], kx, dot);
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
    if (e < epl) s_acc[warp][lane * epl + e] = acc[e];
  if (lane == 0) {
    s_m[warp] = m;
    s_l[warp] = l;
  }
  __syncthreads();
  for (int c = threadIdx.x; c < hd; c += 128) {
    float M = -CUDART_INF_F;
#pragma unroll
    for (int w = 0; w < 4; ++w) M = fmaxf(M, s_m[w]);
    float L = 0.f, A = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float wgt = s_m[w] == -CUDART_INF_F ? 0.f : __expf(s_m[w] - M);
      L = fmaf(s_l[w], wgt, L);
      A = fmaf(s_acc[w][c], wgt, A);
    }
    bt_put3(X, term_stride, (size_t)blockIdx.x * d + head * hd + c, A / L);
  }
}

// One request per block (512 threads): the request's row of logits goes to its own buffer; warp 0 ranks the whole
// vocabulary (KeepTopK with log-probabilities under temperature tau, Algorithm 1); then Eq. 5-7, Eq. 2 and Eq. 4 on
// the request's own draft state, as block 0 of the single-request kernel does.
__global__ void __launch_bounds__(kConsumerThreads) spd_batch_tail_kernel(const KParams *kps, const float *Y, int V) {
  extern __shared__ __align__(16) uint8_t bt_smem[];
  __shared__ int s_dead, s_quit;
  const KParams &p = kps[blockIdx.x];
  const float *row = Y + (size_t)blockIdx.x * V;
  for (int c = threadIdx.x; c < V; c += kConsumerThreads) p.logits[c] = row[c];
  if (threadIdx.x == 0) s_dead = s_quit = 0;
  __syncthreads();
  State *st = p.st;
  if (threadIdx.x < 32) {
    block_topk(p, 0, V);  // the k best logits and (max, sum exp) of z / tau over the whole vocabulary, into this block's list
    __syncwarp();
    if (threadIdx.x == 0) {
      const float2 ms = p.pk_ms[blockIdx.x];
      const float lse = ms.x + __logf(ms.y);
      for (int j = 0; j < p.k; ++j) {
        const int id = p.pk_id[(size_t)blockIdx.x * p.k + j];
        st->cand_tok[j] = id < 0 ? 0 : id;
        st->cand_lp[j] = p.pk_val[(size_t)blockIdx.x * p.k + j] * p.inv_tau - lse;
      }
    }
  }
  __syncthreads();
  Blk b;
  b.p = &p;
  b.ring = nullptr;
  b.part = reinterpret_cast<float *>(bt_smem);
  b.full = b.empty = nullptr;
  b.red = nullptr;
  b.dead = &s_dead;
  b.quit = &s_quit;
  b.bar_target = 0;
  b.c_stage = b.c_phase = 0;
  tail_score_select(b, false, st->n_gen);
}

}  // namespace spd

namespace {
constexpr size_t kBatchTailSmem = 20480;
}

// Enqueues one batched timestep of n requests (kps: their parameters in device memory, in row order) on stream s.
// job: the buffers of the context that lends its long-prefix workspace (h, y, q, x, tensor maps); y_logits: [128][V]
// floats; lm_tmap: the LM head's tensor map.  *launches receives the number of kernels enqueued.
extern "C" cudaError_t spd_internal_batch_step(const spd::TcJob *job, const spd::KParams *kps, int n, int V, const __nv_bfloat16 *final_norm,
                                               float *y_logits, cudaStream_t s, int *launches) {
  const spd::TcJob &j = *job;
  const int d = j.d, f = j.f;
  const size_t ts_d = (size_t)j.x_term_rows * d, ts_f = (size_t)j.x_term_rows * f;
  const uint8_t *xmap_d = j.x_tmaps, *xmap_f = j.x_tmaps + spd::kTensorMapBytes;
  int count = 0;
  cudaError_t e = cudaSuccess;
  auto gemm = [&](const uint8_t *xmap, int which, float *Y, int N, int C) {
    if (e != cudaSuccess) return;
    e = spd_internal_tc_gemm(xmap, j.w_tmaps + (size_t)which * spd::kTensorMapBytes, Y, n, N, C, j.x_term_rows, j.st, s);
    ++count;
  };
  auto resid = [&](const __nv_bfloat16 *gain) {
    if (e != cudaSuccess) return;
    e = spd_internal_tc_resid_norm(j.h, j.y, gain, j.x, ts_d, n, d, j.eps, s);
    ++count;
  };
  spd::spd_batch_input_kernel<<<n, 256, 0, s>>>(kps, j.h, j.layers[0].attn_norm, j.x, ts_d, d, j.eps);
  e = cudaGetLastError();
  ++count;
  for (int l = 0; l < j.L && e == cudaSuccess; ++l) {
    gemm(xmap_d, 4 * l, j.y, 3 * d, d);
    if (e != cudaSuccess) break;
    spd::spd_batch_rope_cache_kernel<<<n, 256, 0, s>>>(j.y, j.q, kps, d, j.hd, l);
    if ((e = cudaGetLastError()) != cudaSuccess) break;
    spd::spd_batch_attn_kernel<<<dim3(n, j.H), 128, 0, s>>>(j.q, kps, j.x, ts_d, d, j.hd, l);
    if ((e = cudaGetLastError()) != cudaSuccess) break;
    count += 2;
    gemm(xmap_d, 4 * l + 1, j.y, d, d);
    resid(j.layers[l].ffn_norm);
    gemm(xmap_d, 4 * l + 2, j.y, 2 * f, d);
    if (e != cudaSuccess) break;
    e = spd_internal_tc_swiglu(j.y, j.x, ts_f, n, f, s);
    ++count;
    gemm(xmap_f, 4 * l + 3, j.y, d, f);
    resid(l + 1 < j.L ? j.layers[l + 1].attn_norm : final_norm);
  }
  gemm(xmap_d, 4 * j.L, y_logits, V, d);
  if (e == cudaSuccess) {
    spd::spd_batch_tail_kernel<<<n, spd::kConsumerThreads, kBatchTailSmem, s>>>(kps, y_logits, V);
    e = cudaGetLastError();
    ++count;
  }
  if (launches) *launches = count;
  return e;
}
