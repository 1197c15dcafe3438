// Batched Superposed Decoding: one timestep of up to 128 requests per pass over the weights (the paper's closing
// remark: batching is complementary to the method, since each request still needs one pass for its k drafts).
//
// A request is a context of its own (prefix, KV cache, draft state); the requests of a batch share the weights and
// the n-gram tables.  Their superposed inputs (Eq. 3) are the token rows of a tensor-core product made for few rows
// (spd_batch_gemm_kernel in spd_prefill_tc.cu: the 128 weight rows of a tile are the wide tcgen05.mma operand, the
// requests' activations, as three exact bf16 terms, the narrow one, TMEM accumulators, columns split among blocks),
// so the weights are streamed once per timestep whatever the number of requests.  Between the products run
// element-wise kernels spread over requests and columns: the superposed embedding, the rotary embedding and the
// append to the request's own cache at its own position, attention over that cache (a block per request and head),
// residual add and SwiGLU; RMSNorm's 1 / rms is applied behind the product that follows it.  After the LM head (one
// more product, a row of logits per request) a block per request runs the method's tail on the request's own draft
// state: KeepTopK, Eq. 5-7 with the n-gram probes, Eq. 2, Eq. 4.
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

// A batch has few token rows, so the row-wise work between the products is spread over the columns: a block takes
// kBtCols columns of one request's row.  RMSNorm's factor 1 / rms(h) is common to a row's columns and moves behind
// the product (as in the single-request kernel): the kernels that write a residual row h store h * gain as the next
// product's terms and the sum of squares of their columns (ss[request][chunk]); the kernels that read that product
// multiply its rows by rsqrt(sum of the row's chunks / d + eps).
constexpr int kBtCols = 512;      // columns per block: two per thread
constexpr int kBtMaxChunks = 32;  // d_model <= 16384
static_assert(8 + 3 * kMaxK <= kBtResultWords, "a request's row of results holds the head and three lists of k");

__device__ __forceinline__ float bt_block_sum(float v, float *scratch) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
  __syncthreads();
  float s = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) s += scratch[w];
  return s;
}

__device__ __forceinline__ float bt_rs(const float *ss, int request, int d, float eps) {
  const int nch = (d + kBtCols - 1) / kBtCols;
  float s = 0.f;
  for (int c = 0; c < nch; ++c) s += ss[request * kBtMaxChunks + c];
  return rsqrtf(s / (float)d + eps);
}

// Position of the request's next input: the prefix's m positions, then one per superposed input so far.  The
// device copy of a request's parameters keeps m - 1 in pos0; n_gen counts the tokens generated per draft.
__device__ __forceinline__ int bt_pos(const KParams &p) { return p.pos0 + p.st->n_gen; }

// grid (requests, column chunks): the superposed input of Eq. 3, h = sum_i gamma_i E[last token of draft i], stored as
// the request's residual row; h * gain of the first layer's norm as three bf16 terms; the chunk's sum of squares.
__global__ void __launch_bounds__(256) spd_batch_input_kernel(const KParams *kps, float *h, const __nv_bfloat16 *gain, uint16_t *X,
                                                              size_t term_stride, int d, float *ss) {
  dep_wait();    // the kernel before this one in the stream wrote what this one reads
  dep_launch();  // the next one may set itself up meanwhile
  __shared__ float scratch[8];
  const KParams &p = kps[blockIdx.x];
  const State *st = p.st;
  float sq = 0.f;
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const int c = blockIdx.y * kBtCols + e * 256 + threadIdx.x;
    if (c < d) {
      float acc = 0.f;
      for (int i = 0; i < p.k; ++i) acc = fmaf(st->gamma[i], __bfloat162float(p.tok_emb[(size_t)st->win[i][kWin - 1] * d + c]), acc);
      h[(size_t)blockIdx.x * d + c] = acc;
      sq = fmaf(acc, acc, sq);
      bt_put3(X, term_stride, (size_t)blockIdx.x * d + c, acc * __bfloat162float(gain[c]));
    }
  }
  sq = bt_block_sum(sq, scratch);
  if (threadIdx.x == 0) ss[blockIdx.x * kBtMaxChunks + blockIdx.y] = sq;
}

// grid (requests, column chunks): residual add h += y (y = the sum of nz partial products zs floats apart), h * gain
// of the next norm as terms, the chunk's sum of squares.
__global__ void __launch_bounds__(256) spd_batch_resid_kernel(float *h, const float *y, int nz, size_t zs, const __nv_bfloat16 *gain, uint16_t *X,
                                                              size_t term_stride, int d, float *ss) {
  dep_wait();    // the kernel before this one in the stream wrote what this one reads
  dep_launch();  // the next one may set itself up meanwhile
  __shared__ float scratch[8];
  float sq = 0.f;
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const int c = blockIdx.y * kBtCols + e * 256 + threadIdx.x;
    if (c < d) {
      const size_t at = (size_t)blockIdx.x * d + c;
      float v = h[at];
      for (int z = 0; z < nz; ++z) v += y[z * zs + at];
      h[at] = v;
      sq = fmaf(v, v, sq);
      bt_put3(X, term_stride, at, v * __bfloat162float(gain[c]));
    }
  }
  sq = bt_block_sum(sq, scratch);
  if (threadIdx.x == 0) ss[blockIdx.x * kBtMaxChunks + blockIdx.y] = sq;
}

// One column pair of one token row: the QKV product's row (the sum of its nz partial sums) times 1 / rms, rotary
// embedding of q and k (adjacent pairs) at position pos, q to Q, k and v into the cache.  Y row = [q | k | v].
__device__ __forceinline__ void bt_rope_cache_pair(const float *Y, int nz, size_t zs, float rs, float *Q, void *kcache, void *vcache,
                                                   const float2 *rope, int max_pos, int kv_bf16, int d, int hd, int layer, int t, int pos,
                                                   int i) {
  const float *yr = Y + (size_t)t * 3 * d;
  const size_t crow = ((size_t)layer * max_pos + pos) * d;
  const float2 cs = rope[(size_t)pos * (hd / 2) + (i % (hd / 2))];
  float2 qq = make_float2(0.f, 0.f), kk = qq, vv = qq;
  for (int z = 0; z < nz; ++z) {  // the product's partial sums over column ranges, in order
    const float *yz = yr + z * zs;
    qq.x += yz[2 * i]; qq.y += yz[2 * i + 1];
    kk.x += yz[d + 2 * i]; kk.y += yz[d + 2 * i + 1];
    vv.x += yz[2 * d + 2 * i]; vv.y += yz[2 * d + 2 * i + 1];
  }
  const float qe = qq.x * rs, qo = qq.y * rs, ke = kk.x * rs, ko = kk.y * rs;
  Q[(size_t)t * d + 2 * i] = qe * cs.x - qo * cs.y;
  Q[(size_t)t * d + 2 * i + 1] = qe * cs.y + qo * cs.x;
  const float k0 = ke * cs.x - ko * cs.y, k1 = ke * cs.y + ko * cs.x;
  const float v0 = vv.x * rs, v1 = vv.y * rs;
  if (kv_bf16) {
    reinterpret_cast<__nv_bfloat162 *>(kcache)[(crow >> 1) + i] = __halves2bfloat162(__float2bfloat16_rn(k0), __float2bfloat16_rn(k1));
    reinterpret_cast<__nv_bfloat162 *>(vcache)[(crow >> 1) + i] = __halves2bfloat162(__float2bfloat16_rn(v0), __float2bfloat16_rn(v1));
  } else {
    reinterpret_cast<float2 *>(kcache)[(crow >> 1) + i] = make_float2(k0, k1);
    reinterpret_cast<float2 *>(vcache)[(crow >> 1) + i] = make_float2(v0, v1);
  }
}

// grid (requests, chunks of 256 column pairs): each request at its own position, into its own cache.
__global__ void __launch_bounds__(256) spd_batch_rope_cache_kernel(const float *Y, int nz, size_t zs, const float *ss, float eps, float *Q,
                                                                   const KParams *kps, int d, int hd, int layer) {
  dep_wait();    // the kernel before this one in the stream wrote what this one reads
  dep_launch();  // the next one may set itself up meanwhile
  const KParams &p = kps[blockIdx.x];
  const int i = blockIdx.y * 256 + threadIdx.x;  // column pair
  if (i >= d / 2) return;
  bt_rope_cache_pair(Y, nz, zs, bt_rs(ss, blockIdx.x, d, eps), Q, p.kcache, p.vcache, p.rope, p.max_pos, p.kv_bf16, d, hd, layer, blockIdx.x,
                     bt_pos(p), i);
}

// The same for a job of prefix tokens of one request (token t at position pos0 + t, one cache).
__global__ void __launch_bounds__(256) spd_job_rope_cache_kernel(const float *Y, int nz, size_t zs, const float *ss, float eps, float *Q,
                                                                 void *kcache, void *vcache, const float2 *rope, int max_pos, int kv_bf16, int d,
                                                                 int hd, int layer, int pos0) {
  dep_wait();
  dep_launch();
  const int i = blockIdx.y * 256 + threadIdx.x;
  if (i >= d / 2) return;
  bt_rope_cache_pair(Y, nz, zs, bt_rs(ss, blockIdx.x, d, eps), Q, kcache, vcache, rope, max_pos, kv_bf16, d, hd, layer, blockIdx.x,
                     pos0 + blockIdx.x, i);
}

// grid (tokens, column chunks): a job's residual rows start as its tokens' embeddings; h * gain of the first layer's
// norm as three bf16 terms; the chunk's sum of squares.
__global__ void __launch_bounds__(256) spd_job_input_kernel(const int32_t *ids, const __nv_bfloat16 *tok_emb, float *h, const __nv_bfloat16 *gain,
                                                            uint16_t *X, size_t term_stride, int d, float *ss) {
  dep_wait();
  dep_launch();
  __shared__ float scratch[8];
  const __nv_bfloat16 *row = tok_emb + (size_t)ids[blockIdx.x] * d;
  float sq = 0.f;
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const int c = blockIdx.y * kBtCols + e * 256 + threadIdx.x;
    if (c < d) {
      const float v = __bfloat162float(row[c]);
      h[(size_t)blockIdx.x * d + c] = v;
      sq = fmaf(v, v, sq);
      bt_put3(X, term_stride, (size_t)blockIdx.x * d + c, v * __bfloat162float(gain[c]));
    }
  }
  sq = bt_block_sum(sq, scratch);
  if (threadIdx.x == 0) ss[blockIdx.x * kBtMaxChunks + blockIdx.y] = sq;
}

// grid (requests, chunks of 256 rows of the FFN): u = SiLU(gate) * up from the gate / up product's row times 1 / rms
// (Y row = [gate_0, up_0, gate_1, up_1, ...]), as three bf16 terms.
__global__ void __launch_bounds__(256) spd_batch_swiglu_kernel(const float *Y, int nz, size_t zs, const float *ss, float eps, int d, uint16_t *X,
                                                               size_t term_stride, int f) {
  dep_wait();    // the kernel before this one in the stream wrote what this one reads
  dep_launch();  // the next one may set itself up meanwhile
  const int t = blockIdx.x, j = blockIdx.y * 256 + threadIdx.x;
  if (j >= f) return;
  const float rs = bt_rs(ss, t, d, eps);
  const float2 *yr = reinterpret_cast<const float2 *>(Y + (size_t)t * 2 * f);
  float2 gu = make_float2(0.f, 0.f);
  for (int z = 0; z < nz; ++z) {
    const float2 more = yr[z * (zs / 2) + j];
    gu.x += more.x;
    gu.y += more.y;
  }
  const float g = gu.x * rs, up = gu.y * rs;
  bt_put3(X, term_stride, (size_t)t * f + j, g / (1.f + __expf(-g)) * up);
}

// One (request, head) per block of four warps: softmax attention of the request's query over its own cache, a warp
// per position with an online softmax, the warps' states merged in shared memory; output as three bf16 terms.
__global__ void __launch_bounds__(128) spd_batch_attn_kernel(const float *Q, const KParams *kps, uint16_t *X, size_t term_stride, int d,
                                                             int hd, int layer) {
  dep_wait();    // the kernel before this one in the stream wrote what this one reads
  dep_launch();  // the next one may set itself up meanwhile
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

// One request per block (512 threads): the request's row of logits (the LM head's partial products added, times
// 1 / rms of the final norm) goes to its own buffer; every warp ranks a sixteenth of the vocabulary, warp 0 merges
// the sixteen lists (KeepTopK with log-probabilities under temperature tau, Algorithm 1); then Eq. 5-7, Eq. 2 and
// Eq. 4 on the request's own draft state, as block 0 of the single-request kernel does.
__global__ void __launch_bounds__(kConsumerThreads) spd_batch_tail_kernel(const KParams *kps, const float *Y, int nz, size_t zs, const float *ss,
                                                                          float eps, int V, int32_t *results) {
  dep_wait();    // the kernel before this one in the stream wrote what this one reads
  dep_launch();  // the next one may set itself up meanwhile
  extern __shared__ __align__(16) uint8_t bt_smem[];
  __shared__ int s_dead, s_quit;
  const KParams &p = kps[blockIdx.x];
  const float rs = bt_rs(ss, blockIdx.x, p.d, eps);
  const float *row = Y + (size_t)blockIdx.x * V;
  for (int c = threadIdx.x; c < V; c += kConsumerThreads) {
    float z = row[c];
    for (int i = 1; i < nz; ++i) z += row[i * zs + c];
    p.logits[c] = z * rs;
  }
  if (threadIdx.x == 0) s_dead = s_quit = 0;
  __syncthreads();
  {
    const int warp = threadIdx.x >> 5;
    const int r0 = (int)((long long)V * warp / kConsumerWarps), r1 = (int)((long long)V * (warp + 1) / kConsumerWarps);
    block_topk(p, r0, r1, warp);  // this warp's list: slot `warp` of the request's own partial lists
  }
  __threadfence_block();
  __syncthreads();
  if (threadIdx.x < 32) tail_keep_topk(p, kConsumerWarps);
  __syncthreads();
  Blk b;
  b.p = &p;
  b.part = reinterpret_cast<float *>(bt_smem);
  b.dead = &s_dead;
  b.quit = &s_quit;
  b.bar_target = 0;
  b.c_stage = b.c_phase = 0;
  const int step = p.st->n_gen;
  tail_score_select(b, false, step);
  // The request's row of the batch's results, which the host fetches with one copy for all requests: the state's
  // first words (stop, abort flag, error, error info, window length, tokens generated), then the k new tokens, their
  // parents and gamma.
  __syncthreads();
  if (threadIdx.x < kBtResultWords) {
    const State *st = p.st;
    const int i = threadIdx.x;
    int32_t v = 0;
    if (i == 0) v = (int32_t)st->stop;
    else if (i == 1) v = (int32_t)st->abort_flag;
    else if (i == 2) v = st->err;
    else if (i == 3) v = st->err_info;
    else if (i == 4) v = st->win_len;
    else if (i == 5) v = st->n_gen;
    else if (i >= 8 && i < 8 + p.k) v = p.hist_tok[(size_t)step * p.k + (i - 8)];
    else if (i >= 8 + kMaxK && i < 8 + kMaxK + p.k) v = p.hist_par[(size_t)step * p.k + (i - 8 - kMaxK)];
    else if (i >= 8 + 2 * kMaxK && i < 8 + 2 * kMaxK + p.k) v = __float_as_int(st->gamma[i - 8 - 2 * kMaxK]);
    results[(size_t)blockIdx.x * kBtResultWords + i] = v;
  }
}

}  // namespace spd

namespace {
constexpr size_t kBatchTailSmem = 20480;
}

// Enqueues one batched timestep of n requests (kps: their parameters in device memory, in row order) on stream s.
// job: the buffers of the context that lends its long-prefix workspace (h, y, q, x, tensor maps); y_logits: [128][V]
// floats; lm_tmap: the LM head's tensor map.  *launches receives the number of kernels enqueued.
extern "C" cudaError_t spd_internal_batch_step(const spd::TcJob *job, const spd::KParams *kps, int n, int V, const __nv_bfloat16 *final_norm,
                                               float *y_logits, size_t y_floats, size_t y_logits_floats, float *ss, int32_t *results,
                                               int sm_count, cudaStream_t s, int *launches) {
  const spd::TcJob &j = *job;
  const int d = j.d, f = j.f;
  const size_t ts_d = (size_t)j.x_term_rows * d, ts_f = (size_t)j.x_term_rows * f;
  const uint8_t *xmap_d = j.x_tmaps, *xmap_f = j.x_tmaps + spd::kTensorMapBytes;
  int count = 0;
  cudaError_t e = cudaSuccess;
  // The product built for few token rows (weights as the wide operand, columns split among blocks): its output is nz
  // partial sums zs floats apart.
  int nz = 1;
  size_t zs = 0;
  auto gemm = [&](const uint8_t *xmap, int which, float *Y, size_t room, int N, int C) {
    if (e != cudaSuccess) return;
    const uint8_t *wmap = j.w_tmaps + (size_t)which * spd::kTensorMapBytes;
    e = spd_internal_batch_gemm(j.x_tmaps, xmap != xmap_d, wmap, Y, room, n, N, C, j.x_term_rows, j.st, sm_count, s, 1, &nz, &zs);
    ++count;
  };
  const int nch = (d + spd::kBtCols - 1) / spd::kBtCols;
  auto resid = [&](const __nv_bfloat16 *gain) {
    if (e != cudaSuccess) return;
    e = spd::launch_dep(spd::spd_batch_resid_kernel, dim3(n, nch), dim3(256), 0, s, j.h, j.y, nz, zs, gain, j.x, ts_d, d, ss);
    ++count;
  };
  e = spd::launch_dep(spd::spd_batch_input_kernel, dim3(n, nch), dim3(256), 0, s, kps, j.h, j.layers[0].attn_norm, j.x, ts_d, d, ss);
  ++count;
  for (int l = 0; l < j.L && e == cudaSuccess; ++l) {
    gemm(xmap_d, 4 * l, j.y, y_floats, 3 * d, d);
    if (e != cudaSuccess) break;
    e = spd::launch_dep(spd::spd_batch_rope_cache_kernel, dim3(n, (d / 2 + 255) / 256), dim3(256), 0, s, j.y, nz, zs, ss, j.eps, j.q, kps, d, j.hd, l);
    if (e != cudaSuccess) break;
    e = spd::launch_dep(spd::spd_batch_attn_kernel, dim3(n, j.H), dim3(128), 0, s, j.q, kps, j.x, ts_d, d, j.hd, l);
    if (e != cudaSuccess) break;
    count += 2;
    gemm(xmap_d, 4 * l + 1, j.y, y_floats, d, d);
    resid(j.layers[l].ffn_norm);
    gemm(xmap_d, 4 * l + 2, j.y, y_floats, 2 * f, d);
    if (e != cudaSuccess) break;
    e = spd::launch_dep(spd::spd_batch_swiglu_kernel, dim3(n, (f + 255) / 256), dim3(256), 0, s, j.y, nz, zs, ss, j.eps, d, j.x, ts_f, f);
    ++count;
    gemm(xmap_f, 4 * l + 3, j.y, y_floats, d, f);
    resid(l + 1 < j.L ? j.layers[l + 1].attn_norm : final_norm);
  }
  gemm(xmap_d, 4 * j.L, y_logits, y_logits_floats, V, d);
  if (e == cudaSuccess) {
    e = spd::launch_dep(spd::spd_batch_tail_kernel, dim3(n), dim3(spd::kConsumerThreads), kBatchTailSmem, s, kps, y_logits, nz, zs, ss, j.eps, V, results);
    ++count;
  }
  if (launches) *launches = count;
  return e;
}

// The row-wise kernels of a job of up to 128 prefix tokens of one request (the long-prefix path's small jobs): the same
// column-parallel kernels as a batched timestep's, token t at position job.pos0 + t.  ss: [128][32] floats.
extern "C" cudaError_t spd_internal_job_input(const spd::TcJob *job, float *ss, cudaStream_t s) {
  const spd::TcJob &j = *job;
  return spd::launch_dep(spd::spd_job_input_kernel, dim3(j.n_tok, (j.d + spd::kBtCols - 1) / spd::kBtCols), dim3(256), 0, s, j.ids, j.tok_emb, j.h,
                         j.layers[0].attn_norm, j.x, (size_t)j.x_term_rows * j.d, j.d, ss);
}
extern "C" cudaError_t spd_internal_job_rope_cache(const spd::TcJob *job, float *ss, int nz, size_t zs, int layer, cudaStream_t s) {
  const spd::TcJob &j = *job;
  return spd::launch_dep(spd::spd_job_rope_cache_kernel, dim3(j.n_tok, (j.d / 2 + 255) / 256), dim3(256), 0, s, j.y, nz, zs, ss, j.eps, j.q, j.kcache,
                         j.vcache, j.rope, j.max_pos, j.kv_bf16, j.d, j.hd, layer, j.pos0);
}
extern "C" cudaError_t spd_internal_job_resid(const spd::TcJob *job, float *ss, int nz, size_t zs, const __nv_bfloat16 *gain, cudaStream_t s) {
  const spd::TcJob &j = *job;
  return spd::launch_dep(spd::spd_batch_resid_kernel, dim3(j.n_tok, (j.d + spd::kBtCols - 1) / spd::kBtCols), dim3(256), 0, s, j.h, j.y, nz, zs, gain,
                         j.x, (size_t)j.x_term_rows * j.d, j.d, ss);
}
extern "C" cudaError_t spd_internal_job_swiglu(const spd::TcJob *job, float *ss, int nz, size_t zs, cudaStream_t s) {
  const spd::TcJob &j = *job;
  return spd::launch_dep(spd::spd_batch_swiglu_kernel, dim3(j.n_tok, (j.f + 255) / 256), dim3(256), 0, s, j.y, nz, zs, ss, j.eps, j.d, j.x,
                         (size_t)j.x_term_rows * j.f, j.f);
}
