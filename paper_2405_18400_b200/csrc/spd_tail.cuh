// Pieces of the method's tail that both kernels of the library run: per-block top-k of the logits with
// softmax statistics, KeepTopK over the blocks' partial lists (Algorithm 1), the first timestep's
// assignment (Eq. 1) and the drafts' weights (Eq. 4).  Each runs on one warp.
#pragma once
#include <cuda_runtime.h>
#include <math_constants.h>

#include "spd_params.h"

namespace spd {

// ---------------------------------------------------------------- LM head: block-level top-k and softmax statistics
// Ranking order everywhere: larger value first, then smaller index.
__device__ __forceinline__ bool ranks_before(float v, int i, float w, int j) { return v > w || (v == w && i < j); }

__device__ __forceinline__ void warp_best(float &v, int &i) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, v, o);
    const int oi = __shfl_xor_sync(0xffffffffu, i, o);
    if (oi >= 0 && (i < 0 || ranks_before(ov, oi, v, i))) { v = ov; i = oi; }
  }
}

// One warp: the k best logits among rows [r0, r1) and (max, sum exp) of z / tau over them, into list `slot` of the
// partial lists (the decode and prefill kernels: warp 0 of each block, slot = the block).
static __device__ void block_topk(const KParams &p, int r0, int r1, int slot) {
  const int lane = threadIdx.x & 31;
  float pv = 0.f;
  int pi = -1;
  float mx = -CUDART_INF_F;
  for (int j = 0; j < p.k; ++j) {
    float bv = 0.f;
    int bi = -1;
    for (int r = r0 + lane; r < r1; r += 32) {
      const float z = p.logits[r];
      if (j > 0 && !ranks_before(pv, pi, z, r)) continue;  // already taken (or is the previous winner)
      if (bi < 0 || ranks_before(z, r, bv, bi)) { bv = z; bi = r; }
    }
    warp_best(bv, bi);
    if (lane == 0) {
      p.pk_val[(size_t)slot * p.k + j] = bi >= 0 ? bv : -CUDART_INF_F;
      p.pk_id[(size_t)slot * p.k + j] = bi;
    }
    pv = bv;
    pi = bi;
    if (j == 0) mx = bi >= 0 ? bv * p.inv_tau : -CUDART_INF_F;
    if (bi < 0) {  // fewer rows than k: the rest stay empty
      for (int jj = j + 1; jj < p.k; ++jj)
        if (lane == 0) {
          p.pk_val[(size_t)slot * p.k + jj] = -CUDART_INF_F;
          p.pk_id[(size_t)slot * p.k + jj] = -1;
        }
      break;
    }
  }
  float s = 0.f;
  for (int r = r0 + lane; r < r1; r += 32) s += __expf(p.logits[r] * p.inv_tau - mx);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) p.pk_ms[slot] = make_float2(mx, s);
}

// KeepTopK over the whole vocabulary from the n_lists partial lists (Algorithm 1), with
// log-probabilities under temperature tau.  Warp 0.
static __device__ void tail_keep_topk(const KParams &p, int n_lists) {
  const int lane = threadIdx.x & 31;
  State *st = p.st;
  const int ncand = n_lists * p.k;
  float M = -CUDART_INF_F;
  for (int g = lane; g < n_lists; g += 32) M = fmaxf(M, __ldcg(&p.pk_ms[g]).x);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  float S = 0.f;
  for (int g = lane; g < n_lists; g += 32) {
    const float2 ms = __ldcg(&p.pk_ms[g]);
    if (ms.x > -CUDART_INF_F) S = fmaf(ms.y, __expf(ms.x - M), S);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) S += __shfl_xor_sync(0xffffffffu, S, o);
  const float lse = M + __logf(S);
  float pv = 0.f;
  int pi = -1;
  for (int j = 0; j < p.k; ++j) {
    float bv = 0.f;
    int bi = -1;
    for (int c = lane; c < ncand; c += 32) {
      const int id = __ldcg(&p.pk_id[c]);
      if (id < 0) continue;
      const float z = __ldcg(&p.pk_val[c]);
      if (j > 0 && !ranks_before(pv, pi, z, id)) continue;
      if (bi < 0 || ranks_before(z, id, bv, bi)) { bv = z; bi = id; }
    }
    warp_best(bv, bi);
    if (lane == 0) {
      // non-finite logits can leave a round without a winner: keep the token id valid
      st->cand_tok[j] = bi < 0 ? 0 : bi;
      st->cand_lp[j] = bv * p.inv_tau - lse;
    }
    pv = bv;
    pi = bi;
  }
  __syncwarp();
}

// gamma_i = p_i / sum_j p_j (Eq. 4), from the drafts' log-probabilities; the step is then complete: the
// history windows have grown by one token.  One warp.
__device__ __forceinline__ void tail_gamma(const KParams &p, int lane) {
  State *st = p.st;
  const int k = p.k;
  const float lp = lane < k ? st->logP[lane] : -CUDART_INF_F;
  float mx = lp;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  const float e = lane < k ? expf(lp - mx) : 0.f;
  float den = e;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
  if (lane < k) st->gamma[lane] = e / den;
  if (lane == 0) {
    st->win_len = min(st->win_len + 1, kWin);
    st->n_gen += 1;
  }
}

// First timestep (Eq. 1): draft i takes the i-th kept token and its log-probability; no n-gram term.  Thread
// i < k of one warp.
__device__ __forceinline__ void tail_first(const KParams &p, int i, int step) {
  State *st = p.st;
  const int k = p.k;
  if (i < k) {
    const int tok = st->cand_tok[i];
    st->logP_in[i] = 0.f;
    int w[kWin];
#pragma unroll
    for (int j = 0; j < kWin; ++j) w[j] = st->win[i][j];
#pragma unroll
    for (int j = 0; j < kWin; ++j) st->win_in[i][j] = w[j];
#pragma unroll
    for (int j = 0; j + 1 < kWin; ++j) st->win[i][j] = w[j + 1];
    st->win[i][kWin - 1] = tok;
    st->logP[i] = st->cand_lp[i];
    st->sel[i] = i;
    p.hist_tok[(size_t)step * k + i] = tok;
    p.hist_par[(size_t)step * k + i] = i;
  }
}

}  // namespace spd
