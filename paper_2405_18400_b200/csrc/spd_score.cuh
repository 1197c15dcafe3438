// The scoring stage of a timestep (Eq. 5-7, Eq. 2, Eq. 4) on one block, and the block context the kernels that
// run it share: n-gram hash probes, interpolation, selection of the k best options, update of the draft state.
#pragma once
#include <cuda_runtime.h>
#include <math_constants.h>

#include "spd_params.h"
#include "spd_ptx.cuh"
#include "spd_tail.cuh"

namespace spd {

constexpr unsigned long long kWaitNs = 1500ull * 1000ull * 1000ull;  // 1.5 s per wait
constexpr int kErrTable = -6, kErrTimeout = -7;
constexpr uint32_t kSkipped = 0xffffffffu;  // in the count / total arrays: this order does not apply to the draft

// ---------------------------------------------------------------- block context
struct Blk {
  const KParams *p;
  float *part;       // scratch of the scoring stage (the decode kernel's row partials live there between steps)
  volatile int *dead;
  volatile int *quit;  // block-uniform copy of *dead, refreshed inside every grid barrier
  unsigned int bar_target;
  // consumer ring cursor
  uint32_t c_stage, c_phase;
};

__device__ __forceinline__ void give_up(Blk &b, int code, int info) {
  State *st = b.p->st;
  if (atomicCAS(&st->err, 0, code) == 0) st->err_info = info;
  atomicExch(&st->abort_flag, 1u);
  *b.dead = 1;
}

// ---------------------------------------------------------------- the method's tail (block 0)
// Count stored under the key (1 .. 2^32 - 2), 0 when the key is absent.
__device__ __forceinline__ uint32_t probe(Blk &b, const SpdSlot *tab, uint64_t mask, uint32_t w0, uint32_t w1, uint32_t w2) {
  uint64_t idx = spd_key_hash(w0, w1, w2) & mask;
  const uint64_t limit = mask + 1 < 16384 ? mask + 1 : 16384;
  for (uint64_t i = 0; i < limit; ++i) {
    const uint4 s = __ldg(reinterpret_cast<const uint4 *>(tab + idx));
    if (s.w == 0u) return 0;
    if (s.x == w0 && s.y == w1 && s.z == w2) return s.w;
    idx = (idx + 1) & mask;
  }
  if (mask + 1 > limit) give_up(b, kErrTable, 400);
  return 0;
}

// Scores the k*k options, keeps the k best, updates the draft state.  `first` = first timestep: draft i
// simply takes kept token i (Eq. 1).  All consumer threads of block 0.
static __device__ void tail_score_select(Blk &b, bool first, int step) {
  const KParams &p = *b.p;
  State *st = p.st;
  const int tid = threadIdx.x, k = p.k, nt = p.n_tables;
  uint32_t *s_cnt = reinterpret_cast<uint32_t *>(b.part);  // [k*k][8]; kSkipped where the order does not apply
  uint32_t *s_tot = s_cnt + kMaxK * kMaxK * kMaxTables;    // [k][8]
  float *s_png = reinterpret_cast<float *>(s_tot + kMaxK * kMaxTables);  // [k*k]
  float *s_score = s_png + kMaxK * kMaxK;                  // [k*k]
  named_sync(1, kConsumerThreads);
  if (first) {
    tail_first(p, tid, step);
  } else {
    // Eq. 5 lookups: one thread per (draft, token, table) count and per (draft, table) context total
    const int n_cnt = k * k * nt, n_all = n_cnt + k * nt;
    const int wl = st->win_len;
    for (int qi = tid; qi < n_all; qi += kConsumerThreads) {
      int i, j, ti;
      if (qi < n_cnt) {
        i = qi / (k * nt);
        j = (qi / nt) % k;
        ti = qi % nt;
      } else {
        const int r = qi - n_cnt;
        i = r / nt;
        j = -1;
        ti = r % nt;
      }
      const TableDev &tb = p.tab[ti];
      uint32_t res = kSkipped;
      if (tb.n >= p.n_min && tb.n <= p.n_max && wl >= tb.n - 1) {
        int32_t key[6];
#pragma unroll
        for (int e = 0; e < 6; ++e) key[e] = 0;
        for (int e = 0; e < tb.n - 1; ++e) key[e] = st->win[i][kWin - (tb.n - 1) + e];
        int len = tb.n - 1;
        if (j >= 0) key[len++] = st->cand_tok[j];
        uint32_t w0, w1, w2;
        spd_pack_key(key, len, w0, w1, w2);
        res = j >= 0 ? probe(b, tb.ngram, tb.ngram_mask, w0, w1, w2) : probe(b, tb.ctx, tb.ctx_mask, w0, w1, w2);
      }
      if (j >= 0) s_cnt[(i * k + j) * kMaxTables + ti] = res;
      else s_tot[i * kMaxTables + ti] = res;
    }
    named_sync(1, kConsumerThreads);
    if (tid < k * k) {
      const int i = tid / k;
      float png = 0.f;
      for (int ti = 0; ti < nt; ++ti) {
        const uint32_t c = s_cnt[tid * kMaxTables + ti], t = s_tot[i * kMaxTables + ti];
        st->cnt[tid][ti] = c;
        if (tid % k == 0) st->tot[i][ti] = t;
        if (t != kSkipped && t > 0u) png = fmaf(p.lambda[p.tab[ti].n - 2], (float)c / (float)t, png);
      }
      s_png[tid] = png;
      st->png[tid] = png;
    }
    named_sync(1, kConsumerThreads);
    if (tid < k * k) {
      const int i = tid / k, j = tid - i * k;
      bool overlap = false;
      for (int jj = 0; jj < k; ++jj) overlap |= s_png[i * k + jj] > 0.f;
      const float base = st->logP[i] + (1.f - p.alpha) * st->cand_lp[j];
      float sc;
      if (!overlap) sc = base + p.log_delta;                                   // Eq. 7
      else if (s_png[tid] > 0.f) sc = base + p.alpha * logf(s_png[tid]);       // Eq. 6
      else sc = -CUDART_INF_F;                                                 // token absent from the n-gram distribution
      s_score[tid] = sc;
      st->score[tid] = sc;
    }
    named_sync(1, kConsumerThreads);
    if (tid < 32) {
      // the k best options, best first (Eq. 2); then the state moves to the new drafts
      const int lane = tid;
      float pv = 0.f;
      int pi = -1;
      int my_sel = -1;
      float my_score = 0.f;
      for (int r = 0; r < k; ++r) {
        float bv = 0.f;
        int bi = -1;
        for (int c = lane; c < k * k; c += 32) {
          const float z = s_score[c];
          if (r > 0 && !ranks_before(pv, pi, z, c)) continue;
          if (bi < 0 || ranks_before(z, c, bv, bi)) { bv = z; bi = c; }
        }
        warp_best(bv, bi);
        if (lane == r) { my_sel = bi; my_score = bv; }
        pv = bv;
        pi = bi;
      }
      int w[kWin];
      float old_lp = 0.f;
      if (lane < k) {
        old_lp = st->logP[lane];
        const int par = my_sel / k;
#pragma unroll
        for (int j = 0; j < kWin; ++j) w[j] = st->win[par][j];
      }
      int own[kWin];
      if (lane < k) {
#pragma unroll
        for (int j = 0; j < kWin; ++j) own[j] = st->win[lane][j];
      }
      __syncwarp();
      if (lane < k) {
        const int par = my_sel / k, tok = st->cand_tok[my_sel - par * k];
        st->logP_in[lane] = old_lp;
#pragma unroll
        for (int j = 0; j < kWin; ++j) st->win_in[lane][j] = own[j];
#pragma unroll
        for (int j = 0; j + 1 < kWin; ++j) st->win[lane][j] = w[j + 1];
        st->win[lane][kWin - 1] = tok;
        st->logP[lane] = my_score;
        st->sel[lane] = my_sel;
        p.hist_tok[(size_t)step * k + lane] = tok;
        p.hist_par[(size_t)step * k + lane] = par;
      }
    }
  }
  named_sync(1, kConsumerThreads);
  if (tid < 32) tail_gamma(p, tid);
  named_sync(1, kConsumerThreads);
}

}  // namespace spd
