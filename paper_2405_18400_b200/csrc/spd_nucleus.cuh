// Nucleus sampling over the LM-head output (Section 2: the smallest set of most probable tokens whose
// probability mass reaches p; one token is drawn from it in proportion to its probability), for splicing
// Superposed Decoding onto nucleus-sampled prefixes (Section 4.5).  Runs on one block, all consumer threads.
//
// Tokens are ordered by logit, descending, equal logits by ascending id.  With e_i = exp(z_i / T - max) the
// nucleus is the shortest head of that order whose sum reaches p * sum_i e_i, and the draw u in [0, 1) picks
// the first token whose running sum exceeds u * (mass of the nucleus).  All sums are taken in 64-bit fixed
// point (e_i * 2^40, rounded down), so they are exact, independent of the order of summation, and every
// comparison is an integer comparison.  Both thresholds are located by a radix search over the logits'
// order-preserving 32-bit keys: six passes (6,6,6,6,6,2 bits), each a histogram of mass and count per digit
// among the logits that share the digits fixed so far, scanned from the top digit down.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "spd_params.h"
#include "spd_ptx.cuh"

namespace spd {

constexpr int kNsBins = 64;
constexpr int kNsBatch = 8;  // logits a thread loads before it looks at them

struct NsShared {
  // per warp and digit: mass as two 20-bit halves (32-bit shared-memory atomics are native, 64-bit ones are
  // not; a warp adds at most 2016 values below 2^20 to a cell) and count
  unsigned int hi[kConsumerWarps][kNsBins], lo[kConsumerWarps][kNsBins];
  unsigned int cnts[kConsumerWarps][kNsBins];
  unsigned long long park[3];   // values carried from the first search to the second
  unsigned long long tot[kNsBins];
  unsigned int ctot[kNsBins];
  // search state and results (thread 0 writes, everyone reads after a barrier)
  unsigned long long above;     // mass of the logits above the digits fixed so far
  unsigned long long total;     // mass of all logits
  unsigned long long target;    // the running sum to reach
  unsigned long long tie_mass;  // mass of the logits equal to the located one
  unsigned int tie_cnt;
  unsigned int prefix;          // digits fixed so far
  float zmax;
  int warp_cnt[kConsumerWarps];
  int token;
};
static_assert(sizeof(NsShared) <= 20480, "nucleus scratch must fit the block's scratch area");

__device__ __forceinline__ uint32_t ns_key(float z) {
  const uint32_t u = __float_as_uint(z + 0.f);  // -0 and +0 are one value
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
// e = exp(z / T - max) in 2^-40 units, rounded down, as two 20-bit halves (e * 2^20 and the remainder * 2^20 are
// exact in float32, so the halves are exact)
__device__ __forceinline__ void ns_mass(float z, float inv_t, float m, unsigned int &hi, unsigned int &lo) {
  const float e20 = __expf(fmaf(z, inv_t, -m)) * 1048576.f;
  const float fh = floorf(e20);
  hi = (unsigned int)fh;
  lo = (unsigned int)((e20 - fh) * 1048576.f);
}

// Locates the first token (in the order above) whose running sum reaches s.target (>= 1): leaves its key in
// s.prefix, the mass above it in s.above, and mass and count of the logits equal to it in s.tie_*.  With
// `fraction` > 0 the target is first set to ceil(fraction * total mass).  If rounding left the target above
// the total, the last token is located.
static __device__ void ns_search(NsShared &s, const float *logits, int V, float inv_t, float m, float fraction) {
  const int tid = threadIdx.x, warp = tid >> 5;
  int decided = 0;
  for (int pass = 0; pass < 6; ++pass) {
    const int width = pass < 5 ? 6 : 2, shift = 32 - decided - width;
    for (int i = tid; i < kConsumerWarps * kNsBins; i += kConsumerThreads) {
      (&s.hi[0][0])[i] = 0u;
      (&s.lo[0][0])[i] = 0u;
      (&s.cnts[0][0])[i] = 0u;
    }
    named_sync(1, kConsumerThreads);
    const uint32_t prefix = s.prefix;
    int cur = -1;  // a run of logits with one digit is summed in registers: at most 63 values of at most 2^20
    unsigned int cur_hi = 0u, cur_lo = 0u, cur_c = 0u;
    for (int r0 = tid; r0 < V; r0 += kNsBatch * kConsumerThreads) {
      float zb[kNsBatch];  // a batch of loads in flight: the logits come from L2
#pragma unroll
      for (int e = 0; e < kNsBatch; ++e) {
        const int r = r0 + e * kConsumerThreads;
        zb[e] = r < V ? __ldcg(logits + r) : 0.f;
      }
#pragma unroll
      for (int e = 0; e < kNsBatch; ++e) {
        if (r0 + e * kConsumerThreads >= V) break;
        const float z = zb[e];
        const uint32_t key = ns_key(z);
        if (decided == 0 || (key >> (32 - decided)) == prefix) {
          const int d = (int)((key >> shift) & ((1u << width) - 1u));
          if (d != cur) {
            if (cur >= 0) {
              atomicAdd(&s.hi[warp][cur], cur_hi + (cur_lo >> 20));
              atomicAdd(&s.lo[warp][cur], cur_lo & 0xfffffu);
              atomicAdd(&s.cnts[warp][cur], cur_c);
            }
            cur = d;
            cur_hi = cur_lo = cur_c = 0u;
          }
          unsigned int h, l;
          ns_mass(z, inv_t, m, h, l);
          cur_hi += h;
          cur_lo += l;
          cur_c += 1u;
        }
      }
    }
    if (cur >= 0) {
      atomicAdd(&s.hi[warp][cur], cur_hi + (cur_lo >> 20));
      atomicAdd(&s.lo[warp][cur], cur_lo & 0xfffffu);
      atomicAdd(&s.cnts[warp][cur], cur_c);
    }
    named_sync(1, kConsumerThreads);
    if (tid < kNsBins) {
      unsigned long long q = 0ull;
      unsigned int c = 0u;
      for (int w = 0; w < kConsumerWarps; ++w) {
        q += ((unsigned long long)s.hi[w][tid] << 20) + s.lo[w][tid];
        c += s.cnts[w][tid];
      }
      s.tot[tid] = q;
      s.ctot[tid] = c;
    }
    named_sync(1, kConsumerThreads);
    if (tid == 0) {
      if (pass == 0) {
        unsigned long long all = 0ull;
        for (int d = 0; d < kNsBins; ++d) all += s.tot[d];
        s.total = all;
        if (fraction > 0.f) {
          unsigned long long t = __double2ull_ru((double)fraction * (double)all);
          s.target = t < 1ull ? 1ull : (t > all ? all : t);
        }
      }
      unsigned long long cum = s.above, last_tot = 0ull;
      int g = -1, last = -1;
      for (int d = (1 << width) - 1; d >= 0; --d) {
        if (s.ctot[d] == 0u) continue;
        if (cum + s.tot[d] >= s.target) {
          g = d;
          break;
        }
        cum += s.tot[d];
        last = d;
        last_tot = s.tot[d];
      }
      if (g < 0) {  // the target lies above the total: the last token in the order
        g = last < 0 ? 0 : last;
        cum -= last_tot;
      }
      s.above = cum;
      s.prefix = (decided == 0 ? 0u : (s.prefix << width)) | (uint32_t)g;
      s.tie_mass = s.tot[g];
      s.tie_cnt = s.ctot[g];
    }
    named_sync(1, kConsumerThreads);
    decided += width;
  }
}

// Draws one token from the nucleus of softmax(logits / T) with the uniform number u in [0, 1).  Every
// consumer thread of the block calls it; all get the token.
static __device__ __noinline__ int ns_sample(const float *logits, int V, float inv_t, float top_p, float u, uint8_t *scratch) {
  NsShared &s = *reinterpret_cast<NsShared *>(scratch);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  named_sync(1, kConsumerThreads);
  // largest logit
  float zm = -3.402823466e38f;
  for (int r0 = tid; r0 < V; r0 += kNsBatch * kConsumerThreads) {
#pragma unroll
    for (int e = 0; e < kNsBatch; ++e) {
      const int r = r0 + e * kConsumerThreads;
      if (r < V) zm = fmaxf(zm, __ldcg(logits + r));
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) zm = fmaxf(zm, __shfl_xor_sync(0xffffffffu, zm, o));
  float *wmax = reinterpret_cast<float *>(&s.tot[0]);
  if (lane == 0) wmax[warp] = zm;
  named_sync(1, kConsumerThreads);
  if (tid == 0) {
    float z = wmax[0];
    for (int w = 1; w < kConsumerWarps; ++w) z = fmaxf(z, wmax[w]);
    s.zmax = z;
    s.above = 0ull;
    s.prefix = 0u;
    s.target = 1ull;
  }
  named_sync(1, kConsumerThreads);
  const float m = s.zmax * inv_t;
  // where the nucleus ends
  ns_search(s, logits, V, inv_t, m, top_p);
  if (tid == 0) {
    const uint32_t cut_key = s.prefix;
    const unsigned long long q = s.tie_cnt ? s.tie_mass / s.tie_cnt : 0ull;  // equal logits have equal mass
    unsigned long long take = s.tie_cnt;  // how many of the equal logits at the cut belong to the nucleus
    if (q > 0ull) {
      const unsigned long long need = s.target > s.above ? s.target - s.above : 1ull;
      take = (need + q - 1ull) / q;
      if (take > s.tie_cnt) take = s.tie_cnt;
      if (take < 1ull) take = 1ull;
    }
    const unsigned long long mass = s.above + take * q;
    unsigned long long t = mass ? __double2ull_rd((double)u * (double)mass) : 0ull;
    if (mass && t >= mass) t = mass - 1ull;
    // second search: first token whose running sum exceeds t
    s.park[0] = t;
    s.park[1] = take;
    s.park[2] = (unsigned long long)cut_key;
    s.above = 0ull;
    s.prefix = 0u;
    s.target = t + 1ull;
  }
  named_sync(1, kConsumerThreads);
  const unsigned long long t = s.park[0], take = s.park[1];
  const uint32_t cut_key = (uint32_t)s.park[2];
  ns_search(s, logits, V, inv_t, m, 0.f);
  // which of the logits equal to the located one: the j-th by ascending id
  const uint32_t hit_key = s.prefix;
  unsigned long long j = 0ull;
  {
    const unsigned long long q = s.tie_cnt ? s.tie_mass / s.tie_cnt : 0ull;
    if (q > 0ull && t >= s.above) j = (t - s.above) / q;
    if (j >= s.tie_cnt) j = s.tie_cnt ? s.tie_cnt - 1ull : 0ull;
    if (hit_key == cut_key && j >= take) j = take - 1ull;
  }
  const int seg = (V + kConsumerThreads - 1) / kConsumerThreads;
  const int lo = tid * seg, hi = min(V, lo + seg);
  int mine = 0;
  for (int r0 = lo; r0 < hi; r0 += kNsBatch) {
#pragma unroll
    for (int e = 0; e < kNsBatch; ++e)
      if (r0 + e < hi) mine += ns_key(__ldcg(logits + r0 + e)) == hit_key ? 1 : 0;
  }
  int incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) s.warp_cnt[warp] = incl;
  if (tid == 0) s.token = 0;
  named_sync(1, kConsumerThreads);
  int before = incl - mine;
  for (int w = 0; w < warp; ++w) before += s.warp_cnt[w];
  if (mine > 0 && (unsigned long long)before <= j && j < (unsigned long long)(before + mine)) {
    int left = (int)(j - (unsigned long long)before);
    for (int r = lo; r < hi; ++r)
      if (ns_key(__ldcg(logits + r)) == hit_key && left-- == 0) s.token = r;
  }
  named_sync(1, kConsumerThreads);
  const int tok = s.token;
  named_sync(1, kConsumerThreads);
  return tok;
}

}  // namespace spd
