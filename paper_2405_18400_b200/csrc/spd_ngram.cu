// Host-side construction of the n-gram hash tables (see include/spd.h, spd_ngram_plan / spd_ngram_build).
#include <cstring>

#include "spd.h"
#include "spd_hash.h"

namespace {

uint64_t pow2_at_least(uint64_t x) {
  uint64_t p = 16;
  while (p < x) p <<= 1;
  return p;
}

int compare_rows(const int32_t *a, const int32_t *b, int n) {
  for (int j = 0; j < n; ++j) {
    if (a[j] < b[j]) return -1;
    if (a[j] > b[j]) return 1;
  }
  return 0;
}

// Linear probing insert; the table is never more than half full, so a free slot exists.
void insert(SpdSlot *tab, uint64_t mask, uint32_t w0, uint32_t w1, uint32_t w2, uint32_t count) {
  uint64_t idx = spd_key_hash(w0, w1, w2) & mask;
  while (tab[idx].count != 0) idx = (idx + 1) & mask;
  tab[idx] = SpdSlot{w0, w1, w2, count};
}

}  // namespace

extern "C" {

int spd_ngram_plan(int32_t n, int64_t n_entries, const int32_t *keys, uint64_t *ngram_slots, uint64_t *ctx_slots) {
  if (n < 2 || n > SPD_MAX_N || n_entries < 0 || (n_entries > 0 && !keys) || !ngram_slots || !ctx_slots) return SPD_EINVAL;
  int64_t n_ctx = 0;
  for (int64_t i = 0; i < n_entries; ++i) {
    const int32_t *row = keys + i * n;
    for (int j = 0; j < n; ++j)
      if (row[j] < 0 || row[j] > 65535) return SPD_ERANGE;
    if (i > 0 && compare_rows(row - n, row, n) >= 0) return SPD_EINVAL;
    if (i == 0 || compare_rows(row - n, row, n - 1) != 0) ++n_ctx;
  }
  *ngram_slots = pow2_at_least(2 * (uint64_t)n_entries);
  *ctx_slots = pow2_at_least(2 * (uint64_t)n_ctx);
  return SPD_OK;
}

int spd_ngram_build(int32_t n, int64_t n_entries, const int32_t *keys, const int64_t *counts, uint64_t ngram_slots,
                    void *ngram_out, uint64_t ctx_slots, void *ctx_out) {
  uint64_t need_ng = 0, need_ctx = 0;
  int rc = spd_ngram_plan(n, n_entries, keys, &need_ng, &need_ctx);
  if (rc) return rc;
  if (!ngram_out || !ctx_out || (n_entries > 0 && !counts)) return SPD_EINVAL;
  if (ngram_slots < need_ng || ctx_slots < need_ctx) return SPD_ENOMEM;
  if ((ngram_slots & (ngram_slots - 1)) || (ctx_slots & (ctx_slots - 1))) return SPD_EINVAL;
  SpdSlot *ng = static_cast<SpdSlot *>(ngram_out), *cx = static_cast<SpdSlot *>(ctx_out);
  std::memset(ng, 0, ngram_slots * sizeof(SpdSlot));
  std::memset(cx, 0, ctx_slots * sizeof(SpdSlot));
  uint64_t total = 0;
  for (int64_t i = 0; i < n_entries; ++i) {
    const int32_t *row = keys + i * n;
    if (counts[i] <= 0 || counts[i] > 0xfffffffell) return SPD_ERANGE;
    uint32_t w0, w1, w2;
    spd_pack_key(row, n, w0, w1, w2);
    insert(ng, ngram_slots - 1, w0, w1, w2, (uint32_t)counts[i]);
    total += (uint64_t)counts[i];
    // the context's total is written when its run of entries ends
    if (i + 1 == n_entries || compare_rows(row, row + n, n - 1) != 0) {
      if (total > 0xfffffffeull) return SPD_ERANGE;
      spd_pack_key(row, n - 1, w0, w1, w2);
      insert(cx, ctx_slots - 1, w0, w1, w2, (uint32_t)total);
      total = 0;
    }
  }
  return SPD_OK;
}

}  // extern "C"
