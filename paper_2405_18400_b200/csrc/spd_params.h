// Structures shared by the host API and the decode kernel (device side of the library only).
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

#include "spd_hash.h"

namespace spd {

constexpr int kMaxK = 16;
constexpr int kMaxTables = 8;
constexpr int kWin = 8;             // tokens of history kept per draft (n_max - 1 <= 5 are used)
constexpr int kConsumerWarps = 16;  // warps that multiply; one more warp streams weights
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;
constexpr int kTile = 128;          // rows between two epilogues
constexpr int kMaxRowsPerChunk = 8;
constexpr int kMaxStages = 16;
constexpr int kMaxVec = 4;          // 16-byte column vectors per thread: columns <= 4 * 512 * 8
constexpr int kMaxSplit = 8;        // attention splits per head
constexpr int kTensorMapBytes = 128; // size of one tensor map object (CUtensorMap)
constexpr int kPfTokens = 16;       // prefix tokens one prefill launch takes
constexpr int kUnitRows = 8;        // rows of a unit of a matrix in fragment order (the granularity of the blocks' shares; 4 was
                                    // measured too: the shares come out more even, but a 7B timestep took 4.16 ms against 2.65 ms)
constexpr int kScratchBytes = 20480; // per-block scratch after the decode kernel's ring: row partials / attention merge / tail

enum Mode { kModePrefill = 0, kModeDecode = 1, kModeScoreOnly = 2, kModeSample = 3, kModeNucleusOnly = 4 };

struct LayerW {
  const __nv_bfloat16 *attn_norm, *wqkv, *wo, *ffn_norm, *wgate_up, *wdown;
  // the same matrices in the decode kernel's fragment order (spd_pack_image), or null
  const __nv_bfloat16 *wqkv_img, *wo_img, *wgate_up_img;
};

struct TableDev {
  const SpdSlot *ngram, *ctx;
  uint64_t ngram_mask, ctx_mask;
  int32_t n, pad;
};

// Draft state and the last step's intermediates, in device memory.
struct State {
  unsigned int bar;         // grid barrier counter (zeroed by the host before every launch)
  unsigned int stop;        // set once the most probable draft's new token is the stop token (zeroed with `bar`)
  unsigned int abort_flag;  // set by any thread that gave up a wait
  int32_t err, err_info;
  int32_t win_len;          // valid tokens in each history window
  int32_t n_gen;            // tokens generated per draft so far
  int32_t win[kMaxK][kWin]; // right-aligned: win[i][kWin-1] is draft i's last token
  float logP[kMaxK], gamma[kMaxK];
  // intermediates of the last step
  int32_t cand_tok[kMaxK];
  float cand_lp[kMaxK];
  float logP_in[kMaxK];
  int32_t win_in[kMaxK][kWin];
  float score[kMaxK * kMaxK], png[kMaxK * kMaxK];
  uint32_t cnt[kMaxK * kMaxK][kMaxTables];  // 0xffffffff: order skipped
  uint32_t tot[kMaxK][kMaxTables];
  int32_t sel[kMaxK];
};

struct KParams {
  // model
  int32_t L, d, H, hd, f, V, max_pos;
  float eps;
  int32_t kv_bf16;
  const LayerW *layers;
  const __nv_bfloat16 *tok_emb, *final_norm, *lm_head;
  // method
  int32_t k, n_min, n_max, n_tables;
  float lambda[8];
  float alpha, inv_tau, log_delta;
  TableDev tab[kMaxTables];
  // workspace
  void *kcache, *vcache;     // [L][max_pos][d] float or bf16
  const float2 *rope;        // [max_pos][hd/2] (cos, sin)
  float *h, *q, *u, *logits; // [d], [d], [f], [V]
  float *opart;              // [H * kMaxSplit][hd] unnormalised attention partials
  float2 *oml;               // [H * kMaxSplit] (running max, running sum)
  float *pk_val;             // [grid][k] per-block top logits
  int32_t *pk_id;            // [grid][k]
  float2 *pk_ms;             // [grid] (max of z/tau, sum of exp(z/tau - max))
  State *st;
  int32_t *hist_tok, *hist_par;  // [max_pos][k]
  int32_t *prefix;           // [max_pos]; kModeSample appends the sampled tokens
  float *trace;              // [L][2][d] or null
  float *pf_h, *pf_q;        // [kPfTokens][d] prefill: residual rows, rotated queries
  const void *pf_tmaps;      // [4 L + 1] tensor maps (128 bytes each) of the layers' matrices and the LM head, for the prefill's tiled copies
  // prefill activations as mma fragments, three bf16 terms each: [ceil(C/16)][2][3][32] x 8 bytes
  uint16_t *pf_xh, *pf_xo;   // gain-scaled residual (C = d), attention output (C = d)
  uint16_t *pf_xu;           // SwiGLU output (C = f)
  // prefill attention split over position ranges: per (head, token half, range) unnormalised sums and (max, sum),
  // arrivals per (head, token half)
  float *pf_part;            // [H * 2 * 8][8][hd]
  float2 *pf_ml;             // [H * 2 * 8][8]
  unsigned int *pf_cnt;      // [H * 2], zero between phases
  // nucleus sampling (kModeSample): one uniform number per sampled token
  const float *ns_u;         // [max_pos]
  float ns_p, ns_inv_temp;
  // launch
  int32_t mode, n_iters, pos0, step0;
  int32_t pf_head;           // prefill kernel: the launch ends the prefix: LM head on its last token and first timestep
  int32_t stage_bytes, n_stages;
  // prefill kernel only (kept behind the fields the decode kernel reads: its code is sensitive to their offsets)
  float *pf_ss;              // [grid][kPfTokens] per block: sums of squares of the residual values it produced
  int32_t pf_stall;          // prefill kernel, test hook: block 0 withholds its arrival at the grid barriers
  int32_t eos_id;            // stop token (-1: none): decoding ends with the step in which the most probable draft emits it
  const __nv_bfloat16 *lm_head_img;  // the LM head in fragment order, or null
};

}  // namespace spd
