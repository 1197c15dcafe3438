/*
 * spd.h - C ABI of the B200 (sm_100a) Superposed Decoding library.
 *
 * Superposed Decoding (Shen et al., arXiv 2405.18400) produces k drafts from ONE batch-1
 * inference pass per timestep: the input of the language model is the gamma-weighted sum of the k
 * drafts' last-token embeddings (Section 3.1), the k most probable next tokens expand the k
 * drafts into k*k options, each option is scored by the draft's probability times an
 * interpolation of the model's probability with n-gram probabilities (Section 3.2), and the k
 * best options become the drafts of the next timestep (Section 3, Algorithm 1).
 *
 * All entry points return an int status (0 = SPD_OK, negative = error); none throws, aborts or
 * traps the device.  "DEVICE" pointers are CUDA device addresses of the current device, "HOST"
 * pointers are ordinary host addresses.  The library never allocates or frees device memory:
 * weights, n-gram tables and the workspace are allocated by the caller and only borrowed; they
 * must stay valid and unchanged until spd_destroy.  A context is not thread-safe; calls on one
 * context must be serialised by the caller.  Work is enqueued on the stream given in spd_config.
 */
#ifndef SPD_H_
#define SPD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPD_MAX_K 16       /* drafts per context                        */
#define SPD_MAX_ORDERS 8   /* lambda entries: orders 2..9 addressable   */
#define SPD_MAX_N 6        /* largest n-gram order a table slot can hold */

enum {
  SPD_OK = 0,
  SPD_EINVAL = -1,   /* null pointer, bad shape, k out of range, vocab > 65535, misaligned pointer   */
  SPD_ESTATE = -2,   /* spd_step / spd_generate before spd_prefill                                   */
  SPD_ERANGE = -3,   /* prefix empty or too long, token id outside the vocabulary, out of positions  */
  SPD_ENOMEM = -4,   /* workspace (or a caller-provided buffer) too small                            */
  SPD_ECUDA = -5,    /* a CUDA runtime call failed; spd_last_cuda_error() gives its text             */
  SPD_ETABLE = -6,   /* an n-gram table probe ran past its bound (malformed table)                   */
  SPD_ETIMEOUT = -7  /* a bounded wait inside the decode kernel expired                              */
};

typedef struct spd_ctx spd_ctx; /* opaque; small host object owned by the library */

/*
 * Model and method configuration.
 * Decoder (the paper uses Llama-2 unchanged, Section 4): n_layers pre-norm blocks of RMSNorm ->
 * multi-head attention with rotary embedding on adjacent pairs (2i, 2i+1), angle
 * pos * rope_theta^(-2i/head_dim) -> residual -> RMSNorm -> SwiGLU feed-forward -> residual; final
 * RMSNorm; untied output projection.  head_dim = d_model / n_heads must be a multiple of 32, at
 * most 256; d_model and d_ffn multiples of 8; vocab <= 65535; max_pos = positions the KV cache holds.
 * Method: k drafts (1..SPD_MAX_K); n-gram orders n_min..n_max (2..SPD_MAX_N) with interpolation
 * weights lambda[n-2] (Eq. 5, Appendix B); alpha of Eq. 6; tau = softmax temperature applied to
 * the logits before anything else; delta of Eq. 7 (0 < delta <= 1; the paper gives no value).
 * eos_id: the stop token, -1 for none (Section 3 and Algorithm 1 generate "until max generation length or stop
 * token"; which draft's token counts is not said: here decoding ends with the timestep in which the most
 * probable draft emits it, see spd_finished).  kv_dtype: 0 = float32 cache, 1 = bf16
 * cache (keys after the rotary embedding and values are rounded to nearest even when stored).
 * stream: a cudaStream_t (NULL = the legacy default stream).
 */
typedef struct {
  int32_t n_layers, d_model, n_heads, d_ffn, vocab, max_pos;
  float rms_eps, rope_theta;
  int32_t k;
  int32_t n_min, n_max;
  float lambda[SPD_MAX_ORDERS];
  float alpha, tau, delta;
  int32_t eos_id;
  int32_t kv_dtype;
  void *stream;
} spd_config;

/*
 * Model parameters: DEVICE pointers to bf16 data, row-major [out][in], each 16-byte aligned,
 * BORROWED.  The per-layer members are HOST arrays of n_layers DEVICE pointers.
 *   tok_emb   [vocab][d_model]      final_norm [d_model]      lm_head [vocab][d_model]
 *   attn_norm [d_model]             ffn_norm   [d_model]
 *   wqkv      [3*d_model][d_model]  rows 0..d-1 = W_q, d..2d-1 = W_k, 2d..3d-1 = W_v
 *   wo        [d_model][d_model]
 *   wgate_up  [2*d_ffn][d_model]    row 2j = gate row j, row 2j+1 = up row j (interleaved)
 *   wdown     [d_model][d_ffn]
 * Optional second images of lm_head, wqkv, wo and wgate_up in fragment order (spd_pack_image), same sizes: with all
 * four present (every layer), d_model a multiple of 32, d_ffn of 4 and vocab of 8, the decode timesteps (Section 3,
 * "Next Timesteps") multiply these matrices on the tensor cores; the row-major ones are still what the first
 * timestep's kernels read.  Null members: every timestep uses the row-major matrices.
 */
typedef struct {
  const void *tok_emb, *final_norm, *lm_head;
  const void *const *attn_norm, *const *wqkv, *const *wo;
  const void *const *ffn_norm, *const *wgate_up, *const *wdown;
  const void *lm_head_img;
  const void *const *wqkv_img, *const *wo_img, *const *wgate_up_img;
} spd_weights;

/*
 * One n-gram order's frequency store (Section 4: a table of the distinct n-grams with how often each occurs) as two
 * open-addressing hash tables in DEVICE memory, BORROWED, produced by spd_ngram_build.  A slot is
 * 16 bytes: six uint16 token ids (unused ones 0) then a uint32 count; count 0 marks an empty slot.
 * `ngram` maps n tokens -> count; `ctx` maps the first n-1 tokens -> sum of the counts of all stored
 * n-grams that start with them.  Slot numbers are powers of two.
 */
typedef struct {
  int32_t n;
  int32_t reserved;
  uint64_t ngram_slots, ctx_slots;
  const void *ngram, *ctx;
} spd_ngram_table;

/* Bytes of DEVICE workspace spd_create needs for this configuration (KV cache, activations,
 * draft state, history).  HOST pointers.  SPD_EINVAL on a bad configuration. */
int spd_workspace_bytes(const spd_config *cfg, size_t *bytes);

/*
 * Creates a context.  cfg, weights, tables: HOST structs (copied).  n_tables may be 0 (then every
 * draft takes the delta path of Eq. 7).  workspace: DEVICE memory of at least spd_workspace_bytes,
 * 256-byte aligned, BORROWED; its contents are initialised here (this call enqueues copies on the
 * stream and synchronises it).  *out receives the context.  The calling thread's current device
 * is the device used for every later call.
 */
int spd_create(const spd_config *cfg, const spd_weights *weights, const spd_ngram_table *tables, int32_t n_tables,
               void *workspace, size_t workspace_bytes, spd_ctx **out);

/*
 * First timestep (Section 3 "First Timestep", Eq. 1; Algorithm 1's first branch): runs the decoder
 * over the m prefix tokens (HOST int32 ids, 1 <= m < max_pos), draft i takes the i-th most probable
 * next token and its probability, no n-gram term.  out_ids / out_gamma: HOST arrays of k entries
 * (token of draft i; gamma_i of Eq. 4), either may be NULL.  Restarts the context from scratch.
 * Synchronises the stream before returning.  Prefixes of more than 32 tokens (head size 64 or 128,
 * max_pos >= 130) run all but their last 1..16 tokens through the long-prefix path (tensor-core
 * products over up to 512 tokens at a time, many small launches); its buffers are part of the
 * workspace.  The result does not depend on which path a token took beyond float rounding.
 */
int spd_prefill(spd_ctx *ctx, const int32_t *prefix_ids, int32_t m, int32_t *out_ids, float *out_gamma);

/*
 * One later timestep (Section 3 "Next Timesteps", Eq. 2-7; Algorithm 1's second branch).  HOST
 * outputs of k entries each, any may be NULL: out_ids[r] = new last token of draft r, out_parent[r]
 * = index of the previous-step draft that draft r extends, out_gamma[r] = its weight (Eq. 4).
 * Drafts are ordered by probability, most probable first.  Synchronises the stream.
 */
int spd_step(spd_ctx *ctx, int32_t *out_ids, int32_t *out_parent, float *out_gamma);

/*
 * n_steps timesteps in one device launch with a single synchronisation at the end (the timed call).
 * HOST outputs, any may be NULL: out_tokens [k][*out_len] row-major = all tokens generated so far
 * by each surviving draft (the first-timestep token included, the prefix excluded); out_len = that
 * length; out_logp [k] = log of the draft probabilities P of Eq. 2; out_gamma [k].
 * out_tokens must have room for k * (tokens generated so far + n_steps) entries.  With a stop token the launch
 * ends after the timestep in which the most probable draft emits it: *out_len is then smaller than asked for
 * (rows of out_tokens are *out_len apart), and spd_finished turns 1.
 */
int spd_generate(spd_ctx *ctx, int32_t n_steps, int32_t *out_tokens, int32_t *out_len, float *out_logp,
                 float *out_gamma);

/*
 * Reset (Section 5.3 "Superposed Decoding Resets"): one of the k drafts is chosen - by the caller; the paper
 * samples one every s timesteps - and draft generation restarts from it.  The chosen draft's tokens are
 * appended to the prefix, the cache positions that were filled from superposed inputs are recomputed from
 * those tokens (the original prefix's positions are kept), and the first timestep (Eq. 1) runs on the longer
 * prefix.  Afterwards the context is exactly as after spd_prefill on prefix + chosen draft.  draft: 0..k-1;
 * out_ids / out_gamma as for spd_prefill.  SPD_ESTATE before spd_prefill.  Synchronises the stream.
 */
int spd_reset(spd_ctx *ctx, int32_t draft, int32_t *out_ids, float *out_gamma);

/*
 * Nucleus sampling spliced in front of Superposed Decoding (Section 4.5: a nucleus-sampled generation serves
 * as the prefix of k superposed drafts; Section 2 for the sampler: the smallest set of most probable tokens
 * whose probability reaches top_p, one token drawn from it in proportion to its probability).  Extends the
 * prefix by n_new tokens, each drawn from softmax(logits / temperature) restricted to its nucleus - tokens
 * ordered by probability, equal ones by ascending id; the draw u picks the first token whose running
 * probability exceeds u times the nucleus' mass - then runs the first timestep (Eq. 1) on the longer prefix:
 * afterwards the context is as after spd_prefill on prefix + sampled tokens.  The random numbers are the
 * caller's: uniforms = HOST array of n_new floats in [0, 1).  0 < top_p <= 1, temperature > 0.  HOST outputs,
 * any may be NULL: out_new [n_new] sampled ids; out_ids / out_gamma [k] as for spd_prefill.  Needs a context
 * fresh from spd_prefill, spd_reset or spd_sample (no spd_step since), else SPD_ESTATE; SPD_ERANGE when the
 * prefix would not fit or an argument is out of range.  One launch; synchronises the stream.
 */
int spd_sample(spd_ctx *ctx, int32_t n_new, float top_p, float temperature, const float *uniforms, int32_t *out_new,
               int32_t *out_ids, float *out_gamma);

/* Same as spd_generate but only enqueues the launch: no synchronisation, no outputs.  For callers
 * that time the launch with their own CUDA events; follow with spd_sync. */
int spd_generate_async(spd_ctx *ctx, int32_t n_steps);

/* Synchronises the stream and reports any error the device recorded (SPD_ETABLE, SPD_ETIMEOUT). */
int spd_sync(spd_ctx *ctx);

/* Frees the host object.  Device memory stays the caller's. */
int spd_destroy(spd_ctx *ctx);

/* Static text for a status code. */
const char *spd_strerror(int status);
/* Text of the last CUDA runtime error seen by this thread's calls ("" if none). */
const char *spd_last_cuda_error(void);

/*
 * Fragment order of a weight matrix for the decode timesteps' products y = W x (Section 3: every later timestep is
 * one pass of the superposed input through the decoder).  w: DEVICE, bf16 row-major [rows][cols], rows a multiple
 * of 8, cols a multiple of 32; out: DEVICE, rows * cols * 2 bytes, 16-byte aligned, not overlapping w.  Every block
 * of 8 rows x 32 columns is stored as 32 vectors of 16 bytes, vector 4 g + t = row g's column pairs 2t, 2t+8,
 * 2t+16, 2t+24 of the block (the operand registers of two m16n8k16 tensor-core instructions for that lane); blocks
 * of one 8-row unit follow one another in column order, units in row order.  Enqueued on `stream` (a cudaStream_t,
 * may be null), not synchronised.  SPD_EINVAL for null pointers or sizes that do not divide; SPD_ECUDA.
 */
int spd_pack_image(const void *w, int32_t rows, int32_t cols, void *out, void *stream);

/*
 * N-gram table construction (host side; the tables of Section 4 re-laid as hash tables).
 * Input: n_entries unique n-grams as HOST int32 keys [n_entries][n] in lexicographic order with
 * HOST int64 counts (> 0).  spd_ngram_plan reports the slot numbers to allocate (powers of two, at
 * least twice the entries); spd_ngram_build fills caller-provided HOST buffers of ngram_slots*16 and
 * ctx_slots*16 bytes, which the caller then copies to the device.  SPD_ERANGE if a token id exceeds
 * 65535 or a count or context total exceeds 2^32-2 (counts are unsigned 32-bit on the device and
 * 2^32-1 is reserved); SPD_EINVAL if keys are not strictly increasing.
 */
int spd_ngram_plan(int32_t n, int64_t n_entries, const int32_t *keys, uint64_t *ngram_slots, uint64_t *ctx_slots);
int spd_ngram_build(int32_t n, int64_t n_entries, const int32_t *keys, const int64_t *counts, uint64_t ngram_slots,
                    void *ngram_out, uint64_t ctx_slots, void *ctx_out);

/*
 * Test hook: copies an internal buffer to HOST memory after synchronising the stream.  `what`:
 *   SPD_DBG_LOGITS    float [vocab]        logits of the last LM pass
 *   SPD_DBG_CAND_TOK  int32 [k]            kept tokens (KeepTopK), most probable first
 *   SPD_DBG_CAND_LP   float [k]            their log-probabilities z/tau - logsumexp(z/tau)
 *   SPD_DBG_LOGP_IN   float [k]            draft log-probabilities before the last step's selection
 *   SPD_DBG_SCORE     float [k*k]          score of option i*k+j (-inf = dropped)
 *   SPD_DBG_PNG       float [k*k]          Eq. 5 value of option i*k+j
 *   SPD_DBG_CNT       uint32 [k*k][8]      n-gram count per option and table (0xffffffff = order skipped)
 *   SPD_DBG_TOT       uint32 [k][8]        context total per draft and table (0xffffffff = order skipped)
 *   SPD_DBG_SEL       int32 [k]            chosen options i*k+j, best first
 *   SPD_DBG_LOGP      float [k]            current draft log-probabilities
 *   SPD_DBG_HIST_IN   int32 [k][8]         last 8 tokens of each draft before the last step's selection (right-aligned)
 *   SPD_DBG_TRACE     float [n_layers][2][d_model]  residual after attention / after the FFN of the last LM pass
 *                     (recorded only while spd_debug_trace has switched it on; zeros otherwise)
 *   SPD_DBG_HIDDEN    float [d_model]      residual stream after the last LM pass
 *   SPD_DBG_KCACHE    float [n_layers][T][d_model]  cached keys of the T positions written so far (T = prefix
 *                     length + tokens generated - 1), widened to float32;  SPD_DBG_VCACHE likewise for values
 * SPD_ENOMEM if `bytes` is smaller than the buffer.
 */
enum {
  SPD_DBG_LOGITS = 0, SPD_DBG_CAND_TOK, SPD_DBG_CAND_LP, SPD_DBG_LOGP_IN, SPD_DBG_SCORE, SPD_DBG_PNG, SPD_DBG_CNT,
  SPD_DBG_TOT, SPD_DBG_SEL, SPD_DBG_LOGP, SPD_DBG_HIST_IN, SPD_DBG_TRACE, SPD_DBG_HIDDEN, SPD_DBG_KCACHE, SPD_DBG_VCACHE
};
int spd_debug_read(spd_ctx *ctx, int what, void *host_buf, size_t bytes);

/*
 * Test hook: switches the recording of the per-layer residual trace (SPD_DBG_TRACE) on (on != 0) or off for the
 * launches that follow.  Off after spd_create, so that the decoding path writes no instrumentation.
 */
int spd_debug_trace(spd_ctx *ctx, int on);

/*
 * Test hook for the scoring stage alone (Eq. 2, 4-7): overwrites the draft state with the given
 * HOST values - hist int32 [k][hist_len] = each draft's most recent tokens (hist_len <= 8, oldest
 * first), logp float [k] - and runs KeepTopK-to-selection on the given kept tokens cand_tok int32 [k]
 * and log-probabilities cand_lp float [k] without an LM pass.  Results are read with spd_debug_read.
 */
int spd_debug_score(spd_ctx *ctx, const int32_t *hist, int32_t hist_len, const float *logp, const int32_t *cand_tok,
                    const float *cand_lp);

/*
 * Test hook for the nucleus sampler alone (the draw that spd_sample makes per token): HOST logits float
 * [vocab], one uniform number u in [0, 1); *out_token (HOST) receives the drawn id.  No LM pass.  The
 * context must be prefilled again before decoding continues.
 */
int spd_debug_nucleus(spd_ctx *ctx, const float *logits, float top_p, float temperature, float u, int32_t *out_token);

/*
 * The scoring stage of one timestep (what spd_debug_score runs) without any device allocation.  The
 * paper has no counterpart to this call; it exists for callers that cannot allocate device memory
 * at the point where they need a score: code running inside a memory-budgeted serving process whose
 * pool is already carved up, plug-ins that are handed device pointers but no allocator, or code on a
 * path where cudaMalloc's implicit device synchronisation is not acceptable.  Such callers have no
 * workspace to give spd_create, so the draft state the kernel needs as scratch lives in a fixed 16 KB
 * array inside the library image; every GPU that loads the library holds those 16 KB until the process
 * exits.  The call neither allocates nor frees anything (no cudaMalloc / cudaFree, no allocating library).
 *   cfg      HOST; only k, vocab, n_min, n_max, lambda, alpha, delta and stream are read.
 *   tables   HOST array of n_tables descriptors whose ngram / ctx members are DEVICE pointers, ascending n.
 *   hist     HOST int32 [k][hist_len], each draft's most recent tokens, oldest first;  logp HOST float [k];
 *   cand_tok HOST int32 [k], cand_lp HOST float [k]: the kept tokens and their log-probabilities.
 *   outputs  HOST, any may be NULL: out_sel int32 [k] chosen options i*k+j (best first), out_logp float [k],
 *            out_gamma float [k] (Eq. 4), out_score float [k*k] (-inf = dropped option).
 * Limits of the fixed scratch: k <= SPD_MAX_K (16), n_tables <= 8, hist_len <= 8; anything larger is
 * refused with SPD_ERANGE.  The first call on each device looks up the array's device address (that
 * device must be current); make that first call before any stream capture begins (which says nothing about
 * whether a later call can be captured: no claim is made either way).  All calls on a
 * device share the one array, which still holds the previous call's data when the next begins (each
 * call overwrites it completely before launching); two calls whose device work overlaps, from
 * different streams or threads, race on it, so serialise them.  Synchronises the stream before returning.
 */
int spd_score_static(const spd_config *cfg, const spd_ngram_table *tables, int32_t n_tables, const int32_t *hist,
                     int32_t hist_len, const float *logp, const int32_t *cand_tok, const float *cand_lp,
                     int32_t *out_sel, float *out_logp, float *out_gamma, float *out_score);

/*
 * Test hook for the bounded device waits: launches the prefill kernel on one token with one block withholding
 * its arrival at the first grid barrier, so that the other blocks' waits (1.5 s) run out.  The kernel then
 * ends by itself (every block gives up, drains its copies in flight and returns) and the call returns what the
 * device recorded, which must be SPD_ETIMEOUT.  The context stays usable: prefill it again.
 */
int spd_debug_expire(spd_ctx *ctx);

/*
 * The same for the long-prefix path's products (tcgen05 kernel): one tile is launched whose producer announces
 * its first stage of operands but never copies it, so that the issuing thread's wait for that stage (1.5 s) runs
 * out; the block records SPD_ETIMEOUT, waits for the copies it did issue, frees its tensor memory and returns.
 * Returns what the device recorded.  SPD_ESTATE when the context has no long-prefix path (max_pos < 130 or a head
 * size other than 64 or 128).  The context stays usable: prefill it again.
 */
int spd_debug_expire_products(spd_ctx *ctx);

/*
 * Batched timesteps (the paper's closing remark that batching is complementary to Superposed Decoding: every
 * request of a batch still needs only one pass for its k drafts).  ctxs: HOST array of n different contexts
 * (1 <= n <= 128) over the same weights, device and stream, each prefilled on its own prefix, none with a stop
 * token; the first one lends its workspace and must have the long-prefix path (max_pos >= 130, head size 64 or
 * 128).  One timestep of all n requests streams the weights once: the requests' superposed inputs (Eq. 3) are the
 * token rows of the tensor-core products, each request keeps its own KV cache, position and draft state, and its
 * step is the one spd_step takes (Eq. 2-7).  spd_batch_generate enqueues n_steps timesteps and synchronises once;
 * every context can afterwards be read (spd_debug_read), stepped alone or in another batch.  spd_batch_step takes
 * one timestep and returns HOST rows of SPD_MAX_K entries per request (the first k used, any array may be NULL):
 * out_ids[r][i], out_parent[r][i], out_gamma[r][i] as spd_step gives them for request r.
 * SPD_ERANGE: n beyond 128 or the leading context without the long-prefix path, or a request out of positions;
 * SPD_EINVAL: contexts of different models, devices or streams, a context twice, a stop token configured;
 * SPD_ESTATE: a request not prefilled.  A device error of any request is returned (the first one found).
 */
int spd_batch_generate(spd_ctx *const *ctxs, int32_t n, int32_t n_steps);
int spd_batch_step(spd_ctx *const *ctxs, int32_t n, int32_t *out_ids, int32_t *out_parent, float *out_gamma);

/*
 * 1 once the most probable draft has ended with the stop token (cfg.eos_id; always 0 without one), as seen by the
 * last synchronising call.  spd_step / spd_generate / spd_generate_async then return SPD_ESTATE until the context is
 * prefilled or reset again.  The drafts stay readable; the paper does not say what happens to the other drafts.
 */
int spd_finished(const spd_ctx *ctx);

/* Number of kernel launches this context has enqueued so far. */
int64_t spd_launch_count(const spd_ctx *ctx);

/* Tuning knobs of the weight-streaming ring (bytes per stage, stages); 0 keeps the default.  Takes
 * effect from the next launch.  SPD_EINVAL if a matrix row does not fit a stage or shared memory
 * would overflow. */
int spd_set_ring(spd_ctx *ctx, int32_t stage_bytes, int32_t n_stages);

/* The ring spd_create chooses for a model (host only, no device needed): bytes per stage and stages of the decode
 * kernel's weight ring, for a context whose weights come with fragment-order images (with_images != 0) or without.
 * A stage takes two of the model's longest rows when four such stages fit beside the scratch area (and, with
 * images, the fragments of x), else one row (rows over 16 KB) or 32 KB.  SPD_EINVAL for an invalid configuration or
 * a row that fits no ring. */
int spd_ring_plan(const spd_config *cfg, int32_t with_images, int32_t *stage_bytes, int32_t *n_stages);

#ifdef __cplusplus
}
#endif
#endif /* SPD_H_ */
