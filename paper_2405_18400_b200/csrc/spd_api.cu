// Host side of the C ABI declared in include/spd.h: argument checks, workspace layout, launches.
#include <cuda.h>  // tensor-map types and the encoder's signature only; the entry point comes from the runtime
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "spd.h"
#include "spd_params.h"
#include "spd_prefill_tc.h"

extern "C" cudaError_t spd_internal_launch(const spd::KParams *p, int grid, size_t dyn_smem, cudaStream_t stream);
extern "C" cudaError_t spd_internal_prepare(size_t dyn_smem, int *blocks_per_sm);
extern "C" cudaError_t spd_internal_prefill_prepare(int *blocks_per_sm);
extern "C" cudaError_t spd_internal_prefill_launch(const spd::KParams *p, int grid, cudaStream_t stream);
extern "C" cudaError_t spd_internal_pack_image(const void *w, void *out, int rows, int cols, cudaStream_t stream);
extern "C" cudaError_t spd_internal_batch_step(const spd::TcJob *job, const spd::KParams *kps, int n, int V, const __nv_bfloat16 *final_norm,
                                               float *y_logits, size_t y_floats, size_t y_logits_floats, float *ss, int32_t *results,
                                               int sm_count, cudaStream_t s, int *launches);

namespace {

thread_local char g_cuda_err[256] = "";

int cuda_fail(cudaError_t e, const char *what) {
  std::snprintf(g_cuda_err, sizeof g_cuda_err, "%s: %s", what, cudaGetErrorString(e));
  cudaGetLastError();
  return SPD_ECUDA;
}
#define SPD_CUDA(call)                                 \
  do {                                                 \
    cudaError_t e_ = (call);                           \
    if (e_ != cudaSuccess) return cuda_fail(e_, #call); \
  } while (0)

constexpr size_t kPartBytes = spd::kScratchBytes;  // per-block scratch after the ring: row partials / attention merge / tail
constexpr size_t kSmemLimit = 232448; // 227 KB opt-in maximum per block on sm_100

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Layout {
  size_t kcache, vcache, rope, layers, h, q, u, logits, opart, oml, pk_val, pk_id, pk_ms, state, hist_tok, hist_par, prefix,
      trace, ns_u, pf_tmaps, pf_h, pf_q, pf_ss, pf_part, pf_ml, pf_cnt, pf_xh, pf_xo, pf_xu, tc_tmaps, tc_h, tc_q, tc_y, tc_x, bt_kp, bt_y,
      bt_ss, bt_out, total;
};

// Tokens one long-prefix job takes at most (0: the context never runs one): prefixes of more than 64 tokens send
// all but their last 1..16 tokens through the tensor-core path.
int tc_rows(const spd_config &c) {
  const int hd = c.d_model / c.n_heads;
  if (hd != 64 && hd != 128) return 0;  // the head sizes its attention kernel is built for
  const int full = (c.max_pos - 2) / spd::kTcTile * spd::kTcTile;
  return full < spd::kTcMaxTokens ? full : spd::kTcMaxTokens;
}

bool valid_config(const spd_config *c) {
  if (!c) return false;
  if (c->n_layers < 1 || c->d_model < 8 || c->n_heads < 1 || c->d_ffn < 8 || c->vocab < 1 || c->max_pos < 2) return false;
  if (c->d_model % 8 || c->d_ffn % 8 || c->d_model % c->n_heads) return false;
  const int hd = c->d_model / c->n_heads;
  if (hd % 32 || hd > 256) return false;
  if (c->vocab > 65535) return false;
  if (c->d_model > spd::kMaxVec * spd::kConsumerThreads * 8 || c->d_ffn > spd::kMaxVec * spd::kConsumerThreads * 8) return false;
  if (c->k < 1 || c->k > SPD_MAX_K) return false;
  if (c->n_min < 2 || c->n_max > SPD_MAX_N) return false;
  if (!(c->tau > 0.f) || !(c->delta > 0.f) || c->delta > 1.f || !(c->alpha >= 0.f) || c->alpha > 1.f) return false;
  if (!(c->rms_eps >= 0.f) || !(c->rope_theta > 0.f)) return false;
  if (c->eos_id < -1 || c->eos_id >= c->vocab) return false;
  if (c->kv_dtype != 0 && c->kv_dtype != 1) return false;
  return true;
}

// Bytes of a prefill fragment buffer for C columns: per 16 columns, 2 token tiles x 3 terms x 32 lanes x 8 bytes.
size_t frag_bytes(int C) { return (size_t)((C + 15) / 16) * 2 * 3 * 32 * 8; }

Layout make_layout(const spd_config &c, int grid) {
  Layout L{};
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t at = off;
    off = align_up(off + bytes, 256);
    return at;
  };
  const size_t kvb = (size_t)c.n_layers * c.max_pos * c.d_model * (c.kv_dtype ? 2 : 4);
  const int hd = c.d_model / c.n_heads;
  L.kcache = take(kvb);
  L.vcache = take(kvb);
  L.rope = take((size_t)c.max_pos * (hd / 2) * sizeof(float2));
  L.layers = take((size_t)c.n_layers * sizeof(spd::LayerW));
  L.h = take((size_t)c.d_model * 4);
  L.q = take((size_t)c.d_model * 4);
  L.u = take((size_t)c.d_ffn * 4);
  L.logits = take((size_t)c.vocab * 4);
  L.opart = take((size_t)c.n_heads * spd::kMaxSplit * hd * 4);
  L.oml = take((size_t)c.n_heads * spd::kMaxSplit * sizeof(float2));
  L.pk_val = take((size_t)grid * c.k * 4);
  L.pk_id = take((size_t)grid * c.k * 4);
  L.pk_ms = take((size_t)grid * sizeof(float2));
  L.state = take(sizeof(spd::State));
  L.hist_tok = take((size_t)c.max_pos * c.k * 4);
  L.hist_par = take((size_t)c.max_pos * c.k * 4);
  L.prefix = take((size_t)c.max_pos * 4);
  L.trace = take((size_t)c.n_layers * 2 * c.d_model * 4);
  L.ns_u = take((size_t)c.max_pos * 4);
  L.pf_tmaps = take((size_t)(4 * c.n_layers + 1) * sizeof(CUtensorMap));
  L.pf_h = take((size_t)spd::kPfTokens * c.d_model * 4);
  L.pf_q = take((size_t)spd::kPfTokens * c.d_model * 4);
  L.pf_ss = take((size_t)grid * spd::kPfTokens * 4);
  L.pf_part = take((size_t)c.n_heads * 8 * spd::kPfTokens * hd * 4);
  L.pf_ml = take((size_t)c.n_heads * 8 * spd::kPfTokens * sizeof(float2));
  L.pf_cnt = take((size_t)c.n_heads * 2 * 4);
  L.pf_xh = take(frag_bytes(c.d_model));
  L.pf_xo = take(frag_bytes(c.d_model));
  L.pf_xu = take(frag_bytes(c.d_ffn));
  const size_t tcr = (size_t)tc_rows(c);
  const size_t wide = (size_t)(3 * c.d_model > 2 * c.d_ffn ? 3 * c.d_model : 2 * c.d_ffn);
  L.tc_tmaps = take(8 * sizeof(CUtensorMap));  // term buffer as [..][d] and [..][f] in boxes of 128, 16, 32 and 64 rows
  L.tc_h = take(tcr * c.d_model * 4);
  L.tc_q = take(tcr * c.d_model * 4);
  L.tc_y = take(tcr * wide * 4);
  L.tc_x = take(3 * tcr * (size_t)(c.d_model > c.d_ffn ? c.d_model : c.d_ffn) * 2);
  // batched timesteps led by this context: the requests' parameters and their rows of logits
  L.bt_kp = take(tcr ? (size_t)spd::kTcTile * sizeof(spd::KParams) : 0);
  L.bt_y = take(tcr ? (size_t)spd::kTcTile * c.vocab * 4 : 0);
  L.bt_ss = take(tcr ? (size_t)spd::kTcTile * 32 * 4 : 0);  // per request and 512-column chunk: sums of squares of the residual row
  L.bt_out = take(tcr ? (size_t)spd::kTcTile * spd::kBtResultWords * 4 : 0);  // per request: a timestep's results
  L.total = off;
  return L;
}

// Tensor map of a bf16 matrix [rows][cols] for the prefill kernel's tiled copies: boxes of 64 columns x 32 rows
// (128 bytes per row), 128-byte shared-memory swizzle, zeros outside the matrix.
using TensorMapEncode = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                     const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                     CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool weight_map(TensorMapEncode encode, const void *w, int rows, int cols, CUtensorMap *out) {
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {64, 32};
  const cuuint32_t step[2] = {1, 1};
  return encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(w), dims, strides, box, step,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map of the term buffer of the long-prefix path seen as a bf16 matrix [rows][cols]: boxes of 64 columns x
// box_rows rows, 128-byte swizzle, zeros outside.
bool term_map(TensorMapEncode encode, const void *x, int rows, int cols, int box_rows, CUtensorMap *out) {
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  const cuuint32_t step[2] = {1, 1};
  return encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(x), dims, strides, box, step,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static_assert(sizeof(CUtensorMap) == spd::kTensorMapBytes, "the prefill kernel steps through the tensor maps by this size");

constexpr int kLayoutGrid = 1024;  // workspace is sized for up to this many blocks

}  // namespace

struct spd_ctx {
  spd_config cfg;
  spd::KParams kp;
  Layout lay;
  uint8_t *ws;
  cudaStream_t stream;
  int device;
  int grid;
  size_t dyn_smem;
  bool prefilled;
  int32_t m;       // prefix length
  std::vector<int32_t> prefix;  // host copy of the prefix (spd_reset extends it)
  std::vector<spd::LayerW> layers_host;  // the layer table, for the long-prefix path's launches
  int tc_rows;     // tokens one long-prefix job takes (0: path unused)
  int32_t n_gen;   // tokens generated per draft
  bool stopped;    // the most probable draft ended with the stop token: no further steps until the next prefill
  bool decoding;   // the last launch was a run of decode steps (the device's token count is the one to take over)
  int64_t launches;
};

namespace {

// Shared memory behind the scratch area that the fragment-order multiply loop needs for the activation vector: 12
// vectors of 16 bytes per 32 columns.
size_t frag_bytes(const spd_config &c) { return (size_t)c.d_model / 32 * 192; }

// reserve: bytes of shared memory kept back behind the ring and the scratch area.
int pick_ring(const spd_config &c, int32_t stage_bytes, int32_t n_stages, size_t reserve, int32_t *out_stage, int32_t *out_n) {
  const size_t maxrow = (size_t)2 * (c.d_model > c.d_ffn ? c.d_model : c.d_ffn);
  if (reserve + kPartBytes + 4096 >= kSmemLimit) return SPD_EINVAL;
  const size_t avail = kSmemLimit - kPartBytes - 4096 - reserve;  // 4096: static shared memory and alignment slack
  size_t sb = stage_bytes > 0 ? (size_t)stage_bytes : 32768;
  if (stage_bytes <= 0) {
    // Default: a stage takes two of the longest rows when four such stages fit (a chunk of two rows halves the
    // float32 loop's cost per row of folding and handing back the stage: 7B shape 2.65 -> 2.58 ms per step; the
    // number of stages matters little from four on), else one row.
    // (13B shape, where four two-row stages do not fit: six one-row stages of 28 KB 4.56 ms per step, five stages
    // of 32 KB 4.64 ms, three two-row stages 4.66 ms)
    const size_t two = align_up(2 * maxrow, 1024);
    if (two > sb && avail / two >= 4) sb = two;
    else if (maxrow > sb / 2) sb = align_up(maxrow, 1024);
  }
  if (sb % 128 || sb < maxrow) return SPD_EINVAL;
  int ns = n_stages > 0 ? n_stages : (int)(avail / sb);
  if (ns > spd::kMaxStages) ns = spd::kMaxStages;
  if (ns < 2 || (size_t)ns * sb > avail) return SPD_EINVAL;
  *out_stage = (int32_t)sb;
  *out_n = ns;
  return SPD_OK;
}

// Waits for the stream and returns what the device recorded; with a stop token configured, also takes over the
// device's count of generated tokens and its stop flag (a launch may have ended before its last step).
int check_device_error(spd_ctx *ctx) {
  int32_t head[6] = {0, 0, 0, 0, 0, 0};  // stop, abort flag, err, err_info, win_len, n_gen
  static_assert(offsetof(spd::State, n_gen) - offsetof(spd::State, stop) == 5 * sizeof(int32_t), "the fields read here are adjacent");
  SPD_CUDA(cudaMemcpyAsync(head, ctx->ws + ctx->lay.state + offsetof(spd::State, stop), sizeof head, cudaMemcpyDeviceToHost,
                           ctx->stream));
  SPD_CUDA(cudaStreamSynchronize(ctx->stream));
  if (head[2] == 0 && ctx->cfg.eos_id >= 0 && ctx->decoding) {
    ctx->n_gen = head[5];
    if (head[0]) ctx->stopped = true;
  }
  return head[2];
}

// Bytes of the state's head that every launch zeroes: with `keep_err` (later launches of a multi-launch call)
// the error words of the earlier launches survive (the first error sticks), else they are cleared too.
size_t head_bytes(bool keep_err) { return keep_err ? offsetof(spd::State, err) : offsetof(spd::State, win_len); }

int launch(spd_ctx *ctx, int mode, int n_iters, int pos0, int step0) {
  spd::KParams &kp = ctx->kp;
  kp.mode = mode;
  kp.n_iters = n_iters;
  kp.pos0 = pos0;
  kp.step0 = step0;
  // barrier counters, abort flag and error word start from zero at every launch
  SPD_CUDA(cudaMemsetAsync(ctx->ws + ctx->lay.state, 0, head_bytes(false), ctx->stream));
  SPD_CUDA(spd_internal_launch(&kp, ctx->grid, ctx->dyn_smem, ctx->stream));
  ctx->launches += 1;
  return SPD_OK;
}

// The long-prefix path's view of a context (tokens and positions are filled in per job).
spd::TcJob tc_job(spd_ctx *ctx) {
  const spd::KParams &kp = ctx->kp;
  spd::TcJob job;
  job.L = kp.L; job.d = kp.d; job.H = kp.H; job.hd = kp.hd; job.f = kp.f; job.max_pos = kp.max_pos; job.kv_bf16 = kp.kv_bf16;
  job.eps = kp.eps;
  job.layers = ctx->layers_host.data();
  job.tok_emb = kp.tok_emb;
  job.w_tmaps = ctx->ws + ctx->lay.pf_tmaps;
  job.x_tmaps = ctx->ws + ctx->lay.tc_tmaps;
  job.kcache = kp.kcache; job.vcache = kp.vcache; job.rope = kp.rope;
  job.h = reinterpret_cast<float *>(ctx->ws + ctx->lay.tc_h);
  job.y = reinterpret_cast<float *>(ctx->ws + ctx->lay.tc_y);
  job.q = reinterpret_cast<float *>(ctx->ws + ctx->lay.tc_q);
  job.x = reinterpret_cast<uint16_t *>(ctx->ws + ctx->lay.tc_x);
  job.x_term_rows = ctx->tc_rows;
  job.st = kp.st;
  job.sm_count = ctx->grid;
  job.y_floats = (size_t)ctx->tc_rows * (size_t)(3 * kp.d > 2 * kp.f ? 3 * kp.d : 2 * kp.f);
  job.ss = reinterpret_cast<float *>(ctx->ws + ctx->lay.bt_ss);
  job.ids = nullptr;
  job.pos0 = job.n_tok = 0;
  return job;
}

// Runs prefix tokens [first, first + count) (positions alike), the last of which ends the prefix, through the
// prefill kernel, kPfTokens at a time: their keys and values enter the cache, and the last launch goes on to
// the LM head on the prefix's last token and the first timestep (Eq. 1).
int prefill_tokens(spd_ctx *ctx, int first, int count) {
  spd::KParams &kp = ctx->kp;
  int32_t *base = kp.prefix;
  int rc = SPD_OK;
  // Long run of tokens: all but the last 1..16 go through the tensor-core path, in jobs of up to tc_rows tokens.
  int tc_done = 0;
  if (ctx->tc_rows > 0 && count > spd::kTcMinPrefix) {
    const int tc_total = count - ((count - 1) % spd::kPfTokens + 1);
    SPD_CUDA(cudaMemsetAsync(ctx->ws + ctx->lay.state, 0, head_bytes(false), ctx->stream));
    spd::TcJob job = tc_job(ctx);
    while (tc_done < tc_total) {
      const int n = tc_total - tc_done < ctx->tc_rows ? tc_total - tc_done : ctx->tc_rows;
      job.ids = base + first + tc_done;
      job.pos0 = first + tc_done;
      job.n_tok = n;
      int launched = 0;
      const cudaError_t e = spd_internal_tc_prefill(&job, ctx->stream, &launched);
      ctx->launches += launched;
      if (e != cudaSuccess) return cuda_fail(e, "long-prefix launch");
      tc_done += n;
    }
    first += tc_done;
    count -= tc_done;
  }
  for (int done = 0; done < count && rc == SPD_OK; done += spd::kPfTokens) {
    const int n = count - done < spd::kPfTokens ? count - done : spd::kPfTokens;
    kp.mode = spd::kModePrefill;
    kp.n_iters = n;
    kp.pos0 = first + done;
    kp.step0 = 0;
    kp.pf_head = done + n == count ? 1 : 0;
    kp.prefix = base + first + done;
    cudaError_t e = cudaMemsetAsync(ctx->ws + ctx->lay.state, 0, head_bytes(done > 0 || tc_done > 0), ctx->stream);
    if (e == cudaSuccess) e = spd_internal_prefill_launch(&kp, ctx->grid, ctx->stream);
    if (e != cudaSuccess) rc = cuda_fail(e, "prefill launch");
    else ctx->launches += 1;
  }
  kp.prefix = base;
  kp.pf_head = 0;
  return rc;
}

int set_device(const spd_ctx *ctx) {
  int dev = -1;
  SPD_CUDA(cudaGetDevice(&dev));
  if (dev != ctx->device) SPD_CUDA(cudaSetDevice(ctx->device));
  return SPD_OK;
}

int read_state(spd_ctx *ctx, size_t field_off, void *dst, size_t bytes) {
  SPD_CUDA(cudaMemcpyAsync(dst, ctx->ws + ctx->lay.state + field_off, bytes, cudaMemcpyDeviceToHost, ctx->stream));
  return SPD_OK;
}

}  // namespace

extern "C" {

const char *spd_strerror(int status) {
  switch (status) {
    case SPD_OK: return "ok";
    case SPD_EINVAL: return "invalid argument";
    case SPD_ESTATE: return "call out of order (prefill first)";
    case SPD_ERANGE: return "value out of range";
    case SPD_ENOMEM: return "buffer too small";
    case SPD_ECUDA: return "CUDA runtime error";
    case SPD_ETABLE: return "n-gram table probe exceeded its bound";
    case SPD_ETIMEOUT: return "bounded device wait expired";
    default: return "unknown status";
  }
}

const char *spd_last_cuda_error(void) { return g_cuda_err; }

int spd_workspace_bytes(const spd_config *cfg, size_t *bytes) {
  if (!valid_config(cfg) || !bytes) return SPD_EINVAL;
  *bytes = make_layout(*cfg, kLayoutGrid).total;
  return SPD_OK;
}

int spd_create(const spd_config *cfg, const spd_weights *w, const spd_ngram_table *tables, int32_t n_tables, void *workspace,
               size_t workspace_bytes, spd_ctx **out) {
  if (!valid_config(cfg) || !w || !workspace || !out) return SPD_EINVAL;
  if (n_tables < 0 || n_tables > spd::kMaxTables || (n_tables > 0 && !tables)) return SPD_EINVAL;
  if ((uintptr_t)workspace % 256) return SPD_EINVAL;
  if (!w->tok_emb || !w->final_norm || !w->lm_head || !w->attn_norm || !w->wqkv || !w->wo || !w->ffn_norm || !w->wgate_up ||
      !w->wdown)
    return SPD_EINVAL;
  auto misaligned = [](const void *p) { return p == nullptr || ((uintptr_t)p % 16) != 0; };
  if (misaligned(w->tok_emb) || misaligned(w->final_norm) || misaligned(w->lm_head)) return SPD_EINVAL;
  for (int l = 0; l < cfg->n_layers; ++l)
    if (misaligned(w->attn_norm[l]) || misaligned(w->wqkv[l]) || misaligned(w->wo[l]) || misaligned(w->ffn_norm[l]) ||
        misaligned(w->wgate_up[l]) || misaligned(w->wdown[l]))
      return SPD_EINVAL;
  for (int t = 0; t < n_tables; ++t) {
    const spd_ngram_table &tb = tables[t];
    if (tb.n < 2 || tb.n > SPD_MAX_N || misaligned(tb.ngram) || misaligned(tb.ctx)) return SPD_EINVAL;
    if (!tb.ngram_slots || (tb.ngram_slots & (tb.ngram_slots - 1)) || !tb.ctx_slots || (tb.ctx_slots & (tb.ctx_slots - 1)))
      return SPD_EINVAL;
    for (int s = 0; s < t; ++s)
      if (tables[s].n >= tb.n) return SPD_EINVAL;  // ascending orders, one table per order
  }
  const Layout lay = make_layout(*cfg, kLayoutGrid);
  if (workspace_bytes < lay.total) return SPD_ENOMEM;

  spd_ctx *ctx = new (std::nothrow) spd_ctx();
  if (!ctx) return SPD_ENOMEM;
  ctx->cfg = *cfg;
  ctx->lay = lay;
  ctx->ws = static_cast<uint8_t *>(workspace);
  ctx->stream = static_cast<cudaStream_t>(cfg->stream);
  ctx->prefilled = false;
  ctx->decoding = false;
  ctx->stopped = ctx->decoding = false;
  ctx->m = ctx->n_gen = 0;
  ctx->launches = 0;
  auto fail = [&](int rc) {
    delete ctx;
    return rc;
  };
  cudaError_t e = cudaGetDevice(&ctx->device);
  if (e != cudaSuccess) return fail(cuda_fail(e, "cudaGetDevice"));
  cudaDeviceProp prop;
  e = cudaGetDeviceProperties(&prop, ctx->device);
  if (e != cudaSuccess) return fail(cuda_fail(e, "cudaGetDeviceProperties"));
  if (!prop.cooperativeLaunch) return fail(SPD_EINVAL);
  ctx->grid = prop.multiProcessorCount < kLayoutGrid ? prop.multiProcessorCount : kLayoutGrid;

  spd::KParams &kp = ctx->kp;
  std::memset(&kp, 0, sizeof kp);
  // Fragment-order images: all or none, and only for shapes the tensor-core multiply loop serves.
  bool img = w->lm_head_img && w->wqkv_img && w->wo_img && w->wgate_up_img && cfg->d_model % 32 == 0 && cfg->vocab % spd::kUnitRows == 0 &&
             (2 * cfg->d_ffn) % spd::kUnitRows == 0;
  for (int l = 0; l < cfg->n_layers && img; ++l) img = w->wqkv_img[l] && w->wo_img[l] && w->wgate_up_img[l];
  int rc = pick_ring(*cfg, 0, 0, img ? frag_bytes(*cfg) : 0, &kp.stage_bytes, &kp.n_stages);
  if (rc && img) {  // no room for the fragments: the float32 multiply loop
    img = false;
    rc = pick_ring(*cfg, 0, 0, 0, &kp.stage_bytes, &kp.n_stages);
  }
  if (rc) return fail(rc);
  ctx->dyn_smem = (size_t)kp.stage_bytes * kp.n_stages + kPartBytes + (img ? frag_bytes(*cfg) : 0);
  int per_sm = 0;
  e = spd_internal_prepare(ctx->dyn_smem, &per_sm);
  if (e != cudaSuccess) return fail(cuda_fail(e, "kernel attributes"));
  if (per_sm < 1) return fail(SPD_EINVAL);
  e = spd_internal_prefill_prepare(&per_sm);
  if (e != cudaSuccess) return fail(cuda_fail(e, "prefill kernel attributes"));
  if (per_sm < 1) return fail(SPD_EINVAL);
  ctx->tc_rows = tc_rows(*cfg);
  if (ctx->tc_rows > 0) {
    e = spd_internal_tc_prepare();
    if (e != cudaSuccess) return fail(cuda_fail(e, "long-prefix kernel attributes"));
  }

  const int hd = cfg->d_model / cfg->n_heads;
  kp.L = cfg->n_layers; kp.d = cfg->d_model; kp.H = cfg->n_heads; kp.hd = hd; kp.f = cfg->d_ffn; kp.V = cfg->vocab;
  kp.max_pos = cfg->max_pos; kp.eps = cfg->rms_eps; kp.kv_bf16 = cfg->kv_dtype;
  kp.tok_emb = static_cast<const __nv_bfloat16 *>(w->tok_emb);
  kp.final_norm = static_cast<const __nv_bfloat16 *>(w->final_norm);
  kp.lm_head = static_cast<const __nv_bfloat16 *>(w->lm_head);
  kp.k = cfg->k; kp.n_min = cfg->n_min; kp.n_max = cfg->n_max; kp.n_tables = n_tables;
  for (int i = 0; i < 8; ++i) kp.lambda[i] = cfg->lambda[i];
  kp.alpha = cfg->alpha;
  kp.inv_tau = 1.0f / cfg->tau;
  kp.log_delta = std::log(cfg->delta);
  for (int t = 0; t < n_tables; ++t) {
    kp.tab[t].n = tables[t].n;
    kp.tab[t].ngram = static_cast<const SpdSlot *>(tables[t].ngram);
    kp.tab[t].ctx = static_cast<const SpdSlot *>(tables[t].ctx);
    kp.tab[t].ngram_mask = tables[t].ngram_slots - 1;
    kp.tab[t].ctx_mask = tables[t].ctx_slots - 1;
  }
  uint8_t *ws = ctx->ws;
  kp.kcache = ws + lay.kcache; kp.vcache = ws + lay.vcache;
  kp.rope = reinterpret_cast<const float2 *>(ws + lay.rope);
  kp.layers = reinterpret_cast<const spd::LayerW *>(ws + lay.layers);
  kp.h = reinterpret_cast<float *>(ws + lay.h); kp.q = reinterpret_cast<float *>(ws + lay.q);
  kp.u = reinterpret_cast<float *>(ws + lay.u); kp.logits = reinterpret_cast<float *>(ws + lay.logits);
  kp.opart = reinterpret_cast<float *>(ws + lay.opart); kp.oml = reinterpret_cast<float2 *>(ws + lay.oml);
  kp.pk_val = reinterpret_cast<float *>(ws + lay.pk_val); kp.pk_id = reinterpret_cast<int32_t *>(ws + lay.pk_id);
  kp.pk_ms = reinterpret_cast<float2 *>(ws + lay.pk_ms);
  kp.st = reinterpret_cast<spd::State *>(ws + lay.state);
  kp.hist_tok = reinterpret_cast<int32_t *>(ws + lay.hist_tok); kp.hist_par = reinterpret_cast<int32_t *>(ws + lay.hist_par);
  kp.prefix = reinterpret_cast<int32_t *>(ws + lay.prefix);
  kp.ns_u = reinterpret_cast<const float *>(ws + lay.ns_u);
  kp.trace = nullptr;  // the per-layer residual trace is test instrumentation: spd_debug_trace switches it on
  kp.pf_h = reinterpret_cast<float *>(ws + lay.pf_h); kp.pf_q = reinterpret_cast<float *>(ws + lay.pf_q);
  kp.pf_xh = reinterpret_cast<uint16_t *>(ws + lay.pf_xh); kp.pf_xo = reinterpret_cast<uint16_t *>(ws + lay.pf_xo);
  kp.pf_xu = reinterpret_cast<uint16_t *>(ws + lay.pf_xu);
  kp.pf_tmaps = ws + lay.pf_tmaps;
  kp.pf_ss = reinterpret_cast<float *>(ws + lay.pf_ss);
  kp.pf_part = reinterpret_cast<float *>(ws + lay.pf_part); kp.pf_ml = reinterpret_cast<float2 *>(ws + lay.pf_ml);
  kp.pf_cnt = reinterpret_cast<unsigned int *>(ws + lay.pf_cnt);
  kp.eos_id = cfg->eos_id;

  // rotary table: cos / sin of pos * theta^(-2i/hd), evaluated in double and rounded once
  std::vector<float2> rope((size_t)cfg->max_pos * (hd / 2));
  for (int pos = 0; pos < cfg->max_pos; ++pos)
    for (int i = 0; i < hd / 2; ++i) {
      const double ang = (double)pos * std::pow((double)cfg->rope_theta, -2.0 * i / hd);
      rope[(size_t)pos * (hd / 2) + i] = make_float2((float)std::cos(ang), (float)std::sin(ang));
    }
  std::vector<spd::LayerW> layers(cfg->n_layers);
  for (int l = 0; l < cfg->n_layers; ++l) {
    layers[l].attn_norm = static_cast<const __nv_bfloat16 *>(w->attn_norm[l]);
    layers[l].wqkv = static_cast<const __nv_bfloat16 *>(w->wqkv[l]);
    layers[l].wo = static_cast<const __nv_bfloat16 *>(w->wo[l]);
    layers[l].ffn_norm = static_cast<const __nv_bfloat16 *>(w->ffn_norm[l]);
    layers[l].wgate_up = static_cast<const __nv_bfloat16 *>(w->wgate_up[l]);
    layers[l].wdown = static_cast<const __nv_bfloat16 *>(w->wdown[l]);
    layers[l].wqkv_img = layers[l].wo_img = layers[l].wgate_up_img = nullptr;
  }
  if (img) {
    for (int l = 0; l < cfg->n_layers; ++l) {
      layers[l].wqkv_img = static_cast<const __nv_bfloat16 *>(w->wqkv_img[l]);
      layers[l].wo_img = static_cast<const __nv_bfloat16 *>(w->wo_img[l]);
      layers[l].wgate_up_img = static_cast<const __nv_bfloat16 *>(w->wgate_up_img[l]);
    }
    kp.lm_head_img = static_cast<const __nv_bfloat16 *>(w->lm_head_img);
  }
  // tensor maps of the matrices in the order the prefill kernel walks them
  std::vector<CUtensorMap> tmaps((size_t)4 * cfg->n_layers + 1);
  CUtensorMap xmaps[8];
  std::memset(xmaps, 0, sizeof xmaps);
  ctx->layers_host = layers;
  {
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult found = cudaDriverEntryPointSymbolNotFound;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &found);
    if (e != cudaSuccess) return fail(cuda_fail(e, "cudaGetDriverEntryPoint(cuTensorMapEncodeTiled)"));
    if (found != cudaDriverEntryPointSuccess || !fn) return fail(SPD_EINVAL);
    const TensorMapEncode encode = reinterpret_cast<TensorMapEncode>(fn);
    const int d = cfg->d_model, f = cfg->d_ffn;
    bool ok = true;
    for (int l = 0; l < cfg->n_layers && ok; ++l) {
      ok = weight_map(encode, w->wqkv[l], 3 * d, d, &tmaps[4 * l]) && weight_map(encode, w->wo[l], d, d, &tmaps[4 * l + 1]) &&
           weight_map(encode, w->wgate_up[l], 2 * f, d, &tmaps[4 * l + 2]) && weight_map(encode, w->wdown[l], d, f, &tmaps[4 * l + 3]);
    }
    ok = ok && weight_map(encode, w->lm_head, cfg->vocab, d, &tmaps[(size_t)4 * cfg->n_layers]);
    if (ok && ctx->tc_rows > 0)
      for (int i = 0; i < 4 && ok; ++i) {
        const int box_rows = i == 0 ? spd::kTcTile : 8 << i;  // 128, then 16, 32, 64 for the products of a small batch
        ok = term_map(encode, ws + lay.tc_x, 3 * ctx->tc_rows, d, box_rows, &xmaps[2 * i]) &&
             term_map(encode, ws + lay.tc_x, 3 * ctx->tc_rows, f, box_rows, &xmaps[2 * i + 1]);
      }
    if (!ok) return fail(SPD_EINVAL);
  }
  cudaStream_t s = ctx->stream;
  e = cudaMemcpyAsync(ws + lay.pf_tmaps, tmaps.data(), tmaps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(ws + lay.rope, rope.data(), rope.size() * sizeof(float2), cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(ws + lay.layers, layers.data(), layers.size() * sizeof(spd::LayerW), cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(ws + lay.state, 0, sizeof(spd::State), s);
  if (e == cudaSuccess) e = cudaMemsetAsync(ws + lay.trace, 0, (size_t)cfg->n_layers * 2 * cfg->d_model * 4, s);
  // columns past the row's end inside the last 16-column step of a fragment buffer are never written: zero
  if (e == cudaSuccess) e = cudaMemsetAsync(ws + lay.pf_cnt, 0, lay.tc_tmaps - lay.pf_cnt, s);  // also the arrival counters
  if (e == cudaSuccess) e = cudaMemcpyAsync(ws + lay.tc_tmaps, xmaps, sizeof xmaps, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return fail(cuda_fail(e, "workspace initialisation"));
  *out = ctx;
  return SPD_OK;
}

int spd_destroy(spd_ctx *ctx) {
  delete ctx;
  return SPD_OK;
}

int spd_ring_plan(const spd_config *cfg, int32_t with_images, int32_t *stage_bytes, int32_t *n_stages) {
  if (!valid_config(cfg) || !stage_bytes || !n_stages) return SPD_EINVAL;
  return pick_ring(*cfg, 0, 0, with_images ? frag_bytes(*cfg) : 0, stage_bytes, n_stages);
}

int spd_set_ring(spd_ctx *ctx, int32_t stage_bytes, int32_t n_stages) {
  if (!ctx) return SPD_EINVAL;
  int32_t sb, ns;
  const size_t reserve = ctx->kp.lm_head_img ? frag_bytes(ctx->cfg) : 0;
  int rc = pick_ring(ctx->cfg, stage_bytes, n_stages, reserve, &sb, &ns);
  if (rc) return rc;
  if ((rc = set_device(ctx))) return rc;
  const size_t dyn = (size_t)sb * ns + kPartBytes + reserve;
  int per_sm = 0;
  SPD_CUDA(spd_internal_prepare(dyn > ctx->dyn_smem ? dyn : ctx->dyn_smem, &per_sm));
  if (per_sm < 1) return SPD_EINVAL;
  ctx->kp.stage_bytes = sb;
  ctx->kp.n_stages = ns;
  ctx->dyn_smem = dyn;
  return SPD_OK;
}

int spd_prefill(spd_ctx *ctx, const int32_t *prefix_ids, int32_t m, int32_t *out_ids, float *out_gamma) {
  if (!ctx || !prefix_ids) return SPD_EINVAL;
  const spd_config &c = ctx->cfg;
  if (m < 1 || m >= c.max_pos) return SPD_ERANGE;
  for (int i = 0; i < m; ++i)
    if (prefix_ids[i] < 0 || prefix_ids[i] >= c.vocab) return SPD_ERANGE;
  int rc = set_device(ctx);
  if (rc) return rc;
  // fresh draft state: every history window holds the end of the prefix
  spd::State st;
  std::memset(&st, 0, sizeof st);
  st.win_len = m < spd::kWin ? m : spd::kWin;
  for (int i = 0; i < c.k; ++i)
    for (int j = 0; j < st.win_len; ++j) st.win[i][spd::kWin - st.win_len + j] = prefix_ids[m - st.win_len + j];
  SPD_CUDA(cudaMemcpyAsync(ctx->ws + ctx->lay.state, &st, sizeof st, cudaMemcpyHostToDevice, ctx->stream));
  SPD_CUDA(cudaMemcpyAsync(ctx->ws + ctx->lay.prefix, prefix_ids, (size_t)m * 4, cudaMemcpyHostToDevice, ctx->stream));
  SPD_CUDA(cudaStreamSynchronize(ctx->stream));  // st and the caller's ids may go out of scope
  ctx->prefilled = false;
  ctx->decoding = false;
  if ((rc = prefill_tokens(ctx, 0, m))) return rc;
  int32_t ids[SPD_MAX_K];
  float gamma[SPD_MAX_K];
  if ((rc = read_state(ctx, offsetof(spd::State, cand_tok), ids, sizeof ids))) return rc;
  if ((rc = read_state(ctx, offsetof(spd::State, gamma), gamma, sizeof gamma))) return rc;
  if ((rc = check_device_error(ctx))) return rc;
  ctx->prefilled = true;
  ctx->m = m;
  ctx->n_gen = 1;
  ctx->stopped = c.eos_id >= 0 && ids[0] == c.eos_id;
  ctx->prefix.assign(prefix_ids, prefix_ids + m);
  for (int i = 0; i < c.k; ++i) {
    if (out_ids) out_ids[i] = ids[i];
    if (out_gamma) out_gamma[i] = gamma[i];
  }
  return SPD_OK;
}

int spd_reset(spd_ctx *ctx, int32_t draft, int32_t *out_ids, float *out_gamma) {
  if (!ctx) return SPD_EINVAL;
  if (!ctx->prefilled) return SPD_ESTATE;
  const spd_config &c = ctx->cfg;
  if (draft < 0 || draft >= c.k) return SPD_ERANGE;
  const int k = c.k, n = ctx->n_gen, m = ctx->m;
  if (m + n >= c.max_pos) return SPD_ERANGE;
  int rc = set_device(ctx);
  if (rc) return rc;
  // the chosen draft's tokens, by its parent links
  std::vector<int32_t> tok((size_t)n * k), par((size_t)n * k), seq(n);
  SPD_CUDA(cudaMemcpyAsync(tok.data(), ctx->ws + ctx->lay.hist_tok, tok.size() * 4, cudaMemcpyDeviceToHost, ctx->stream));
  SPD_CUDA(cudaMemcpyAsync(par.data(), ctx->ws + ctx->lay.hist_par, par.size() * 4, cudaMemcpyDeviceToHost, ctx->stream));
  if ((rc = spd_sync(ctx))) return rc;
  for (int s = n - 1, cur = draft; s >= 0; --s) {
    seq[s] = tok[(size_t)s * k + cur];
    cur = par[(size_t)s * k + cur];
  }
  ctx->prefix.insert(ctx->prefix.end(), seq.begin(), seq.end());
  const int m2 = m + n;
  // fresh draft state on the longer prefix; positions 0..m-1 of the cache stay, positions m..m2-1 (so far
  // computed from superposed inputs) are recomputed from the draft's own tokens
  spd::State st;
  std::memset(&st, 0, sizeof st);
  st.win_len = m2 < spd::kWin ? m2 : spd::kWin;
  for (int i = 0; i < k; ++i)
    for (int j = 0; j < st.win_len; ++j) st.win[i][spd::kWin - st.win_len + j] = ctx->prefix[m2 - st.win_len + j];
  SPD_CUDA(cudaMemcpyAsync(ctx->ws + ctx->lay.state, &st, sizeof st, cudaMemcpyHostToDevice, ctx->stream));
  SPD_CUDA(cudaMemcpyAsync(ctx->ws + ctx->lay.prefix + (size_t)m * 4, seq.data(), (size_t)n * 4, cudaMemcpyHostToDevice, ctx->stream));
  SPD_CUDA(cudaStreamSynchronize(ctx->stream));
  ctx->prefilled = false;
  ctx->decoding = false;
  if ((rc = prefill_tokens(ctx, m, n))) return rc;
  int32_t ids[SPD_MAX_K];
  float gamma[SPD_MAX_K];
  if ((rc = read_state(ctx, offsetof(spd::State, cand_tok), ids, sizeof ids))) return rc;
  if ((rc = read_state(ctx, offsetof(spd::State, gamma), gamma, sizeof gamma))) return rc;
  if ((rc = check_device_error(ctx))) return rc;
  ctx->prefilled = true;
  ctx->m = m2;
  ctx->n_gen = 1;
  ctx->stopped = c.eos_id >= 0 && ids[0] == c.eos_id;
  for (int i = 0; i < k; ++i) {
    if (out_ids) out_ids[i] = ids[i];
    if (out_gamma) out_gamma[i] = gamma[i];
  }
  return SPD_OK;
}

int spd_sample(spd_ctx *ctx, int32_t n_new, float top_p, float temperature, const float *uniforms, int32_t *out_new,
               int32_t *out_ids, float *out_gamma) {
  if (!ctx || !uniforms) return SPD_EINVAL;
  if (!ctx->prefilled || ctx->n_gen != 1) return SPD_ESTATE;
  const spd_config &c = ctx->cfg;
  const int m = ctx->m;
  if (n_new < 1 || m + n_new >= c.max_pos) return SPD_ERANGE;
  if (!(top_p > 0.f) || top_p > 1.f || !(temperature > 0.f)) return SPD_ERANGE;
  for (int i = 0; i < n_new; ++i)
    if (!(uniforms[i] >= 0.f) || !(uniforms[i] < 1.f)) return SPD_ERANGE;
  int rc = set_device(ctx);
  if (rc) return rc;
  SPD_CUDA(cudaMemcpyAsync(ctx->ws + ctx->lay.ns_u, uniforms, (size_t)n_new * 4, cudaMemcpyHostToDevice, ctx->stream));
  SPD_CUDA(cudaStreamSynchronize(ctx->stream));  // the caller's array may go out of scope
  ctx->prefilled = false;
  ctx->decoding = false;
  // pass i draws token m + i from the logits of the pass before (the first from those the prefill left),
  // feeds it at position m + i; the last pass ends with the first-timestep decision
  spd::KParams &kp = ctx->kp;
  int32_t *base = kp.prefix;
  kp.prefix = base + m;
  kp.ns_p = top_p;
  kp.ns_inv_temp = 1.0f / temperature;
  rc = launch(ctx, spd::kModeSample, n_new, m, 0);
  kp.prefix = base;
  if (rc) return rc;
  std::vector<int32_t> fresh(n_new);
  int32_t ids[SPD_MAX_K];
  float gamma[SPD_MAX_K];
  SPD_CUDA(cudaMemcpyAsync(fresh.data(), ctx->ws + ctx->lay.prefix + (size_t)m * 4, (size_t)n_new * 4, cudaMemcpyDeviceToHost,
                           ctx->stream));
  if ((rc = read_state(ctx, offsetof(spd::State, cand_tok), ids, sizeof ids))) return rc;
  if ((rc = read_state(ctx, offsetof(spd::State, gamma), gamma, sizeof gamma))) return rc;
  if ((rc = check_device_error(ctx))) return rc;
  ctx->prefix.insert(ctx->prefix.end(), fresh.begin(), fresh.end());
  ctx->prefilled = true;
  ctx->m = m + n_new;
  ctx->n_gen = 1;
  ctx->stopped = c.eos_id >= 0 && ids[0] == c.eos_id;
  for (int i = 0; i < n_new; ++i)
    if (out_new) out_new[i] = fresh[i];
  for (int i = 0; i < c.k; ++i) {
    if (out_ids) out_ids[i] = ids[i];
    if (out_gamma) out_gamma[i] = gamma[i];
  }
  return SPD_OK;
}

int spd_generate_async(spd_ctx *ctx, int32_t n_steps) {
  if (!ctx) return SPD_EINVAL;
  if (!ctx->prefilled || ctx->stopped) return SPD_ESTATE;
  if (n_steps < 1) return SPD_ERANGE;
  const int pos0 = ctx->m + ctx->n_gen - 1;  // position of the first superposed input of this launch
  if (pos0 + n_steps > ctx->cfg.max_pos || ctx->n_gen + n_steps > ctx->cfg.max_pos) return SPD_ERANGE;
  int rc = set_device(ctx);
  if (rc) return rc;
  if ((rc = launch(ctx, spd::kModeDecode, n_steps, pos0, ctx->n_gen))) return rc;
  ctx->n_gen += n_steps;  // with a stop token: until spd_sync reads the device's count
  ctx->decoding = true;
  return SPD_OK;
}

int spd_sync(spd_ctx *ctx) {
  if (!ctx) return SPD_EINVAL;
  int rc = set_device(ctx);
  if (rc) return rc;
  rc = check_device_error(ctx);
  if (rc) ctx->prefilled = false;
  return rc;
}

int spd_step(spd_ctx *ctx, int32_t *out_ids, int32_t *out_parent, float *out_gamma) {
  int rc = spd_generate_async(ctx, 1);
  if (rc) return rc;
  const int k = ctx->cfg.k;
  int32_t ids[SPD_MAX_K], par[SPD_MAX_K];
  float gamma[SPD_MAX_K];
  const size_t row = (size_t)(ctx->n_gen - 1) * k * 4;  // a launch always completes its first step
  SPD_CUDA(cudaMemcpyAsync(ids, ctx->ws + ctx->lay.hist_tok + row, (size_t)k * 4, cudaMemcpyDeviceToHost, ctx->stream));
  SPD_CUDA(cudaMemcpyAsync(par, ctx->ws + ctx->lay.hist_par + row, (size_t)k * 4, cudaMemcpyDeviceToHost, ctx->stream));
  if ((rc = read_state(ctx, offsetof(spd::State, gamma), gamma, sizeof gamma))) return rc;
  if ((rc = spd_sync(ctx))) return rc;
  for (int i = 0; i < k; ++i) {
    if (out_ids) out_ids[i] = ids[i];
    if (out_parent) out_parent[i] = par[i];
    if (out_gamma) out_gamma[i] = gamma[i];
  }
  return SPD_OK;
}

int spd_generate(spd_ctx *ctx, int32_t n_steps, int32_t *out_tokens, int32_t *out_len, float *out_logp, float *out_gamma) {
  int rc = spd_generate_async(ctx, n_steps);
  if (rc) return rc;
  if ((rc = spd_sync(ctx))) return rc;  // with a stop token the run may have ended early: n_gen is the device's from here on
  const int k = ctx->cfg.k, len = ctx->n_gen;
  std::vector<int32_t> tok((size_t)len * k), par((size_t)len * k);
  float logp[SPD_MAX_K], gamma[SPD_MAX_K];
  SPD_CUDA(cudaMemcpyAsync(tok.data(), ctx->ws + ctx->lay.hist_tok, tok.size() * 4, cudaMemcpyDeviceToHost, ctx->stream));
  SPD_CUDA(cudaMemcpyAsync(par.data(), ctx->ws + ctx->lay.hist_par, par.size() * 4, cudaMemcpyDeviceToHost, ctx->stream));
  if ((rc = read_state(ctx, offsetof(spd::State, logP), logp, sizeof logp))) return rc;
  if ((rc = read_state(ctx, offsetof(spd::State, gamma), gamma, sizeof gamma))) return rc;
  SPD_CUDA(cudaStreamSynchronize(ctx->stream));
  if (out_tokens) {
    // follow each surviving draft's parent links back to the first timestep
    for (int r = 0; r < k; ++r) {
      int cur = r;
      for (int s = len - 1; s >= 0; --s) {
        out_tokens[(size_t)r * len + s] = tok[(size_t)s * k + cur];
        cur = par[(size_t)s * k + cur];
      }
    }
  }
  if (out_len) *out_len = len;
  for (int i = 0; i < k; ++i) {
    if (out_logp) out_logp[i] = logp[i];
    if (out_gamma) out_gamma[i] = gamma[i];
  }
  return SPD_OK;
}

namespace {

// Checks a batch and enqueues n_steps timesteps of it; the requests' host-side counters move on.
int batch_enqueue(spd_ctx *const *ctxs, int32_t n, int32_t n_steps) {
  if (!ctxs || n < 1 || !ctxs[0]) return SPD_EINVAL;
  spd_ctx *lead = ctxs[0];
  if (lead->tc_rows < 1 || n > spd::kTcTile || n > lead->tc_rows) return SPD_ERANGE;
  if (n_steps < 1) return SPD_ERANGE;
  const spd_config &c0 = lead->cfg;
  for (int r = 0; r < n; ++r) {
    spd_ctx *x = ctxs[r];
    if (!x) return SPD_EINVAL;
    for (int q = 0; q < r; ++q)
      if (ctxs[q] == x) return SPD_EINVAL;  // a request appears once
    const spd_config &c = x->cfg;
    if (c.n_layers != c0.n_layers || c.d_model != c0.d_model || c.n_heads != c0.n_heads || c.d_ffn != c0.d_ffn || c.vocab != c0.vocab ||
        c.rms_eps != c0.rms_eps || x->device != lead->device || x->stream != lead->stream || x->kp.tok_emb != lead->kp.tok_emb ||
        x->kp.lm_head != lead->kp.lm_head || x->layers_host[0].wqkv != lead->layers_host[0].wqkv)
      return SPD_EINVAL;  // one model, one device, one stream
    if (c.eos_id != -1) return SPD_EINVAL;  // stopping on a token is a single-request feature
    if (!x->prefilled || x->stopped) return SPD_ESTATE;
    const int pos0 = x->m + x->n_gen - 1;
    if (pos0 + n_steps > c.max_pos || x->n_gen + n_steps > c.max_pos) return SPD_ERANGE;
  }
  int rc = set_device(lead);
  if (rc) return rc;
  // the requests' parameters in row order; pos0 = m - 1, so that a request's next position is pos0 + n_gen on the device
  std::vector<spd::KParams> kps(n);
  for (int r = 0; r < n; ++r) {
    kps[r] = ctxs[r]->kp;
    kps[r].pos0 = ctxs[r]->m - 1;
    SPD_CUDA(cudaMemsetAsync(ctxs[r]->ws + ctxs[r]->lay.state, 0, head_bytes(false), lead->stream));
  }
  spd::KParams *dkp = reinterpret_cast<spd::KParams *>(lead->ws + lead->lay.bt_kp);
  SPD_CUDA(cudaMemcpyAsync(dkp, kps.data(), kps.size() * sizeof(spd::KParams), cudaMemcpyHostToDevice, lead->stream));
  SPD_CUDA(cudaStreamSynchronize(lead->stream));  // `kps` leaves scope
  const spd::TcJob job = tc_job(lead);
  for (int s = 0; s < n_steps; ++s) {
    int launched = 0;
    const int wide = 3 * c0.d_model > 2 * c0.d_ffn ? 3 * c0.d_model : 2 * c0.d_ffn;
    const cudaError_t e = spd_internal_batch_step(&job, dkp, n, c0.vocab, lead->kp.final_norm,
                                                  reinterpret_cast<float *>(lead->ws + lead->lay.bt_y), (size_t)lead->tc_rows * wide,
                                                  (size_t)spd::kTcTile * c0.vocab, reinterpret_cast<float *>(lead->ws + lead->lay.bt_ss),
                                                  reinterpret_cast<int32_t *>(lead->ws + lead->lay.bt_out), lead->grid, lead->stream, &launched);
    lead->launches += launched;
    if (e != cudaSuccess) return cuda_fail(e, "batched timestep");
  }
  for (int r = 0; r < n; ++r) {
    ctxs[r]->n_gen += n_steps;
    ctxs[r]->decoding = false;
  }
  return SPD_OK;
}

int batch_wait(spd_ctx *const *ctxs, int32_t n) {
  int first = SPD_OK;
  for (int r = 0; r < n; ++r) {
    const int rc = check_device_error(ctxs[r]);
    if (rc) {
      ctxs[r]->prefilled = false;
      if (!first) first = rc;
    }
  }
  return first;
}

}  // namespace

int spd_batch_generate(spd_ctx *const *ctxs, int32_t n, int32_t n_steps) {
  int rc = batch_enqueue(ctxs, n, n_steps);
  if (rc) return rc;
  return batch_wait(ctxs, n);
}

int spd_batch_step(spd_ctx *const *ctxs, int32_t n, int32_t *out_ids, int32_t *out_parent, float *out_gamma) {
  int rc = batch_enqueue(ctxs, n, 1);
  if (rc) return rc;
  // One copy and one wait for the whole batch: the tail kernel left every request's state words and new tokens in
  // its row of the leading context's results.  (The products record a wait that ran out in the leading context's
  // state, which is row 0's.)
  spd_ctx *lead = ctxs[0];
  static_assert(SPD_MAX_K == spd::kMaxK, "the rows' lists are kMaxK apart");
  std::vector<int32_t> rows((size_t)n * spd::kBtResultWords);
  SPD_CUDA(cudaMemcpyAsync(rows.data(), lead->ws + lead->lay.bt_out, rows.size() * 4, cudaMemcpyDeviceToHost, lead->stream));
  SPD_CUDA(cudaStreamSynchronize(lead->stream));
  int first = SPD_OK;
  for (int r = 0; r < n; ++r) {
    const int32_t *row = rows.data() + (size_t)r * spd::kBtResultWords;
    if (row[2]) {
      ctxs[r]->prefilled = false;
      if (!first) first = row[2];
    }
  }
  if (first) return first;
  for (int r = 0; r < n; ++r) {
    const int32_t *row = rows.data() + (size_t)r * spd::kBtResultWords;
    const int k = ctxs[r]->cfg.k;
    for (int i = 0; i < k; ++i) {
      if (out_ids) out_ids[r * SPD_MAX_K + i] = row[8 + i];
      if (out_parent) out_parent[r * SPD_MAX_K + i] = row[8 + spd::kMaxK + i];
      if (out_gamma) std::memcpy(&out_gamma[r * SPD_MAX_K + i], &row[8 + 2 * spd::kMaxK + i], 4);
    }
  }
  return SPD_OK;
}

int64_t spd_launch_count(const spd_ctx *ctx) { return ctx ? ctx->launches : 0; }

int spd_pack_image(const void *w, int32_t rows, int32_t cols, void *out, void *stream) {
  if (!w || !out || rows < spd::kUnitRows || cols < 32 || rows % spd::kUnitRows || cols % 32 || ((uintptr_t)w % 16) || ((uintptr_t)out % 16)) return SPD_EINVAL;
  const cudaError_t e = spd_internal_pack_image(w, out, rows, cols, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(e, "spd_pack_image");
  return SPD_OK;
}

int spd_finished(const spd_ctx *ctx) { return ctx && ctx->stopped ? 1 : 0; }

int spd_debug_read(spd_ctx *ctx, int what, void *host_buf, size_t bytes) {
  if (!ctx || !host_buf) return SPD_EINVAL;
  int rc = set_device(ctx);
  if (rc) return rc;
  const spd_config &c = ctx->cfg;
  const int k = c.k;
  const uint8_t *st = ctx->ws + ctx->lay.state;
  SPD_CUDA(cudaStreamSynchronize(ctx->stream));
  auto copy = [&](const void *src, size_t n) -> int {
    if (bytes < n) return SPD_ENOMEM;
    SPD_CUDA(cudaMemcpy(host_buf, src, n, cudaMemcpyDeviceToHost));
    return SPD_OK;
  };
  auto copy_rows = [&](const void *src, int rows, size_t row_bytes, size_t row_stride) -> int {
    if (bytes < (size_t)rows * row_bytes) return SPD_ENOMEM;
    SPD_CUDA(cudaMemcpy2D(host_buf, row_bytes, src, row_stride, row_bytes, rows, cudaMemcpyDeviceToHost));
    return SPD_OK;
  };
  switch (what) {
    case SPD_DBG_LOGITS: return copy(ctx->ws + ctx->lay.logits, (size_t)c.vocab * 4);
    case SPD_DBG_CAND_TOK: return copy(st + offsetof(spd::State, cand_tok), (size_t)k * 4);
    case SPD_DBG_CAND_LP: return copy(st + offsetof(spd::State, cand_lp), (size_t)k * 4);
    case SPD_DBG_LOGP_IN: return copy(st + offsetof(spd::State, logP_in), (size_t)k * 4);
    case SPD_DBG_SCORE: return copy(st + offsetof(spd::State, score), (size_t)k * k * 4);
    case SPD_DBG_PNG: return copy(st + offsetof(spd::State, png), (size_t)k * k * 4);
    case SPD_DBG_CNT: return copy(st + offsetof(spd::State, cnt), (size_t)k * k * spd::kMaxTables * 4);
    case SPD_DBG_TOT: return copy(st + offsetof(spd::State, tot), (size_t)k * spd::kMaxTables * 4);
    case SPD_DBG_SEL: return copy(st + offsetof(spd::State, sel), (size_t)k * 4);
    case SPD_DBG_LOGP: return copy(st + offsetof(spd::State, logP), (size_t)k * 4);
    case SPD_DBG_HIST_IN: return copy_rows(st + offsetof(spd::State, win_in), k, spd::kWin * 4, spd::kWin * 4);
    case SPD_DBG_TRACE: return copy(ctx->ws + ctx->lay.trace, (size_t)c.n_layers * 2 * c.d_model * 4);
    case SPD_DBG_HIDDEN: return copy(ctx->ws + ctx->lay.h, (size_t)c.d_model * 4);
    case SPD_DBG_KCACHE:
    case SPD_DBG_VCACHE: {
      const int T = ctx->prefilled ? ctx->m + ctx->n_gen - 1 : 0;
      const size_t rows = (size_t)c.n_layers, row_elems = (size_t)T * c.d_model, esz = c.kv_dtype ? 2 : 4;
      if (bytes < rows * row_elems * 4) return SPD_ENOMEM;
      if (T == 0) return SPD_OK;
      const uint8_t *src = ctx->ws + (what == SPD_DBG_KCACHE ? ctx->lay.kcache : ctx->lay.vcache);
      // the raw rows land in the tail of the caller's buffer, then are widened in place from the front
      uint8_t *raw = static_cast<uint8_t *>(host_buf) + rows * row_elems * (4 - esz);
      SPD_CUDA(cudaMemcpy2D(raw, row_elems * esz, src, (size_t)c.max_pos * c.d_model * esz, row_elems * esz, rows,
                            cudaMemcpyDeviceToHost));
      if (esz == 2) {
        const uint16_t *in = reinterpret_cast<const uint16_t *>(raw);
        uint32_t *out = static_cast<uint32_t *>(host_buf);
        for (size_t i = 0; i < rows * row_elems; ++i) out[i] = (uint32_t)in[i] << 16;
      }
      return SPD_OK;
    }
    default: return SPD_EINVAL;
  }
}

int spd_debug_trace(spd_ctx *ctx, int on) {
  if (!ctx) return SPD_EINVAL;
  ctx->kp.trace = on ? reinterpret_cast<float *>(ctx->ws + ctx->lay.trace) : nullptr;
  return SPD_OK;
}

int spd_debug_score(spd_ctx *ctx, const int32_t *hist, int32_t hist_len, const float *logp, const int32_t *cand_tok,
                    const float *cand_lp) {
  if (!ctx || !hist || !logp || !cand_tok || !cand_lp) return SPD_EINVAL;
  if (hist_len < 0 || hist_len > spd::kWin) return SPD_ERANGE;
  const spd_config &c = ctx->cfg;
  for (int i = 0; i < c.k; ++i) {
    if (cand_tok[i] < 0 || cand_tok[i] >= c.vocab) return SPD_ERANGE;
    for (int j = 0; j < hist_len; ++j)
      if (hist[i * hist_len + j] < 0 || hist[i * hist_len + j] >= c.vocab) return SPD_ERANGE;
  }
  int rc = set_device(ctx);
  if (rc) return rc;
  spd::State st;
  std::memset(&st, 0, sizeof st);
  st.win_len = hist_len;
  for (int i = 0; i < c.k; ++i) {
    for (int j = 0; j < hist_len; ++j) st.win[i][spd::kWin - hist_len + j] = hist[i * hist_len + j];
    st.logP[i] = logp[i];
    st.cand_tok[i] = cand_tok[i];
    st.cand_lp[i] = cand_lp[i];
  }
  SPD_CUDA(cudaMemcpyAsync(ctx->ws + ctx->lay.state, &st, sizeof st, cudaMemcpyHostToDevice, ctx->stream));
  SPD_CUDA(cudaStreamSynchronize(ctx->stream));
  ctx->prefilled = false;  // the draft state no longer belongs to a decoding run
  // launch() zeroes the head of the state only; the fields set above lie behind it
  if ((rc = launch(ctx, spd::kModeScoreOnly, 0, 0, 0))) return rc;
  return spd_sync(ctx);
}

int spd_debug_nucleus(spd_ctx *ctx, const float *logits, float top_p, float temperature, float u, int32_t *out_token) {
  if (!ctx || !logits || !out_token) return SPD_EINVAL;
  if (!(top_p > 0.f) || top_p > 1.f || !(temperature > 0.f) || !(u >= 0.f) || !(u < 1.f)) return SPD_ERANGE;
  int rc = set_device(ctx);
  if (rc) return rc;
  SPD_CUDA(cudaMemcpyAsync(ctx->ws + ctx->lay.logits, logits, (size_t)ctx->cfg.vocab * 4, cudaMemcpyHostToDevice, ctx->stream));
  SPD_CUDA(cudaMemcpyAsync(ctx->ws + ctx->lay.ns_u, &u, 4, cudaMemcpyHostToDevice, ctx->stream));
  SPD_CUDA(cudaStreamSynchronize(ctx->stream));
  ctx->prefilled = false;  // the logits no longer belong to a decoding run
  ctx->kp.ns_p = top_p;
  ctx->kp.ns_inv_temp = 1.0f / temperature;
  if ((rc = launch(ctx, spd::kModeNucleusOnly, 0, 0, 0))) return rc;
  if ((rc = read_state(ctx, offsetof(spd::State, cand_tok), out_token, 4))) return rc;
  return spd_sync(ctx);
}

int spd_debug_expire(spd_ctx *ctx) {
  if (!ctx) return SPD_EINVAL;
  int rc = set_device(ctx);
  if (rc) return rc;
  ctx->prefilled = false;
  ctx->decoding = false;
  SPD_CUDA(cudaMemsetAsync(ctx->ws + ctx->lay.prefix, 0, 4, ctx->stream));  // token 0 at position 0
  ctx->kp.pf_stall = 1;
  spd::KParams &kp = ctx->kp;
  kp.mode = spd::kModePrefill;
  kp.n_iters = 1;
  kp.pos0 = 0;
  kp.step0 = 0;
  kp.pf_head = 0;
  cudaError_t e = cudaMemsetAsync(ctx->ws + ctx->lay.state, 0, head_bytes(false), ctx->stream);
  if (e == cudaSuccess) e = spd_internal_prefill_launch(&kp, ctx->grid, ctx->stream);
  kp.pf_stall = 0;
  if (e != cudaSuccess) return cuda_fail(e, "prefill launch");
  ctx->launches += 1;
  return check_device_error(ctx);
}

int spd_debug_expire_products(spd_ctx *ctx) {
  if (!ctx) return SPD_EINVAL;
  if (ctx->tc_rows == 0) return SPD_ESTATE;
  int rc = set_device(ctx);
  if (rc) return rc;
  ctx->prefilled = false;
  ctx->decoding = false;
  const spd::TcJob job = tc_job(ctx);
  cudaError_t e = cudaMemsetAsync(ctx->ws + ctx->lay.state, 0, head_bytes(false), ctx->stream);
  if (e == cudaSuccess) e = spd_internal_tc_stall(&job, ctx->stream);
  if (e != cudaSuccess) return cuda_fail(e, "long-prefix launch");
  ctx->launches += 1;
  return check_device_error(ctx);
}

}  // extern "C"
