// Host-side description of one long-prefix prefill job (see spd_prefill_tc.cu).
#pragma once
#include "spd_params.h"

namespace spd {

constexpr int kTcTile = 128;      // tokens per tile of the tensor-core products
constexpr int kTcMaxTokens = 512; // tokens one job takes at most
constexpr int kTcMinPrefix = 32;  // runs of more tokens than this take the path: a job of up to 128 tokens costs about 1.5 launches
                                  // of the 16-token kernel, so two launches before the last pay for it

struct TcJob {
  int32_t L, d, H, hd, f, max_pos, kv_bf16;
  float eps;
  const LayerW *layers;              // HOST copy of the layer table [L]
  const __nv_bfloat16 *tok_emb;
  const uint8_t *w_tmaps;            // device: tensor maps of the layers' matrices, four per layer
  const uint8_t *x_tmaps;            // device: tensor maps of the term buffer seen as [3 * x_term_rows][d] and [..][f], boxes of 128 rows;
                                     // then three more pairs with boxes of 16, 32 and 64 rows (products of a small batch)
  void *kcache, *vcache;
  const float2 *rope;
  float *h, *y, *q;                  // [x_term_rows][d], [x_term_rows][max(3d, 2f)], [x_term_rows][d]
  uint16_t *x;                       // [3][x_term_rows][max(d, f)] bf16 terms
  int32_t x_term_rows;
  const int32_t *ids;                // device: the job's token ids
  int32_t pos0, n_tok;               // first position; tokens (<= x_term_rows)
  State *st;
  int32_t sm_count;                  // SMs of the device
  size_t y_floats;                   // room of y in floats (partial sums of a column-split product)
  float *ss;                         // [128][32]: sums of squares of the residual rows per 512-column chunk (jobs of up to 128 tokens)
};

// Words of a request's row in a batched timestep's results (written by the tail kernel, fetched by the host in one copy).
constexpr int kBtResultWords = 64;

// Programmatic dependent launch.  dep_wait: returns once the kernel before this one in the stream has completed and
// its writes are visible (at once when the launch did not ask for the overlap).  dep_launch: the kernel after this
// one may be brought onto the SMs, where it runs up to its own dep_wait, as soon as every block of this kernel has
// said so or has ended.
#ifdef __CUDACC__
__device__ __forceinline__ void dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif

// Launch with programmatic stream serialization: the kernel may be brought onto the SMs while the one before it in the
// stream still runs, and waits there (dep_wait) until that one has completed.  The kernels launched this way start
// with dep_wait (the small-batch product: before its first read of the terms), so that the launch latency, the
// set-up of a block and the product's first weight copies overlap the tail of the kernel before.
template <typename... P, typename... A>
inline cudaError_t launch_dep(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, A... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...);
}

}  // namespace spd

extern "C" cudaError_t spd_internal_tc_prepare(void);
extern "C" cudaError_t spd_internal_tc_stall(const spd::TcJob *job, cudaStream_t stream);
extern "C" cudaError_t spd_internal_tc_prefill(const spd::TcJob *job, cudaStream_t stream, int *launches);
// Row-wise kernels of a job of up to 128 tokens (column-parallel, 1 / rms applied behind the product; spd_batch.cu).
extern "C" cudaError_t spd_internal_job_input(const spd::TcJob *job, float *ss, cudaStream_t s);
extern "C" cudaError_t spd_internal_job_rope_cache(const spd::TcJob *job, float *ss, int nz, size_t zs, int layer, cudaStream_t s);
extern "C" cudaError_t spd_internal_job_resid(const spd::TcJob *job, float *ss, int nz, size_t zs, const __nv_bfloat16 *gain, cudaStream_t s);
extern "C" cudaError_t spd_internal_job_swiglu(const spd::TcJob *job, float *ss, int nz, size_t zs, cudaStream_t s);
// The product of a batched timestep's few token rows.  dep: launch it so that it may start while the kernel before it
// in the stream still runs (it then copies weights only, until that kernel has completed).
extern "C" cudaError_t spd_internal_batch_gemm(const uint8_t *xmaps, int wide, const void *wmap, float *Y, size_t y_floats, int n_tok, int N, int C,
                                               int x_term_rows, spd::State *st, int sm_count, cudaStream_t s, int dep, int *out_nz, size_t *out_zs);
