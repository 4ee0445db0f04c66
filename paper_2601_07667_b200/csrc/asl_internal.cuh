// Internal declarations shared by the translation units of the library.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <vector>

#include "asl.h"
#include "score_tc.cuh"

// Per-request table entry, one per request, resident on the device.
struct AslReq {
  int32_t n;         // tokens, window included
  int32_t T;         // past tokens n - W
  int32_t k;         // past tokens kept: min(budget, n) - W
  int32_t kept;      // k + W
  int32_t tok_off;   // cu_seqlens[b]
  int32_t t_off;     // offset of the request's past segment in packed score vectors
  int32_t kept_off;  // offset of the request's segment in packed kept lists
  int32_t pad;
};

// Scratch layout inside the caller's workspace (byte offsets, 256-aligned).
struct AslWorkspace {
  size_t score_partials;   // pass-1 partial row statistics
  size_t score_offsets;    // per-row log2 normalisers
  size_t score_u[2];       // un-pooled column sums, two slots
  size_t score_q8;         // fp8 K: the window queries as two E4M3 terms [2][B][H_q][W][d] bytes
  size_t score_end;
  size_t rank_keys[2];     // ping-pong sort keys
  size_t rank_idx[2];      // ping-pong sort payload
  size_t rank_hist;        // per-block digit histograms / offsets
  size_t rank_end;
  size_t topk_scratch;     // per-segment digit histograms, pick state and per-tile counts
  size_t topk_end;
  size_t total;
};

struct asl_ctx {
  int device = 0;
  int sm_count = 0;
  bool planned = false;
  int controller = 0;                 // ASL_CONTROLLER_*: asl_set_controller
  const asl_stat* latch_stat = nullptr;   // under ASL_CONTROLLER_LATCH: the records of the latest asl_rank_stat call (device)
  int32_t cur_layer = -1;             // layer the next calls belong to (asl_set_layer / asl_rank_stat)
  asl_params p{};
  std::vector<int32_t> cu, budgets;
  std::vector<float> k_scale;         // per kv head (fp8 K), else empty
  int k_elem_bytes = 2;               // bytes per K element
  std::vector<AslReq> req;
  int64_t sum_tokens = 0, sum_T = 0, sum_kept = 0;
  int32_t max_n = 0, max_T = 0, max_kept = 0;
  AslReq* d_req = nullptr;            // device [B]
  unsigned long long* d_acc = nullptr;  // device [B][2] integer accumulators of the statistic + a block counter
  int32_t* d_err = nullptr;           // device error word of bounded waits
  // scorer plan
  int32_t rows_per_kv = 0;            // G*W
  int32_t n_key_tiles = 0;            // sum over requests of ceil(n_b / tile)
  int32_t u_rows_per_kv = 1;          // rows of un-pooled column sums per kv head (average pooling: all are added;
                                      // max pooling: G * u_parts, u_parts consecutive rows per query head)
  int32_t u_parts = 1;                // partial rows per query head under max pooling
  AslTcPlan tc;                       // tensor-core scorer plan (enabled when the shape fits)
  bool topk_one_cta = false;          // the per-head top-k runs as one CTA per segment (asl_topk_plan)
  AslWorkspace ws{};
  int64_t launches = 0;
};

// Under ASL_CONTROLLER_LATCH a request is finished at layer `cur` once its record selected at an
// earlier layer: Algorithm 2 has returned its one-shot selection and the method does nothing more for it.
// The record may be being written by an asl_rank_stat of the same layer on another stream: the writer
// stores `selected` last, behind a fence, and the reader looks at layer_idx only after it has seen
// `selected`, so a record in the middle of its update reads as "not finished" or with its final layer.
#ifdef __CUDACC__
__device__ inline bool asl_finished(const asl_stat* s, int32_t cur) {
  const volatile asl_stat* v = s;
  if (!v->selected) return false;
  __threadfence();
  return v->layer_idx < cur;
}
#endif
// Programmatic dependent launch between consecutive kernels of one stream: a kernel lets its successor's
// blocks become resident as soon as its own have all started, and a kernel launched with launch_after()
// waits (for the whole grid before it, memory included) where it first touches what that grid may write.
// What a kernel reads before the wait must have been complete before its predecessor was launched.
// Launched the plain way both instructions do nothing.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_release_successor() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_wait_predecessor() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_after(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif
constexpr int ASL_SKIP_MAX_BATCH = 4096;  // requests the scorer's per-launch phase list covers (larger batches are scored in full)

#define ASL_CUDA(expr)                          \
  do {                                          \
    cudaError_t e__ = (expr);                   \
    if (e__ != cudaSuccess) return ASL_ERR_CUDA; \
  } while (0)

static inline size_t asl_align256(size_t x) { return (x + 255) & ~size_t(255); }

// ---- kernels' host launchers (one per translation unit) ----
asl_status asl_launch_score_simt(asl_ctx* c, const void* q, const void* k, const float* lse, float* u, char* ws,
                                 cudaStream_t st);
asl_status asl_launch_window_lse(asl_ctx* c, const char* ws, float* lse_out, cudaStream_t st);
bool asl_tc_plan(asl_ctx* c);
void asl_tc_free(asl_ctx* c);
size_t asl_tc_partial_bytes(const asl_ctx* c);
asl_status asl_tc_reset_sync(asl_ctx* c, cudaStream_t st);
asl_status asl_launch_wait_selftest(asl_ctx* c, int which, unsigned long long limit_ns, cudaStream_t st);
asl_status asl_launch_score_tc(asl_ctx* c, const void* q, const void* k, const float* lse, float* u, char* ws,
                               cudaStream_t st);
asl_status asl_launch_pool(asl_ctx* c, const float* u, float* scores_kv, float* scores_agg, cudaStream_t st);
asl_status asl_launch_live_phases(asl_ctx* c, bool two_pass, cudaStream_t st);
asl_status asl_launch_rank(asl_ctx* c, const float* agg, int32_t layer_idx, int32_t n_rows, int32_t* ring,
                           asl_stat* stat, char* ws, cudaStream_t st);
asl_status asl_launch_topk(asl_ctx* c, const float* scores, int32_t n_heads, int32_t* idx_out, const asl_stat* gate,
                           int32_t gate_layer, char* ws, cudaStream_t st);
bool asl_topk_plan(asl_ctx* c);
size_t asl_topk_scratch_bytes(int64_t segments, int64_t max_T);
asl_status asl_launch_compact(asl_ctx* c, const void* k, const void* v, const int32_t* idx, void* k_out, void* v_out,
                              cudaStream_t st);

asl_status asl_launch_compact_rows(asl_ctx* c, const void* x, const int32_t* idx, void* out, int64_t row_bytes,
                                   cudaStream_t st);

constexpr int ASL_SIMT_KEY_TILE = 128;   // keys per block in the SIMT scorer
constexpr int ASL_RANK_TILE = 2048;      // keys per block in the radix sort
