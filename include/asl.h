/* asl.h -- C ABI of the ASL prefill hot path for NVIDIA B200 (sm_100a).
 *
 * ASL (adaptive selection layer) watches, layer by layer during prefill, how
 * the ranking of context tokens by observation-window attention settles, and
 * prunes the KV cache to a budget.  This library is the per-layer data path:
 *
 *   asl_score_layer   Algorithm 1: window softmax A, past-only column sum U, 1-D
 *                     pooling, SumGroups; plus the "scores" sum of Section 4.1
 *   asl_rank_stat     Algorithm 1: RankDesc; Algorithm 2 up to the threshold test
 *                     (rank rows R, TopKIndices J, Unique U, RelNormVar; Section 4.1)
 *   asl_select_topk   Algorithm 1: k, TopK and the window append
 *   asl_compact_kv    Algorithm 1: the returned K[I], V[I]
 *
 * Conventions
 *   - Every entry point returns an asl_status; nothing throws, aborts or prints.
 *   - "device" pointers are CUDA global-memory addresses on the context's
 *     device; "host" pointers are ordinary process memory.  The caller owns
 *     every buffer it passes; the library keeps no reference after the call's
 *     work has finished on the stream.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*);
 *     no entry point synchronises with the host.
 *   - The library allocates device memory only inside asl_create/asl_plan
 *     (a few KB of per-request tables); scratch comes from the caller's
 *     workspace, whose size asl_plan reports.  The workspace is split into
 *     disjoint regions per entry point, so asl_rank_stat may run on another
 *     stream concurrently with asl_select_topk / asl_compact_kv of the same
 *     layer.  Two calls of the SAME entry point on one context must not overlap.
 *   - At most ONE scoring call (asl_score_layer, asl_score_layer_lse,
 *     asl_score_columns) may be in flight per DEVICE, whatever the context,
 *     stream or process: the scorer is one persistent kernel whose CTAs wait for
 *     one another, so all of them have to be resident at the same time.  Its grid
 *     never exceeds the SM count and one CTA fills an SM, which makes that true
 *     when it has the SMs it asks for; two scorers started side by side could each
 *     hold part of the SMs and wait for CTAs that cannot start.  Such a wait is
 *     bounded (2 s) and ends in ASL_ERR_TIMEOUT, never in a hang, but the results
 *     of both calls are then void.  Order scoring calls of different contexts on
 *     one device with events.  Every other entry point may overlap freely.
 *   - bf16 tensors are passed as raw 16-bit patterns; the channel (head_dim)
 *     axis is contiguous and every row starts on a 16-byte boundary.
 *   - Token indices are request-local, 0-based, int32.
 *   - Requests are packed back to back: request b owns tokens
 *     [cu_seqlens[b], cu_seqlens[b+1]) of K/V, n_b of them, the last `window`
 *     being the observation window; T_b = n_b - window past tokens.
 *     Score vectors are packed the same way over past tokens only: request b's
 *     segment starts at cu_seqlens[b] - b*window and has T_b entries
 *     (sum_T in total).  Kept lists are packed over kept_b = min(budget_b, n_b).
 */
#ifndef ASL_H_
#define ASL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct asl_ctx asl_ctx;   /* opaque: plan, device tables, cached tensor maps */

typedef enum {
  ASL_OK = 0,
  ASL_ERR_INVALID = -1,      /* bad argument (null, shape, alignment, budget < window ...) */
  ASL_ERR_UNSUPPORTED = -2,  /* valid request this build cannot run                         */
  ASL_ERR_WORKSPACE = -3,    /* workspace pointer null or too small                         */
  ASL_ERR_CUDA = -4,         /* a CUDA runtime/driver call failed                           */
  ASL_ERR_TIMEOUT = -5,      /* a bounded device-side wait gave up (see asl_device_status)  */
  ASL_ERR_ARCH = -6          /* device is not sm_100: there is no fallback path             */
} asl_status;

enum { ASL_POOL_AVG = 0, ASL_POOL_MAX = 1 };
enum { ASL_K_BF16 = 0, ASL_K_FP8_E4M3 = 1 };   /* element type of K */

/* Problem statement of Algorithm 1 (W, S, KV_budget) and Algorithm 2
 * (L_min, L_obs, tau).  Host arrays are copied by asl_plan. */
typedef struct {
  int32_t n_q_heads;      /* H_q                                                     */
  int32_t n_kv_heads;     /* H_k, divides H_q; query head a reads kv head a / G      */
  int32_t head_dim;       /* d (128 in this build)                                    */
  int32_t window;         /* W >= 1: observation window = last W query rows           */
  int32_t pool_kernel;    /* S, odd >= 1; stride 1, pad floor(S/2)                    */
  int32_t pool_mode;      /* ASL_POOL_AVG (the paper) or ASL_POOL_MAX                 */
  int32_t batch;          /* B >= 1 requests                                          */
  int32_t l_min;          /* first layer at which the statistic is evaluated          */
  int32_t l_obs;          /* rank rows kept (ring depth), >= 2                        */
  int32_t score_ctas;     /* CTAs of the persistent scorer kernel; 0 = one per SM.  A   */
                          /* smaller number leaves SMs to kernels of other streams    */
                          /* (the previous layer's statistic, top-k and compaction)   */
  double tau;             /* selection fires when relative variance < tau             */
  const int32_t* cu_seqlens; /* host [B+1] token offsets, cu_seqlens[0] = 0           */
  const int32_t* budgets;    /* host [B] KV_budget per request, window included       */
  int64_t q_stride[3];    /* q_obs element strides: request, head, row                */
  int64_t k_stride[2];    /* K element strides: token, head                           */
  int64_t v_stride[2];    /* V element strides: token, head                           */
  int32_t k_dtype;        /* ASL_K_BF16, or ASL_K_FP8_E4M3: a quantised K cache.  K then  */
                          /* holds 8-bit E4M3 codes (finite variant: no infinities) and   */
                          /* the key the method sees is code x k_scale[kv head]; k_stride */
                          /* counts 1-byte elements, rows still start on 16-byte          */
                          /* boundaries; asl_compact_kv copies the codes (k_out is        */
                          /* [H_k][sum_kept][d] bytes), V stays bf16.  The queries stay   */
                          /* bf16: the scorer splits each into two E4M3 terms (exact for  */
                          /* 1/64 <= |q| <= 28, else to 2^-13 / saturated) and runs the   */
                          /* contraction on the 8-bit tensor-core path.  Shapes the       */
                          /* tensor-core scorer does not take are ASL_ERR_UNSUPPORTED.    */
  int32_t reserved0;
  const float* k_scale;   /* host [H_k], finite and > 0; read only for ASL_K_FP8_E4M3     */
} asl_params;

/* Result of Algorithm 2 for one request; lives in device memory, [B] of them,
 * and carries init_var from layer to layer.  Zero it before a new prompt. */
typedef struct {
  int64_t num;        /* sum over the union of rows*sum(r^2) - (sum r)^2, exact           */
  int32_t m;          /* |U|: size of the union of per-row top-k sets                     */
  int32_t rows;       /* rank rows the statistic was taken over                           */
  int32_t k;          /* min(KV_budget - W, T)                                            */
  int32_t layer_idx;  /* layer of the latest call                                         */
  int32_t evaluated;  /* 1 if layer_idx >= L_min and rows >= 2, else 0 (fields above 0)    */
  int32_t selected;   /* 1 if rel < tau at this layer                                     */
  int32_t has_init;   /* init_var holds a value                                           */
  int32_t reserved;
  double var_top;     /* num / (rows^2 * m)                                               */
  double init_var;    /* var_top at the first evaluated layer                             */
  double rel;         /* var_top / init_var (NaN, which never selects, if init_var is 0)  */
} asl_stat;

/* Context bound to CUDA device `device`.  ASL_ERR_ARCH unless it is sm_100. */
asl_status asl_create(asl_ctx** out, int device);
asl_status asl_destroy(asl_ctx* ctx);

/* Validates the parameters, copies the host arrays, builds the per-request
 * tables on the device and reports the workspace size every later call needs.
 * ASL_ERR_INVALID for: null pointers, H_q % H_k != 0, even or zero S, W < 1,
 * n_b <= W (Algorithm 1 needs a non-empty past), budget_b < W, l_obs < 2,
 * strides that break 16-byte row alignment.  budget_b >= n_b is valid (keep all).
 * May be called again on the same context to re-plan. */
asl_status asl_plan(asl_ctx* ctx, const asl_params* params, size_t* workspace_bytes);

/* Derived sizes of the current plan (host values): sum_T = sum of past tokens,
 * sum_kept = sum of min(budget_b, n_b). */
asl_status asl_plan_sizes(const asl_ctx* ctx, int64_t* sum_tokens, int64_t* sum_T, int64_t* sum_kept);

/* Algorithm 1 up to SumGroups: A = softmax over all n keys of the last W query rows
 * (causal mask on the last W x W block), U = column sums over the W rows for
 * past columns, pooled per query head, summed over each GQA group:
 *   scores_kv  device [H_k][sum_T] fp32   P of Algorithm 1 (SumGroups)
 *   scores_agg device [sum_T]      fp32   sum over kv heads (the "scores" of Section 4.1)
 * q_obs device bf16 [B][H_q][W][d] (strides q_stride), k device bf16 packed
 * [sum n_b][H_k][d] (strides k_stride). */
asl_status asl_score_layer(asl_ctx* ctx, const void* q_obs, const void* k, float* scores_kv,
                           float* scores_agg, void* workspace, size_t workspace_bytes, void* stream);

/* The same scores when the caller already holds the softmax denominators of the
 * window rows (Algorithm 1 (window softmax A) is a softmax: A = exp(s - lse) with
 * lse = log sum over the visible keys of exp(s), s = q.k/sqrt(d); a fused
 * attention forward keeps exactly this value per query row).  One pass over K
 * instead of two.  lse: device fp32 [B][H_q][W], natural logarithm. */
asl_status asl_score_layer_lse(asl_ctx* ctx, const void* q_obs, const void* k, const float* lse, float* scores_kv,
                               float* scores_agg, void* workspace, size_t workspace_bytes, void* stream);

/* asl_score_layer in two halves, for callers that pipeline layers: the first
 * half is the scoring proper (the window softmax and the past-only column sums
 * of Algorithm 1; lse null = two passes, else as asl_score_layer_lse) and leaves
 * its un-pooled sums in slot 0 or 1 of the workspace; the second half is the
 * pooling, SumGroups and the aggregate.  The second half of layer l may run on
 * another stream while the first half of layer l+1 fills the other slot.
 * asl_score_layer = both halves on slot 0. */
asl_status asl_score_columns(asl_ctx* ctx, const void* q_obs, const void* k, const float* lse, void* workspace,
                             size_t workspace_bytes, int32_t slot, void* stream);
asl_status asl_pool_scores(asl_ctx* ctx, void* workspace, size_t workspace_bytes, int32_t slot, float* scores_kv,
                           float* scores_agg, void* stream);

/* Denominators found by the latest asl_score_layer call on this workspace, in
 * the layout asl_score_layer_lse takes: lse_out device fp32 [B][H_q][W]. */
asl_status asl_window_lse(asl_ctx* ctx, const void* workspace, size_t workspace_bytes, float* lse_out, void* stream);

/* Algorithm 1 (RankDesc) + Algorithm 2: writes rank row RankDesc(scores_agg)
 * (0-based, ties to the lower index) into ring slot layer_idx % L_obs of
 * rank_ring (device int32 [L_obs][sum_T]), then, if layer_idx >= L_min and
 * n_rows >= 2, takes the statistic over the latest n_rows rows (the rows of
 * layers layer_idx-n_rows+1 .. layer_idx, n_rows <= L_obs, this one included):
 * union of the per-row k smallest ranks, mean population variance of ranks,
 * relative variance against init_var, comparison with tau.  stat: device [B]. */
asl_status asl_rank_stat(asl_ctx* ctx, const float* scores_agg, int32_t layer_idx, int32_t n_rows,
                         int32_t* rank_ring, asl_stat* stat, void* workspace, size_t workspace_bytes,
                         void* stream);

/* Algorithm 1 (k, TopK and window append) per (request, head): the k_b = min(budget_b, n_b) - W
 * past tokens with the largest score, ties to the lower index, written in
 * ascending index order and followed by the window indices T_b .. n_b-1.
 * scores device [n_heads][sum_T] fp32; idx_out device int32 [n_heads][sum_kept].
 * n_heads is H_k for the per-head cache, 1 for a selection on the aggregate
 * (1 <= n_heads <= H_k, else ASL_ERR_INVALID). */
asl_status asl_select_topk(asl_ctx* ctx, const float* scores, int32_t n_heads, int32_t* idx_out,
                           void* workspace, size_t workspace_bytes, void* stream);

/* Algorithm 2 as a state machine on the device, for callers that issue all layers ahead of time (one CUDA
 * graph of the prompt's layers) and cannot branch on a layer's result on the host.
 *   ASL_CONTROLLER_REPORT (default): every asl_rank_stat call sorts and evaluates its layer.
 *   ASL_CONTROLLER_LATCH: once a request's record says `selected`, it is final: later asl_rank_stat calls
 *     leave the request's record (layer_idx = the selection layer) and its rank rows as they are and their
 *     blocks exit at once; the host reads the records once, after the last layer.
 * asl_select_topk_gated is asl_select_topk for the requests whose record (`stat`, device [B], as written by
 * the asl_rank_stat call of layer `layer_idx` ordered before it) selected at exactly that layer; the lists of
 * all other requests are left untouched.  With n_heads = 1 on scores_agg, called after every layer's
 * asl_rank_stat, it leaves in idx_out the one-shot selection of Algorithm 2 for every request that selected.
 *
 * Under ASL_CONTROLLER_LATCH the work of a finished request is skipped as well (Algorithm 2 ends the
 * method for a request at its selection layer: only select_idx goes on and the rank cache is released).
 * A request is finished at layer l when its record selected at a layer before l.  asl_set_layer tells
 * the context which layer the calls that follow belong to (call it at the start of every layer); the
 * records consulted are those passed to the latest asl_rank_stat call.  Then, for a finished request,
 *   - the scorer leaves out its phases (a one-block kernel ahead of the launch reads the flags once and
 *     writes the launch's phase list without them, so a record that a
 *     still-running asl_rank_stat of the previous layer is about to set takes effect one layer later);
 *   - asl_pool_scores, asl_select_topk and asl_compact_kv leave its scores, kept list and compacted
 *     cache as its selection layer wrote them; they read the records on the device, so issue them after
 *     (on the same stream as, or ordered behind) the asl_rank_stat call of the previous layer;
 *   - its rows of the rank ring are dead: nothing reads or writes them again, the caller may reuse them.
 * Batches of more than 4096 requests are scored in full (the other calls still skip).  Without
 * asl_set_layer (or in ASL_CONTROLLER_REPORT) nothing is skipped. */
enum { ASL_CONTROLLER_REPORT = 0, ASL_CONTROLLER_LATCH = 1 };
asl_status asl_set_controller(asl_ctx* ctx, int32_t mode);
asl_status asl_set_layer(asl_ctx* ctx, int32_t layer_idx);
asl_status asl_select_topk_gated(asl_ctx* ctx, const float* scores, int32_t n_heads, int32_t* idx_out,
                                 const asl_stat* stat, int32_t layer_idx, void* workspace, size_t workspace_bytes,
                                 void* stream);

/* Algorithm 1 (K[I], V[I]): k_out[h][r][:] = k[cu_seqlens[b] + idx[h][r]][h][:] and
 * the same for v, r running over request b's kept segment.
 * k_out, v_out: device bf16 dense [H_k][sum_kept][d]. */
asl_status asl_compact_kv(asl_ctx* ctx, const void* k, const void* v, const int32_t* idx, void* k_out,
                          void* v_out, void* stream);

/* Algorithm 2 (one-shot selection), the one-shot selection at the selection layer: once
 * asl_rank_stat reports `selected`, the tokens that go on to the deeper layers
 * are select_idx = Unique(J_last u I_w): the k tokens with the best aggregate
 * score of THIS layer plus the window.  That index list is asl_select_topk with
 * scores = scores_agg and n_heads = 1 (ascending, window appended: already
 * unique); this call gathers any per-token tensor with it, for example the
 * hidden states:  out[kept_off_b + r][:] = x[cu_seqlens[b] + idx[kept_off_b + r]][:].
 *   x    device, packed [sum n_b] rows of row_bytes bytes (multiple of 16, 16-byte aligned)
 *   idx  device int32 [sum_kept], as written by asl_select_topk(n_heads = 1)
 *   out  device, [sum_kept] rows of row_bytes bytes */
asl_status asl_compact_rows(asl_ctx* ctx, const void* x, const int32_t* idx, void* out, int64_t row_bytes,
                            void* stream);

/* Rank row without any allocation.  (The paper has no counterpart: this is a
 * packaging of Algorithm 1 (RankDesc) for hosts that may not allocate.)
 *
 * Who needs it: a caller that cannot obtain device memory at the time it wants
 * a rank row -- an inference server whose memory pool was handed over to its
 * own allocator at start-up, a plugin invoked inside another runtime's
 * callback, a process run under a "no cudaMalloc after initialisation" rule.
 * Such a caller can use neither asl_create/asl_plan (both allocate small device
 * tables) nor a workspace it has nowhere to take from.  This call needs no
 * context and no workspace: its sort scratch is a fixed array compiled into
 * the library (about 4.5 MiB of device memory on every GPU that loads the
 * library, held until the process exits).
 *
 *   scores    device fp32 [T]   one request's aggregate scores
 *   rank_out  device int32 [T]  rank_out[j] = 0-based rank of token j by
 *                               descending score, ties to the lower index --
 *                               the same row asl_rank_stat writes into its ring
 *   T         1 .. ASL_RANK_STATIC_MAX_T; larger -> ASL_ERR_WORKSPACE (the fixed
 *             scratch is too small; use asl_rank_stat with a workspace instead)
 *
 * Runs on the calling thread's current device, asynchronously on `stream`;
 * calls no cudaMalloc/cudaFree and no allocating library routine.  The first
 * call on each device also looks up the scratch array's device address and
 * checks the architecture (ASL_ERR_ARCH unless sm_100); make that first call
 * outside any stream capture.  All calls on a device share the one scratch
 * array, which keeps whatever the last call left in it (every call overwrites
 * what it reads, nothing needs clearing): two calls whose kernels can overlap
 * on the GPU -- different streams, no ordering between them -- race on it and
 * give wrong ranks.  Issue them on one stream or order them with events.
 * ASL_ERR_INVALID for null pointers or T < 1. */
#define ASL_RANK_STATIC_MAX_T 262144
asl_status asl_rank_desc_static(const float* scores, int32_t T, int32_t* rank_out, void* stream);

/* Reads the device error word written by bounded waits (host-synchronising:
 * it waits for `stream` first).  ASL_OK, or ASL_ERR_TIMEOUT with *where set to
 * the code of the wait that gave up; the word is cleared. */
asl_status asl_device_status(asl_ctx* ctx, void* stream, int32_t* where);

/* Self-test of the bounded waits (no counterpart in the paper: a diagnostic of this library).  The
 * scorer's kernels wait on shared-memory barriers and on counters in device memory; every such wait
 * gives up after a time limit, records a code in the context's error word and lets the kernel finish,
 * so that a wait that can never end surfaces as ASL_ERR_TIMEOUT instead of a hung device.  This call
 * launches one warp that runs one of those two waits -- which = 0: a barrier nobody arrives on;
 * which = 1: a counter nobody advances -- with the limit `limit_ns` (1 us .. 1 ms), so the path can be
 * exercised without any fault: afterwards asl_device_status returns ASL_ERR_TIMEOUT with *where = 91
 * (barrier) or 92 (counter), and the query after that ASL_OK.  Needs a planned context; asynchronous
 * on `stream`. */
asl_status asl_selftest_bounded_wait(asl_ctx* ctx, int32_t which, int64_t limit_ns, void* stream);

/* Number of kernels this context has launched so far (host counter). */
int64_t asl_launch_count(const asl_ctx* ctx);

const char* asl_strerror(asl_status s);

#ifdef __cplusplus
}
#endif
#endif /* ASL_H_ */
