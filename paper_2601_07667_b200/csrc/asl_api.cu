// C-ABI entry points: argument checks, planning, workspace layout, dispatch.
#include <math.h>
#include <stdlib.h>
#include <new>

#include "asl_internal.cuh"

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

void free_plan(asl_ctx* c) {
  asl_tc_free(c);
  if (c->d_req) cudaFree(c->d_req);
  if (c->d_acc) cudaFree(c->d_acc);
  c->d_req = nullptr;
  c->d_acc = nullptr;
  c->latch_stat = nullptr;
  c->cur_layer = -1;
  c->planned = false;
}

}  // namespace

extern "C" {

asl_status asl_create(asl_ctx** out, int device) {
  if (!out) return ASL_ERR_INVALID;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return ASL_ERR_CUDA;
  cudaDeviceProp prop;
  ASL_CUDA(cudaGetDeviceProperties(&prop, device));
  if (prop.major != 10) return ASL_ERR_ARCH;      // sm_100 only: no fallback path
  asl_ctx* c = new (std::nothrow) asl_ctx();
  if (!c) return ASL_ERR_CUDA;
  c->device = device;
  c->sm_count = prop.multiProcessorCount;
  int prev = 0;
  cudaGetDevice(&prev);
  cudaSetDevice(device);
  cudaError_t e = cudaMalloc(&c->d_err, sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMemset(c->d_err, 0, sizeof(int32_t));
  cudaSetDevice(prev);
  if (e != cudaSuccess) { delete c; return ASL_ERR_CUDA; }
  *out = c;
  return ASL_OK;
}

asl_status asl_destroy(asl_ctx* c) {
  if (!c) return ASL_ERR_INVALID;
  free_plan(c);
  if (c->d_err) cudaFree(c->d_err);
  delete c;
  return ASL_OK;
}

asl_status asl_plan(asl_ctx* c, const asl_params* p, size_t* workspace_bytes) {
  if (!c || !p || !workspace_bytes || !p->cu_seqlens || !p->budgets) return ASL_ERR_INVALID;
  if (p->n_q_heads < 1 || p->n_kv_heads < 1 || p->n_q_heads % p->n_kv_heads) return ASL_ERR_INVALID;
  if (p->window < 1 || p->batch < 1) return ASL_ERR_INVALID;
  if (p->pool_kernel < 1 || p->pool_kernel % 2 == 0) return ASL_ERR_INVALID;
  if (p->pool_mode != ASL_POOL_AVG && p->pool_mode != ASL_POOL_MAX) return ASL_ERR_INVALID;
  if (p->l_obs < 2 || p->l_min < 0 || p->score_ctas < 0) return ASL_ERR_INVALID;
  if (p->head_dim < 8 || p->head_dim % 8) return ASL_ERR_INVALID;
  if (p->head_dim != 128) return ASL_ERR_UNSUPPORTED;
  if (p->k_dtype != ASL_K_BF16 && p->k_dtype != ASL_K_FP8_E4M3) return ASL_ERR_INVALID;
  const bool fp8 = p->k_dtype == ASL_K_FP8_E4M3;
  if (fp8) {
    if (!p->k_scale) return ASL_ERR_INVALID;
    for (int h = 0; h < p->n_kv_heads; ++h)
      if (!(p->k_scale[h] > 0.0f) || !(p->k_scale[h] < INFINITY)) return ASL_ERR_INVALID;
    if (p->k_stride[0] % 16 || p->k_stride[1] % 16) return ASL_ERR_INVALID;     // 16-byte rows of 1-byte elements
  }
  // rows must start on 16-byte boundaries: every stride a multiple of 8 elements
  const int64_t strides[] = {p->q_stride[0], p->q_stride[1], p->q_stride[2], p->k_stride[0],
                             p->k_stride[1], p->v_stride[0], p->v_stride[1]};
  for (int64_t s : strides)
    if (s < 0 || s % 8) return ASL_ERR_INVALID;
  if (p->q_stride[2] < p->head_dim || p->k_stride[1] < p->head_dim || p->v_stride[1] < p->head_dim) return ASL_ERR_INVALID;
  if (p->cu_seqlens[0] != 0) return ASL_ERR_INVALID;

  std::vector<AslReq> req(p->batch);
  int64_t sum_T = 0, sum_kept = 0, tiles = 0;
  int32_t max_n = 0, max_T = 0, max_kept = 0;
  for (int b = 0; b < p->batch; ++b) {
    const int64_t n = (int64_t)p->cu_seqlens[b + 1] - p->cu_seqlens[b];
    const int64_t budget = p->budgets[b];
    if (n <= p->window || budget < p->window) return ASL_ERR_INVALID;
    AslReq& r = req[b];
    r.n = (int32_t)n;
    r.T = (int32_t)(n - p->window);
    r.kept = (int32_t)(budget < n ? budget : n);
    r.k = r.kept - p->window;
    r.tok_off = p->cu_seqlens[b];
    r.t_off = (int32_t)sum_T;
    r.kept_off = (int32_t)sum_kept;
    r.pad = (int32_t)tiles;                       // first key tile of the request (SIMT scorer partials)
    sum_T += r.T;
    sum_kept += r.kept;
    tiles += (n + ASL_SIMT_KEY_TILE - 1) / ASL_SIMT_KEY_TILE;
    max_n = r.n > max_n ? r.n : max_n;
    max_T = r.T > max_T ? r.T : max_T;
    max_kept = r.kept > max_kept ? r.kept : max_kept;
    // the integer numerator of the statistic must fit 63 bits: m * rows^2 * T^2 / 4
    const double m_max = fmin((double)r.T, (double)(r.k > 0 ? r.k : 1) * p->l_obs);
    if (m_max * p->l_obs * p->l_obs * (double)r.T * (double)r.T / 4.0 >= 9.0e18) return ASL_ERR_UNSUPPORTED;
  }
  if (sum_T >= (int64_t)1 << 31 || (int64_t)p->cu_seqlens[p->batch] >= (int64_t)1 << 31) return ASL_ERR_UNSUPPORTED;

  int prev = 0;
  cudaGetDevice(&prev);
  ASL_CUDA(cudaSetDevice(c->device));
  free_plan(c);
  cudaError_t e = cudaMalloc(&c->d_req, sizeof(AslReq) * p->batch);
  if (e == cudaSuccess) e = cudaMemcpy(c->d_req, req.data(), sizeof(AslReq) * p->batch, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMalloc(&c->d_acc, sizeof(unsigned long long) * (2 * p->batch + 1));
  if (e == cudaSuccess) e = cudaMemset(c->d_acc, 0, sizeof(unsigned long long) * (2 * p->batch + 1));

  cudaSetDevice(prev);
  if (e != cudaSuccess) { free_plan(c); return ASL_ERR_CUDA; }

  c->p = *p;
  c->cu.assign(p->cu_seqlens, p->cu_seqlens + p->batch + 1);
  c->budgets.assign(p->budgets, p->budgets + p->batch);
  c->p.cu_seqlens = c->cu.data();
  c->p.budgets = c->budgets.data();
  c->k_scale.clear();
  if (fp8) c->k_scale.assign(p->k_scale, p->k_scale + p->n_kv_heads);
  c->p.k_scale = fp8 ? c->k_scale.data() : nullptr;
  c->k_elem_bytes = fp8 ? 1 : 2;
  c->req = req;
  c->sum_tokens = p->cu_seqlens[p->batch];
  c->sum_T = sum_T;
  c->sum_kept = sum_kept;
  c->max_n = max_n; c->max_T = max_T; c->max_kept = max_kept;
  c->rows_per_kv = (p->n_q_heads / p->n_kv_heads) * p->window;
  c->n_key_tiles = (int32_t)tiles;

  cudaGetDevice(&prev);
  cudaSetDevice(c->device);
  const bool tc = asl_tc_plan(c);
  asl_topk_plan(c);
  cudaSetDevice(prev);
  if (fp8 && !tc) { free_plan(c); return ASL_ERR_UNSUPPORTED; }     // only the tensor-core scorer reads 8-bit keys
  const int G = p->n_q_heads / p->n_kv_heads;
  // the tensor-core scorer writes two partial column sums per chunk (one per half of the chunk's rows);
  // under max pooling they belong to different query heads unless a chunk is a single head
  c->u_parts = (tc && p->pool_mode == ASL_POOL_MAX && p->window > c->tc.NC / 2) ? 2 : 1;
  c->u_rows_per_kv = p->pool_mode == ASL_POOL_MAX ? G * c->u_parts : (tc ? 2 * c->tc.nchunk : 1);

  AslWorkspace& w = c->ws;
  size_t off = 0;
  size_t partial_bytes = (size_t)tiles * p->n_kv_heads * c->rows_per_kv * sizeof(float2);
  if (tc && asl_tc_partial_bytes(c) > partial_bytes) partial_bytes = asl_tc_partial_bytes(c);
  w.score_partials = off; off = asl_align256(off + partial_bytes);
  const size_t rows_padded = tc && c->tc.nchunk * c->tc.NC > c->rows_per_kv ? (size_t)c->tc.nchunk * c->tc.NC : (size_t)c->rows_per_kv;
  w.score_offsets = off;  off = asl_align256(off + (size_t)p->batch * p->n_kv_heads * rows_padded * sizeof(float));
  const size_t u_rows = (size_t)p->n_kv_heads * c->u_rows_per_kv;
  for (int i = 0; i < 2; ++i) { w.score_u[i] = off; off = asl_align256(off + u_rows * (size_t)sum_T * sizeof(float)); }
  w.score_q8 = off;
  if (fp8) off = asl_align256(off + (size_t)2 * p->batch * p->n_q_heads * p->window * p->head_dim);
  w.score_end = off;
  for (int i = 0; i < 2; ++i) { w.rank_keys[i] = off; off = asl_align256(off + (size_t)sum_T * 4); }
  for (int i = 0; i < 2; ++i) { w.rank_idx[i] = off; off = asl_align256(off + (size_t)sum_T * 4); }
  const size_t nblk = (max_T + ASL_RANK_TILE - 1) / ASL_RANK_TILE;
  w.rank_hist = off;      off = asl_align256(off + (size_t)4 * p->batch * 256 * nblk * sizeof(int32_t));
  w.rank_end = off;
  w.topk_scratch = off;   off = asl_align256(off + asl_topk_scratch_bytes((int64_t)p->batch * p->n_kv_heads, max_T));
  w.topk_end = off;
  w.total = off;
  *workspace_bytes = w.total;
  c->planned = true;
  return ASL_OK;
}

asl_status asl_plan_sizes(const asl_ctx* c, int64_t* sum_tokens, int64_t* sum_T, int64_t* sum_kept) {
  if (!c || !c->planned) return ASL_ERR_INVALID;
  if (sum_tokens) *sum_tokens = c->sum_tokens;
  if (sum_T) *sum_T = c->sum_T;
  if (sum_kept) *sum_kept = c->sum_kept;
  return ASL_OK;
}

// scoring alone: un-pooled column sums into slot `slot` of the workspace
static asl_status score_columns_impl(asl_ctx* c, const void* q_obs, const void* k, const float* lse, void* workspace,
                                     size_t workspace_bytes, int slot, void* stream) {
  if (!c || !c->planned || !q_obs || !k || slot < 0 || slot > 1) return ASL_ERR_INVALID;
  if (!aligned16(q_obs) || !aligned16(k)) return ASL_ERR_INVALID;
  if (!workspace || workspace_bytes < c->ws.total || !aligned16(workspace)) return ASL_ERR_WORKSPACE;
  char* ws = static_cast<char*>(workspace);
  float* u = reinterpret_cast<float*>(ws + c->ws.score_u[slot]);
  if (c->tc.enabled) {
    // requests that have finished are not scored any more: a small kernel ahead of the launch reads their
    // flags once and writes the launch's phase list without their phases, so that every CTA of the
    // persistent kernel walks the same list
    if (c->latch_stat && c->cur_layer >= 0 && c->p.batch <= ASL_SKIP_MAX_BATCH) {
      const asl_status s = asl_launch_live_phases(c, lse == nullptr, static_cast<cudaStream_t>(stream));
      if (s != ASL_OK) return s;
    }
    return asl_launch_score_tc(c, q_obs, k, lse, u, ws, static_cast<cudaStream_t>(stream));
  }
  return asl_launch_score_simt(c, q_obs, k, lse, u, ws, static_cast<cudaStream_t>(stream));
}

static asl_status pool_scores_impl(asl_ctx* c, void* workspace, size_t workspace_bytes, int slot, float* scores_kv,
                                   float* scores_agg, void* stream) {
  if (!c || !c->planned || !scores_kv || !scores_agg || slot < 0 || slot > 1) return ASL_ERR_INVALID;
  if (!workspace || workspace_bytes < c->ws.total || !aligned16(workspace)) return ASL_ERR_WORKSPACE;
  const float* u = reinterpret_cast<const float*>(static_cast<char*>(workspace) + c->ws.score_u[slot]);
  return asl_launch_pool(c, u, scores_kv, scores_agg, static_cast<cudaStream_t>(stream));
}

asl_status asl_score_layer(asl_ctx* c, const void* q_obs, const void* k, float* scores_kv, float* scores_agg,
                           void* workspace, size_t workspace_bytes, void* stream) {
  if (!scores_kv || !scores_agg) return ASL_ERR_INVALID;
  const asl_status s = score_columns_impl(c, q_obs, k, nullptr, workspace, workspace_bytes, 0, stream);
  return s != ASL_OK ? s : pool_scores_impl(c, workspace, workspace_bytes, 0, scores_kv, scores_agg, stream);
}

asl_status asl_score_layer_lse(asl_ctx* c, const void* q_obs, const void* k, const float* lse, float* scores_kv,
                               float* scores_agg, void* workspace, size_t workspace_bytes, void* stream) {
  if (!lse || !scores_kv || !scores_agg) return ASL_ERR_INVALID;
  const asl_status s = score_columns_impl(c, q_obs, k, lse, workspace, workspace_bytes, 0, stream);
  return s != ASL_OK ? s : pool_scores_impl(c, workspace, workspace_bytes, 0, scores_kv, scores_agg, stream);
}

asl_status asl_score_columns(asl_ctx* c, const void* q_obs, const void* k, const float* lse, void* workspace,
                             size_t workspace_bytes, int32_t slot, void* stream) {
  return score_columns_impl(c, q_obs, k, lse, workspace, workspace_bytes, slot, stream);
}

asl_status asl_pool_scores(asl_ctx* c, void* workspace, size_t workspace_bytes, int32_t slot, float* scores_kv,
                           float* scores_agg, void* stream) {
  return pool_scores_impl(c, workspace, workspace_bytes, slot, scores_kv, scores_agg, stream);
}

asl_status asl_window_lse(asl_ctx* c, const void* workspace, size_t workspace_bytes, float* lse_out, void* stream) {
  if (!c || !c->planned || !lse_out) return ASL_ERR_INVALID;
  if (!workspace || workspace_bytes < c->ws.total || !aligned16(workspace)) return ASL_ERR_WORKSPACE;
  return asl_launch_window_lse(c, static_cast<const char*>(workspace), lse_out, static_cast<cudaStream_t>(stream));
}

asl_status asl_rank_stat(asl_ctx* c, const float* scores_agg, int32_t layer_idx, int32_t n_rows, int32_t* rank_ring,
                         asl_stat* stat, void* workspace, size_t workspace_bytes, void* stream) {
  if (!c || !c->planned || !scores_agg || !rank_ring || !stat) return ASL_ERR_INVALID;
  if (layer_idx < 0 || n_rows < 1 || n_rows > c->p.l_obs || n_rows > layer_idx + 1) return ASL_ERR_INVALID;
  if (!workspace || workspace_bytes < c->ws.total || !aligned16(workspace)) return ASL_ERR_WORKSPACE;
  if (c->controller == ASL_CONTROLLER_LATCH) c->latch_stat = stat;
  return asl_launch_rank(c, scores_agg, layer_idx, n_rows, rank_ring, stat, static_cast<char*>(workspace),
                         static_cast<cudaStream_t>(stream));
}

asl_status asl_select_topk(asl_ctx* c, const float* scores, int32_t n_heads, int32_t* idx_out, void* workspace,
                           size_t workspace_bytes, void* stream) {
  if (!c || !c->planned || !scores || !idx_out || n_heads < 1) return ASL_ERR_INVALID;
  if (!workspace || workspace_bytes < c->ws.total || !aligned16(workspace)) return ASL_ERR_WORKSPACE;
  return asl_launch_topk(c, scores, n_heads, idx_out, nullptr, 0, static_cast<char*>(workspace),
                         static_cast<cudaStream_t>(stream));
}

asl_status asl_select_topk_gated(asl_ctx* c, const float* scores, int32_t n_heads, int32_t* idx_out, const asl_stat* stat,
                                 int32_t layer_idx, void* workspace, size_t workspace_bytes, void* stream) {
  if (!c || !c->planned || !scores || !idx_out || !stat || n_heads < 1 || layer_idx < 0) return ASL_ERR_INVALID;
  if (!workspace || workspace_bytes < c->ws.total || !aligned16(workspace)) return ASL_ERR_WORKSPACE;
  return asl_launch_topk(c, scores, n_heads, idx_out, stat, layer_idx, static_cast<char*>(workspace),
                         static_cast<cudaStream_t>(stream));
}

asl_status asl_set_controller(asl_ctx* c, int32_t mode) {
  if (!c || (mode != ASL_CONTROLLER_REPORT && mode != ASL_CONTROLLER_LATCH)) return ASL_ERR_INVALID;
  c->controller = mode;
  if (mode != ASL_CONTROLLER_LATCH) c->latch_stat = nullptr;
  return ASL_OK;
}

asl_status asl_set_layer(asl_ctx* c, int32_t layer_idx) {
  if (!c || layer_idx < 0) return ASL_ERR_INVALID;
  c->cur_layer = layer_idx;
  return ASL_OK;
}

asl_status asl_compact_kv(asl_ctx* c, const void* k, const void* v, const int32_t* idx, void* k_out, void* v_out,
                          void* stream) {
  if (!c || !c->planned || !k || !v || !idx || !k_out || !v_out) return ASL_ERR_INVALID;
  if (!aligned16(k) || !aligned16(v) || !aligned16(k_out) || !aligned16(v_out)) return ASL_ERR_INVALID;
  return asl_launch_compact(c, k, v, idx, k_out, v_out, static_cast<cudaStream_t>(stream));
}

asl_status asl_compact_rows(asl_ctx* c, const void* x, const int32_t* idx, void* out, int64_t row_bytes, void* stream) {
  if (!c || !c->planned || !x || !idx || !out) return ASL_ERR_INVALID;
  if (row_bytes < 16 || row_bytes % 16 || row_bytes / 16 > 0x7fffffff) return ASL_ERR_INVALID;
  if (!aligned16(x) || !aligned16(out)) return ASL_ERR_INVALID;
  return asl_launch_compact_rows(c, x, idx, out, row_bytes, static_cast<cudaStream_t>(stream));
}

asl_status asl_device_status(asl_ctx* c, void* stream, int32_t* where) {
  if (!c) return ASL_ERR_INVALID;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t word = 0;
  ASL_CUDA(cudaMemcpyAsync(&word, c->d_err, sizeof(word), cudaMemcpyDeviceToHost, st));
  ASL_CUDA(cudaStreamSynchronize(st));
  if (where) *where = word;
  if (word == 0) return ASL_OK;
  ASL_CUDA(cudaMemsetAsync(c->d_err, 0, sizeof(word), st));
  if (asl_tc_reset_sync(c, st) != ASL_OK) return ASL_ERR_CUDA;
  return ASL_ERR_TIMEOUT;
}

asl_status asl_selftest_bounded_wait(asl_ctx* c, int32_t which, int64_t limit_ns, void* stream) {
  if (!c || !c->planned || (which != 0 && which != 1) || limit_ns < 1000 || limit_ns > 1000000) return ASL_ERR_INVALID;
  return asl_launch_wait_selftest(c, which, (unsigned long long)limit_ns, static_cast<cudaStream_t>(stream));
}

int64_t asl_launch_count(const asl_ctx* c) { return c ? c->launches : 0; }

const char* asl_strerror(asl_status s) {
  switch (s) {
    case ASL_OK: return "ok";
    case ASL_ERR_INVALID: return "invalid argument";
    case ASL_ERR_UNSUPPORTED: return "unsupported configuration";
    case ASL_ERR_WORKSPACE: return "workspace missing or too small";
    case ASL_ERR_CUDA: return "CUDA call failed";
    case ASL_ERR_TIMEOUT: return "bounded device wait expired";
    case ASL_ERR_ARCH: return "device is not sm_100";
  }
  return "unknown status";
}

}  // extern "C"
