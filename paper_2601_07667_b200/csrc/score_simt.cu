// Observation-window scorer on the CUDA cores (Algorithm 1 (window softmax A, past-only column sum U)).
//
// Two passes over K, both in the log2 domain x = (q.k) * log2(e)/sqrt(d):
//   pass 1  thread = query row: online row max / row sum over one key tile,
//           one (max, sum) partial per (row, tile); a combine kernel folds the
//           partials of a row, in tile order, into offset = max + log2(sum).
//   pass 2  thread = past key: exp2(x - offset[row]) summed over the window
//           rows of each query head = that key's column sum U.
// This is the general-shape path (any window, any group size); the tensor-core
// scorer replaces it for the shapes it supports.
#include "asl_internal.cuh"

namespace {

constexpr int D = 128;
constexpr int KT = ASL_SIMT_KEY_TILE;

__device__ __forceinline__ float bf16lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf16hi(uint32_t x) { return __uint_as_float(x & 0xFFFF0000u); }

// dot of a register-resident fp32 vector with a bf16 row in shared memory (all
// threads read the same row: broadcast loads).
__device__ __forceinline__ float dot_row(const float (&v)[D], const uint4* row) {
  float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
  for (int i = 0; i < D / 8; ++i) {
    uint4 p = row[i];
    acc0 = fmaf(v[8 * i + 0], bf16lo(p.x), acc0);
    acc1 = fmaf(v[8 * i + 1], bf16hi(p.x), acc1);
    acc0 = fmaf(v[8 * i + 2], bf16lo(p.y), acc0);
    acc1 = fmaf(v[8 * i + 3], bf16hi(p.y), acc1);
    acc0 = fmaf(v[8 * i + 4], bf16lo(p.z), acc0);
    acc1 = fmaf(v[8 * i + 5], bf16hi(p.z), acc1);
    acc0 = fmaf(v[8 * i + 6], bf16lo(p.w), acc0);
    acc1 = fmaf(v[8 * i + 7], bf16hi(p.w), acc1);
  }
  return acc0 + acc1;
}

__device__ __forceinline__ void load_row(float (&v)[D], const uint16_t* src) {
  const uint4* s = reinterpret_cast<const uint4*>(src);
#pragma unroll
  for (int i = 0; i < D / 8; ++i) {
    uint4 p = s[i];
    v[8 * i + 0] = bf16lo(p.x); v[8 * i + 1] = bf16hi(p.x);
    v[8 * i + 2] = bf16lo(p.y); v[8 * i + 3] = bf16hi(p.y);
    v[8 * i + 4] = bf16lo(p.z); v[8 * i + 5] = bf16hi(p.z);
    v[8 * i + 6] = bf16lo(p.w); v[8 * i + 7] = bf16hi(p.w);
  }
}

struct ScoreArgs {
  const uint16_t* q;
  const uint16_t* k;
  const AslReq* req;
  int64_t qs_b, qs_h, qs_r, ks_t, ks_h;
  int32_t Hk, G, W, R;       // R = G*W rows per kv head
  float scale_log2;
};

// ---- pass 1: partial row statistics ---------------------------------------
__global__ void __launch_bounds__(256) score_pass1_simt(ScoreArgs a, float2* __restrict__ partials) {
  __shared__ uint4 ks[KT * D / 8];
  const int b = blockIdx.z, h = blockIdx.y, tile = blockIdx.x;
  const AslReq rq = a.req[b];
  const int j0 = tile * KT;
  if (j0 >= rq.n) return;
  // stage the key tile (rows past the request's end are zero and never visible)
  for (int i = threadIdx.x; i < KT * D / 8; i += blockDim.x) {
    int jj = i / (D / 8), c = i % (D / 8);
    int j = j0 + jj;
    uint4 val = make_uint4(0, 0, 0, 0);
    if (j < rq.n)
      val = *reinterpret_cast<const uint4*>(a.k + (int64_t)(rq.tok_off + j) * a.ks_t + (int64_t)h * a.ks_h + c * 8);
    ks[i] = val;
  }
  __syncthreads();
  float2* out = partials + ((int64_t)(rq.pad + tile) * a.Hk + h) * a.R;
  for (int r = threadIdx.x; r < a.R; r += blockDim.x) {
    const int g = r / a.W, t = r % a.W;
    float qv[D];
    load_row(qv, a.q + (int64_t)b * a.qs_b + (int64_t)(h * a.G + g) * a.qs_h + (int64_t)t * a.qs_r);
    const int last = rq.T + t;                 // row t sits at position T+t and sees keys j <= T+t
    float m = -INFINITY, l = 0.f;
    for (int jj = 0; jj < KT; ++jj) {
      if (j0 + jj > last) break;
      float x = dot_row(qv, ks + jj * (D / 8)) * a.scale_log2;
      if (x > m) { l = l * exp2f(m - x) + 1.f; m = x; }
      else       { l += exp2f(x - m); }
    }
    out[r] = make_float2(m, l);
  }
}

// ---- combine: offset[row] = max + log2(sum) over the request's tiles --------
__global__ void score_combine_simt(const float2* __restrict__ partials, const AslReq* __restrict__ req, int Hk, int R,
                                   float* __restrict__ offsets) {
  const int b = blockIdx.y, h = blockIdx.x;
  const AslReq rq = req[b];
  const int tiles = (rq.n + KT - 1) / KT;
  for (int r = threadIdx.x; r < R; r += blockDim.x) {
    float M = -INFINITY;
    for (int t = 0; t < tiles; ++t) M = fmaxf(M, partials[((int64_t)(rq.pad + t) * Hk + h) * R + r].x);
    float L = 0.f;
    for (int t = 0; t < tiles; ++t) {
      float2 p = partials[((int64_t)(rq.pad + t) * Hk + h) * R + r];
      if (p.y > 0.f) L += p.y * exp2f(p.x - M);
    }
    offsets[((int64_t)b * Hk + h) * R + r] = M + log2f(L);
  }
}

// ---- pass 2: normalised column sums ----------------------------------------
// per_q_head = 0: u[h][t_off + j]       = sum over all G*W rows   (group sum folded in)
// per_q_head = 1: u[h*G+g][t_off + j]   = sum over the W rows of query head g
__global__ void __launch_bounds__(128) score_pass2_simt(ScoreArgs a, const float* __restrict__ offsets, int per_q_head,
                                                        int64_t sum_T, float* __restrict__ u) {
  constexpr int RC = 64;                        // query rows staged per round
  __shared__ uint4 qs[RC * D / 8];
  __shared__ float offs[RC];
  const int b = blockIdx.z, h = blockIdx.y;
  const AslReq rq = a.req[b];
  const int j0 = blockIdx.x * KT;
  if (j0 >= rq.T) return;
  const int j = j0 + threadIdx.x;
  const bool live = j < rq.T;
  float kv[D];
  if (live) load_row(kv, a.k + (int64_t)(rq.tok_off + j) * a.ks_t + (int64_t)h * a.ks_h);
  else {
#pragma unroll
    for (int c = 0; c < D; ++c) kv[c] = 0.f;
  }
  const float* off = offsets + ((int64_t)b * a.Hk + h) * a.R;
  float total = 0.f, acc = 0.f;
  int cur_g = 0;
  for (int r0 = 0; r0 < a.R; r0 += RC) {
    __syncthreads();
    for (int i = threadIdx.x; i < RC * D / 8; i += blockDim.x) {
      int rr = i / (D / 8), c = i % (D / 8);
      int r = r0 + rr;
      uint4 val = make_uint4(0, 0, 0, 0);
      if (r < a.R) {
        int g = r / a.W, t = r % a.W;
        val = *reinterpret_cast<const uint4*>(a.q + (int64_t)b * a.qs_b + (int64_t)(h * a.G + g) * a.qs_h +
                                              (int64_t)t * a.qs_r + c * 8);
      }
      qs[i] = val;
    }
    for (int i = threadIdx.x; i < RC; i += blockDim.x) offs[i] = (r0 + i < a.R) ? off[r0 + i] : 0.f;
    __syncthreads();
    const int lim = min(RC, a.R - r0);
    for (int rr = 0; rr < lim; ++rr) {
      const int g = (r0 + rr) / a.W;
      if (g != cur_g) {
        if (per_q_head && live) u[(int64_t)(h * a.G + cur_g) * sum_T + rq.t_off + j] = acc;
        total += acc; acc = 0.f; cur_g = g;
      }
      float x = dot_row(kv, qs + rr * (D / 8)) * a.scale_log2 - offs[rr];
      acc += exp2f(x);
    }
  }
  if (live) {
    if (per_q_head) u[(int64_t)(h * a.G + cur_g) * sum_T + rq.t_off + j] = acc;
    else            u[(int64_t)h * sum_T + rq.t_off + j] = total + acc;
  }
}

// offsets[b][h][r] (log2 domain, row r = g*W + t of kv head h) <-> lse[b][h*G + g][t] (natural log)
__global__ void lse_to_offsets(const float* __restrict__ lse, float* __restrict__ offsets, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) offsets[i] = lse[i] * 1.4426950408889634f;
}
// `stride`: offsets per kv head (the tensor-core scorer pads a kv head's rows to whole chunks)
__global__ void offsets_to_lse(const float* __restrict__ offsets, float* __restrict__ lse, int n, int R, int stride) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) lse[i] = __ldcg(offsets + (int64_t)(i / R) * stride + i % R) * 0.6931471805599453f;
}

}  // namespace

// The row offsets of the latest asl_score_layer call, as natural-log softmax denominators.
// [b][h][g*W + t] and [b][h*G + g][t] are the same linear order: contiguous groups.
asl_status asl_launch_window_lse(asl_ctx* c, const char* ws, float* lse_out, cudaStream_t st) {
  const int n = c->p.batch * c->p.n_kv_heads * c->rows_per_kv;
  const int stride = c->tc.enabled ? c->tc.nchunk * c->tc.NC : c->rows_per_kv;
  offsets_to_lse<<<(n + 255) / 256, 256, 0, st>>>(reinterpret_cast<const float*>(ws + c->ws.score_offsets), lse_out, n,
                                                  c->rows_per_kv, stride);
  c->launches += 1;
  ASL_CUDA(cudaGetLastError());
  return ASL_OK;
}

asl_status asl_launch_score_simt(asl_ctx* c, const void* q, const void* k, const float* lse, float* u, char* ws,
                                 cudaStream_t st) {
  const asl_params& p = c->p;
  ScoreArgs a;
  a.q = static_cast<const uint16_t*>(q);
  a.k = static_cast<const uint16_t*>(k);
  a.req = c->d_req;
  a.qs_b = p.q_stride[0]; a.qs_h = p.q_stride[1]; a.qs_r = p.q_stride[2];
  a.ks_t = p.k_stride[0]; a.ks_h = p.k_stride[1];
  a.Hk = p.n_kv_heads; a.G = p.n_q_heads / p.n_kv_heads; a.W = p.window; a.R = c->rows_per_kv;
  a.scale_log2 = (float)(1.4426950408889634 / sqrt((double)p.head_dim));
  float2* partials = reinterpret_cast<float2*>(ws + c->ws.score_partials);
  float* offsets = reinterpret_cast<float*>(ws + c->ws.score_offsets);
  if (lse) {                                    // supplied denominators: pass 2 alone
    const int n = p.batch * p.n_kv_heads * c->rows_per_kv;
    lse_to_offsets<<<(n + 255) / 256, 256, 0, st>>>(lse, offsets, n);
    c->launches += 1;
  } else {
    const int max_tiles = (c->max_n + KT - 1) / KT;
    dim3 g1(max_tiles, p.n_kv_heads, p.batch);
    score_pass1_simt<<<g1, 256, 0, st>>>(a, partials);
    score_combine_simt<<<dim3(p.n_kv_heads, p.batch), 256, 0, st>>>(partials, c->d_req, a.Hk, a.R, offsets);
    c->launches += 2;
  }
  dim3 g2((c->max_T + KT - 1) / KT, p.n_kv_heads, p.batch);
  score_pass2_simt<<<g2, 128, 0, st>>>(a, offsets, p.pool_mode == ASL_POOL_MAX ? 1 : 0, c->sum_T, u);
  c->launches += 1;
  ASL_CUDA(cudaGetLastError());
  return ASL_OK;
}
