// 1-D pooling, GQA group sum and all-head aggregate (Algorithm 1 (1-D pooling, SumGroups) and
// the "scores" sum of Section 4.1).  One thread per past token walks the kv
// heads, so the aggregate needs no atomics and is bit-reproducible.
//   average pooling: input is group-summed column sums, `urows` rows per kv head
//                    (one per row chunk of the scorer) that are added first
//                    (pooling is linear, so summing the group first is the same
//                    up to rounding); zero padding, divisor always S.
//   max pooling:     input is per query head, `parts` consecutive rows of partial
//                    sums each, u[H_q][parts][sum_T]; each head is pooled over its
//                    in-range taps, then the group is summed.
// Taps never cross a request's past segment [0, T_b).
#include "asl_internal.cuh"

namespace {

constexpr int PT = 256;          // tokens per block
constexpr int MAX_HALO = 16;     // pooling kernels up to 33 taps go through shared memory

// One block pools PT consecutive past tokens of one request.  Row by row, the
// un-pooled sums of the tile and its halo are staged in shared memory (partial
// rows added on the way), pooled from there, and added up per kv head and over
// all heads in a fixed order: no atomics, bit-reproducible.
__global__ void __launch_bounds__(PT) pool_group_kernel(const float* __restrict__ u, const AslReq* __restrict__ req,
                                                        int Hk, int G, int S, int mode, int urows, int parts, int64_t sum_T,
                                                        float* __restrict__ scores_kv, float* __restrict__ scores_agg) {
  __shared__ float tile[PT + 2 * MAX_HALO];
  const int b = blockIdx.y;
  const AslReq rq = req[b];
  const int j0 = blockIdx.x * PT;
  if (j0 >= rq.T) return;
  const int r = S / 2;
  const int j = j0 + threadIdx.x;
  const bool live = j < rq.T;
  const int lo = max(0, j - r), hi = min(rq.T - 1, j + r);
  const float inv = 1.0f / (float)S;
  // stage sum over `nrows` consecutive rows starting at `row0` for tokens j0-r .. j0+PT-1+r (zero outside [0, T))
  auto stage = [&](int row0, int nrows) {
    __syncthreads();
    for (int i = threadIdx.x; i < PT + 2 * r; i += PT) {
      const int t = j0 - r + i;
      float v = 0.f;
      if (t >= 0 && t < rq.T) {
        const float* src = u + (int64_t)row0 * sum_T + rq.t_off + t;
        for (int c = 0; c < nrows; ++c) v += src[(int64_t)c * sum_T];
      }
      tile[i] = v;
    }
    __syncthreads();
  };
  float agg = 0.f;
  for (int h = 0; h < Hk; ++h) {
    float p = 0.f;
    if (mode == ASL_POOL_AVG) {
      stage(h * urows, urows);
      if (live) {
        float s = 0.f;
        for (int i = lo; i <= hi; ++i) s += tile[i - j0 + r];
        p = s * inv;
      }
    } else {
      for (int g = 0; g < G; ++g) {
        stage((h * G + g) * parts, parts);
        if (live) {
          float mx = tile[lo - j0 + r];
          for (int i = lo + 1; i <= hi; ++i) mx = fmaxf(mx, tile[i - j0 + r]);
          p += mx;
        }
      }
    }
    if (live) scores_kv[(int64_t)h * sum_T + rq.t_off + j] = p;
    agg += p;
  }
  if (live) scores_agg[rq.t_off + j] = agg;
}

}  // namespace

asl_status asl_launch_pool(asl_ctx* c, const float* u, float* scores_kv, float* scores_agg, cudaStream_t st) {
  const asl_params& p = c->p;
  if (p.pool_kernel / 2 > MAX_HALO) return ASL_ERR_UNSUPPORTED;
  dim3 grid((c->max_T + PT - 1) / PT, p.batch);
  pool_group_kernel<<<grid, PT, 0, st>>>(u, c->d_req, p.n_kv_heads, p.n_q_heads / p.n_kv_heads, p.pool_kernel,
                                          p.pool_mode, c->u_rows_per_kv, c->u_parts, c->sum_T, scores_kv, scores_agg);
  c->launches += 1;
  ASL_CUDA(cudaGetLastError());
  return ASL_OK;
}
