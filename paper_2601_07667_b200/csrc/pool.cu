// 1-D pooling, GQA group sum and all-head aggregate (Algorithm 1 lines 5-6 and
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

__global__ void __launch_bounds__(256) pool_group_kernel(const float* __restrict__ u, const AslReq* __restrict__ req,
                                                         int Hk, int G, int S, int mode, int urows, int parts, int64_t sum_T,
                                                         float* __restrict__ scores_kv, float* __restrict__ scores_agg) {
  const int b = blockIdx.y;
  const AslReq rq = req[b];
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= rq.T) return;
  const int r = S / 2;
  const int lo = max(0, j - r), hi = min(rq.T - 1, j + r);
  const float inv = 1.0f / (float)S;
  float agg = 0.f;
  for (int h = 0; h < Hk; ++h) {
    float p;
    if (mode == ASL_POOL_AVG) {
      float s = 0.f;
      for (int c = 0; c < urows; ++c) {
        const float* row = u + (int64_t)(h * urows + c) * sum_T + rq.t_off;
        for (int i = lo; i <= hi; ++i) s += row[i];
      }
      p = s * inv;
    } else {
      p = 0.f;
      for (int g = 0; g < G; ++g) {
        const float* row = u + (int64_t)(h * G + g) * parts * sum_T + rq.t_off;
        float mx = -INFINITY;
        for (int i = lo; i <= hi; ++i) {
          float v = row[i];
          for (int c = 1; c < parts; ++c) v += row[(int64_t)c * sum_T + i];     // partial sums of one head come first
          mx = fmaxf(mx, v);
        }
        p += mx;
      }
    }
    scores_kv[(int64_t)h * sum_T + rq.t_off + j] = p;
    agg += p;
  }
  scores_agg[rq.t_off + j] = agg;
}

}  // namespace

asl_status asl_launch_pool(asl_ctx* c, const float* u, float* scores_kv, float* scores_agg, cudaStream_t st) {
  const asl_params& p = c->p;
  dim3 grid((c->max_T + 255) / 256, p.batch);
  pool_group_kernel<<<grid, 256, 0, st>>>(u, c->d_req, p.n_kv_heads, p.n_q_heads / p.n_kv_heads, p.pool_kernel,
                                          p.pool_mode, c->u_rows_per_kv, c->u_parts, c->sum_T, scores_kv, scores_agg);
  c->launches += 1;
  ASL_CUDA(cudaGetLastError());
  return ASL_OK;
}
