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

constexpr int HB = 8;            // staged rows per round: their loads are all in flight together

// One block pools PT consecutive past tokens of one request.  A "unit" is what
// gets pooled as one row: a kv head's group-summed sums (average pooling) or one
// query head's sums (max pooling); it is stored as `nrows` consecutive partial
// rows of u that are added on the way into shared memory.  HB units are staged
// per round with their halo, pooled from there, and added up per kv head and
// over all heads in a fixed order: no atomics, bit-reproducible.
__global__ void __launch_bounds__(PT + 2 * MAX_HALO) pool_group_kernel(const float* __restrict__ u, const AslReq* __restrict__ req,
                                                        int Hk, int G, int S, int mode, int urows, int parts, int64_t sum_T,
                                                        const asl_stat* __restrict__ latch, int cur_layer,
                                                        float* __restrict__ scores_kv, float* __restrict__ scores_agg) {
  __shared__ float tile[HB][PT + 2 * MAX_HALO];
  const int b = blockIdx.y;
  if (latch && asl_finished(latch + b, cur_layer)) return;      // the request's scores stay as its selection layer left them
  const AslReq rq = req[b];
  const int j0 = blockIdx.x * PT;
  if (j0 >= rq.T) return;
  const int r = S / 2;
  const int j = j0 + threadIdx.x;
  const bool live = threadIdx.x < PT && j < rq.T;      // the last 2 * MAX_HALO threads only load halo columns
  const int lo = max(0, j - r), hi = min(rq.T - 1, j + r);
  const float inv = 1.0f / (float)S;
  const bool avg = mode == ASL_POOL_AVG;
  const int units = avg ? Hk : Hk * G;
  const int nrows = avg ? urows : parts;
  const int per_head = avg ? 1 : G;
  float agg = 0.f, p = 0.f;
  for (int u0 = 0; u0 < units; u0 += HB) {
    const int nb = min(HB, units - u0);
    const int tot = nb * nrows;                       // rows u0*nrows .. u0*nrows + tot - 1 of u
    __syncthreads();
    if (threadIdx.x < PT + 2 * r) {                     // one column of the tile per thread, halo included
      const int i = threadIdx.x;
      const int t = j0 - r + i;
      const bool inside = t >= 0 && t < rq.T;
      const float* src = u + (int64_t)u0 * nrows * sum_T + rq.t_off + t;
#pragma unroll
      for (int q = 0; q < HB; ++q) tile[q][i] = 0.f;
      for (int e0 = 0; e0 < tot; e0 += 16) {            // sixteen loads in flight
        float x[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) x[k] = (inside && e0 + k < tot) ? __ldcg(src + (int64_t)(e0 + k) * sum_T) : 0.f;
#pragma unroll
        for (int k = 0; k < 16; ++k)
          if (e0 + k < tot) tile[(e0 + k) / nrows][i] += x[k];
      }
    }
    __syncthreads();
    for (int q = 0; q < nb; ++q) {
      if (live) {
        if (avg) {
          float s = 0.f;
          for (int i = lo; i <= hi; ++i) s += tile[q][i - j0 + r];
          p = s * inv;
        } else {
          float mx = tile[q][lo - j0 + r];
          for (int i = lo + 1; i <= hi; ++i) mx = fmaxf(mx, tile[q][i - j0 + r]);
          p += mx;
        }
      }
      const int unit = u0 + q;
      if ((unit + 1) % per_head == 0) {
        if (live) scores_kv[(int64_t)(unit / per_head) * sum_T + rq.t_off + j] = p;
        agg += p;
        p = 0.f;
      }
    }
  }
  if (live) scores_agg[rq.t_off + j] = agg;
}

// Average pooling without shared memory, for plans whose segments all start and end on 16-byte boundaries of the
// score rows (T_b and the rows' length multiples of 4) and whose pooling window reaches at most 4 tokens to a
// side.  A lane owns 4 consecutive tokens: one 16-byte load per partial row, all of a batch of rows in flight, the
// rows of a kv head added in order, the neighbours' sums fetched by warp shuffles; the first and the last lane of
// a warp only supply the halo, so a warp pools 120 tokens.  One round trip to memory and no block-wide barrier; the
// sums are formed in the same order as in the kernel above, so the two give identical bits.
constexpr int PV_ROWS = 16;      // partial rows in flight per lane

__global__ void __launch_bounds__(PT) pool_avg_vec4_kernel(const float* __restrict__ u, const AslReq* __restrict__ req, int Hk, int S,
                                                           int urows, int64_t sum_T, const asl_stat* __restrict__ latch, int cur_layer,
                                                           float* __restrict__ scores_kv, float* __restrict__ scores_agg) {
  const int b = blockIdx.y;
  if (latch && asl_finished(latch + b, cur_layer)) return;
  const AslReq rq = req[b];
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const int warp_of_segment = blockIdx.x * (PT / 32) + wid;
  if (warp_of_segment * 120 >= rq.T) return;                           // the whole warp is past the segment
  const int g = warp_of_segment * 30 + lane - 1;                       // group of 4 tokens; lanes 0 and 31: halo only
  const int j0 = 4 * g;
  const bool inside = g >= 0 && j0 < rq.T;
  const bool owner = inside && lane >= 1 && lane <= 30;
  const int r = S / 2;
  const float inv = 1.0f / (float)S;
  const float* base = u + rq.t_off + j0;
  float agg[4] = {0.f, 0.f, 0.f, 0.f};
  const int heads_per_batch = PV_ROWS / urows;                         // urows divides PV_ROWS (checked by the launcher)
  for (int h0 = 0; h0 < Hk; h0 += heads_per_batch) {
    float4 x[PV_ROWS];
#pragma unroll
    for (int e = 0; e < PV_ROWS; ++e) {
      const int row = h0 * urows + e;
      x[e] = (inside && row < Hk * urows) ? __ldcg(reinterpret_cast<const float4*>(base + (int64_t)row * sum_T)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    for (int hh = 0; hh < heads_per_batch && h0 + hh < Hk; ++hh) {
      float v[12];                                                     // sums of tokens j0-4 .. j0+7
      float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int e = 0; e < PV_ROWS; ++e)
        if (e / urows == hh) { sum.x += x[e].x; sum.y += x[e].y; sum.z += x[e].z; sum.w += x[e].w; }
      v[4] = sum.x; v[5] = sum.y; v[6] = sum.z; v[7] = sum.w;
      v[0] = __shfl_up_sync(0xffffffffu, sum.x, 1); v[1] = __shfl_up_sync(0xffffffffu, sum.y, 1);
      v[2] = __shfl_up_sync(0xffffffffu, sum.z, 1); v[3] = __shfl_up_sync(0xffffffffu, sum.w, 1);
      v[8] = __shfl_down_sync(0xffffffffu, sum.x, 1); v[9] = __shfl_down_sync(0xffffffffu, sum.y, 1);
      v[10] = __shfl_down_sync(0xffffffffu, sum.z, 1); v[11] = __shfl_down_sync(0xffffffffu, sum.w, 1);
      float p[4];
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        float acc = 0.f;
#pragma unroll
        for (int d = -4; d <= 4; ++d)
          if (d >= -r && d <= r) acc += v[4 + t + d];                  // tokens outside the segment hold 0: zero padding
        p[t] = acc * inv;
        agg[t] += p[t];
      }
      if (owner) *reinterpret_cast<float4*>(scores_kv + (int64_t)(h0 + hh) * sum_T + rq.t_off + j0) = make_float4(p[0], p[1], p[2], p[3]);
    }
  }
  if (owner) *reinterpret_cast<float4*>(scores_agg + rq.t_off + j0) = make_float4(agg[0], agg[1], agg[2], agg[3]);
}

}  // namespace

asl_status asl_launch_pool(asl_ctx* c, const float* u, float* scores_kv, float* scores_agg, cudaStream_t st) {
  const asl_params& p = c->p;
  if (p.pool_kernel / 2 > MAX_HALO) return ASL_ERR_UNSUPPORTED;
  const int urows = c->u_rows_per_kv;
  bool vec4 = p.pool_mode == ASL_POOL_AVG && p.pool_kernel / 2 <= 4 && urows <= PV_ROWS && PV_ROWS % urows == 0 && c->sum_T % 4 == 0 &&
              ((reinterpret_cast<uintptr_t>(u) | reinterpret_cast<uintptr_t>(scores_kv) | reinterpret_cast<uintptr_t>(scores_agg)) & 15) == 0;
  for (const AslReq& r : c->req) vec4 = vec4 && r.T % 4 == 0 && r.t_off % 4 == 0;
  if (vec4) {
    const int warps = c->max_T > 0 ? (c->max_T + 119) / 120 : 1;
    pool_avg_vec4_kernel<<<dim3((warps + PT / 32 - 1) / (PT / 32), p.batch), PT, 0, st>>>(
        u, c->d_req, p.n_kv_heads, p.pool_kernel, urows, c->sum_T, c->latch_stat, c->cur_layer, scores_kv, scores_agg);
    c->launches += 1;
    ASL_CUDA(cudaGetLastError());
    return ASL_OK;
  }
  dim3 grid((c->max_T + PT - 1) / PT, p.batch);
  pool_group_kernel<<<grid, PT + 2 * MAX_HALO, 0, st>>>(u, c->d_req, p.n_kv_heads, p.n_q_heads / p.n_kv_heads, p.pool_kernel,
                                          p.pool_mode, c->u_rows_per_kv, c->u_parts, c->sum_T, c->latch_stat, c->cur_layer,
                                          scores_kv, scores_agg);
  c->launches += 1;
  ASL_CUDA(cudaGetLastError());
  return ASL_OK;
}
