// Per-(request, head) top-k with the window appended (Algorithm 1 lines 7-8).
//
// Radix select on an order-preserving 32-bit image of the fp32 score: four
// most-significant-digit passes (8 bits each) find the exact k-th largest key;
// every token with a larger key is kept, and of the tokens that equal it the
// lowest-indexed ones fill the remainder.  An ordered block scan then emits the
// kept indices in ascending order, followed by T .. n-1.
#include "asl_internal.cuh"

namespace {

constexpr int THREADS = 1024;
constexpr int PER_THREAD = 4;
constexpr int CHUNK = THREADS * PER_THREAD;

__device__ __forceinline__ uint32_t asc_key(float s) {
  uint32_t u = __float_as_uint(s);
  if (u == 0x80000000u) u = 0;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__global__ void __launch_bounds__(THREADS) topk_select_kernel(const float* __restrict__ scores,
                                                              const AslReq* __restrict__ req, int64_t sum_T,
                                                              int64_t sum_kept, int32_t* __restrict__ idx_out) {
  __shared__ int hist[256];
  __shared__ uint32_t s_prefix;
  __shared__ int s_remaining;
  __shared__ int warp_sums[THREADS / 32];
  const int b = blockIdx.y, h = blockIdx.x;
  const AslReq rq = req[b];
  const float* row = scores + (int64_t)h * sum_T + rq.t_off;
  int32_t* out = idx_out + (int64_t)h * sum_kept + rq.kept_off;
  const int T = rq.T, k = rq.k;
  const int tid = threadIdx.x;

  // window indices (Algorithm 1 line 8)
  for (int t = tid; t < rq.kept - k; t += THREADS) out[k + t] = T + t;
  if (k == 0) return;

  // ---- exact k-th largest key -------------------------------------------------
  uint32_t prefix = 0, mask = 0;
  int remaining = k;     // rank of the wanted key among keys matching the prefix (1 = largest)
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    for (int i = tid; i < T; i += THREADS) {
      const uint32_t u = asc_key(row[i]);
      if ((u & mask) == prefix) atomicAdd(&hist[(u >> shift) & 255], 1);
    }
    __syncthreads();
    if (tid == 0) {
      int rem = remaining, d = 255;
      for (; d > 0; --d) {
        if (hist[d] >= rem) break;
        rem -= hist[d];
      }
      s_prefix = prefix | ((uint32_t)d << shift);
      s_remaining = rem;
    }
    __syncthreads();
    prefix = s_prefix;
    remaining = s_remaining;
    mask |= 0xFFu << shift;
    __syncthreads();
  }
  const uint32_t thr = prefix;       // k-th largest key
  const int need = remaining;        // how many keys equal to thr are kept (lowest indices)

  // ---- ordered emit -------------------------------------------------------------
  const int lane = tid & 31, wid = tid >> 5;
  int run_gt = 0, run_eq = 0;        // kept-larger / equal counts before this chunk
  for (int c0 = 0; c0 < T; c0 += CHUNK) {
    const int i0 = c0 + tid * PER_THREAD;
    uint32_t u[PER_THREAD];
    int packed = 0;                  // (larger << 16) | equal, each <= 4096*... per chunk <= CHUNK < 65536
#pragma unroll
    for (int e = 0; e < PER_THREAD; ++e) {
      const int i = i0 + e;
      u[e] = (i < T) ? asc_key(row[i]) : 0u;
      if (i < T) packed += (u[e] > thr) ? (1 << 16) : ((u[e] == thr) ? 1 : 0);
    }
    int incl = packed;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) warp_sums[wid] = incl;
    __syncthreads();
    int base = 0, total = 0;
    for (int w2 = 0; w2 < THREADS / 32; ++w2) {
      const int v = warp_sums[w2];
      if (w2 < wid) base += v;
      total += v;
    }
    int excl = base + incl - packed;
    int gt_before = run_gt + (excl >> 16), eq_before = run_eq + (excl & 0xFFFF);
#pragma unroll
    for (int e = 0; e < PER_THREAD; ++e) {
      const int i = i0 + e;
      if (i < T) {
        if (u[e] > thr) {
          out[gt_before + min(eq_before, need)] = i;
          ++gt_before;
        } else if (u[e] == thr) {
          if (eq_before < need) out[gt_before + eq_before] = i;
          ++eq_before;
        }
      }
    }
    run_gt += total >> 16;
    run_eq += total & 0xFFFF;
    __syncthreads();
  }
}

}  // namespace

asl_status asl_launch_topk(asl_ctx* c, const float* scores, int32_t n_heads, int32_t* idx_out, cudaStream_t st) {
  topk_select_kernel<<<dim3(n_heads, c->p.batch), THREADS, 0, st>>>(scores, c->d_req, c->sum_T, c->sum_kept, idx_out);
  c->launches += 1;
  ASL_CUDA(cudaGetLastError());
  return ASL_OK;
}
