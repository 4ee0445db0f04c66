// Per-(request, head) top-k with the window appended (Algorithm 1 (k, TopK and window append)).
//
// Radix select on an order-preserving 32-bit image of the fp32 score, 11+11+10
// bits from the top: the exact k-th largest key is found; every token with a
// larger key is kept, and of the tokens equal to it the lowest-indexed fill the
// remainder.  One thread-block cluster (up to 8 CTAs of 1024 threads) works on
// one (request, head): each thread keeps 16 consecutive scores in registers,
// CTAs histogram their slices in shared memory, read each other's histograms
// through distributed shared memory and agree on the digit; an ordered scan
// then emits the kept indices in ascending order, followed by T .. n-1.
// Segments longer than cluster x 16384 are walked in rounds and re-read from L2.
#include <cooperative_groups.h>

#include "asl_internal.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int THREADS = 1024;
constexpr int PER_THREAD = 16;
constexpr int SLICE = THREADS * PER_THREAD;   // scores per CTA per round
constexpr int BINS = 2048;
constexpr int MAX_CL = 8;
constexpr int MAX_ROUNDS = 64;

__device__ __forceinline__ uint32_t asc_key(float s) {
  uint32_t u = __float_as_uint(s);
  if (u == 0x80000000u) u = 0;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct Shared {
  int hist[BINS];
  int tot[BINS];
  int warp_a[32], warp_b[32];
  int counts[MAX_ROUNDS][2];     // this CTA's (larger, equal) counts per round
  uint32_t prefix;
  int remaining;
};

template <bool CACHED>
__global__ void __launch_bounds__(THREADS) topk_cluster_kernel(const float* __restrict__ scores,
                                                               const AslReq* __restrict__ req, int64_t sum_T,
                                                               int64_t sum_kept, int32_t* __restrict__ idx_out) {
  __shared__ Shared sh;
  cg::cluster_group cluster = cg::this_cluster();
  const int CL = (int)cluster.num_blocks();
  const int r = (int)cluster.block_rank();
  const int b = blockIdx.z, h = blockIdx.y;
  const AslReq rq = req[b];
  const float* row = scores + (int64_t)h * sum_T + rq.t_off;
  int32_t* out = idx_out + (int64_t)h * sum_kept + rq.kept_off;
  const int T = rq.T, k = rq.k;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int rounds = (T + CL * SLICE - 1) / (CL * SLICE);

  // window indices (Algorithm 1 (TopK and window append))
  for (int t = r * THREADS + tid; t < rq.kept - k; t += CL * THREADS) out[k + t] = T + t;
  if (k == 0) return;                      // uniform over the cluster: nobody waits for anybody

  uint32_t key[PER_THREAD];
  auto load_round = [&](int rho) {
    const int i0 = (rho * CL + r) * SLICE + tid * PER_THREAD;
#pragma unroll
    for (int e = 0; e < PER_THREAD; ++e) key[e] = (i0 + e < T) ? asc_key(__ldg(row + i0 + e)) : 0u;
  };
  if (CACHED) load_round(0);

  // ---- exact k-th largest key: three digit passes ---------------------------------
  uint32_t prefix = 0, mask = 0;
  int remaining = k;
  const int shifts[3] = {21, 10, 0};
  const int widths[3] = {11, 11, 10};
  for (int pass = 0; pass < 3; ++pass) {
    const int shift = shifts[pass];
    const uint32_t dmask = (1u << widths[pass]) - 1u;
    for (int i = tid; i < BINS; i += THREADS) sh.hist[i] = 0;
    __syncthreads();
    for (int rho = 0; rho < rounds; ++rho) {
      if (!CACHED) load_round(rho);
      const int i0 = (rho * CL + r) * SLICE + tid * PER_THREAD;
#pragma unroll
      for (int e = 0; e < PER_THREAD; ++e) {
        const bool in = (i0 + e < T) && ((key[e] & mask) == prefix);
        if (in) atomicAdd(&sh.hist[(key[e] >> shift) & dmask], 1);     // shared-memory atomic: conflicts replay in hardware
      }
    }
    cluster.sync();                        // every CTA's histogram is complete
    for (int i = tid; i < BINS; i += THREADS) {
      int s = 0;
      for (int c = 0; c < CL; ++c) s += cluster.map_shared_rank(sh.hist, c)[i];
      sh.tot[i] = s;
    }
    cluster.sync();                        // remote reads done: histograms may be cleared again
    // suffix sums from the top bin: thread t owns bins 2047-2t and 2046-2t
    const int hi = BINS - 1 - 2 * tid, lo = hi - 1;
    const int c_hi = sh.tot[hi], c_lo = sh.tot[lo];
    int incl = c_hi + c_lo;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) sh.warp_a[wid] = incl;
    __syncthreads();
    int base = 0;
    for (int w2 = 0; w2 < wid; ++w2) base += sh.warp_a[w2];
    const int before_hi = base + incl - (c_hi + c_lo);     // keys in bins above `hi`
    const int before_lo = before_hi + c_hi;
    if (before_hi < remaining && remaining <= before_hi + c_hi) {
      sh.prefix = prefix | ((uint32_t)hi << shift);
      sh.remaining = remaining - before_hi;
    } else if (before_lo < remaining && remaining <= before_lo + c_lo) {
      sh.prefix = prefix | ((uint32_t)lo << shift);
      sh.remaining = remaining - before_lo;
    }
    __syncthreads();
    prefix = sh.prefix;
    remaining = sh.remaining;
    mask |= dmask << shift;
    __syncthreads();
  }
  const uint32_t thr = prefix;             // the k-th largest key
  const int need = remaining;              // keys equal to thr that are kept (lowest indices first)

  // ---- counts per (round, CTA), then the ordered emit -------------------------------
  for (int rho = 0; rho < rounds; ++rho) {
    if (!CACHED) load_round(rho);
    const int i0 = (rho * CL + r) * SLICE + tid * PER_THREAD;
    int gt = 0, eq = 0;
#pragma unroll
    for (int e = 0; e < PER_THREAD; ++e) {
      if (i0 + e < T) { gt += key[e] > thr; eq += key[e] == thr; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      gt += __shfl_down_sync(0xffffffffu, gt, o);
      eq += __shfl_down_sync(0xffffffffu, eq, o);
    }
    if (lane == 0) { sh.warp_a[wid] = gt; sh.warp_b[wid] = eq; }
    __syncthreads();
    if (tid == 0) {
      int g = 0, q = 0;
      for (int w2 = 0; w2 < 32; ++w2) { g += sh.warp_a[w2]; q += sh.warp_b[w2]; }
      sh.counts[rho][0] = g;
      sh.counts[rho][1] = q;
    }
    __syncthreads();
  }
  cluster.sync();                          // every CTA's counts are visible
  int run_gt = 0, run_eq = 0;              // kept-larger / equal keys before this CTA's slice of round 0
  for (int c = 0; c < r; ++c) {
    const int(*rc)[2] = cluster.map_shared_rank(sh.counts, c);
    run_gt += rc[0][0];
    run_eq += rc[0][1];
  }
  for (int rho = 0; rho < rounds; ++rho) {
    if (!CACHED) load_round(rho);
    const int i0 = (rho * CL + r) * SLICE + tid * PER_THREAD;
    int gt = 0, eq = 0;
#pragma unroll
    for (int e = 0; e < PER_THREAD; ++e) {
      if (i0 + e < T) { gt += key[e] > thr; eq += key[e] == thr; }
    }
    int ig = gt, ie = eq;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int vg = __shfl_up_sync(0xffffffffu, ig, o), ve = __shfl_up_sync(0xffffffffu, ie, o);
      if (lane >= o) { ig += vg; ie += ve; }
    }
    __syncthreads();
    if (lane == 31) { sh.warp_a[wid] = ig; sh.warp_b[wid] = ie; }
    __syncthreads();
    int gt_before = run_gt + ig - gt, eq_before = run_eq + ie - eq;
    for (int w2 = 0; w2 < wid; ++w2) { gt_before += sh.warp_a[w2]; eq_before += sh.warp_b[w2]; }
#pragma unroll
    for (int e = 0; e < PER_THREAD; ++e) {
      const int i = i0 + e;
      if (i < T) {
        if (key[e] > thr) {
          out[gt_before + min(eq_before, need)] = i;
          ++gt_before;
        } else if (key[e] == thr) {
          if (eq_before < need) out[gt_before + eq_before] = i;
          ++eq_before;
        }
      }
    }
    if (rho + 1 < rounds) {                // counts of the slices between this one and ours in the next round
      for (int c = r; c < CL; ++c) {
        const int(*rc)[2] = cluster.map_shared_rank(sh.counts, c);
        run_gt += rc[rho][0];
        run_eq += rc[rho][1];
      }
      for (int c = 0; c < r; ++c) {
        const int(*rc)[2] = cluster.map_shared_rank(sh.counts, c);
        run_gt += rc[rho + 1][0];
        run_eq += rc[rho + 1][1];
      }
    }
  }
  cluster.sync();                          // no CTA leaves while its shared memory may still be read
}

}  // namespace

asl_status asl_launch_topk(asl_ctx* c, const float* scores, int32_t n_heads, int32_t* idx_out, cudaStream_t st) {
  int cl = (c->max_T + SLICE - 1) / SLICE;
  if (cl < 1) cl = 1;
  if (cl > MAX_CL) cl = MAX_CL;
  const int rounds = (c->max_T + cl * SLICE - 1) / (cl * SLICE);
  if (rounds > MAX_ROUNDS) return ASL_ERR_UNSUPPORTED;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(cl, n_heads, c->p.batch);
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cl;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const AslReq* req = c->d_req;
  int64_t sum_T = c->sum_T, sum_kept = c->sum_kept;
  cudaError_t e;
  if (rounds == 1) e = cudaLaunchKernelEx(&cfg, topk_cluster_kernel<true>, scores, req, sum_T, sum_kept, idx_out);
  else             e = cudaLaunchKernelEx(&cfg, topk_cluster_kernel<false>, scores, req, sum_T, sum_kept, idx_out);
  c->launches += 1;
  if (e != cudaSuccess) return ASL_ERR_CUDA;
  return ASL_OK;
}
