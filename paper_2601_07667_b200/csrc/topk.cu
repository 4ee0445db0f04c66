// Per-(request, head) top-k with the window appended (Algorithm 1 (k, TopK and window append)).
//
// Radix select on an order-preserving 32-bit image of the fp32 score, 11+11+10
// bits from the top: the exact k-th largest key is found; every token with a
// larger key is kept, and of the tokens equal to it the lowest-indexed fill the
// remainder.  The work is cut into tiles of 4096 scores, one 256-thread CTA per
// tile with its 16 scores per thread in registers, and into five short kernels
// that meet only through global memory:
//
//   digit 1 histogram -> pick + digit 2 histogram -> pick + digit 3 histogram
//   -> pick + per-tile counts of larger / equal keys -> ordered emit
//
// Every CTA of a kernel repeats the (cheap) pick of the previous digit from the
// segment's global histogram, so no kernel waits for another CTA, and no CTA
// needs a neighbour on a particular SM: the kernels run on whatever SMs a
// concurrently running persistent kernel leaves free.  The emit writes the kept
// indices in ascending order, followed by T .. n-1.
#include "asl_internal.cuh"

namespace {

constexpr int THREADS = 256;
constexpr int PER_THREAD = 16;
constexpr int TILE = THREADS * PER_THREAD;    // scores per CTA
constexpr int BINS = 2048;
constexpr int STATE_INTS = 8;                 // per segment: prefix/remaining after each digit
constexpr int SEG_INTS = 3 * BINS + STATE_INTS;

__device__ __forceinline__ uint32_t asc_key(float s) {
  uint32_t u = __float_as_uint(s);
  if (u == 0x80000000u) u = 0;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct TopkArgs {
  const float* scores;
  const AslReq* req;
  int32_t* scratch;      // [segments][SEG_INTS]
  int32_t* counts;       // [segments][max_tiles][2]
  int32_t* idx_out;
  int64_t sum_T, sum_kept;
  int32_t n_heads, max_tiles;
  const asl_stat* gate;  // null, or: only requests whose statistic selected at layer `gate_layer` are worked on
  int32_t gate_layer;
  const asl_stat* latch; // null, or: requests that finished before layer `cur_layer` are left alone
  int32_t cur_layer;
};

struct Segment {
  const float* row;
  int32_t* hist;         // three tables of BINS
  int32_t* state;
  int32_t* counts;
  int32_t* out;
  int T, k, kept, tile;
  bool open;             // false: the gate keeps this request's list as it is
};

__device__ __forceinline__ Segment segment_of(const TopkArgs& a) {
  const int b = blockIdx.z, h = blockIdx.y;
  const AslReq rq = a.req[b];
  const int64_t seg = (int64_t)b * a.n_heads + h;
  Segment s;
  s.open = !a.gate || (a.gate[b].selected && a.gate[b].layer_idx == a.gate_layer);
  if (a.latch && asl_finished(a.latch + b, a.cur_layer)) s.open = false;
  s.row = a.scores + (int64_t)h * a.sum_T + rq.t_off;
  s.hist = a.scratch + seg * SEG_INTS;
  s.state = s.hist + 3 * BINS;
  s.counts = a.counts + seg * a.max_tiles * 2;
  s.out = a.idx_out + (int64_t)h * a.sum_kept + rq.kept_off;
  s.T = rq.T; s.k = rq.k; s.kept = rq.kept; s.tile = blockIdx.x;
  return s;
}

__device__ __forceinline__ void load_keys(const Segment& s, uint32_t (&key)[PER_THREAD]) {
  const int i0 = s.tile * TILE + threadIdx.x * PER_THREAD;
  if (i0 + PER_THREAD <= s.T && ((reinterpret_cast<uintptr_t>(s.row + i0) & 15) == 0)) {
#pragma unroll
    for (int q = 0; q < PER_THREAD / 4; ++q) {
      const float4 v = __ldg(reinterpret_cast<const float4*>(s.row + i0) + q);
      key[4 * q] = asc_key(v.x); key[4 * q + 1] = asc_key(v.y); key[4 * q + 2] = asc_key(v.z); key[4 * q + 3] = asc_key(v.w);
    }
  } else {
#pragma unroll
    for (int e = 0; e < PER_THREAD; ++e) key[e] = (i0 + e < s.T) ? asc_key(__ldg(s.row + i0 + e)) : 0u;
  }
}

// The bin (counted from the top) that holds the `remaining`-th largest key of a
// table of `bins` counts, and how many keys of that bin are still wanted.
// Thread t owns the bins/THREADS bins just below bins-1-t*(bins/THREADS).
template <int PER>
__device__ __forceinline__ void pick(const int32_t* __restrict__ table, int remaining, int& bin, int& rem_out) {
  __shared__ int warp_tot[THREADS / 32];
  __shared__ int found[2];
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int top = PER * THREADS - 1 - PER * tid;       // highest bin of this thread
  int c[PER];
  int sum = 0;
#pragma unroll
  for (int j = 0; j < PER; ++j) { c[j] = __ldcg(table + top - j); sum += c[j]; }
  int incl = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) warp_tot[wid] = incl;
  __syncthreads();
  int above = incl - sum;                              // keys in bins above this thread's
  for (int w2 = 0; w2 < wid; ++w2) above += warp_tot[w2];
  if (above < remaining && remaining <= above + sum) {
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      if (above < remaining && remaining <= above + c[j]) { found[0] = top - j; found[1] = remaining - above; }
      above += c[j];
    }
  }
  __syncthreads();
  bin = found[0];
  rem_out = found[1];
  __syncthreads();
}

// counts the digit (key >> shift) & dmask of the keys whose bits under `mask` equal `prefix`
__device__ __forceinline__ void tile_histogram(const Segment& s, const uint32_t (&key)[PER_THREAD], uint32_t mask,
                                               uint32_t prefix, int shift, uint32_t dmask, int32_t* __restrict__ table) {
  __shared__ int hist[BINS];
  const int tid = threadIdx.x;
  for (int i = tid; i < BINS; i += THREADS) hist[i] = 0;
  __syncthreads();
  const int i0 = s.tile * TILE + tid * PER_THREAD;
  int run_bin = -1, run = 0;                           // neighbouring scores often share a digit: one atomic per run
#pragma unroll
  for (int e = 0; e < PER_THREAD; ++e) {
    const bool in = (i0 + e < s.T) && ((key[e] & mask) == prefix);
    const int d = (int)((key[e] >> shift) & dmask);
    if (in && d == run_bin) { ++run; continue; }
    if (run) atomicAdd(&hist[run_bin], run);
    run_bin = in ? d : -1;
    run = in ? 1 : 0;
  }
  if (run) atomicAdd(&hist[run_bin], run);
  __syncthreads();
  for (int i = tid; i < BINS; i += THREADS) {
    const int v = hist[i];
    if (v) atomicAdd(table + i, v);
  }
}

// stage 0: digit 1 histogram; stage 1 / 2: pick the previous digit, histogram the next
template <int STAGE>
__global__ void __launch_bounds__(THREADS) topk_digit_kernel(TopkArgs a) {
  const Segment s = segment_of(a);
  if (!s.open || s.k == 0 || s.tile * TILE >= s.T) return;
  uint32_t key[PER_THREAD];
  load_keys(s, key);
  if (STAGE == 0) {
    tile_histogram(s, key, 0u, 0u, 21, 2047u, s.hist);
  } else if (STAGE == 1) {
    int bin, rem;
    pick<8>(s.hist, s.k, bin, rem);
    if (s.tile == 0 && threadIdx.x == 0) { s.state[0] = bin; s.state[1] = rem; }
    tile_histogram(s, key, 2047u << 21, (uint32_t)bin << 21, 10, 2047u, s.hist + BINS);
  } else {
    const int bin1 = __ldcg(s.state + 0), rem1 = __ldcg(s.state + 1);
    int bin, rem;
    pick<8>(s.hist + BINS, rem1, bin, rem);
    if (s.tile == 0 && threadIdx.x == 0) { s.state[2] = bin; s.state[3] = rem; }
    const uint32_t prefix = ((uint32_t)bin1 << 21) | ((uint32_t)bin << 10);
    tile_histogram(s, key, 0xfffffc00u, prefix, 0, 1023u, s.hist + 2 * BINS);
  }
}

// the k-th largest key and the number of keys equal to it that are kept; per-tile counts
__global__ void __launch_bounds__(THREADS) topk_count_kernel(TopkArgs a) {
  __shared__ int w_gt[THREADS / 32], w_eq[THREADS / 32];
  const Segment s = segment_of(a);
  if (!s.open || s.k == 0 || s.tile * TILE >= s.T) return;
  uint32_t key[PER_THREAD];
  load_keys(s, key);
  const int bin1 = __ldcg(s.state + 0), bin2 = __ldcg(s.state + 2), rem2 = __ldcg(s.state + 3);
  int bin, need;
  pick<4>(s.hist + 2 * BINS, rem2, bin, need);
  const uint32_t thr = ((uint32_t)bin1 << 21) | ((uint32_t)bin2 << 10) | (uint32_t)bin;
  if (s.tile == 0 && threadIdx.x == 0) { s.state[4] = (int32_t)thr; s.state[5] = need; }
  const int i0 = s.tile * TILE + threadIdx.x * PER_THREAD;
  int gt = 0, eq = 0;
#pragma unroll
  for (int e = 0; e < PER_THREAD; ++e) {
    if (i0 + e < s.T) { gt += key[e] > thr; eq += key[e] == thr; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    gt += __shfl_down_sync(0xffffffffu, gt, o);
    eq += __shfl_down_sync(0xffffffffu, eq, o);
  }
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  if (lane == 0) { w_gt[wid] = gt; w_eq[wid] = eq; }
  __syncthreads();
  if (threadIdx.x == 0) {
    int g = 0, q = 0;
    for (int w2 = 0; w2 < THREADS / 32; ++w2) { g += w_gt[w2]; q += w_eq[w2]; }
    s.counts[2 * s.tile] = g;
    s.counts[2 * s.tile + 1] = q;
  }
}

// ordered emit (Algorithm 1 (TopK and window append))
__global__ void __launch_bounds__(THREADS) topk_emit_kernel(TopkArgs a) {
  __shared__ int w_gt[THREADS / 32], w_eq[THREADS / 32];
  const Segment s = segment_of(a);
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int tiles = max(1, (s.T + TILE - 1) / TILE);
  if (!s.open || s.tile >= tiles) return;
  for (int t = s.tile * THREADS + tid; t < s.kept - s.k; t += tiles * THREADS) s.out[s.k + t] = s.T + t;   // the window
  if (s.k == 0) return;
  uint32_t key[PER_THREAD];
  load_keys(s, key);
  const uint32_t thr = (uint32_t)__ldcg(s.state + 4);
  const int need = __ldcg(s.state + 5);
  // larger / equal keys in the tiles before this one
  int run_gt = 0, run_eq = 0;
  for (int t = tid; t < s.tile; t += THREADS) { run_gt += __ldcg(s.counts + 2 * t); run_eq += __ldcg(s.counts + 2 * t + 1); }
  const int i0 = s.tile * TILE + tid * PER_THREAD;
  int gt = 0, eq = 0;
#pragma unroll
  for (int e = 0; e < PER_THREAD; ++e) {
    if (i0 + e < s.T) { gt += key[e] > thr; eq += key[e] == thr; }
  }
  // block totals of the look-behind sums, block-exclusive scans of this tile's counts
  int tg = run_gt, te = run_eq, ig = gt, ie = eq;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    tg += __shfl_xor_sync(0xffffffffu, tg, o);
    te += __shfl_xor_sync(0xffffffffu, te, o);
  }
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int vg = __shfl_up_sync(0xffffffffu, ig, o), ve = __shfl_up_sync(0xffffffffu, ie, o);
    if (lane >= o) { ig += vg; ie += ve; }
  }
  __shared__ int b_gt[THREADS / 32], b_eq[THREADS / 32];
  if (lane == 31) { w_gt[wid] = ig; w_eq[wid] = ie; }
  if (lane == 0) { b_gt[wid] = tg; b_eq[wid] = te; }
  __syncthreads();
  int gt_before = ig - gt, eq_before = ie - eq;
  for (int w2 = 0; w2 < THREADS / 32; ++w2) {
    gt_before += b_gt[w2];
    eq_before += b_eq[w2];
    if (w2 < wid) { gt_before += w_gt[w2]; eq_before += w_eq[w2]; }
  }
#pragma unroll
  for (int e = 0; e < PER_THREAD; ++e) {
    const int i = i0 + e;
    if (i < s.T) {
      if (key[e] > thr) {
        s.out[gt_before + min(eq_before, need)] = i;
        ++gt_before;
      } else if (key[e] == thr) {
        if (eq_before < need) s.out[gt_before + eq_before] = i;
        ++eq_before;
      }
    }
  }
}

}  // namespace

size_t asl_topk_scratch_bytes(int64_t segments, int64_t max_T) {
  const int64_t tiles = (max_T + TILE - 1) / TILE > 0 ? (max_T + TILE - 1) / TILE : 1;
  return (size_t)(segments * SEG_INTS + segments * tiles * 2) * sizeof(int32_t);
}

asl_status asl_launch_topk(asl_ctx* c, const float* scores, int32_t n_heads, int32_t* idx_out, const asl_stat* gate,
                           int32_t gate_layer, char* ws, cudaStream_t st) {
  if (n_heads > c->p.n_kv_heads) return ASL_ERR_INVALID;      // the scratch is sized for H_k heads
  const int tiles = c->max_T > 0 ? (c->max_T + TILE - 1) / TILE : 1;
  const int64_t segments = (int64_t)c->p.batch * n_heads;
  TopkArgs a;
  a.scores = scores;
  a.req = c->d_req;
  a.scratch = reinterpret_cast<int32_t*>(ws + c->ws.topk_scratch);
  a.counts = a.scratch + segments * SEG_INTS;
  a.idx_out = idx_out;
  a.sum_T = c->sum_T;
  a.sum_kept = c->sum_kept;
  a.n_heads = n_heads;
  a.max_tiles = tiles;
  a.gate = gate;
  a.gate_layer = gate_layer;
  a.latch = gate ? nullptr : c->latch_stat;      // the gated call has its own rule
  a.cur_layer = c->cur_layer;
  ASL_CUDA(cudaMemsetAsync(a.scratch, 0, (size_t)segments * SEG_INTS * sizeof(int32_t), st));
  const dim3 grid(tiles, n_heads, c->p.batch);
  topk_digit_kernel<0><<<grid, THREADS, 0, st>>>(a);
  topk_digit_kernel<1><<<grid, THREADS, 0, st>>>(a);
  topk_digit_kernel<2><<<grid, THREADS, 0, st>>>(a);
  topk_count_kernel<<<grid, THREADS, 0, st>>>(a);
  topk_emit_kernel<<<grid, THREADS, 0, st>>>(a);
  c->launches += 5;
  ASL_CUDA(cudaGetLastError());
  return ASL_OK;
}
