// Per-(request, head) top-k with the window appended (Algorithm 1 (k, TopK and window append)).
//
// Radix select on an order-preserving 32-bit image of the fp32 score, 11+11+10
// bits from the top: the exact k-th largest key is found; every token with a
// larger key is kept, and of the tokens equal to it the lowest-indexed fill the
// remainder.  Two forms.  Plans whose longest segment has 8 K to 256 K scores
// and whose k is a small part of it run one CTA per segment in a single launch
// (second half of this file).  Everything else is cut into tiles of 4096 scores,
// one 256-thread CTA per tile with its 16 scores per thread in registers, and
// into five short kernels that meet only through global memory:
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
  int32_t n_heads, max_tiles, max_T;
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
  pdl_release_successor();
  const Segment s = segment_of(a);
  if (!s.open || s.k == 0 || s.tile * TILE >= s.T) return;
  uint32_t key[PER_THREAD];
  load_keys(s, key);                      // the scores were complete before the first of these kernels started
  pdl_wait_predecessor();
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
  pdl_release_successor();
  const Segment s = segment_of(a);
  if (!s.open || s.k == 0 || s.tile * TILE >= s.T) return;
  uint32_t key[PER_THREAD];
  load_keys(s, key);
  pdl_wait_predecessor();
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
  pdl_release_successor();
  if (!s.open || s.tile >= tiles) return;
  uint32_t key[PER_THREAD];
  if (s.k) load_keys(s, key);
  pdl_wait_predecessor();
  for (int t = s.tile * THREADS + tid; t < s.kept - s.k; t += tiles * THREADS) s.out[s.k + t] = s.T + t;   // the window
  if (s.k == 0) return;
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

// ---------------------------------------------------------------------------
// One CTA per segment.
//
// For segments of a few thousand to a few hundred thousand scores the whole
// selection runs in one 1024-thread CTA with no scratch in global memory:
//
//   sample 4096 scores -> a lower bound L that, with a wide margin, at least k
//   scores reach -> ONE pass over the segment that keeps every (key, index) with
//   key >= L in shared memory -> exact radix select of the k-th largest key among
//   them -> two bitmaps over the segment (keys above the k-th, keys equal to it)
//   -> ordered emit from the bitmaps.
//
// The bound is only a way to look at few keys: the pass counts what it keeps, and
// if fewer than k scores reached L, or more than the shared-memory list holds
// (long runs of equal scores, a k that is a large part of T), the CTA takes the
// same 11+11+10-bit radix select as the tiled kernels over the whole segment
// (three more passes and one to fill the bitmaps).  Both ways end in the exact
// k-th key and the same tie rule, so the kept list does not depend on which ran.
// ---------------------------------------------------------------------------
constexpr int SEG_THREADS = 1024;
constexpr int SEG_WARPS = SEG_THREADS / 32;
constexpr int SEG_CAP = 12288;                 // (key, index) pairs the shared-memory list holds
constexpr int SEG_SAMPLE = 2048;
constexpr int SEG_MIN_T = 8192;                // shorter segments: the full select at once (a sample would be most of them)
constexpr int SEG_MAX_T = 262144;              // the bitmaps cover this many scores
constexpr int SEG_UNROLL = 8;                  // 16-byte loads in flight per thread

struct SegSmem {
  int hist[BINS];
  uint32_t cand_key[SEG_CAP];
  int32_t cand_idx[SEG_CAP];
  // behind this struct, sized for the plan's longest segment (seg_smem_bytes): two bitmaps over the segment
  // and, per bitmap word, the kept scores before it (short-list emit)
  int warp_a[SEG_WARPS], warp_b[SEG_WARPS];
  int found[2][2];
  int n_cand;
};

// dynamic shared memory of the kernel for segments of up to max_T scores
__host__ __device__ inline int seg_words(int max_T) { return ((max_T + 31) / 32 + 3) & ~3; }
inline size_t seg_smem_bytes(int max_T) { return sizeof(SegSmem) + (size_t)seg_words(max_T) * (2 * sizeof(uint32_t) + 2 * sizeof(uint16_t)); }

// The sample rank whose key is taken as the lower bound: the expected number of sampled scores among
// the k largest, plus four standard deviations and two.
__host__ __device__ inline int seg_sample_rank(int T, int k) {
  const float mean = (float)SEG_SAMPLE * (float)k / (float)T;
  return (int)ceilf(mean + 4.f * sqrtf(mean)) + 2;
}

// Warp `wid` walks a contiguous run of 16-byte vectors of the segment; the vectors are aligned in
// memory, so the first and the last may hold fewer than four scores of the segment.
struct SegWalk {
  const float* row;
  const float4* base4;
  int T, mis, per, v_begin, v_end;
  __device__ SegWalk(const float* row_, int T_, int wid) : row(row_), T(T_) {
    mis = (int)((reinterpret_cast<uintptr_t>(row_) >> 2) & 3);
    base4 = reinterpret_cast<const float4*>(row_ - mis);
    const int nv = (T + mis + 3) >> 2;
    per = (((nv + SEG_WARPS - 1) / SEG_WARPS) + 32 * SEG_UNROLL - 1) / (32 * SEG_UNROLL) * (32 * SEG_UNROLL);   // whole load blocks
    v_begin = min(nv, wid * per);
    v_end = min(nv, v_begin + per);
  }
  __device__ __forceinline__ int first_index(int v) const { return v * 4 - mis; }
  // keys of vector v; bit c of the result: element c is a score of the segment
  __device__ __forceinline__ uint32_t load(int v, uint32_t (&key)[4]) const {
    key[0] = key[1] = key[2] = key[3] = 0u;
    if (v >= v_end) return 0u;
    const int e0 = v * 4 - mis;
    if (e0 >= 0 && e0 + 4 <= T) {
      const float4 x = __ldcg(base4 + v);
      key[0] = asc_key(x.x); key[1] = asc_key(x.y); key[2] = asc_key(x.z); key[3] = asc_key(x.w);
      return 15u;
    }
    uint32_t m = 0u;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int e = e0 + c;
      if (e >= 0 && e < T) { key[c] = asc_key(__ldcg(row + e)); m |= 1u << c; }
    }
    return m;
  }
  // SEG_UNROLL vectors per lane from vector s0 on (s0 is the same for the whole warp).  Away from the ends of
  // the warp's run and of the segment every load is a full vector: all of them are issued before the first is used.
  // all SEG_UNROLL x 32 vectors from s0 on are full vectors of the segment inside this warp's run
  __device__ __forceinline__ bool interior(int s0) const {
    return s0 + 32 * SEG_UNROLL <= v_end && s0 * 4 - mis >= 0 && (s0 + 32 * SEG_UNROLL) * 4 - mis <= T;
  }
  __device__ __forceinline__ void load_block(int s0, int lane, uint32_t (&key)[SEG_UNROLL][4], uint32_t (&m)[SEG_UNROLL]) const {
    if (interior(s0)) {
      float4 x[SEG_UNROLL];
#pragma unroll
      for (int u = 0; u < SEG_UNROLL; ++u) x[u] = __ldcg(base4 + s0 + 32 * u + lane);
#pragma unroll
      for (int u = 0; u < SEG_UNROLL; ++u) {
        key[u][0] = asc_key(x[u].x); key[u][1] = asc_key(x[u].y); key[u][2] = asc_key(x[u].z); key[u][3] = asc_key(x[u].w);
        m[u] = 15u;
      }
    } else {
#pragma unroll
      for (int u = 0; u < SEG_UNROLL; ++u) m[u] = load(s0 + 32 * u + lane, key[u]);
    }
  }
};

// exclusive prefix, at position `wid`, of the 32 per-warp totals in `tot` (every warp computes it for itself)
__device__ __forceinline__ int seg_warp_base(const int* tot, int lane, int wid) {
  const int t = tot[lane];
  int incl = t;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  return __shfl_sync(0xffffffffu, incl - t, wid);
}

// pick() for 1024 threads over a table in shared memory (NB = 2048 or 1024 bins); `par` alternates between
// consecutive calls (the result of a call stays readable while the next one runs)
template <int NB>
__device__ __forceinline__ void seg_pick(SegSmem& sm, int remaining, int par, int& bin, int& rem_out) {
  constexpr int PER = NB / SEG_THREADS;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int top = NB - 1 - PER * tid;
  int c[PER];
  int sum = 0;
#pragma unroll
  for (int j = 0; j < PER; ++j) { c[j] = sm.hist[top - j]; sum += c[j]; }
  int incl = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) sm.warp_a[wid] = incl;
  __syncthreads();
  int above = incl - sum + seg_warp_base(sm.warp_a, lane, wid);
  if (above < remaining && remaining <= above + sum) {
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      if (above < remaining && remaining <= above + c[j]) { sm.found[par][0] = top - j; sm.found[par][1] = remaining - above; }
      above += c[j];
    }
  }
  __syncthreads();
  bin = sm.found[par][0];
  rem_out = sm.found[par][1];
}

__device__ __forceinline__ void seg_clear_hist(SegSmem& sm) {
  for (int i = threadIdx.x; i < BINS; i += SEG_THREADS) sm.hist[i] = 0;
  __syncthreads();
}

// digit histogram of the listed keys whose bits under `mask` equal `prefix`
__device__ __forceinline__ void seg_list_hist(SegSmem& sm, int n, uint32_t mask, uint32_t prefix, int shift, uint32_t dmask) {
  seg_clear_hist(sm);
  for (int i = threadIdx.x; i < n; i += SEG_THREADS) {
    const uint32_t key = sm.cand_key[i];
    if ((key & mask) == prefix) atomicAdd(&sm.hist[(key >> shift) & dmask], 1);
  }
  __syncthreads();
}

// the same over the whole segment (one pass over its scores)
__device__ __forceinline__ void seg_full_hist(SegSmem& sm, const SegWalk& w, uint32_t mask, uint32_t prefix, int shift,
                                              uint32_t dmask) {
  seg_clear_hist(sm);
  const int lane = threadIdx.x & 31;
  for (int s = w.v_begin; s < w.v_end; s += 32 * SEG_UNROLL) {
    uint32_t key[SEG_UNROLL][4], m[SEG_UNROLL];
    w.load_block(s, lane, key, m);
    int run_bin = -1, run = 0;
#pragma unroll
    for (int u = 0; u < SEG_UNROLL; ++u) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const bool in = ((m[u] >> c) & 1u) && ((key[u][c] & mask) == prefix);
        const int d = (int)((key[u][c] >> shift) & dmask);
        if (in && d == run_bin) { ++run; continue; }
        if (run) atomicAdd(&sm.hist[run_bin], run);
        run_bin = in ? d : -1;
        run = in ? 1 : 0;
      }
    }
    if (run) atomicAdd(&sm.hist[run_bin], run);
  }
  __syncthreads();
}

__global__ void __launch_bounds__(SEG_THREADS, 1) topk_segment_kernel(TopkArgs a) {
  extern __shared__ __align__(16) uint8_t seg_smem_raw[];
  SegSmem& sm = *reinterpret_cast<SegSmem*>(seg_smem_raw);
  const int cap_words = seg_words(a.max_T);
  uint32_t* const bm_gt = reinterpret_cast<uint32_t*>(seg_smem_raw + sizeof(SegSmem));
  uint32_t* const bm_eq = bm_gt + cap_words;
  uint16_t* const pre_gt = reinterpret_cast<uint16_t*>(bm_eq + cap_words);
  uint16_t* const pre_eq = pre_gt + cap_words;
  const Segment s = segment_of(a);
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  if (!s.open) return;
  for (int t = tid; t < s.kept - s.k; t += SEG_THREADS) s.out[s.k + t] = s.T + t;   // the window
  if (s.k == 0) return;
  const SegWalk w(s.row, s.T, wid);

  // ---- the short list: every score that reaches a sampled lower bound
  bool listed = false;
  int n = 0;
  if (s.T >= SEG_MIN_T) {
    if (tid == 0) sm.n_cand = 0;
    {
      float x[SEG_SAMPLE / SEG_THREADS];
#pragma unroll
      for (int j = 0; j < SEG_SAMPLE / SEG_THREADS; ++j) x[j] = __ldcg(s.row + (int)(((long long)(tid + j * SEG_THREADS) * s.T) / SEG_SAMPLE));
#pragma unroll
      for (int j = 0; j < SEG_SAMPLE / SEG_THREADS; ++j) sm.cand_key[tid + j * SEG_THREADS] = asc_key(x[j]);
    }
    __syncthreads();
    int b1, b2, rem1, rem2;
    seg_list_hist(sm, SEG_SAMPLE, 0u, 0u, 21, 2047u);
    seg_pick<2048>(sm, min(SEG_SAMPLE, seg_sample_rank(s.T, s.k)), 0, b1, rem1);
    seg_list_hist(sm, SEG_SAMPLE, 2047u << 21, (uint32_t)b1 << 21, 10, 2047u);
    seg_pick<2048>(sm, rem1, 1, b2, rem2);
    const uint32_t bound = ((uint32_t)b1 << 21) | ((uint32_t)b2 << 10);
    // A strictly positive bound is compared on the raw bits: key >= bound <=> bits - lo < 2^31 - lo (unsigned).
    const bool raw = bound > 0x80000000u;
    const uint32_t lo = bound & 0x7fffffffu, span = 0x80000000u - lo;
    for (int s0 = w.v_begin; s0 < w.v_end; s0 += 32 * SEG_UNROLL) {
      uint32_t hit = 0u;                                  // bit 4u+c: element c of the lane's u-th vector is listed
      if (raw && w.interior(s0)) {
        float4 x[SEG_UNROLL];
#pragma unroll
        for (int u = 0; u < SEG_UNROLL; ++u) x[u] = __ldcg(w.base4 + s0 + 32 * u + lane);
#pragma unroll
        for (int u = 0; u < SEG_UNROLL; ++u) {
          hit |= (__float_as_uint(x[u].x) - lo < span ? 1u : 0u) << (4 * u);
          hit |= (__float_as_uint(x[u].y) - lo < span ? 2u : 0u) << (4 * u);
          hit |= (__float_as_uint(x[u].z) - lo < span ? 4u : 0u) << (4 * u);
          hit |= (__float_as_uint(x[u].w) - lo < span ? 8u : 0u) << (4 * u);
        }
      } else {
        uint32_t key[SEG_UNROLL][4], m[SEG_UNROLL];
        w.load_block(s0, lane, key, m);
#pragma unroll
        for (int u = 0; u < SEG_UNROLL; ++u)
#pragma unroll
          for (int c = 0; c < 4; ++c)
            if (((m[u] >> c) & 1u) && key[u][c] >= bound) hit |= 1u << (4 * u + c);
      }
      const int cnt = __popc(hit);
      int incl = cnt;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      const int total = __shfl_sync(0xffffffffu, incl, 31);
      if (total == 0) continue;                         // the same for the whole warp
      int base = 0;
      if (lane == 31) base = atomicAdd(&sm.n_cand, total);
      base = __shfl_sync(0xffffffffu, base, 31);
      int slot = base + incl - cnt;
      while (hit) {
        const int bpos = __ffs(hit) - 1;
        hit &= hit - 1;
        if (slot < SEG_CAP) sm.cand_idx[slot] = w.first_index(s0 + 32 * (bpos >> 2) + lane) + (bpos & 3);
        ++slot;
      }
    }
    __syncthreads();
    n = sm.n_cand;
    listed = n >= s.k && n <= SEG_CAP;
    if (listed) {
      for (int i0 = 0; i0 < n; i0 += 4 * SEG_THREADS) {
        float x[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int i = i0 + j * SEG_THREADS + tid;
          x[j] = i < n ? __ldcg(s.row + sm.cand_idx[i]) : 0.f;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int i = i0 + j * SEG_THREADS + tid;
          if (i < n) sm.cand_key[i] = asc_key(x[j]);
        }
      }
      __syncthreads();
    }
  }

  // ---- the exact k-th largest key and how many keys equal to it are kept
  int bin1, bin2, bin3, rem1, rem2, need;
  if (listed) {
    seg_list_hist(sm, n, 0u, 0u, 21, 2047u);
    seg_pick<2048>(sm, s.k, 0, bin1, rem1);
    seg_list_hist(sm, n, 2047u << 21, (uint32_t)bin1 << 21, 10, 2047u);
    seg_pick<2048>(sm, rem1, 1, bin2, rem2);
    seg_list_hist(sm, n, 0xfffffc00u, ((uint32_t)bin1 << 21) | ((uint32_t)bin2 << 10), 0, 1023u);
    seg_pick<1024>(sm, rem2, 0, bin3, need);
  } else {
    seg_full_hist(sm, w, 0u, 0u, 21, 2047u);
    seg_pick<2048>(sm, s.k, 0, bin1, rem1);
    seg_full_hist(sm, w, 2047u << 21, (uint32_t)bin1 << 21, 10, 2047u);
    seg_pick<2048>(sm, rem1, 1, bin2, rem2);
    seg_full_hist(sm, w, 0xfffffc00u, ((uint32_t)bin1 << 21) | ((uint32_t)bin2 << 10), 0, 1023u);
    seg_pick<1024>(sm, rem2, 0, bin3, need);
  }
  const uint32_t thr = ((uint32_t)bin1 << 21) | ((uint32_t)bin2 << 10) | (uint32_t)bin3;

  // ---- bitmaps over the segment: keys above the k-th, keys equal to it
  const int words = (s.T + 31) >> 5;
  for (int i = tid; i < words; i += SEG_THREADS) { bm_gt[i] = 0u; bm_eq[i] = 0u; }
  __syncthreads();
  if (listed) {
    for (int i = tid; i < n; i += SEG_THREADS) {
      const uint32_t key = sm.cand_key[i];
      const int e = sm.cand_idx[i];
      if (key > thr) atomicOr(&bm_gt[e >> 5], 1u << (e & 31));
      else if (key == thr) atomicOr(&bm_eq[e >> 5], 1u << (e & 31));
    }
  } else {
    for (int s0 = w.v_begin; s0 < w.v_end; s0 += 32 * SEG_UNROLL) {
      uint32_t key[SEG_UNROLL][4], m[SEG_UNROLL];
      w.load_block(s0, lane, key, m);
#pragma unroll
      for (int u = 0; u < SEG_UNROLL; ++u)
#pragma unroll
        for (int c = 0; c < 4; ++c)
          if ((m[u] >> c) & 1u) {
            const int e = w.first_index(s0 + 32 * u + lane) + c;
            if (key[u][c] > thr) atomicOr(&bm_gt[e >> 5], 1u << (e & 31));
            else if (key[u][c] == thr) atomicOr(&bm_eq[e >> 5], 1u << (e & 31));
          }
    }
  }
  __syncthreads();

  // ---- ordered emit (Algorithm 1 (TopK and window append)): thread t owns a run of bitmap words
  const int wpt = (words + SEG_THREADS - 1) / SEG_THREADS;
  const int w0 = min(words, tid * wpt), w1 = min(words, w0 + wpt);
  int cg = 0, ce = 0;
  for (int i = w0; i < w1; ++i) { cg += __popc(bm_gt[i]); ce += __popc(bm_eq[i]); }
  int ig = cg, ie = ce;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int vg = __shfl_up_sync(0xffffffffu, ig, o), ve = __shfl_up_sync(0xffffffffu, ie, o);
    if (lane >= o) { ig += vg; ie += ve; }
  }
  if (lane == 31) { sm.warp_a[wid] = ig; sm.warp_b[wid] = ie; }
  __syncthreads();
  int gt_before = ig - cg + seg_warp_base(sm.warp_a, lane, wid), eq_before = ie - ce + seg_warp_base(sm.warp_b, lane, wid);
  if (listed) {
    // every listed score finds its own place: kept scores before its word (at most SEG_CAP: 16 bits) plus those
    // before it in its word; the work is spread evenly however the kept tokens cluster
    for (int i = w0; i < w1; ++i) {
      pre_gt[i] = (uint16_t)gt_before;
      pre_eq[i] = (uint16_t)eq_before;
      gt_before += __popc(bm_gt[i]);
      eq_before += __popc(bm_eq[i]);
    }
    __syncthreads();
    // places first (they read the listed keys), then the kept indices into the keys' storage in output order,
    // then one coalesced copy: a scattered store to global memory costs a cache-line access each
    int place[SEG_CAP / SEG_THREADS];
#pragma unroll
    for (int j = 0; j < SEG_CAP / SEG_THREADS; ++j) {
      const int i = tid + j * SEG_THREADS;
      place[j] = -1;
      if (i < n) {
        const uint32_t key = sm.cand_key[i];
        if (key >= thr) {
          const int e = sm.cand_idx[i], wd = e >> 5;
          const uint32_t below = (1u << (e & 31)) - 1u;
          const int g = pre_gt[wd] + __popc(bm_gt[wd] & below), q = pre_eq[wd] + __popc(bm_eq[wd] & below);
          if (key > thr) place[j] = g + min(q, need);
          else if (q < need) place[j] = g + q;
        }
      }
    }
    __syncthreads();
    int32_t* ordered = reinterpret_cast<int32_t*>(sm.cand_key);
#pragma unroll
    for (int j = 0; j < SEG_CAP / SEG_THREADS; ++j)
      if (place[j] >= 0) ordered[place[j]] = sm.cand_idx[tid + j * SEG_THREADS];
    __syncthreads();
    for (int i = tid; i < s.k; i += SEG_THREADS) s.out[i] = ordered[i];
    return;
  }
  for (int i = w0; i < w1; ++i) {
    const uint32_t g = bm_gt[i], q = bm_eq[i];
    uint32_t bits = g | q;
    while (bits) {
      const int bpos = __ffs(bits) - 1;
      bits &= bits - 1;
      const int idx = i * 32 + bpos;
      if ((g >> bpos) & 1u) {
        s.out[gt_before + min(eq_before, need)] = idx;
        ++gt_before;
      } else {
        if (eq_before < need) s.out[gt_before + eq_before] = idx;
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

// Whether the plan's segments go to the one-CTA kernel: the longest fits its bitmaps, is long enough for a
// sample to be a small part of it, and for every long segment the scores expected above the sampled bound
// (sample rank / sample size of the segment, with a fifth on top) fit the shared-memory list.  Called with the
// context's device current.
bool asl_topk_plan(asl_ctx* c) {
  c->topk_one_cta = false;
  if (c->max_T < SEG_MIN_T || c->max_T > SEG_MAX_T) return false;
  for (const AslReq& r : c->req) {
    if (r.T < SEG_MIN_T || r.k == 0) continue;
    const int rank = seg_sample_rank(r.T, r.k) < SEG_SAMPLE ? seg_sample_rank(r.T, r.k) : SEG_SAMPLE;
    if (1.2 * (double)r.T * rank / SEG_SAMPLE > (double)SEG_CAP) return false;
  }
  if (cudaFuncSetAttribute(topk_segment_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)seg_smem_bytes(SEG_MAX_T)) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  c->topk_one_cta = true;
  return true;
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
  a.max_T = c->max_T;
  a.gate = gate;
  a.gate_layer = gate_layer;
  a.latch = gate ? nullptr : c->latch_stat;      // the gated call has its own rule
  a.cur_layer = c->cur_layer;
  if (c->topk_one_cta) {
    topk_segment_kernel<<<dim3(1, n_heads, c->p.batch), SEG_THREADS, seg_smem_bytes(c->max_T), st>>>(a);
    c->launches += 1;
    ASL_CUDA(cudaGetLastError());
    return ASL_OK;
  }
  ASL_CUDA(cudaMemsetAsync(a.scratch, 0, (size_t)segments * SEG_INTS * sizeof(int32_t), st));
  const dim3 grid(tiles, n_heads, c->p.batch);
  topk_digit_kernel<0><<<grid, THREADS, 0, st>>>(a);
  launch_after(topk_digit_kernel<1>, grid, dim3(THREADS), st, a);
  launch_after(topk_digit_kernel<2>, grid, dim3(THREADS), st, a);
  launch_after(topk_count_kernel, grid, dim3(THREADS), st, a);
  launch_after(topk_emit_kernel, grid, dim3(THREADS), st, a);
  c->launches += 5;
  ASL_CUDA(cudaGetLastError());
  return ASL_OK;
}
