// Rank row and rank-variance statistic (Algorithm 1 (RankDesc); Algorithm 2 (stacked rank rows R, k, TopKIndices J, Unique U, RelNormVar, threshold test);
// Section 4.1 "var_top" and "relative variance").
//
// RankDesc: stable least-significant-digit radix sort (8-bit digits, one kernel
// per digit after a first histogram) of
// (key, token index) pairs per request, key = bit pattern that ascends as the
// score descends; equal scores keep ascending index order, so the position of
// a token in the sorted sequence is its 0-based rank with ties to the lower
// index.  The last pass scatters positions straight into the ring row.
//
// Statistic: a token is in the union iff its smallest rank over the rows is < k
// (the k smallest ranks of a row are exactly ranks 0..k-1).  The numerator
// sum_j (rows*sum r^2 - (sum r)^2) is accumulated in 64-bit integers with
// integer atomics, so it does not depend on the order of accumulation.
#include <mutex>

#include "asl_internal.cuh"

namespace {

constexpr int TILE = ASL_RANK_TILE;      // keys per block
constexpr int SORT_THREADS = 256;
constexpr int WARPS = SORT_THREADS / 32;
constexpr int PER_WARP = TILE / WARPS;   // consecutive keys of one warp
constexpr int ROUNDS = PER_WARP / 32;    // walked 32 at a time, all loads issued up front
constexpr int PARTS = SORT_THREADS / 256;  // threads per digit where a thread walks a digit's column of tile counts
static_assert(SORT_THREADS % 256 == 0 && SORT_THREADS <= 1024 && TILE % SORT_THREADS == 0, "a thread per digit; whole rounds");

__device__ __forceinline__ uint32_t desc_key(float s) {
  uint32_t u = __float_as_uint(s);
  if (u == 0x80000000u) u = 0;                           // -0 ranks with +0
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);        // ascending with the score
  return ~u;                                             // ascending as the score descends
}

// Lanes of the warp whose 8-bit digit equals this lane's: eight ballots, no
// data-dependent loop (the hardware match instruction walks distinct values).
__device__ __forceinline__ uint32_t same_digit(uint32_t d, bool valid) {
  uint32_t peers = __ballot_sync(0xffffffffu, valid);
#pragma unroll
  for (int bit = 0; bit < 8; ++bit) {
    const uint32_t b = __ballot_sync(0xffffffffu, (d >> bit) & 1u);
    peers &= ((d >> bit) & 1u) ? b : ~b;
  }
  return peers;
}

// The first pass reads the fp32 scores and forms keys on the fly (token index =
// position); later passes read the (key, index) pairs of the previous pass.
template <bool FIRST>
__device__ __forceinline__ void load_tile(const float* __restrict__ agg, const uint32_t* __restrict__ keys_in,
                                          const int32_t* __restrict__ idx_in, const AslReq& rq, int wstart, int lane,
                                          uint32_t (&key)[ROUNDS], int32_t (&id)[ROUNDS]) {
#pragma unroll
  for (int r = 0; r < ROUNDS; ++r) {
    const int i = wstart + r * 32 + lane;
    key[r] = 0u;
    id[r] = i;
    if (i < rq.T) {
      if (FIRST) key[r] = desc_key(agg[rq.t_off + i]);
      else { key[r] = keys_in[rq.t_off + i]; id[r] = idx_in[rq.t_off + i]; }
    }
  }
}

// hist[0][b][blk][digit]: digit counts of one tile of the scores, lowest digit.  The
// tables of the three later passes are cleared here; each scatter pass counts the
// next digit of what it writes into them.
__global__ void __launch_bounds__(SORT_THREADS) rank_hist_first(const float* __restrict__ agg, const AslReq* __restrict__ req,
                                                                const asl_stat* __restrict__ latch, int nblk, int64_t table,
                                                                int32_t* __restrict__ hist) {
  __shared__ int cnt[256];
  pdl_release_successor();                 // launched the plain way: the scores are complete when it starts
  const int b = blockIdx.y, blk = blockIdx.x;
  const int64_t row = ((int64_t)b * nblk + blk) * 256 + (threadIdx.x & 255);
  if (threadIdx.x < 256) {
#pragma unroll
    for (int t = 1; t < 4; ++t) hist[t * table + row] = 0;
  }
  if (latch && latch[b].selected) return;              // the request's selection is final: no more rank rows
  const AslReq rq = req[b];
  const int start = blk * TILE;
  if (start >= rq.T) return;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  if (threadIdx.x < 256) cnt[threadIdx.x] = 0;
  uint32_t key[ROUNDS];
  int32_t id[ROUNDS];
  load_tile<true>(agg, nullptr, nullptr, rq, start + wid * PER_WARP, lane, key, id);
  __syncthreads();
#pragma unroll
  for (int r = 0; r < ROUNDS; ++r) {
    const bool valid = start + wid * PER_WARP + r * 32 + lane < rq.T;
    const uint32_t d = key[r] & 255u;
    const uint32_t peers = same_digit(d, valid);
    if (valid && (peers & ((1u << lane) - 1u)) == 0) atomicAdd(&cnt[d], __popc(peers));
  }
  __syncthreads();
  if (threadIdx.x < 256) hist[row] = cnt[threadIdx.x];
}

// in place: hist[b][blk][digit] -> first output position of (digit, blk), i.e. the
// exclusive scan in (digit, blk) order.  1024 threads: thread (part, digit) walks a
// quarter of the tiles with its loads batched, the parts are chained through shared memory.
__global__ void __launch_bounds__(1024) rank_scan(int32_t* __restrict__ hist, const AslReq* __restrict__ req,
                                                  const asl_stat* __restrict__ latch, int nblk) {
  __shared__ int part_tot[4][256];
  __shared__ int warp_tot[8];
  pdl_release_successor();
  pdl_wait_predecessor();
  const int b = blockIdx.x;
  if (latch && latch[b].selected) return;
  const int used = (req[b].T + TILE - 1) / TILE;             // tiles of this request
  const int d = threadIdx.x & 255, part = threadIdx.x >> 8;
  const int per = (used + 3) / 4;
  const int b0 = part * per, b1 = min(used, b0 + per);
  int32_t* col = hist + (int64_t)b * nblk * 256 + d;
  int total = 0;
  for (int i0 = b0; i0 < b1; i0 += 8) {
    int v[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) v[k] = (i0 + k < b1) ? col[(int64_t)(i0 + k) * 256] : 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) total += v[k];
  }
  part_tot[part][d] = total;
  __syncthreads();
  int digit_total = 0, before = 0;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int t = part_tot[q][d];
    digit_total += t;
    if (q < part) before += t;
  }
  // exclusive scan of the digit totals over the 256 digits (every part computes it)
  const int lane = threadIdx.x & 31, w8 = d >> 5;
  int incl = digit_total;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (part == 0 && lane == 31) warp_tot[w8] = incl;
  __syncthreads();
  int base = incl - digit_total + before;
  for (int w2 = 0; w2 < w8; ++w2) base += warp_tot[w2];
  for (int i0 = b0; i0 < b1; i0 += 8) {
    int v[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) v[k] = (i0 + k < b1) ? col[(int64_t)(i0 + k) * 256] : 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      if (i0 + k < b1) col[(int64_t)(i0 + k) * 256] = base;
      base += v[k];
    }
  }
}

// Stable scatter of one tile; the last pass writes rank[token] = position.
// SCAN: `counts` holds raw tile counts and the tile's first output positions are
// summed here (thread = digit walks the tiles' rows; used while the request has few
// tiles); otherwise `counts` was turned into positions by rank_scan.  A pass that is
// not the last counts, per destination tile, the next digit of every pair it writes
// (integer atomics: the table does not depend on the order of arrival).
template <bool FIRST, bool SCAN>
__global__ void __launch_bounds__(SORT_THREADS) rank_scatter(const float* __restrict__ agg,
                                                             const uint32_t* __restrict__ keys_in,
                                                             const int32_t* __restrict__ idx_in,
                                                             uint32_t* __restrict__ keys_out, int32_t* __restrict__ idx_out,
                                                             int32_t* __restrict__ rank_row, const int32_t* __restrict__ counts,
                                                             int32_t* __restrict__ next_counts,
                                                             const AslReq* __restrict__ req,
                                                             const asl_stat* __restrict__ latch, int shift, int nblk) {
  constexpr int SCAN_BATCH = 64 / PARTS;       // loads of tile counts in flight per thread
  __shared__ int cnt[WARPS][256];
  __shared__ int warp_tot[8];
  __shared__ int digit_off[256];
  __shared__ int part_tot[PARTS > 1 ? PARTS : 1][PARTS > 1 ? 256 : 1], part_before[PARTS > 1 ? PARTS : 1][PARTS > 1 ? 256 : 1];
  pdl_release_successor();
  const int b = blockIdx.y, blk = blockIdx.x;
  if (latch && latch[b].selected) return;
  const AslReq rq = req[b];
  const int start = blk * TILE;
  if (start >= rq.T) return;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const int wstart = start + wid * PER_WARP;
  const uint32_t lt = (1u << lane) - 1u;
  uint32_t key[ROUNDS];
  int32_t id[ROUNDS];
  // the scores were complete before the first histogram ran: the first pass loads them while that kernel
  // finishes; pairs and counts come from the kernel just before
  if (!FIRST) pdl_wait_predecessor();
  load_tile<FIRST>(agg, keys_in, idx_in, rq, wstart, lane, key, id);
  if (FIRST) pdl_wait_predecessor();
  if (SCAN) {
    // PARTS threads per digit, each over a run of the tiles' counts with all of its loads in flight
    const int d = threadIdx.x & 255, part = threadIdx.x >> 8;
    const int used = (rq.T + TILE - 1) / TILE;
    const int per = (used + PARTS - 1) / PARTS;
    const int b0 = part * per, b1 = min(used, b0 + per);
    const int32_t* col = counts + (int64_t)b * nblk * 256 + d;
    int before = 0, total = 0;
    for (int i0 = b0; i0 < b1; i0 += SCAN_BATCH) {
      int v[SCAN_BATCH];
#pragma unroll
      for (int k = 0; k < SCAN_BATCH; ++k) v[k] = (i0 + k < b1) ? __ldcg(col + (int64_t)(i0 + k) * 256) : 0;
#pragma unroll
      for (int k = 0; k < SCAN_BATCH; ++k) { total += v[k]; if (i0 + k < blk) before += v[k]; }
    }
    if (PARTS > 1) {
      part_tot[part][d] = total;
      part_before[part][d] = before;
      __syncthreads();
      total = 0;
      before = 0;
      if (threadIdx.x < 256) {
#pragma unroll
        for (int q = 0; q < PARTS; ++q) { total += part_tot[q][d]; before += part_before[q][d]; }
      }
    }
    int incl = total;                       // exclusive scan of the digit totals over the 256 digits
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (threadIdx.x < 256 && lane == 31) warp_tot[wid] = incl;
    __syncthreads();
    if (threadIdx.x < 256) {
      int off = incl - total + before;
      for (int w2 = 0; w2 < wid; ++w2) off += warp_tot[w2];
      digit_off[threadIdx.x] = off;
    }
  } else {
    if (threadIdx.x < 256) digit_off[threadIdx.x] = counts[((int64_t)b * nblk + blk) * 256 + threadIdx.x];
  }
  for (int i = threadIdx.x; i < WARPS * 256; i += SORT_THREADS) (&cnt[0][0])[i] = 0;
  __syncthreads();
  // per-warp digit counts; the peer masks are kept for the second walk
  uint32_t peers[ROUNDS];
#pragma unroll
  for (int r = 0; r < ROUNDS; ++r) {
    const bool valid = wstart + r * 32 + lane < rq.T;
    const uint32_t d = (key[r] >> shift) & 255u;
    peers[r] = same_digit(d, valid);
    if (valid && (peers[r] & lt) == 0) cnt[wid][d] += __popc(peers[r]);
    __syncwarp();
  }
  __syncthreads();
  if (threadIdx.x < 256) {  // digit threadIdx.x: bases of the warps, in warp order, after the tile's global offset
    int run = digit_off[threadIdx.x];
#pragma unroll
    for (int w2 = 0; w2 < WARPS; ++w2) {
      const int v = cnt[w2][threadIdx.x];
      cnt[w2][threadIdx.x] = run;
      run += v;
    }
  }
  __syncthreads();
  int32_t* next_b = next_counts ? next_counts + (int64_t)b * nblk * 256 : nullptr;
  const bool top_next = shift == 16;        // the next digit is the sign/exponent byte: few distinct values
#pragma unroll
  for (int r = 0; r < ROUNDS; ++r) {
    const bool valid = wstart + r * 32 + lane < rq.T;
    const uint32_t d = (key[r] >> shift) & 255u;
    int pos = 0;
    if (valid) pos = cnt[wid][d] + __popc(peers[r] & lt);
    __syncwarp();
    if (valid && (peers[r] & lt) == 0) cnt[wid][d] += __popc(peers[r]);
    __syncwarp();
    if (valid) {
      if (rank_row) rank_row[rq.t_off + id[r]] = pos;
      else { keys_out[rq.t_off + pos] = key[r]; idx_out[rq.t_off + pos] = id[r]; }
    }
    if (next_b) {
      const uint32_t slot = valid ? (uint32_t)(pos / TILE) * 256u + ((key[r] >> (shift + 8)) & 255u) : 0xffffffffu;
      if (top_next) {                       // one atomic per distinct counter of the warp
        const uint32_t same = __match_any_sync(0xffffffffu, slot);
        if (valid && (same & lt) == 0) atomicAdd(next_b + slot, __popc(same));
      } else if (valid) {
        atomicAdd(next_b + slot, 1);
      }
    }
  }
}

// the four passes of one rank row; scratch: two key and two index arrays, four tables of tile histograms
constexpr int SCAN_IN_SCATTER_MAX_TILES = 128;

int launch_sort(const float* agg, const AslReq* req, const asl_stat* latch, int batch, int max_T, uint32_t* const keys[2],
                int32_t* const idx[2], int32_t* hist, int32_t* rank_row, cudaStream_t st) {
  const int nblk = (max_T + TILE - 1) / TILE;
  const dim3 grid(nblk, batch);
  const int64_t table = (int64_t)batch * nblk * 256;
  const bool fused_scan = nblk <= SCAN_IN_SCATTER_MAX_TILES;
  int launches = 1;
  rank_hist_first<<<grid, SORT_THREADS, 0, st>>>(agg, req, latch, nblk, table, hist);
  for (int pass = 0; pass < 4; ++pass) {
    const int in = (pass + 1) & 1, out = in ^ 1;           // pass 0 reads the scores, writes buffer 0
    const int shift = pass * 8;
    int32_t* row = pass == 3 ? rank_row : nullptr;
    int32_t* cur = hist + pass * table;
    int32_t* nxt = pass == 3 ? nullptr : hist + (pass + 1) * table;
    if (!fused_scan) { launch_after(rank_scan, dim3(batch), dim3(1024), st, cur, req, latch, nblk); ++launches; }
    ++launches;
    if (pass == 0) {
      if (fused_scan) launch_after(rank_scatter<true, true>, grid, dim3(SORT_THREADS), st, agg, nullptr, nullptr, keys[out], idx[out], row, cur, nxt, req, latch, shift, nblk);
      else launch_after(rank_scatter<true, false>, grid, dim3(SORT_THREADS), st, agg, nullptr, nullptr, keys[out], idx[out], row, cur, nxt, req, latch, shift, nblk);
    } else {
      if (fused_scan) launch_after(rank_scatter<false, true>, grid, dim3(SORT_THREADS), st, nullptr, keys[in], idx[in], keys[out], idx[out], row, cur, nxt, req, latch, shift, nblk);
      else launch_after(rank_scatter<false, false>, grid, dim3(SORT_THREADS), st, nullptr, keys[in], idx[in], keys[out], idx[out], row, cur, nxt, req, latch, shift, nblk);
    }
  }
  return launches;
}


struct StatArgs {
  const int32_t* ring;
  const AslReq* req;
  unsigned long long* acc;   // [B][2]: numerator, union size; then one counter of finished blocks
  asl_stat* stat;
  int64_t sum_T;
  int32_t l_obs, first_layer, n_rows, batch, layer_idx, latch;
  double tau;
};

// Algorithm 2 (threshold test) for request b from the accumulated integers; clears them for the next layer
__device__ void stat_finalize_one(unsigned long long* acc, const AslReq* __restrict__ req, asl_stat* __restrict__ stat, int b,
                                  int layer_idx, int n_rows, int evaluate, double tau, int latch) {
  asl_stat s = stat[b];
  if (latch && s.selected) return;                     // final: the record keeps the selection layer
  s.layer_idx = layer_idx;
  s.k = req[b].k;
  s.rows = n_rows;
  s.evaluated = 0;
  s.selected = 0;
  s.num = 0;
  s.m = 0;
  if (evaluate) {
    const unsigned long long num = __ldcg(acc + 2 * b), m = __ldcg(acc + 2 * b + 1);
    acc[2 * b] = 0;
    acc[2 * b + 1] = 0;
    s.num = (int64_t)num;
    s.m = (int32_t)m;
    s.evaluated = 1;
    s.var_top = (double)num / ((double)n_rows * (double)n_rows * (double)m);   // empty union (k = 0): NaN, never selects
    if (!s.has_init) { s.init_var = s.var_top; s.has_init = 1; }
    s.rel = s.init_var != 0.0 ? s.var_top / s.init_var : __longlong_as_double(0x7ff8000000000000ll);   // zero first variance: undefined, never selects
    s.selected = (s.rel < tau) ? 1 : 0;
  }
  const int32_t selected = s.selected;
  s.selected = 0;
  stat[b] = s;
  if (selected) {                                      // last, behind a fence: see asl_finished
    __threadfence();
    reinterpret_cast<volatile asl_stat*>(stat + b)->selected = 1;
  }
}

// layers before L_min (or with a single rank row): only the bookkeeping fields change
__global__ void rank_stat_skip(unsigned long long* acc, const AslReq* __restrict__ req, asl_stat* __restrict__ stat, int batch,
                               int layer_idx, int n_rows, int latch) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b < batch) stat_finalize_one(acc, req, stat, b, layer_idx, n_rows, 0, 0.0, latch);
}

constexpr int STAT_TOKENS = 4;   // tokens per thread: few, fat blocks (one wave on the SMs a persistent scorer leaves free)

__global__ void __launch_bounds__(256) rank_stat_accumulate(StatArgs a) {
  __shared__ unsigned long long s_num[8];
  __shared__ int s_m[8];
  const int b = blockIdx.y;
  const AslReq rq = a.req[b];
  const bool open = !(a.latch && a.stat[b].selected);
  unsigned long long num = 0;
  int m = 0;
  int j[STAT_TOKENS];
  long long s1[STAT_TOKENS], s2[STAT_TOKENS];
  int mn[STAT_TOKENS];
#pragma unroll
  for (int i = 0; i < STAT_TOKENS; ++i) {
    j[i] = (blockIdx.x * STAT_TOKENS + i) * 256 + threadIdx.x;
    s1[i] = 0; s2[i] = 0; mn[i] = 0x7fffffff;
  }
  // the rows of the earlier layers are read (all of a batch's loads in flight) while the sort of this layer's row ends
  for (int r0 = 0; r0 < a.n_rows - 1; r0 += 8) {
    int v[STAT_TOKENS][8];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int slot = (a.first_layer + r0 + q) % a.l_obs;
#pragma unroll
      for (int i = 0; i < STAT_TOKENS; ++i)
        v[i][q] = (open && j[i] < rq.T && r0 + q < a.n_rows - 1) ? __ldcg(a.ring + (int64_t)slot * a.sum_T + rq.t_off + j[i]) : -1;
    }
#pragma unroll
    for (int i = 0; i < STAT_TOKENS; ++i)
#pragma unroll
      for (int q = 0; q < 8; ++q)
        if (v[i][q] >= 0) { mn[i] = min(mn[i], v[i][q]); s1[i] += v[i][q]; s2[i] += (long long)v[i][q] * v[i][q]; }
  }
  pdl_wait_predecessor();
  {
    const int slot = (a.first_layer + a.n_rows - 1) % a.l_obs;
    int v[STAT_TOKENS];
#pragma unroll
    for (int i = 0; i < STAT_TOKENS; ++i) v[i] = (open && j[i] < rq.T) ? __ldcg(a.ring + (int64_t)slot * a.sum_T + rq.t_off + j[i]) : -1;
#pragma unroll
    for (int i = 0; i < STAT_TOKENS; ++i) {
      if (v[i] < 0) continue;
      mn[i] = min(mn[i], v[i]);
      s1[i] += v[i];
      s2[i] += (long long)v[i] * v[i];
      if (mn[i] < rq.k) {
        m += 1;
        num += (unsigned long long)((long long)a.n_rows * s2[i] - s1[i] * s1[i]);
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    num += __shfl_down_sync(0xffffffffu, num, o);
    m += __shfl_down_sync(0xffffffffu, m, o);
  }
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  if (lane == 0) { s_num[wid] = num; s_m[wid] = m; }
  __syncthreads();
  __shared__ bool last;
  if (threadIdx.x == 0) {
    for (int w2 = 1; w2 < 8; ++w2) { num += s_num[w2]; m += s_m[w2]; }
    if (m) {
      atomicAdd(&a.acc[2 * b], num);
      atomicAdd(&a.acc[2 * b + 1], (unsigned long long)m);
    }
    // the block that finishes last sees every block's sums and closes the statistic
    __threadfence();
    const unsigned long long blocks = (unsigned long long)gridDim.x * gridDim.y;
    last = atomicAdd(&a.acc[2 * a.batch], 1ull) + 1 == blocks;
  }
  __syncthreads();
  if (last) {
    __threadfence();
    for (int bb = threadIdx.x; bb < a.batch; bb += blockDim.x)
      stat_finalize_one(a.acc, a.req, a.stat, bb, a.layer_idx, a.n_rows, 1, a.tau, a.latch);
    if (threadIdx.x == 0) a.acc[2 * a.batch] = 0;
  }
}

}  // namespace

asl_status asl_launch_rank(asl_ctx* c, const float* agg, int32_t layer_idx, int32_t n_rows, int32_t* ring,
                           asl_stat* stat, char* ws, cudaStream_t st) {
  const asl_params& p = c->p;
  uint32_t* keys[2] = {reinterpret_cast<uint32_t*>(ws + c->ws.rank_keys[0]),
                       reinterpret_cast<uint32_t*>(ws + c->ws.rank_keys[1])};
  int32_t* idx[2] = {reinterpret_cast<int32_t*>(ws + c->ws.rank_idx[0]),
                     reinterpret_cast<int32_t*>(ws + c->ws.rank_idx[1])};
  int32_t* hist = reinterpret_cast<int32_t*>(ws + c->ws.rank_hist);
  int32_t* row = ring + (int64_t)(layer_idx % p.l_obs) * c->sum_T;
  const asl_stat* latch = c->controller == ASL_CONTROLLER_LATCH ? stat : nullptr;
  c->launches += launch_sort(agg, c->d_req, latch, p.batch, c->max_T, keys, idx, hist, row, st);
  const int evaluate = (layer_idx >= p.l_min && n_rows >= 2) ? 1 : 0;
  if (evaluate) {
    StatArgs a{ring, c->d_req, c->d_acc, stat, c->sum_T, p.l_obs, layer_idx - n_rows + 1, n_rows, p.batch, layer_idx,
               latch ? 1 : 0, p.tau};
    launch_after(rank_stat_accumulate, dim3((c->max_T + 256 * STAT_TOKENS - 1) / (256 * STAT_TOKENS), p.batch), dim3(256), st, a);
  } else {
    rank_stat_skip<<<(p.batch + 63) / 64, 64, 0, st>>>(c->d_acc, c->d_req, stat, p.batch, layer_idx, n_rows, latch ? 1 : 0);
  }
  c->launches += 1;
  ASL_CUDA(cudaGetLastError());
  return ASL_OK;
}

// ---------------------------------------------------------------------------
// Allocation-free rank row.
//
// Some hosts of this library are not allowed to allocate device memory while
// they run: a serving engine that hands its whole memory pool to its own
// allocator at start-up, a plugin called from inside another runtime's
// execution callback, code running under a "no cudaMalloc after init" rule.
// For them the sort's scratch (two ping-pong key arrays, two payload arrays,
// the per-tile digit histograms and a one-entry request table) lives in this
// file-scope device array.  Every device that loads the library carries these
// bytes until the process exits, which is why the segment length is capped.
//
// In host code `g_rank_static` is only a handle: the device address is asked
// for once per device with cudaGetSymbolAddress and that pointer is what the
// kernels get.
// ---------------------------------------------------------------------------
namespace {

constexpr int STATIC_MAX_T = ASL_RANK_STATIC_MAX_T;
constexpr int STATIC_NBLK = (STATIC_MAX_T + TILE - 1) / TILE;
constexpr int STATIC_MAX_DEVICES = 64;

struct RankStaticScratch {
  AslReq req;                       // the one request the kernels index with blockIdx.y = 0
  uint32_t keys[2][STATIC_MAX_T];
  int32_t idx[2][STATIC_MAX_T];
  int32_t hist[4 * 256 * STATIC_NBLK];
};

static __device__ __align__(256) unsigned char g_rank_static[sizeof(RankStaticScratch)];

// Writes the request record.  Nothing else in the scratch has to start from a
// known value: the sort writes every key, payload and histogram entry before it
// reads it, so what an earlier call left behind is never seen.
__global__ void rank_static_begin(RankStaticScratch* s, int T) {
  AslReq r;
  r.n = T; r.T = T; r.k = 0; r.kept = 0; r.tok_off = 0; r.t_off = 0; r.kept_off = 0; r.pad = 0;
  s->req = r;
}

struct RankStaticDevices {
  RankStaticScratch* ptr[STATIC_MAX_DEVICES] = {};
  asl_status status[STATIC_MAX_DEVICES] = {};
  bool done[STATIC_MAX_DEVICES] = {};
  std::mutex lock;
};

RankStaticDevices& rank_static_devices() {
  static RankStaticDevices d;
  return d;
}

// Once per device, with that device current: architecture check and the
// device address of the scratch array.
asl_status rank_static_setup(int device, RankStaticScratch** out) {
  RankStaticDevices& d = rank_static_devices();
  std::lock_guard<std::mutex> guard(d.lock);
  if (!d.done[device]) {
    asl_status st = ASL_OK;
    int major = 0;
    void* p = nullptr;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess) st = ASL_ERR_CUDA;
    else if (major != 10) st = ASL_ERR_ARCH;
    else if (cudaGetSymbolAddress(&p, g_rank_static) != cudaSuccess || !p) st = ASL_ERR_CUDA;
    d.ptr[device] = static_cast<RankStaticScratch*>(p);
    d.status[device] = st;
    d.done[device] = st == ASL_OK || st == ASL_ERR_ARCH;     // a failed CUDA call is tried again by the next call
    if (st == ASL_ERR_CUDA) cudaGetLastError();
  }
  *out = d.ptr[device];
  return d.status[device];
}

}  // namespace

extern "C" asl_status asl_rank_desc_static(const float* scores, int32_t T, int32_t* rank_out, void* stream) {
  if (!scores || !rank_out || T < 1) return ASL_ERR_INVALID;
  if (T > STATIC_MAX_T) return ASL_ERR_WORKSPACE;      // the fixed scratch cannot hold this segment
  int device = -1;
  ASL_CUDA(cudaGetDevice(&device));
  if (device < 0 || device >= STATIC_MAX_DEVICES) return ASL_ERR_UNSUPPORTED;
  RankStaticScratch* s = nullptr;
  const asl_status ready = rank_static_setup(device, &s);
  if (ready != ASL_OK) return ready;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const AslReq* req = &s->req;
  rank_static_begin<<<1, 1, 0, st>>>(s, T);
  uint32_t* const keys[2] = {s->keys[0], s->keys[1]};
  int32_t* const idx[2] = {s->idx[0], s->idx[1]};
  launch_sort(scores, req, nullptr, 1, T, keys, idx, s->hist, rank_out, st);
  ASL_CUDA(cudaGetLastError());
  return ASL_OK;
}
