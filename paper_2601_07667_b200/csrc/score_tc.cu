// Observation-window scorer on the 5th-generation tensor cores (Algorithm 1 (window softmax A, past-only column sum U)).
//
// One persistent kernel, one CTA per SM, does both softmax passes of every
// (request, kv head, row chunk) "segment":
//
//   pass 1  D[row][key] = Q_chunk . K_tile^T  (query rows in TMEM lanes): each
//           epilogue thread keeps, for its rows, the sum of 2^(x - ref) over the
//           keys of the CTA's tiles (ref: the maximum of the first 32 keys the
//           row met); each epilogue set publishes (ref, sum) per row.  Once every
//           set has published, two helper warps per CTA fold the partials of
//           "their" rows (row r belongs to CTA r mod grid), in a fixed order, into
//           offset[row] = log2 of the row's softmax denominator, off the
//           epilogue's critical path.
//   pass 2  D[key][row] = K_tile . Q_chunk^T  (keys in TMEM lanes): each thread
//           owns one key and sums exp2(x - offset[row]) over the chunk's rows:
//           the key's column sum U, already summed over the GQA group.
//
// All arithmetic is in the log2 domain x = (q.k) * log2(e)/sqrt(d).  A "chunk"
// is up to 256 of the G*W query rows that share a kv head; a "phase" is one pass
// over one segment's 128-key tiles.  Phases are ordered pass1(s0) pass1(s1)
// pass2(s0) pass2(s1) pass1(s2) ... so that the offsets a pass-2 phase needs were
// finished one phase earlier, and so that K of a segment is still in L2 when
// pass 2 reads it again: HBM sees K once.  The tiles of the whole phase list are
// dealt round-robin to the CTAs.
//
// Inside a CTA: warp 0 streams K tiles through a 3-stage TMA ring (128B-swizzled)
// and keeps the Q chunks of two phases resident (the next one is prefetched);
// warp 1 issues tcgen05.mma into two 256-column TMEM accumulators; warps 2-3 fold
// pass-1 partials; two sets of eight epilogue warps take alternate tiles, one
// accumulator each (two warps per TMEM lane quarter, half of the columns each).  The
// exponentials are split between the MUFU unit and a degree-3 polynomial on the
// FMA pipe (packed f32x2 arithmetic).
//
// Every wait (mbarrier, counter) is bounded: when the limit is reached the thread
// records a code in the context's error word and the CTA drains: producers stop,
// the epilogue keeps walking its barrier sequence without waiting or computing,
// in-flight copies are waited for with the same bound and tensor memory is freed.
#include <cuda.h>
#include <cuda_fp8.h>

#include "asl_internal.cuh"

namespace {

constexpr int KT = ASL_TC_KEY_TILE;          // keys per tile
constexpr int NSTAGE = 3;
constexpr int HALF_BYTES = KT * 128;         // one 64-channel block of a K tile: 128 rows x 128 B
constexpr int STAGE_BYTES = 2 * HALF_BYTES;
constexpr int MAX_NC = 256;
constexpr int Q_BLOCK_BYTES = MAX_NC * 128;  // one 64-channel block of a Q chunk
constexpr int Q_BUF_BYTES = 2 * Q_BLOCK_BYTES;
constexpr int THREADS = 640;                 // warp 0: TMA, 1: MMA, 2-3: partial folding, 4-11 / 12-19: epilogue sets
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;   // every wait gives up after 2 s

// shared-memory map (offsets from the 1024-aligned base of dynamic shared memory)
constexpr int SM_Q = 0;                                      // two Q chunk buffers
constexpr int SM_K = SM_Q + 2 * Q_BUF_BYTES;
constexpr int SM_NEGOFF = SM_K + NSTAGE * STAGE_BYTES;       // float[2][256]: -offset per epilogue set
constexpr int SM_BAR = SM_NEGOFF + 2048;                     // mbarriers
constexpr int SM_MISC = SM_BAR + 128;                        // tmem base, abort flag
constexpr int SMEM_BYTES = SM_MISC + 64;
static_assert(SMEM_BYTES <= 232448, "shared memory budget of one CTA");

enum { BAR_FULL = 0, BAR_EMPTY = NSTAGE, BAR_TFULL = 2 * NSTAGE, BAR_TEMPTY = 2 * NSTAGE + 2,
       BAR_QFULL = 2 * NSTAGE + 4, BAR_QEMPTY = 2 * NSTAGE + 6, BAR_DRAIN = 2 * NSTAGE + 8, N_BARS = 2 * NSTAGE + 9 };
static_assert(N_BARS * 8 <= 128, "barrier area");

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long now;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
  return now;
}
// Bounded wait.  `watch_abort`: also give up when another role raised the flag.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int code,
                                          bool watch_abort, unsigned long long limit_ns = WAIT_LIMIT_NS) {
  unsigned long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    if (mbar_try(bar, parity)) return true;
    if ((it & 15u) == 15u) {
      if (watch_abort && *abort_flag) return false;
      const unsigned long long now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) break;
    }
  }
  *abort_flag = code;
  return false;
}
// Bounded wait until the 32-bit word at p equals `want` (acquire).  Lane 0 polls.
__device__ __forceinline__ bool word_wait(const uint32_t* p, uint32_t want, volatile int* abort_flag, int code, int lane,
                                          uint32_t nap_max, unsigned long long limit_ns = WAIT_LIMIT_NS) {
  int gave_up = 0;
  if (lane == 0) {
    unsigned long long t0 = 0;
    uint32_t nap = 64;
    for (uint32_t it = 0;; ++it) {
      uint32_t v;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
      if (v == want) break;
      if ((it & 7u) == 7u) {
        const unsigned long long now = global_ns();
        if (t0 == 0) t0 = now;
        else if (now - t0 > limit_ns || *abort_flag) { gave_up = 1; if (!*abort_flag) *abort_flag = code; break; }
      }
      __nanosleep(nap);
      if (nap < nap_max) nap <<= 1;
    }
  }
  return __shfl_sync(0xffffffffu, gave_up, 0) == 0;
}

// L2 eviction policies for the K stream: pass 1 asks L2 to keep what pass 2 will read again, pass 2
// (and a launch that has only pass 2) marks what it reads as the first to go.
__device__ __forceinline__ uint64_t l2_policy_keep() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t l2_policy_stream() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2,
                                            uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6;" ::"r"(dst),
      "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2,
                                            int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(
          dst),
      "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2,
                                            int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];" ::"r"(
          dst),
      "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem], bf16 x bf16 -> fp32
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accum)
      : "memory");
}
// the same with 8-bit operands (E4M3 x E4M3 -> fp32), 32 channels per instruction
__device__ __forceinline__ void tc_mma_f8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accum)
      : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane: issue only; the
// registers hold the data after tc_ld_wait on the same array.
__device__ __forceinline__ void tc_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
// Waits for every tcgen05.ld this thread has issued.  The array is an in/out
// operand so that no use of its registers can be scheduled above the wait.
__device__ __forceinline__ void tc_ld_wait(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
                 "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]),
                 "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]),
                 "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void bar_sync(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

// ---- two fp32 values in one 64-bit register: the FMA pipe takes fma on such pairs as
//      one instruction, which halves the issue slots of the softmax arithmetic ----
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pk(float lo, float hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ f32x2 pku(uint32_t lo, uint32_t hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
  return r;
}
__device__ __forceinline__ void upk(f32x2 v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ void upku(f32x2 v, uint32_t& lo, uint32_t& hi) { asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v)); }
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ float hsum(f32x2 v) {
  float lo, hi;
  upk(v, lo, hi);
  return lo + hi;
}
// 2^x of a pair on the MUFU unit
__device__ __forceinline__ f32x2 ex2_pair_mufu(f32x2 x) {
  float a, b;
  upk(x, a, b);
  return pk(ex2(a), ex2(b));
}
// 2^x of a pair on the FMA pipe (any x < 128): clamp at -125, round to the nearest
// integer n with the 1.5*2^23 trick, degree-3 minimax polynomial of 2^f on
// f = x - n in [-0.5, 0.5] (relative error 7.5e-5), n added into the exponent field.
// Additions are written as fma(a, 1, b): the packed fma issues faster than the packed add.
__device__ __forceinline__ f32x2 ex2_pair_poly(f32x2 x) {
  float a, b;
  upk(x, a, b);
  const f32x2 xc = pk(fmaxf(a, -125.0f), fmaxf(b, -125.0f));
  const f32x2 one = pk(1.0f, 1.0f);
  const f32x2 t = fma2(xc, one, pk(12582912.0f, 12582912.0f));
  const f32x2 f = fma2(fma2(t, one, pk(-12582912.0f, -12582912.0f)), pk(-1.0f, -1.0f), xc);
  f32x2 p = fma2(pk(0.0551716685f, 0.0551716685f), f, pk(0.2426111400f, 0.2426111400f));
  p = fma2(p, f, pk(0.6932609677f, 0.6932609677f));
  p = fma2(p, f, pk(0.9999280572f, 0.9999280572f));
  uint32_t tl, th, pl, ph;
  upku(t, tl, th);
  upku(p, pl, ph);
  return pku(pl + (tl << 23), ph + (th << 23));
}
// which of a block's 16 column pairs take the polynomial: POLY_PAIRS_OF_8 of every 8, spread out
#ifndef ASL_POLY_PAIRS_OF_8
#define ASL_POLY_PAIRS_OF_8 2
#endif
constexpr int POLY_PAIRS_OF_8 = ASL_POLY_PAIRS_OF_8;
__device__ __forceinline__ constexpr bool pair_is_poly(int pi) {
  return POLY_PAIRS_OF_8 >= 4 ? (pi & 1) == 1
                              : ((POLY_PAIRS_OF_8 >= 1 && (pi & 7) == 1) || (POLY_PAIRS_OF_8 >= 2 && (pi & 7) == 5) ||
                                 (POLY_PAIRS_OF_8 >= 3 && (pi & 7) == 3));
}
// sum over 32 accumulator columns of 2^(v*scale + c), c one pair per column pair
template <typename OffsetPair>
__device__ __forceinline__ float exp_sum32(const uint32_t (&cur)[32], f32x2 scale2, OffsetPair off) {
  f32x2 acc_m = pk(0.f, 0.f), acc_p = pk(0.f, 0.f);
  const f32x2 one = pk(1.0f, 1.0f);
#pragma unroll
  for (int pi = 0; pi < 16; ++pi) {
    const f32x2 x = fma2(pku(cur[2 * pi], cur[2 * pi + 1]), scale2, off(pi));
    if (pair_is_poly(pi)) acc_p = fma2(ex2_pair_poly(x), one, acc_p);
    else                  acc_m = fma2(ex2_pair_mufu(x), one, acc_m);
  }
  return hsum(fma2(acc_m, one, acc_p));
}

// K-major, 128B-swizzled operand: rows of 128 B, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)64 << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}
// kind::f16, A = B = bf16, D = fp32, both operands K-major
__device__ __forceinline__ uint32_t instr_desc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// kind::f8f6f4, A = B = E4M3 (format code 0), D = fp32, both operands K-major
__device__ __forceinline__ uint32_t instr_desc_f8(int M, int N) {
  return (1u << 4) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

struct TcArgs {
  const TcPhase* phases;
  const AslReq* req;
  float2* partials;        // pass 1: [segment][CTA][set][NC] (reference, sum) of each epilogue set
  float* offsets;          // [segment][NC], written by the folding warps, read by pass 2
  const float* lse;        // null, or the rows' natural-log softmax denominators [B][H_q][W]: pass 2 alone
  float* u;                // pass 2 out: column sums
  uint32_t* published;     // [segment] epilogue sets that have published, accumulated over launches
  uint32_t* folded;        // [segment] rows whose offset is written, accumulated over launches
  int32_t* err;
  int64_t sum_T;
  uint32_t* epoch_word;    // two-pass launches completed so far (the counters accumulate over launches); then a ticket word
  uint32_t epoch_limit;    // beyond it the last CTA clears the counters instead of letting them wrap
  int32_t nseg;
  const int32_t* live_hdr; // null, or device {phases, work items} of `phases`, written ahead of the launch (the list without
                           // the phases of finished requests); then n_phases / total_items below are not used
  int32_t n_phases, total_items, NC, W, G, Hk, Hq, u_rows_per_kv, u_parts;
  float scale_log2;
};

// walks the CTA's items (global item g = blockIdx.x + i*gridDim.x) through the phase list.  The
// current phase record and the one after it stay in registers: the next record is requested when a
// phase is entered, so its load latency is hidden behind the phase's tiles.
struct ItemWalk {
  const TcPhase* phases;
  int total, n_phases;
  int g, ph;
  TcPhase cur, nxt;
  __device__ __forceinline__ ItemWalk(const TcArgs& a, int n_phases_, int total_) : phases(a.phases), total(total_), n_phases(n_phases_),
                                                                                g((int)blockIdx.x), ph(0) {
    cur = phases[0];
    nxt = phases[n_phases > 1 ? 1 : 0];
  }
  __device__ __forceinline__ bool valid() const { return g < total; }
  __device__ __forceinline__ const TcPhase& phase() {       // phases are sorted by g0 and cover [0, total)
    while (g >= cur.g0 + cur.ntiles) {
      cur = nxt;
      ++ph;
      nxt = phases[ph + 1 < n_phases ? ph + 1 : ph];
    }
    return cur;
  }
  __device__ __forceinline__ bool last_in_phase() const { return g + (int)gridDim.x >= cur.g0 + cur.ntiles; }
  __device__ __forceinline__ void next() { g += (int)gridDim.x; }
};

// FP8: K tiles hold E4M3 codes (one 128-byte row per key: a tile is one 16 KB box), the query chunk holds
// the two E4M3 terms of every query (term t in the t-th 32 KB block of the chunk's buffer, where bf16
// queries keep their t-th 64-channel block), and a tile takes 2 terms x 4 k-steps of 32 channels.
template <bool PER_Q, bool FP8>
__global__ void __launch_bounds__(THREADS, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k, const TcArgs a) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sbase = smem_u32(smem);
  if (sbase & 1023u) {                       // the swizzled operand layout needs a 1024-byte aligned base
    if (threadIdx.x == 0) atomicCAS(a.err, 0, 901);
    return;
  }
  const uint32_t bars = sbase + SM_BAR;
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + SM_MISC);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + SM_MISC + 4);
  volatile uint32_t* s_epoch = reinterpret_cast<volatile uint32_t*>(smem + SM_MISC + 8);
  volatile int* s_list = reinterpret_cast<volatile int*>(smem + SM_MISC + 16);       // {phases, work items} of this launch

  float* s_negoff = reinterpret_cast<float*>(smem + SM_NEGOFF);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int NC = a.NC;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };

  // ---- set-up: zero the Q buffers (rows past NC feed unused MMA rows), barriers, tensor memory ----
  if (NC & 127)
    for (int i = threadIdx.x; i < 2 * Q_BUF_BYTES / 16; i += THREADS) reinterpret_cast<uint4*>(smem + SM_Q)[i] = make_uint4(0, 0, 0, 0);
  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGE; ++s) { mbar_init(bar(BAR_FULL + s), 1); mbar_init(bar(BAR_EMPTY + s), 1); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(BAR_TFULL + i), 1); mbar_init(bar(BAR_TEMPTY + i), 8);
      mbar_init(bar(BAR_QFULL + i), 1); mbar_init(bar(BAR_QEMPTY + i), 1);
    }
    mbar_init(bar(BAR_DRAIN), 1);
    *s_abort = 0;
    // This launch's number.  It is read on the device, not passed by the host, so that a launch
    // replayed from a CUDA graph still counts: no CTA of this launch can see the increment below,
    // which the last CTA to leave makes.
    uint32_t done = 0;
    if (!a.lse) asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(done) : "l"(a.epoch_word) : "memory");
    *s_epoch = done + 1u;
    s_list[0] = a.live_hdr ? __ldcg(a.live_hdr) : a.n_phases;
    s_list[1] = a.live_hdr ? __ldcg(a.live_hdr + 1) : a.total_items;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(sbase + SM_MISC) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;
  const uint32_t epoch = *s_epoch;
  const int n_phases = s_list[0], total_items = s_list[1];

  if (warp == 0) {
    // =============================== TMA producer ===============================
    // Local phase l (the l-th phase in which this CTA has a tile) uses Q buffer l%2.
    if (lane == 0) {
      ItemWalk w(a, n_phases, total_items);
      const uint64_t pol_keep = l2_policy_keep(), pol_stream = l2_policy_stream();
      int item = 0, lp = -1, cur_ph = -1;
      int q_issued = -1;                       // highest local phase whose Q chunk has been requested
      int loaded_seg[2] = {-1, -1};
      int next_ph = -1;                        // the CTA's next phase after the current one (-1: none)
      int tok_off = 0;                         // first token of the current phase's request
      bool ok = true;
      // requests the Q chunk of local phase `l` (phase record p); `block`: wait for the buffer, else only try
      auto issue_q = [&](int l, const TcPhase& p, bool block) -> bool {
        const int b = l & 1, use = l >> 1;
        if (use >= 1) {
          const uint32_t par = (uint32_t)((use - 1) & 1);
          if (block) { if (!mbar_wait(bar(BAR_QEMPTY + b), par, s_abort, 11, true)) return false; }
          else if (!mbar_try(bar(BAR_QEMPTY + b), par)) return true;
        }
        if (loaded_seg[b] == p.seg) {
          mbar_arrive(bar(BAR_QFULL + b));     // same chunk as the buffer holds: nothing to copy
        } else {
          const int r0 = p.chunk * NC;
          const int head = p.h * a.G + r0 / a.W, t0 = r0 % a.W;
          const uint32_t dst = sbase + SM_Q + (uint32_t)b * Q_BUF_BYTES;
          mbar_expect_tx(bar(BAR_QFULL + b), 2u * 128u * (uint32_t)NC);
          if (FP8) {
            tma_load_5d(dst, &tm_q, bar(BAR_QFULL + b), 0, t0, head, p.b, 0);
            tma_load_5d(dst + Q_BLOCK_BYTES, &tm_q, bar(BAR_QFULL + b), 0, t0, head, p.b, 1);
          } else {
            tma_load_4d(dst, &tm_q, bar(BAR_QFULL + b), 0, t0, head, p.b);
            tma_load_4d(dst + Q_BLOCK_BYTES, &tm_q, bar(BAR_QFULL + b), 64, t0, head, p.b);
          }
          loaded_seg[b] = p.seg;
        }
        q_issued = l;
        return true;
      };
      for (; ok && w.valid(); w.next(), ++item) {
        const TcPhase p = w.phase();
        if (w.ph != cur_ph) {
          cur_ph = w.ph;
          ++lp;
          tok_off = p.tok_off;
          if (q_issued < lp && !issue_q(lp, p, true)) { ok = false; break; }
          // where does this CTA go after this phase?
          const int end = p.g0 + p.ntiles;
          const int gn = w.g + ((end - w.g + (int)gridDim.x - 1) / (int)gridDim.x) * (int)gridDim.x;
          next_ph = -1;
          if (gn < w.total) {
            int q = w.ph + 1;
            while (gn >= a.phases[q].g0 + a.phases[q].ntiles) ++q;
            next_ph = q;
          }
        }
        if (next_ph >= 0 && q_issued == lp) {    // prefetch the next phase's Q chunk once its buffer is free
          if (!issue_q(lp + 1, a.phases[next_ph], false)) { ok = false; break; }
        }
        const int s = item % NSTAGE;
        if (!mbar_wait(bar(BAR_EMPTY + s), ((item / NSTAGE) & 1) ^ 1, s_abort, 12, true)) { ok = false; break; }
        mbar_expect_tx(bar(BAR_FULL + s), FP8 ? HALF_BYTES : STAGE_BYTES);
        const uint32_t dst = sbase + SM_K + s * STAGE_BYTES;
        const int tok = tok_off + (w.g - p.g0) * KT;
        const uint64_t pol = p.pass == 1 ? pol_keep : pol_stream;
        tma_load_3d(dst, &tm_k, bar(BAR_FULL + s), 0, p.h, tok, pol);
        if (!FP8) tma_load_3d(dst + HALF_BYTES, &tm_k, bar(BAR_FULL + s), 64, p.h, tok, pol);
      }
      if (!ok) {
        // let the copies already issued land before the CTA's shared memory is released
        const int armed = item < NSTAGE ? item : NSTAGE;
        for (int i = 0; i < armed; ++i) {
          const int it = item - 1 - i, s = it % NSTAGE;
          mbar_wait(bar(BAR_FULL + s), (it / NSTAGE) & 1, s_abort, 13, false);
        }
        for (int l = q_issued; l >= 0 && l > q_issued - 2; --l)
          mbar_wait(bar(BAR_QFULL + (l & 1)), (l >> 1) & 1, s_abort, 14, false);
      }
    }
  } else if (warp == 1) {
    // =============================== MMA issuer =================================
    if (lane == 0) {
      ItemWalk w(a, n_phases, total_items);
      int item = 0, lp = -1, cur_ph = -1;
      bool ok = true;
      const uint32_t idesc1 = FP8 ? instr_desc_f8(128, KT) : instr_desc(128, KT);
      const uint32_t idesc2 = FP8 ? instr_desc_f8(KT, NC) : instr_desc(KT, NC);
      // byte offset of k-step ks inside a K tile: bf16 tiles are two 64-channel blocks, 8-bit tiles one block
      auto k_off = [](int ks) { return (uint32_t)(FP8 ? (ks & 3) * 32 : (ks >> 2) * HALF_BYTES + (ks & 3) * 32); };
      const int nhalf = (NC > 128) ? 2 : 1;
      uint32_t qbase = 0;
      for (; ok && w.valid(); w.next(), ++item) {
        const TcPhase p = w.phase();
        if (w.ph != cur_ph) {
          cur_ph = w.ph;
          ++lp;
          if (!mbar_wait(bar(BAR_QFULL + (lp & 1)), (lp >> 1) & 1, s_abort, 21, true)) { ok = false; break; }
          qbase = sbase + SM_Q + (uint32_t)(lp & 1) * Q_BUF_BYTES;
        }
        const int s = item % NSTAGE, acc = item & 1;
        if (!mbar_wait(bar(BAR_TEMPTY + acc), ((item >> 1) & 1) ^ 1, s_abort, 22, true)) { ok = false; break; }
        if (!mbar_wait(bar(BAR_FULL + s), (item / NSTAGE) & 1, s_abort, 23, true)) { ok = false; break; }
        tc_fence_after();
        const uint32_t kbase = sbase + SM_K + s * STAGE_BYTES;
        const uint32_t d0 = tmem + (uint32_t)(acc * 256);
        if (p.pass == 2) {
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const uint64_t ad = smem_desc(kbase + k_off(ks));
            const uint64_t bd = smem_desc(qbase + (ks >> 2) * Q_BLOCK_BYTES + (ks & 3) * 32);
            if (FP8) tc_mma_f8(d0, ad, bd, idesc2, ks > 0);
            else     tc_mma(d0, ad, bd, idesc2, ks > 0);
          }
        } else {
          for (int hf = 0; hf < nhalf; ++hf) {
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const uint64_t ad = smem_desc(qbase + (ks >> 2) * Q_BLOCK_BYTES + hf * (128 * 128) + (ks & 3) * 32);
              const uint64_t bd = smem_desc(kbase + k_off(ks));
              if (FP8) tc_mma_f8(d0 + (uint32_t)(hf * 128), ad, bd, idesc1, ks > 0);
              else     tc_mma(d0 + (uint32_t)(hf * 128), ad, bd, idesc1, ks > 0);
            }
          }
        }
        tc_commit(bar(BAR_EMPTY + s));       // smem stage free once these MMAs have read it
        tc_commit(bar(BAR_TFULL + acc));     // accumulator ready for the epilogue
        if (w.last_in_phase()) tc_commit(bar(BAR_QEMPTY + (lp & 1)));   // last tile of the phase here
      }
      if (!ok) {  // make sure nothing is still writing tensor memory before it is freed
        tc_commit(bar(BAR_DRAIN));
        mbar_wait(bar(BAR_DRAIN), 0, s_abort, 24, false);
      }
    }
  } else if (warp < 4) {
    // =============================== partial folding ==============================
    // For every segment, in phase order: wait until all its epilogue sets have
    // published, then fold the partials of this CTA's rows in a fixed order (the
    // result does not depend on timing) and count the rows as done.
    const int hw = warp - 2;
    const int grid = (int)gridDim.x;
    const int entries = 2 * grid;                                  // entry e: CTA e/2, set e%2
    for (int ph = 0; ph < n_phases; ++ph) {
      const TcPhase p = a.phases[ph];
      if (p.pass != 1) continue;
      if ((int)blockIdx.x + hw * grid >= NC) continue;             // no row of this segment is ours
      if (!word_wait(a.published + p.seg, epoch * 2u * (uint32_t)p.ncontrib, s_abort, 41, lane, 256)) break;
      const int first = p.g0 % grid;
      for (int row = blockIdx.x + hw * grid; row < NC; row += 2 * grid) {
        const float2* src = a.partials + (int64_t)p.seg * entries * NC + row;
        auto fetch = [&](int e) {
          int d = (e >> 1) - first;
          if (d < 0) d += grid;
          return (e < entries && d < p.ntiles) ? __ldcg(src + (int64_t)e * NC) : make_float2(-INFINITY, 0.f);
        };
        float M = -INFINITY, L = 0.f;
        for (int e0 = 0; e0 < entries; e0 += 320) {
          float2 v[10];
#pragma unroll
          for (int i = 0; i < 10; ++i) v[i] = fetch(e0 + lane + 32 * i);      // all loads in flight
#pragma unroll
          for (int i = 0; i < 10; ++i) {
            if (v[i].y > 0.f) {
              const float Mn = fmaxf(M, v[i].x);
              L = L * ex2(M - Mn) + v[i].y * ex2(v[i].x - Mn);
              M = Mn;
            }
          }
        }
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {                         // butterfly: every lane ends with the same (M, L)
          const float Mo = __shfl_xor_sync(0xffffffffu, M, o), Lo = __shfl_xor_sync(0xffffffffu, L, o);
          const bool lower = (lane & o) == 0;                      // fold in lane order so both partners agree bitwise
          const float Ma = lower ? M : Mo, La = lower ? L : Lo, Mb = lower ? Mo : M, Lb = lower ? Lo : L;
          const float Mn = fmaxf(Ma, Mb);
          float Ln = 0.f;
          if (La > 0.f) Ln += La * ex2(Ma - Mn);
          if (Lb > 0.f) Ln += Lb * ex2(Mb - Mn);
          M = Mn; L = Ln;
        }
        if (lane == 0) {
          __stcg(a.offsets + (int64_t)p.seg * NC + row, M + log2f(L));
          __threadfence();
          atomicAdd(a.folded + p.seg, 1u);
        }
      }
    }
  } else {
    // =============================== epilogue ===================================
    // 16 warps: set = which accumulator (tiles item%2 == set); within a set two warps share each
    // TMEM lane quarter and split the accumulator's columns in halves (`sub`).
    const int e = warp - 4;
    const int set = e >> 3, sub = (e >> 2) & 1;
    const int quarter = warp & 3;       // TMEM lanes 32*quarter .. +31 are this warp's
    const int lt = quarter * 32 + lane;                        // TMEM lane of this thread, 0..127
    const int st = (e & 7) * 32 + lane;                        // thread of the set, 0..255
    const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(set * 256);
    float scale = a.scale_log2;             // log2(e)/sqrt(d) times the phase's accumulator factor (FP8 keys: per kv head)
    f32x2 scale2 = pk(scale, scale);
    float* negoff = s_negoff + set * 256;
    const int nhalf = (NC > 128) ? 2 : 1;
    ItemWalk w(a, n_phases, total_items);
    int item = 0, cur_ph = -1, mine = 0;    // `mine`: tiles this set has taken
    bool dead = false;                      // a wait expired: keep the barrier sequence, skip the work
    // pass-1 state of row sub*128 + lt: sum of 2^(x - mref) over the keys seen so far.  mref is the
    // maximum of the first 32 keys the row met; later blocks do not track the maximum (their terms may
    // exceed 1, fp32 has the range), unless a sum overflows, in which case the tile is redone with it.
    float mref = -INFINITY, l = 0.f;
    bool first_tile = true;                 // this set has not yet taken a tile of the current pass-1 phase
    for (; w.valid(); w.next(), ++item) {
      const TcPhase p = w.phase();
      if (w.ph != cur_ph) {
        cur_ph = w.ph;
        if (FP8) {
          scale = a.scale_log2 * p.kscale;
          scale2 = pk(scale, scale);
        }
        if (p.pass == 1) {
          mref = -INFINITY;
          l = 0.f;
          first_tile = true;
        } else {
          // the segment's offsets: wait until every row has been folded, then stage -offset for this set
          if (!dead && !a.lse) dead = !word_wait(a.folded + p.seg, epoch * (uint32_t)NC, s_abort, 33, lane, 256);
          bar_sync(2 + set, 256);                                 // the set is done with the previous offsets
          if (st < NC) {
            float off = INFINITY;                                 // a padding row: 2^(x - inf) = 0
            if (st >= p.rows) {
            } else if (a.lse) {                                   // supplied: natural log -> log2 domain
              const int r = p.chunk * NC + st;                    // row within the kv head: query head r / W, window row r % W
              off = __ldg(a.lse + ((int64_t)p.b * a.Hq + p.h * a.G + r / a.W) * a.W + r % a.W) * 1.4426950408889634f;
            } else {
              off = __ldcg(a.offsets + (int64_t)p.seg * NC + st);
            }
            negoff[st] = dead ? 0.f : -off;
          }
          bar_sync(2 + set, 256);
        }
      }
      if ((item & 1) == set) {
        if (!dead) {
          const bool ok = mbar_wait(bar(BAR_TFULL + set), mine & 1, s_abort, 31, true);
          dead = !__all_sync(0xffffffffu, ok);
        }
        ++mine;
        if (!dead) {
          tc_fence_after();
          const int tile = w.g - p.g0;
          uint32_t cur[32];
          auto release = [&]() {                                   // this warp has read its part of the accumulator
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(BAR_TEMPTY + set));
          };
          if (p.pass == 1) {
            // ---- pass 1: sum of 2^(x - mref) of this thread's row over the tile's 128 keys ----
            // Fast walk: every key of the tile is visible to every row; it does not track the maximum.
            // Careful walk (tiles that reach into the window, or after a sum overflowed in the fast
            // walk): per-row masks, block maxima, MUFU only.
            if (sub < nhalf) {
              const uint32_t addr = lane_base + (uint32_t)(sub * 128);
              const float keep_m = mref, keep_l = l;
              bool careful = tile * KT + KT - 1 > p.T;
              if (!careful) {
#pragma unroll 1
                for (int blk = 0; blk < 4; ++blk) {
                  tc_ld32_issue(addr + (uint32_t)(blk * 32), cur);
                  tc_ld_wait(cur);
                  if (first_tile && blk == 0) {                    // first block of the row: its maximum is the reference
                    float c0 = fmaxf(__uint_as_float(cur[0]), __uint_as_float(cur[1]));
                    float c1 = fmaxf(__uint_as_float(cur[2]), __uint_as_float(cur[3]));
#pragma unroll
                    for (int i = 4; i < 32; i += 4) {
                      c0 = fmaxf(c0, fmaxf(__uint_as_float(cur[i]), __uint_as_float(cur[i + 1])));
                      c1 = fmaxf(c1, fmaxf(__uint_as_float(cur[i + 2]), __uint_as_float(cur[i + 3])));
                    }
                    mref = fmaxf(c0, c1) * scale;
                  }
                  const f32x2 nm2 = pk(-mref, -mref);
                  l += exp_sum32(cur, scale2, [&](int) { return nm2; });
                }
                // a term beyond fp32 range (a logit 127 above the reference): redo the tile carefully
                careful = __any_sync(0xffffffffu, !(l < INFINITY));
                if (careful) { mref = keep_m; l = keep_l; }
              }
              if (careful) {
                const int row = sub * 128 + lt;
                const int lastkey = p.T + (p.chunk * NC + row) % a.W;       // last key this row sees
#pragma unroll 1
                for (int blk = 0; blk < 4; ++blk) {
                  tc_ld32_issue(addr + (uint32_t)(blk * 32), cur);
                  tc_ld_wait(cur);
                  const int j0 = tile * KT + blk * 32;
                  if (j0 <= lastkey) {
                    float c = -INFINITY;
#pragma unroll
                    for (int i = 0; i < 32; ++i) c = fmaxf(c, (j0 + i <= lastkey) ? __uint_as_float(cur[i]) : -INFINITY);
                    const float mn = fmaxf(mref, c * scale);
                    float s0 = 0.f, s1 = 0.f;
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                      s0 += (j0 + i <= lastkey) ? ex2(fmaf(__uint_as_float(cur[i]), scale, -mn)) : 0.f;
                      s1 += (j0 + i + 1 <= lastkey) ? ex2(fmaf(__uint_as_float(cur[i + 1]), scale, -mn)) : 0.f;
                    }
                    l = fmaf(l, ex2(mref - mn), s0 + s1);
                    mref = mn;
                  }
                }
              }
              if (l > 0x1p60f) { l *= 0x1p-60f; mref += 60.f; }     // exact: keeps the running sum far from overflow
            }
            release();
            first_tile = false;
          } else {
            // ---- pass 2: this thread's key, exp2(x - offset[row]) summed over its half of the chunk's rows ----
            const int half_cols = NC >> 1, nblk = half_cols >> 5;
            const uint32_t addr = lane_base + (uint32_t)(sub * half_cols);
            const float* no_base = negoff + sub * half_cols;
            float sums[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
            for (int blk = 0; blk < nblk; ++blk) {
              tc_ld32_issue(addr + (uint32_t)(blk * 32), cur);
              tc_ld_wait(cur);
              if (blk + 1 == nblk) release();
              const float4* no = reinterpret_cast<const float4*>(no_base + blk * 32);   // two column pairs per load
              const float bs = exp_sum32(cur, scale2, [&](int pi) {
                const float4 v = no[pi >> 1];
                return (pi & 1) ? pk(v.z, v.w) : pk(v.x, v.y);
              });
              if (PER_Q) {                                         // W is a multiple of 32: a block never straddles heads
                const int slot = (blk * 32) / a.W;
#pragma unroll
                for (int q = 0; q < 4; ++q) sums[q] += (q == slot) ? bs : 0.f;
              } else {
                sums[0] += bs;
              }
            }
            const int j = tile * KT + lt;
            if (j < p.T) {
              if (PER_Q) {
                // heads of this half: half_cols / W of them, or a part of one head when W > half_cols
                const int col0 = p.chunk * NC + sub * half_cols;
                if (a.W > half_cols) {
                  a.u[(int64_t)((p.h * a.G + col0 / a.W) * 2 + sub) * a.sum_T + p.t_off + j] = sums[0];
                } else {
                  const int nslot = half_cols / a.W;
#pragma unroll
                  for (int q = 0; q < 4; ++q)
                    if (q < nslot) a.u[(int64_t)((p.h * a.G + col0 / a.W + q) * a.u_parts) * a.sum_T + p.t_off + j] = sums[q];
                }
              } else {
                a.u[(int64_t)(p.h * a.u_rows_per_kv + p.chunk * 2 + sub) * a.sum_T + p.t_off + j] = sums[0];
              }
            }
          }
        }
      }
      if (w.last_in_phase() && p.pass == 1) {
        // ---- end of a pass-1 phase in this CTA: each set publishes its own (reference, sum) per row ----
        float2* out = a.partials + (((int64_t)p.seg * gridDim.x + blockIdx.x) * 2 + set) * NC;
        const int row = sub * 128 + lt;
        if (sub < nhalf && row < NC) __stcg(out + row, make_float2(mref, dead ? 0.f : l));
        bar_sync(2 + set, 256);
        if (st == 0) {                 // the barrier orders the set's stores before this thread's fence: the release is cumulative
          __threadfence();
          atomicAdd(a.published + p.seg, 1u);
        }
      }
    }
  }

  // ---- teardown ----
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
  if (threadIdx.x == 0 && *s_abort) atomicCAS(a.err, 0, *s_abort);
  if (threadIdx.x == 0 && !a.lse) {
    // the last CTA to leave closes the launch: next launch number, or a fresh start before the counters wrap
    __threadfence();
    if (atomicAdd(a.epoch_word + 1, 1u) == gridDim.x - 1u) {
      a.epoch_word[1] = 0;
      if (epoch >= a.epoch_limit) {
        for (int i = 0; i < 2 * a.nseg; ++i) a.published[i] = 0;      // published and folded are contiguous
        a.epoch_word[0] = 0;
      } else {
        a.epoch_word[0] = epoch;
      }
      __threadfence();
    }
  }
}

// One warp runs one of the kernel's two kinds of bounded wait on something that never happens (a barrier
// nobody arrives on, a counter nobody advances) with a short limit, and reports like the scorer does.
__global__ void bounded_wait_selftest_kernel(int which, unsigned long long limit_ns, const uint32_t* never_written,
                                             int32_t* err) {
  __shared__ __align__(8) unsigned long long s_bar;
  __shared__ int s_flag;
  const int lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&s_bar), 1);
    s_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  volatile int* abort_flag = &s_flag;
  bool ok;
  if (which == 0) ok = mbar_wait(smem_u32(&s_bar), 0, abort_flag, 91, true, limit_ns);
  else            ok = word_wait(never_written, 0xFFFFFFFFu, abort_flag, 92, lane, 256, limit_ns);
  __syncthreads();
  if (threadIdx.x == 0 && !ok && *abort_flag) atomicCAS(err, 0, *abort_flag);
}

// Device-side controller: the phase list of the next launch without the phases of finished requests.
// One block.  The requests' flags are read once (a record may be changing under a statistic kernel of the
// previous layer that is still running: whatever is read here holds for the whole launch), the live
// phases are copied in order with their first work item recomputed, and the header {phases, items} is
// written.  Segments that are left out of a two-pass launch have their publish counters advanced as if
// they had been scored, so that a later launch that scores them again (a new prompt) finds them where
// its launch number expects them.
__global__ void __launch_bounds__(256) live_phase_list_kernel(const TcPhase* __restrict__ all, int n_all, const asl_stat* __restrict__ latch,
                                                             int cur, int batch, int two_pass, int NC, TcPhase* __restrict__ live,
                                                             int32_t* __restrict__ hdr, uint32_t* __restrict__ published,
                                                             uint32_t* __restrict__ folded) {
  __shared__ uint32_t fin[ASL_SKIP_MAX_BATCH / 32];
  __shared__ int w_items[8], w_cnt[8];
  __shared__ int base_items, base_cnt;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  for (int b0 = 0; b0 < batch; b0 += 256) {
    const int b = b0 + tid;
    const uint32_t word = __ballot_sync(0xffffffffu, b < batch && asl_finished(latch + b, cur));
    if (lane == 0) fin[b >> 5] = word;
  }
  if (tid == 0) { base_items = 0; base_cnt = 0; }
  __syncthreads();
  for (int i0 = 0; i0 < n_all; i0 += 256) {
    const int i = i0 + tid;
    TcPhase ph{};
    bool is_live = false;
    if (i < n_all) {
      ph = all[i];
      is_live = ((fin[ph.b >> 5] >> (ph.b & 31)) & 1u) == 0u;
      if (!is_live && two_pass && ph.pass == 1) { published[ph.seg] += 2u * (uint32_t)ph.ncontrib; folded[ph.seg] += (uint32_t)NC; }
    }
    int items = is_live ? ph.ntiles : 0, cnt = is_live ? 1 : 0;
    int inc_items = items, inc_cnt = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int a = __shfl_up_sync(0xffffffffu, inc_items, o), c2 = __shfl_up_sync(0xffffffffu, inc_cnt, o);
      if (lane >= o) { inc_items += a; inc_cnt += c2; }
    }
    if (lane == 31) { w_items[wid] = inc_items; w_cnt[wid] = inc_cnt; }
    __syncthreads();
    int off_items = base_items + inc_items - items, off_cnt = base_cnt + inc_cnt - cnt;
    for (int w2 = 0; w2 < wid; ++w2) { off_items += w_items[w2]; off_cnt += w_cnt[w2]; }
    if (is_live) { ph.g0 = off_items; live[off_cnt] = ph; }
    __syncthreads();
    if (tid == 255) { base_items = off_items + items; base_cnt = off_cnt + cnt; }
    __syncthreads();
  }
  if (tid == 0) { hdr[0] = base_cnt; hdr[1] = base_items; }
}

// FP8 keys: the bf16 window queries, scaled by Q8_SCALE, as two E4M3 terms hi + lo (hi = nearest code,
// lo = nearest code of the remainder; together exact whenever the remainder's bits fit the format, i.e.
// for 1/64 <= |q| <= 28): out[t][b][head][row][c], dense.
constexpr float Q8_SCALE = 16.0f;
__global__ void __launch_bounds__(256) split_queries_e4m3_kernel(const __nv_bfloat16* __restrict__ q, int64_t qs_b, int64_t qs_h,
                                                                 int64_t qs_r, int Hq, int W, int64_t total,
                                                                 uint8_t* __restrict__ out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int c = (int)(i & 127);
  const int64_t r = i >> 7;
  const int row = (int)(r % W), head = (int)((r / W) % Hq);
  const int64_t b = r / ((int64_t)W * Hq);
  const float x = __bfloat162float(q[b * qs_b + head * qs_h + row * qs_r + c]) * Q8_SCALE;
  const __nv_fp8_storage_t hi = __nv_cvt_float_to_fp8(x, __NV_SATFINITE, __NV_E4M3);
  const float xh = __half2float(__half(__nv_cvt_fp8_to_halfraw(hi, __NV_E4M3)));
  const __nv_fp8_storage_t lo = __nv_cvt_float_to_fp8(x - xh, __NV_SATFINITE, __NV_E4M3);
  out[i] = hi;
  out[total + i] = lo;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

bool make_map(CUtensorMap* tm, CUtensorMapDataType dtype, const void* base, int rank, const cuuint64_t* dims,
              const cuuint64_t* strides_bytes, const cuuint32_t* box) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  return fn(tm, dtype, rank, const_cast<void*>(base), dims, strides_bytes, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// ---------------------------------------------------------------- host side
bool asl_tc_plan(asl_ctx* c) {
  const asl_params& p = c->p;
  AslTcPlan& tp = c->tc;
  tp = AslTcPlan();
  const int W = p.window, G = p.n_q_heads / p.n_kv_heads, R = G * W;
  if (p.head_dim != 128 || W % 32 || W > MAX_NC) return false;
  // Chunk of NC query rows (whole heads, a multiple of 64 rows, at most 256).  Max pooling wants the
  // chunks to tile the G*W rows exactly (its column sums are kept per query head).  Average pooling
  // sums all rows of a kv head anyway, so the last chunk may be padded: its extra rows are given an
  // infinite offset in pass 2 and add nothing.  Fewest chunks first, then least padding.
  int NC = 0;
  if (p.pool_mode == ASL_POOL_MAX) {
    for (int m = MAX_NC / W; m >= 1; --m)
      if (R % (m * W) == 0) { NC = m * W; break; }
    if (NC < 64 || NC % 64 || R % NC) return false;
  } else {
    int best_chunks = 0;
    for (int m = 1; m * W <= MAX_NC; ++m) {
      const int nc = m * W;
      if (nc % 64) continue;
      const int chunks = (R + nc - 1) / nc;
      if (!NC || chunks < best_chunks) { NC = nc; best_chunks = chunks; }
    }
    if (!NC) return false;
  }
  tp.NC = NC;
  tp.nchunk = (R + NC - 1) / NC;
  tp.grid = (p.score_ctas > 0 && p.score_ctas < c->sm_count) ? p.score_ctas : c->sm_count;

  // segments in (request, head, chunk) order; phases in groups: pass 1 of `group` segments, then their pass 2
  struct Seg { int b, h, chunk, tiles1, tiles2; };
  std::vector<Seg> segs;
  for (int b = 0; b < p.batch; ++b)
    for (int h = 0; h < p.n_kv_heads; ++h)
      for (int ch = 0; ch < tp.nchunk; ++ch)
        segs.push_back({b, h, ch, (c->req[b].n + KT - 1) / KT, (c->req[b].T + KT - 1) / KT});
  tp.nseg = (int)segs.size();
  // Segments per group: pass 1 of all of them runs before their pass 2, which hides the fold of the
  // row denominators; K of a whole group has to stay in L2 between the passes (72 MB of the 126 MB).
  int group = 0;
  {
    const double seg_bytes = (double)c->sum_tokens * p.k_stride[0] * c->k_elem_bytes / p.n_kv_heads / (double)p.batch;   // one kv head of an average request
    group = (int)(72.0e6 / (seg_bytes > 1.0 ? seg_bytes : 1.0));
    group = group < 1 ? 1 : (group > 16 ? 16 : group);
  }
  tp.group = group;
  int64_t g = 0;
  auto push = [&](int s, int pass) {
    TcPhase ph{};
    ph.g0 = (int32_t)g;
    ph.ntiles = pass == 1 ? segs[s].tiles1 : segs[s].tiles2;
    ph.pass = pass; ph.seg = s; ph.b = segs[s].b; ph.h = segs[s].h; ph.chunk = segs[s].chunk;
    ph.ncontrib = segs[s].tiles1 < tp.grid ? segs[s].tiles1 : tp.grid;    // CTAs with a tile in pass 1
    ph.T = c->req[ph.b].T; ph.t_off = c->req[ph.b].t_off; ph.tok_off = c->req[ph.b].tok_off;
    ph.rows = R - ph.chunk * NC < NC ? R - ph.chunk * NC : NC;
    ph.kscale = p.k_dtype == ASL_K_FP8_E4M3 ? c->k_scale[ph.h] / Q8_SCALE : 1.0f;
    g += ph.ntiles;
    tp.phases.push_back(ph);
  };
  for (int s0 = 0; s0 < tp.nseg; s0 += group) {
    const int s1 = s0 + group < tp.nseg ? s0 + group : tp.nseg;
    for (int s = s0; s < s1; ++s) push(s, 1);
    for (int s = s0; s < s1; ++s) push(s, 2);
  }
  if (g >= ((int64_t)1 << 31) - tp.grid) return false;
  tp.total_items = (int32_t)g;

  std::vector<TcPhase> only2;
  int64_t g2 = 0;
  for (const TcPhase& ph : tp.phases)
    if (ph.pass == 2) { TcPhase q = ph; q.g0 = (int32_t)g2; g2 += q.ntiles; only2.push_back(q); }
  tp.n_phases2 = (int32_t)only2.size();
  tp.total_items2 = (int32_t)g2;

  const size_t sync_bytes = (2 * (size_t)tp.nseg + 2) * sizeof(uint32_t);   // counters, launch number, exit ticket
  cudaError_t e = cudaMalloc(&tp.d_phases, tp.phases.size() * sizeof(TcPhase));
  if (e == cudaSuccess) e = cudaMalloc(&tp.d_phases2, only2.size() * sizeof(TcPhase));
  if (e == cudaSuccess) e = cudaMemcpy(tp.d_phases2, only2.data(), only2.size() * sizeof(TcPhase), cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMalloc(&tp.d_sync, sync_bytes);
  if (e == cudaSuccess) e = cudaMalloc(&tp.d_live, tp.phases.size() * sizeof(TcPhase));
  if (e == cudaSuccess) e = cudaMalloc(&tp.d_live_hdr, 2 * sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMemcpy(tp.d_phases, tp.phases.data(), tp.phases.size() * sizeof(TcPhase), cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemset(tp.d_sync, 0, sync_bytes);
  if (e != cudaSuccess) { asl_tc_free(c); return false; }
  cudaFuncSetAttribute(score_tc_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  cudaFuncSetAttribute(score_tc_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  cudaFuncSetAttribute(score_tc_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  cudaFuncSetAttribute(score_tc_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  if (cudaGetLastError() != cudaSuccess) { asl_tc_free(c); return false; }
  tp.enabled = encode_fn() != nullptr;
  return tp.enabled;
}

size_t asl_tc_partial_bytes(const asl_ctx* c) {
  const AslTcPlan& tp = c->tc;
  return (size_t)tp.nseg * tp.grid * 2 * tp.NC * sizeof(float2);
}

void asl_tc_free(asl_ctx* c) {
  AslTcPlan& tp = c->tc;
  if (tp.d_phases) cudaFree(tp.d_phases);
  if (tp.d_phases2) cudaFree(tp.d_phases2);
  if (tp.d_sync) cudaFree(tp.d_sync);
  if (tp.d_live) cudaFree(tp.d_live);
  if (tp.d_live_hdr) cudaFree(tp.d_live_hdr);
  tp.d_live = nullptr;
  tp.d_live_hdr = nullptr;
  tp.d_phases = nullptr;
  tp.d_phases2 = nullptr;
  tp.d_sync = nullptr;
  tp.enabled = false;
}

asl_status asl_launch_wait_selftest(asl_ctx* c, int which, unsigned long long limit_ns, cudaStream_t st) {
  bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(which, limit_ns, reinterpret_cast<const uint32_t*>(c->d_err), c->d_err);   // the error word is never all ones
  c->launches += 1;
  ASL_CUDA(cudaGetLastError());
  return ASL_OK;
}

asl_status asl_launch_live_phases(asl_ctx* c, bool two_pass, cudaStream_t st) {
  AslTcPlan& tp = c->tc;
  const TcPhase* all = two_pass ? tp.d_phases : tp.d_phases2;
  const int n_all = two_pass ? (int)tp.phases.size() : tp.n_phases2;
  live_phase_list_kernel<<<1, 256, 0, st>>>(all, n_all, c->latch_stat, c->cur_layer, c->p.batch, two_pass ? 1 : 0, tp.NC, tp.d_live,
                                            tp.d_live_hdr, tp.d_sync, tp.d_sync + tp.nseg);
  c->launches += 1;
  ASL_CUDA(cudaGetLastError());
  return ASL_OK;
}

// after a reported device error the publish counters may be inconsistent: start over
asl_status asl_tc_reset_sync(asl_ctx* c, cudaStream_t st) {
  AslTcPlan& tp = c->tc;
  if (!tp.d_sync) return ASL_OK;
  ASL_CUDA(cudaMemsetAsync(tp.d_sync, 0, (2 * (size_t)tp.nseg + 2) * sizeof(uint32_t), st));
  return ASL_OK;
}

asl_status asl_launch_score_tc(asl_ctx* c, const void* q, const void* k, const float* lse, float* u, char* ws,
                               cudaStream_t st) {
  const asl_params& p = c->p;
  AslTcPlan& tp = c->tc;
  const int W = p.window, G = p.n_q_heads / p.n_kv_heads, NC = tp.NC;
  const bool fp8 = p.k_dtype == ASL_K_FP8_E4M3;
  CUtensorMap tm_q, tm_k;
  const cuuint32_t bw = (cuuint32_t)(W < NC ? W : NC);
  if (fp8) {
    // the queries as two E4M3 terms in the workspace, then 8-bit maps: rows of 128 one-byte channels
    uint8_t* q8 = reinterpret_cast<uint8_t*>(ws + c->ws.score_q8);
    const int64_t total = (int64_t)p.batch * p.n_q_heads * W * 128;
    split_queries_e4m3_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(
        static_cast<const __nv_bfloat16*>(q), p.q_stride[0], p.q_stride[1], p.q_stride[2], p.n_q_heads, W, total, q8);
    c->launches += 1;
    const cuuint64_t qdims[5] = {128, (cuuint64_t)W, (cuuint64_t)p.n_q_heads, (cuuint64_t)p.batch, 2};
    const cuuint64_t qstr[4] = {128, (cuuint64_t)W * 128, (cuuint64_t)p.n_q_heads * W * 128, (cuuint64_t)total};
    const cuuint32_t qbox[5] = {128, bw, (cuuint32_t)NC / bw, 1, 1};
    if (!make_map(&tm_q, CU_TENSOR_MAP_DATA_TYPE_UINT8, q8, 5, qdims, qstr, qbox)) return ASL_ERR_CUDA;
    const cuuint64_t kdims[3] = {128, (cuuint64_t)p.n_kv_heads, (cuuint64_t)c->sum_tokens};
    const cuuint64_t kstr[2] = {(cuuint64_t)p.k_stride[1], (cuuint64_t)p.k_stride[0]};
    const cuuint32_t kbox[3] = {128, 1, (cuuint32_t)KT};
    if (!make_map(&tm_k, CU_TENSOR_MAP_DATA_TYPE_UINT8, k, 3, kdims, kstr, kbox)) return ASL_ERR_CUDA;
  } else {
    const cuuint64_t dims[4] = {128, (cuuint64_t)W, (cuuint64_t)p.n_q_heads, (cuuint64_t)p.batch};
    const cuuint64_t strides[3] = {(cuuint64_t)p.q_stride[2] * 2, (cuuint64_t)p.q_stride[1] * 2, (cuuint64_t)p.q_stride[0] * 2};
    const cuuint32_t box[4] = {64, bw, (cuuint32_t)NC / bw, 1};
    if (!make_map(&tm_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, q, 4, dims, strides, box)) return ASL_ERR_CUDA;
    const cuuint64_t kdims[3] = {128, (cuuint64_t)p.n_kv_heads, (cuuint64_t)c->sum_tokens};
    const cuuint64_t kstr[2] = {(cuuint64_t)p.k_stride[1] * 2, (cuuint64_t)p.k_stride[0] * 2};
    const cuuint32_t kbox[3] = {64, 1, (cuuint32_t)KT};
    if (!make_map(&tm_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, k, 3, kdims, kstr, kbox)) return ASL_ERR_CUDA;
  }
  TcArgs a{};
  const bool live_list = c->latch_stat && c->cur_layer >= 0 && p.batch <= ASL_SKIP_MAX_BATCH;   // written by asl_launch_live_phases just before
  a.phases = live_list ? tp.d_live : (lse ? tp.d_phases2 : tp.d_phases);
  a.live_hdr = live_list ? tp.d_live_hdr : nullptr;
  a.lse = lse;
  a.req = c->d_req;
  a.partials = reinterpret_cast<float2*>(ws + c->ws.score_partials);
  a.offsets = reinterpret_cast<float*>(ws + c->ws.score_offsets);
  a.u = u;
  a.published = tp.d_sync;
  a.folded = tp.d_sync + tp.nseg;
  a.err = c->d_err;
  a.sum_T = c->sum_T;
  a.epoch_word = tp.d_sync + 2 * tp.nseg;         // the one-pass launch touches neither the counters nor this
  a.epoch_limit = 0xFFFFFFFFu / (uint32_t)(2 * tp.grid > MAX_NC ? 2 * tp.grid : MAX_NC) - 2u;
  a.nseg = tp.nseg;
  a.n_phases = lse ? tp.n_phases2 : (int32_t)tp.phases.size();
  a.total_items = lse ? tp.total_items2 : tp.total_items;
  a.NC = NC; a.W = W; a.G = G; a.Hk = p.n_kv_heads; a.Hq = p.n_q_heads;
  a.u_rows_per_kv = c->u_rows_per_kv;
  a.u_parts = c->u_parts;
  a.scale_log2 = (float)(1.4426950408889634 / sqrt((double)p.head_dim));
  // every CTA must be resident at once (pass 2 waits for counters other CTAs advance): one CTA per SM at most
  const int grid = tp.grid;
  const bool per_q = p.pool_mode == ASL_POOL_MAX;
  if (fp8) {
    if (per_q) score_tc_kernel<true, true><<<grid, THREADS, SMEM_BYTES, st>>>(tm_q, tm_k, a);
    else       score_tc_kernel<false, true><<<grid, THREADS, SMEM_BYTES, st>>>(tm_q, tm_k, a);
  } else {
    if (per_q) score_tc_kernel<true, false><<<grid, THREADS, SMEM_BYTES, st>>>(tm_q, tm_k, a);
    else       score_tc_kernel<false, false><<<grid, THREADS, SMEM_BYTES, st>>>(tm_q, tm_k, a);
  }
  c->launches += 1;
  ASL_CUDA(cudaGetLastError());
  return ASL_OK;
}
