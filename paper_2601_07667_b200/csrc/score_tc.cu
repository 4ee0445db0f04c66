// Observation-window scorer on the 5th-generation tensor cores (Algorithm 1 lines 3-4).
//
// One persistent CTA per SM streams 128-key tiles of bf16 K through a 4-stage
// TMA ring into 128B-swizzled shared memory; one thread issues tcgen05.mma with
// fp32 accumulators in tensor memory (two 256-column buffers, so the MMAs of
// tile i+1 overlap the exponentials of tile i); eight warps read the
// accumulators back with tcgen05.ld and do the softmax arithmetic in the log2
// domain x = (q.k) * log2(e)/sqrt(d).
//
//   pass 1  D[row][key] = Q_chunk . K_tile^T  (query rows in TMEM lanes): each
//           thread owns one query row and keeps an online (max, sum); one
//           partial per (work unit, row); a combine kernel folds a row's
//           partials in unit order into offset = max + log2(sum).
//   pass 2  D[key][row] = K_tile . Q_chunk^T  (keys in TMEM lanes): each thread
//           owns one key and sums exp2(x - offset[row]) over the chunk's rows:
//           the key's column sum U, already summed over the GQA group.
//
// A "chunk" is up to 256 of the G*W query rows that share a kv head (the MMA's
// N in pass 2); a "work unit" is a run of consecutive key tiles of one
// (request, kv head, chunk).  Units are dealt round-robin to the CTAs in
// (request, head, chunk, tile) order, so all CTAs work on the same kv head at
// the same time.
//
// Every wait on an mbarrier is bounded: when the limit is reached the thread
// records a code in the context's error word, raises the CTA's abort flag and
// all roles fall through to the common teardown (in-flight copies are waited
// for with the same bound, tensor memory is freed).
#include <cuda.h>

#include "asl_internal.cuh"

namespace {

constexpr int KT = ASL_TC_KEY_TILE;          // keys per tile
constexpr int NSTAGE = 4;
constexpr int HALF_BYTES = KT * 128;         // one 64-channel block of a K tile: 128 rows x 128 B
constexpr int STAGE_BYTES = 2 * HALF_BYTES;
constexpr int MAX_NC = 256;
constexpr int Q_BLOCK_BYTES = MAX_NC * 128;  // one 64-channel block of the Q chunk
constexpr int THREADS = 320;                 // warp 0: TMA, warp 1: MMA, warps 2-9: epilogue
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;   // every wait gives up after 2 s

// shared-memory map (offsets from a 1024-aligned base)
constexpr int SM_Q = 0;
constexpr int SM_K = SM_Q + 2 * Q_BLOCK_BYTES;
constexpr int SM_NEGOFF = SM_K + NSTAGE * STAGE_BYTES;       // float[256]
constexpr int SM_SCRATCH = SM_NEGOFF + 1024;                 // float2[2][2][128] = 4 KB
constexpr int SM_BAR = SM_SCRATCH + 4096;                    // mbarriers
constexpr int SM_MISC = SM_BAR + 128;                        // tmem base, abort flag
constexpr int SM_TOTAL = SM_MISC + 64;
constexpr int SMEM_BYTES = SM_TOTAL + 1024;                  // slack for the alignment

enum { BAR_FULL = 0, BAR_EMPTY = NSTAGE, BAR_TFULL = 2 * NSTAGE, BAR_TEMPTY = 2 * NSTAGE + 2,
       BAR_QFULL = 2 * NSTAGE + 4, BAR_QEMPTY = 2 * NSTAGE + 5, BAR_DRAIN = 2 * NSTAGE + 6, N_BARS = 2 * NSTAGE + 7 };
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
// Bounded wait.  `watch_abort`: also give up when another role raised the flag.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int code,
                                          bool watch_abort) {
  unsigned long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    if (mbar_try(bar, parity)) return true;
    if ((it & 15u) == 15u) {
      if (watch_abort && *abort_flag) return false;
      unsigned long long now;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
      if (t0 == 0) t0 = now;
      else if (now - t0 > WAIT_LIMIT_NS) break;
    }
  }
  *abort_flag = code;
  return false;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(dst),
      "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
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
// 32 consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
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
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// K-major, 128B-swizzled operand: rows of 128 B, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)64 << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}
// kind::f16, A = B = bf16, D = fp32, both operands K-major
__device__ __forceinline__ uint32_t instr_desc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

struct TcArgs {
  const TcUnit* units;
  const AslReq* req;
  float2* partials;        // pass 1 out: [unit][NC]
  const float* offsets;    // pass 2 in:  [B][H_k][R]
  float* u;                // pass 2 out: column sums
  int32_t* err;
  int64_t sum_T;
  int32_t n_units, NC, W, G, Hk, R, u_rows_per_kv;
  float scale_log2;
};

template <int PASS, bool PER_Q>
__global__ void __launch_bounds__(THREADS, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k, const TcArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bars = sbase + SM_BAR;
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + SM_MISC);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + SM_MISC + 4);
  float* s_negoff = reinterpret_cast<float*>(smem + SM_NEGOFF);
  float2* s_scratch = reinterpret_cast<float2*>(smem + SM_SCRATCH);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int NC = a.NC;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };

  // ---- set-up: zero the Q area (rows past NC feed unused MMA rows), barriers, tensor memory ----
  for (int i = threadIdx.x; i < 2 * Q_BLOCK_BYTES / 16; i += THREADS) reinterpret_cast<uint4*>(smem + SM_Q)[i] = make_uint4(0, 0, 0, 0);
  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGE; ++s) { mbar_init(bar(BAR_FULL + s), 1); mbar_init(bar(BAR_EMPTY + s), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar(BAR_TFULL + i), 1); mbar_init(bar(BAR_TEMPTY + i), 8); }
    mbar_init(bar(BAR_QFULL), 1);
    mbar_init(bar(BAR_QEMPTY), 1);
    mbar_init(bar(BAR_DRAIN), 1);
    *s_abort = 0;
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

  if (warp == 0) {
    // =============================== TMA producer ===============================
    if (lane == 0) {
      int tile_iter = 0, seg_iter = 0, cur_seg = -1;
      bool ok = true;
      for (int ui = blockIdx.x; ok && ui < a.n_units; ui += gridDim.x) {
        const TcUnit u = a.units[ui];
        if (u.seg != cur_seg) {
          if (seg_iter > 0 && !mbar_wait(bar(BAR_QEMPTY), (seg_iter - 1) & 1, s_abort, 11, true)) { ok = false; break; }
          const int r0 = u.chunk * NC;
          const int head = u.h * a.G + r0 / a.W, t0 = r0 % a.W;
          mbar_expect_tx(bar(BAR_QFULL), 2u * 128u * (uint32_t)NC);
          tma_load_4d(sbase + SM_Q, &tm_q, bar(BAR_QFULL), 0, t0, head, u.b);
          tma_load_4d(sbase + SM_Q + Q_BLOCK_BYTES, &tm_q, bar(BAR_QFULL), 64, t0, head, u.b);
          cur_seg = u.seg;
          ++seg_iter;
        }
        const int tok0 = a.req[u.b].tok_off + u.tile0 * KT;
        for (int t = 0; t < u.ntiles; ++t, ++tile_iter) {
          const int s = tile_iter % NSTAGE;
          if (!mbar_wait(bar(BAR_EMPTY + s), ((tile_iter / NSTAGE) & 1) ^ 1, s_abort, 12, true)) { ok = false; break; }
          mbar_expect_tx(bar(BAR_FULL + s), STAGE_BYTES);
          const uint32_t dst = sbase + SM_K + s * STAGE_BYTES;
          tma_load_3d(dst, &tm_k, bar(BAR_FULL + s), 0, u.h, tok0 + t * KT);
          tma_load_3d(dst + HALF_BYTES, &tm_k, bar(BAR_FULL + s), 64, u.h, tok0 + t * KT);
        }
      }
      if (!ok) {
        // let the copies already issued land before the CTA's shared memory is released
        const int armed = tile_iter < NSTAGE ? tile_iter : NSTAGE;
        for (int i = 0; i < armed; ++i) {
          const int it = tile_iter - 1 - i, s = it % NSTAGE;
          mbar_wait(bar(BAR_FULL + s), (it / NSTAGE) & 1, s_abort, 13, false);
        }
      }
    }
  } else if (warp == 1) {
    // =============================== MMA issuer =================================
    if (lane == 0) {
      int tile_iter = 0, seg_iter = 0, cur_seg = -1;
      bool ok = true;
      const uint32_t idesc = (PASS == 1) ? instr_desc(128, KT) : instr_desc(KT, NC);
      const int nhalf = (NC > 128) ? 2 : 1;
      for (int ui = blockIdx.x; ok && ui < a.n_units; ui += gridDim.x) {
        const TcUnit u = a.units[ui];
        if (u.seg != cur_seg) {
          if (!mbar_wait(bar(BAR_QFULL), seg_iter & 1, s_abort, 21, true)) { ok = false; break; }
          cur_seg = u.seg;
          ++seg_iter;
        }
        for (int t = 0; t < u.ntiles; ++t, ++tile_iter) {
          const int s = tile_iter % NSTAGE, acc = tile_iter & 1;
          if (!mbar_wait(bar(BAR_TEMPTY + acc), ((tile_iter >> 1) & 1) ^ 1, s_abort, 22, true)) { ok = false; break; }
          if (!mbar_wait(bar(BAR_FULL + s), (tile_iter / NSTAGE) & 1, s_abort, 23, true)) { ok = false; break; }
          tc_fence_after();
          const uint32_t kbase = sbase + SM_K + s * STAGE_BYTES;
          const uint32_t d0 = tmem + (uint32_t)(acc * 256);
          if (PASS == 2) {
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const uint64_t ad = smem_desc(kbase + (ks >> 2) * HALF_BYTES + (ks & 3) * 32);
              const uint64_t bd = smem_desc(sbase + SM_Q + (ks >> 2) * Q_BLOCK_BYTES + (ks & 3) * 32);
              tc_mma(d0, ad, bd, idesc, ks > 0);
            }
          } else {
            for (int hf = 0; hf < nhalf; ++hf) {
#pragma unroll
              for (int ks = 0; ks < 8; ++ks) {
                const uint64_t ad = smem_desc(sbase + SM_Q + (ks >> 2) * Q_BLOCK_BYTES + hf * (128 * 128) + (ks & 3) * 32);
                const uint64_t bd = smem_desc(kbase + (ks >> 2) * HALF_BYTES + (ks & 3) * 32);
                tc_mma(d0 + (uint32_t)(hf * 128), ad, bd, idesc, ks > 0);
              }
            }
          }
          tc_commit(bar(BAR_EMPTY + s));       // smem stage free once these MMAs have read it
          tc_commit(bar(BAR_TFULL + acc));     // accumulator ready for the epilogue
        }
        const int nxt = ui + gridDim.x;
        const int next_seg = (nxt < a.n_units) ? a.units[nxt].seg : -1;
        if (ok && next_seg != cur_seg) tc_commit(bar(BAR_QEMPTY));
      }
      if (!ok) {  // make sure nothing is still writing tensor memory before it is freed
        tc_commit(bar(BAR_DRAIN));
        mbar_wait(bar(BAR_DRAIN), 0, s_abort, 24, false);
      }
    }
  } else {
    // =============================== epilogue ===================================
    const int ew = warp - 2;
    const int half = ew >> 2;           // which half of the columns (or rows) this warp takes
    const int quarter = warp & 3;       // TMEM lanes 32*quarter .. +31 are this warp's
    const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
    const float scale = a.scale_log2;
    int tile_iter = 0, cur_seg = -1, unit_iter = 0;
    bool ok = true;
    for (int ui = blockIdx.x; ok && ui < a.n_units; ui += gridDim.x, ++unit_iter) {
      const TcUnit u = a.units[ui];
      const AslReq rq = a.req[u.b];
      if (PASS == 2 && u.seg != cur_seg) {
        epi_sync();                                 // everyone is done with the previous offsets
        const float* off = a.offsets + ((int64_t)u.b * a.Hk + u.h) * a.R + u.chunk * NC;
        for (int i = threadIdx.x - 64; i < NC; i += 256) s_negoff[i] = -off[i];
        epi_sync();
      }
      cur_seg = u.seg;

      if (PASS == 1) {
        const int nhalf = (NC > 128) ? 2 : 1;
        const int ncb = (nhalf == 2) ? 4 : 2;                       // 32-column blocks this thread reads per tile
        const int col0 = (nhalf == 2) ? half * 128 : half * 64;     // first accumulator column
        const int key0 = (nhalf == 2) ? 0 : half * 64;              // key offset of that column inside the tile
        const int row = (nhalf == 2) ? half * 128 + quarter * 32 + lane : quarter * 32 + lane;
        const bool live = row < NC;
        const int last = rq.T + (u.chunk * NC + row) % a.W;         // last key this row sees
        float m = -INFINITY, l = 0.f;
        for (int t = 0; t < u.ntiles; ++t, ++tile_iter) {
          const int acc = tile_iter & 1;
          ok = mbar_wait(bar(BAR_TFULL + acc), (tile_iter >> 1) & 1, s_abort, 31, false);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          const int jt = (u.tile0 + t) * KT + key0;
          for (int cb = 0; cb < ncb; ++cb) {
            float v[32];
            tc_ld32(lane_addr + (uint32_t)(acc * 256 + col0 + cb * 32), v);
            if (!live) continue;
            const int j0 = jt + cb * 32;
            if (j0 > last) continue;
            if (j0 + 31 > last) {
#pragma unroll
              for (int i = 0; i < 32; ++i) v[i] = (j0 + i <= last) ? v[i] : -INFINITY;
            }
            float cmax = v[0];
#pragma unroll
            for (int i = 1; i < 32; ++i) cmax = fmaxf(cmax, v[i]);
            cmax *= scale;
            if (cmax > m) { l *= ex2(m - cmax); m = cmax; }
            float s0 = 0.f, s1 = 0.f;
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              s0 += ex2(fmaf(v[i], scale, -m));
              s1 += ex2(fmaf(v[i + 1], scale, -m));
            }
            l += s0 + s1;
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(BAR_TEMPTY + acc));
        }
        if (!ok) break;
        float2* out = a.partials + (int64_t)ui * NC;
        if (nhalf == 2) {
          out[row] = make_float2(m, l);
        } else {
          float2* sc = s_scratch + (unit_iter & 1) * 256;
          sc[half * 128 + quarter * 32 + lane] = make_float2(m, l);
          epi_sync();
          if (half == 0 && live) {
            const float2 o = sc[128 + row];
            const float M = fmaxf(m, o.x);
            float L = 0.f;
            if (l > 0.f) L += l * ex2(m - M);
            if (o.y > 0.f) L += o.y * ex2(o.x - M);
            out[row] = make_float2(M, L);
          }
        }
      } else {
        // ---- pass 2 ----
        const int hc = NC >> 1;                                   // columns per half
        const int cw = a.W < hc ? a.W : hc;                       // columns of one query head inside a half
        const int nslot = PER_Q ? hc / cw : 1;
        const bool combine = !PER_Q || a.W > hc;                  // both halves feed the same output row
        const int key_lane = quarter * 32 + lane;
        for (int t = 0; t < u.ntiles; ++t, ++tile_iter) {
          const int acc = tile_iter & 1;
          ok = mbar_wait(bar(BAR_TFULL + acc), (tile_iter >> 1) & 1, s_abort, 32, false);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          float sums[4] = {0.f, 0.f, 0.f, 0.f};
          const int ncb = hc / 32;
          for (int cb = 0; cb < ncb; ++cb) {
            float v[32];
            const int c0 = half * hc + cb * 32;
            tc_ld32(lane_addr + (uint32_t)(acc * 256 + c0), v);
            const float4* no = reinterpret_cast<const float4*>(s_negoff + c0);
            float s0 = 0.f, s1 = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float4 o = no[i];
              s0 += ex2(fmaf(v[4 * i + 0], scale, o.x));
              s1 += ex2(fmaf(v[4 * i + 1], scale, o.y));
              s0 += ex2(fmaf(v[4 * i + 2], scale, o.z));
              s1 += ex2(fmaf(v[4 * i + 3], scale, o.w));
            }
            const int slot = PER_Q ? (cb * 32) / cw : 0;
            sums[slot & 3] += s0 + s1;
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(BAR_TEMPTY + acc));
          const int j = (u.tile0 + t) * KT + key_lane;
          if (combine) {
            float* hs = reinterpret_cast<float*>(s_scratch) + acc * 128;
            if (half == 1) hs[key_lane] = sums[0];
            epi_sync();
            if (half == 0 && j < rq.T) {
              const int row_u = PER_Q ? (u.h * a.G + (u.chunk * NC) / a.W) : (u.h * a.u_rows_per_kv + u.chunk);
              a.u[(int64_t)row_u * a.sum_T + rq.t_off + j] = sums[0] + hs[key_lane];
            }
          } else if (j < rq.T) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              if (q < nslot) {
                const int head = u.h * a.G + (u.chunk * NC + half * hc + q * cw) / a.W;
                a.u[(int64_t)head * a.sum_T + rq.t_off + j] = sums[q];
              }
            }
          }
        }
        if (!ok) break;
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
  if (threadIdx.x == 0 && *s_abort) atomicCAS(a.err, 0, *s_abort + 100 * PASS);
}

// offset[row] = max + log2(sum) over the units of the row's (request, head, chunk), in unit order
__global__ void __launch_bounds__(256) score_tc_combine(const float2* __restrict__ partials, const TcSeg* __restrict__ segs,
                                                        int NC, int Hk, int R, float* __restrict__ offsets) {
  const TcSeg sg = segs[blockIdx.x];
  for (int c = threadIdx.x; c < NC; c += blockDim.x) {
    float M = -INFINITY;
    for (int i = 0; i < sg.nunits; ++i) M = fmaxf(M, partials[(int64_t)(sg.unit0 + i) * NC + c].x);
    float L = 0.f;
    for (int i = 0; i < sg.nunits; ++i) {
      const float2 p = partials[(int64_t)(sg.unit0 + i) * NC + c];
      if (p.y > 0.f) L += p.y * exp2f(p.x - M);
    }
    offsets[((int64_t)sg.b * Hk + sg.h) * R + sg.chunk * NC + c] = M + log2f(L);
  }
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

bool make_map(CUtensorMap* tm, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides_bytes,
              const cuuint32_t* box) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(base), dims, strides_bytes, box, estr,
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
  if (p.head_dim != 128 || W % 32) return false;
  int NC = 0;
  if (W <= 256) {
    for (int m = 256 / W; m >= 1; --m)
      if (R % (m * W) == 0) { NC = m * W; break; }
  } else {
    for (int cnd = 256; cnd >= 64; cnd -= 64)
      if (W % cnd == 0) { NC = cnd; break; }
  }
  if (NC < 64 || NC % 64 || R % NC) return false;
  if (p.pool_mode == ASL_POOL_MAX) {            // per-query-head sums: at most 4 heads per column half
    const int hc = NC / 2, cw = W < hc ? W : hc;
    if (hc / cw > 4) return false;
  }
  tp.NC = NC;
  tp.nchunk = R / NC;
  int64_t tiles1 = 0, tiles2 = 0;
  for (const AslReq& r : c->req) {
    tiles1 += (int64_t)p.n_kv_heads * tp.nchunk * ((r.n + KT - 1) / KT);
    tiles2 += (int64_t)p.n_kv_heads * tp.nchunk * ((r.T + KT - 1) / KT);
  }
  auto build = [&](bool past_only, int64_t total_tiles, std::vector<TcUnit>& units, std::vector<TcSeg>& segs) {
    int64_t tps = (total_tiles + 4 * c->sm_count - 1) / (4 * (int64_t)c->sm_count);
    if (tps < 2) tps = 2;
    if (tps > 32) tps = 32;
    for (int b = 0; b < p.batch; ++b) {
      const int len = past_only ? c->req[b].T : c->req[b].n;
      const int tiles = (len + KT - 1) / KT;
      for (int h = 0; h < p.n_kv_heads; ++h)
        for (int ch = 0; ch < tp.nchunk; ++ch) {
          TcSeg sg{};
          sg.unit0 = (int32_t)units.size(); sg.b = b; sg.h = h; sg.chunk = ch;
          for (int t0 = 0, split = 0; t0 < tiles; t0 += (int)tps, ++split) {
            TcUnit u{};
            u.b = b; u.h = h; u.chunk = ch; u.tile0 = t0;
            u.ntiles = (int32_t)((tiles - t0) < tps ? (tiles - t0) : tps);
            u.seg = (int32_t)segs.size(); u.split = split;
            units.push_back(u);
          }
          sg.nunits = (int32_t)units.size() - sg.unit0;
          segs.push_back(sg);
        }
    }
  };
  std::vector<TcSeg> segs2;
  build(false, tiles1, tp.units1, tp.segs1);
  build(true, tiles2, tp.units2, segs2);
  cudaError_t e = cudaMalloc(&tp.d_units1, tp.units1.size() * sizeof(TcUnit));
  if (e == cudaSuccess) e = cudaMalloc(&tp.d_units2, tp.units2.size() * sizeof(TcUnit));
  if (e == cudaSuccess) e = cudaMalloc(&tp.d_segs1, tp.segs1.size() * sizeof(TcSeg));
  if (e == cudaSuccess) e = cudaMemcpy(tp.d_units1, tp.units1.data(), tp.units1.size() * sizeof(TcUnit), cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(tp.d_units2, tp.units2.data(), tp.units2.size() * sizeof(TcUnit), cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(tp.d_segs1, tp.segs1.data(), tp.segs1.size() * sizeof(TcSeg), cudaMemcpyHostToDevice);
  if (e != cudaSuccess) { asl_tc_free(c); return false; }
  cudaFuncSetAttribute(score_tc_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  cudaFuncSetAttribute(score_tc_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  cudaFuncSetAttribute(score_tc_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  if (cudaGetLastError() != cudaSuccess) { asl_tc_free(c); return false; }
  tp.enabled = encode_fn() != nullptr;
  return tp.enabled;
}

void asl_tc_free(asl_ctx* c) {
  AslTcPlan& tp = c->tc;
  if (tp.d_units1) cudaFree(tp.d_units1);
  if (tp.d_units2) cudaFree(tp.d_units2);
  if (tp.d_segs1) cudaFree(tp.d_segs1);
  tp.d_units1 = tp.d_units2 = nullptr;
  tp.d_segs1 = nullptr;
  tp.enabled = false;
}

asl_status asl_launch_score_tc(asl_ctx* c, const void* q, const void* k, float* scores_kv, float* scores_agg, char* ws,
                               cudaStream_t st) {
  const asl_params& p = c->p;
  AslTcPlan& tp = c->tc;
  const int W = p.window, G = p.n_q_heads / p.n_kv_heads, NC = tp.NC;
  CUtensorMap tm_q, tm_k;
  {
    const cuuint64_t dims[4] = {128, (cuuint64_t)W, (cuuint64_t)p.n_q_heads, (cuuint64_t)p.batch};
    const cuuint64_t strides[3] = {(cuuint64_t)p.q_stride[2] * 2, (cuuint64_t)p.q_stride[1] * 2, (cuuint64_t)p.q_stride[0] * 2};
    const cuuint32_t bw = (cuuint32_t)(W < NC ? W : NC);
    const cuuint32_t box[4] = {64, bw, (cuuint32_t)NC / bw, 1};
    if (!make_map(&tm_q, q, 4, dims, strides, box)) return ASL_ERR_CUDA;
  }
  {
    const cuuint64_t dims[3] = {128, (cuuint64_t)p.n_kv_heads, (cuuint64_t)c->sum_tokens};
    const cuuint64_t strides[2] = {(cuuint64_t)p.k_stride[1] * 2, (cuuint64_t)p.k_stride[0] * 2};
    const cuuint32_t box[3] = {64, 1, (cuuint32_t)KT};
    if (!make_map(&tm_k, k, 3, dims, strides, box)) return ASL_ERR_CUDA;
  }
  TcArgs a{};
  a.req = c->d_req;
  a.partials = reinterpret_cast<float2*>(ws + c->ws.score_partials);
  float* offsets = reinterpret_cast<float*>(ws + c->ws.score_offsets);
  float* u = reinterpret_cast<float*>(ws + c->ws.score_u);
  a.offsets = offsets;
  a.u = u;
  a.err = c->d_err;
  a.sum_T = c->sum_T;
  a.NC = NC; a.W = W; a.G = G; a.Hk = p.n_kv_heads; a.R = c->rows_per_kv;
  a.u_rows_per_kv = c->u_rows_per_kv;
  a.scale_log2 = (float)(1.4426950408889634 / sqrt((double)p.head_dim));
  const int grid = c->sm_count;

  a.units = tp.d_units1;
  a.n_units = (int32_t)tp.units1.size();
  score_tc_kernel<1, false><<<grid < a.n_units ? grid : a.n_units, THREADS, SMEM_BYTES, st>>>(tm_q, tm_k, a);
  score_tc_combine<<<(unsigned)tp.segs1.size(), 256, 0, st>>>(a.partials, tp.d_segs1, NC, a.Hk, a.R, offsets);
  a.units = tp.d_units2;
  a.n_units = (int32_t)tp.units2.size();
  const int g2 = grid < a.n_units ? grid : a.n_units;
  if (p.pool_mode == ASL_POOL_MAX) score_tc_kernel<2, true><<<g2, THREADS, SMEM_BYTES, st>>>(tm_q, tm_k, a);
  else                             score_tc_kernel<2, false><<<g2, THREADS, SMEM_BYTES, st>>>(tm_q, tm_k, a);
  c->launches += 3;
  ASL_CUDA(cudaGetLastError());
  return asl_launch_pool(c, u, scores_kv, scores_agg, st);
}
