// K/V compaction (Algorithm 1 (K[I], V[I])): out[h][r][:] = x[tok_off + idx[h][r]][h][:].
// 16 threads move one row (256 bytes of bf16, 128 bytes of FP8 codes) as 16-byte vectors; K and V in one launch.
#include "asl_internal.cuh"

namespace {

__global__ void __launch_bounds__(256) compact_kv_kernel(const uint8_t* __restrict__ k, const uint8_t* __restrict__ v,
                                                         const int32_t* __restrict__ idx, const AslReq* __restrict__ req,
                                                         int64_t ks_t, int64_t ks_h, int64_t vs_t, int64_t vs_h,
                                                         int64_t sum_kept, int k_vec, int v_vec, const asl_stat* __restrict__ latch,
                                                         int cur_layer, uint8_t* __restrict__ k_out,
                                                         uint8_t* __restrict__ v_out) {
  // strides in bytes; a row is k_vec (v_vec) 16-byte vectors; 16 threads per kept row
  const int b = blockIdx.z, h = blockIdx.y;
  if (latch && asl_finished(latch + b, cur_layer)) return;       // finished request: its compacted cache is final
  const AslReq rq = req[b];
  const int r = blockIdx.x * (blockDim.x / 16) + threadIdx.x / 16;
  const int c = threadIdx.x % 16;
  if (r >= rq.kept) return;
  const int64_t orow = (int64_t)h * sum_kept + rq.kept_off + r;
  const int64_t tok = (int64_t)rq.tok_off + idx[orow];
  if (c < k_vec) {
    const uint4 kv = __ldcs(reinterpret_cast<const uint4*>(k + tok * ks_t + (int64_t)h * ks_h + c * 16));
    __stcs(reinterpret_cast<uint4*>(k_out + (orow * k_vec + c) * 16), kv);
  }
  if (c < v_vec) {
    const uint4 vv = __ldcs(reinterpret_cast<const uint4*>(v + tok * vs_t + (int64_t)h * vs_h + c * 16));
    __stcs(reinterpret_cast<uint4*>(v_out + (orow * v_vec + c) * 16), vv);
  }
}

// Row gather of one tensor with rows of `row_bytes` (a multiple of 16): out[kept_off_b + r] = x[tok_off_b + idx[r]].
// A warp moves one row, 16 bytes per lane per trip.
__global__ void __launch_bounds__(256) compact_rows_kernel(const uint4* __restrict__ x, const int32_t* __restrict__ idx,
                                                           const AslReq* __restrict__ req, int vec_per_row,
                                                           uint4* __restrict__ out) {
  const int b = blockIdx.y;
  const AslReq rq = req[b];
  const int r = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (r >= rq.kept) return;
  const int64_t src = ((int64_t)rq.tok_off + idx[rq.kept_off + r]) * vec_per_row;
  const int64_t dst = ((int64_t)rq.kept_off + r) * vec_per_row;
  for (int c = lane; c < vec_per_row; c += 32) out[dst + c] = x[src + c];
}

}  // namespace

asl_status asl_launch_compact_rows(asl_ctx* c, const void* x, const int32_t* idx, void* out, int64_t row_bytes,
                                   cudaStream_t st) {
  dim3 grid((c->max_kept + 7) / 8, c->p.batch);
  compact_rows_kernel<<<grid, 256, 0, st>>>(static_cast<const uint4*>(x), idx, c->d_req, (int)(row_bytes / 16),
                                            static_cast<uint4*>(out));
  c->launches += 1;
  ASL_CUDA(cudaGetLastError());
  return ASL_OK;
}

asl_status asl_launch_compact(asl_ctx* c, const void* k, const void* v, const int32_t* idx, void* k_out, void* v_out,
                              cudaStream_t st) {
  const asl_params& p = c->p;
  const int kb = c->k_elem_bytes;                          // K elements are 2 bytes (bf16) or 1 (FP8 codes), V is bf16
  const int k_vec = p.head_dim * kb / 16, v_vec = p.head_dim * 2 / 16;
  dim3 grid((c->max_kept + 15) / 16, p.n_kv_heads, p.batch);
  compact_kv_kernel<<<grid, 256, 0, st>>>(static_cast<const uint8_t*>(k), static_cast<const uint8_t*>(v), idx, c->d_req,
                                          p.k_stride[0] * kb, p.k_stride[1] * kb, p.v_stride[0] * 2, p.v_stride[1] * 2,
                                          c->sum_kept, k_vec, v_vec, c->latch_stat, c->cur_layer,
                                          static_cast<uint8_t*>(k_out), static_cast<uint8_t*>(v_out));
  c->launches += 1;
  ASL_CUDA(cudaGetLastError());
  return ASL_OK;
}
