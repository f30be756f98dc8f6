// One context split over several GPUs (ranks): every rank caches a slice of the rows of each sequence
// and runs the decode kernels on it; what crosses the link per (sequence, head) is the log2 of the
// slice's softmax denominator and the slice's normalised weighted sum of keys,
//     lse_r = log2 sum_{t in slice r} 2^(s_t),      u_r = sum_t 2^(s_t) K[t] / 2^(lse_r),
// H (d + 1) floats per sequence.  The exact result over the whole context is the same log-sum-exp
// combine that joins the context splits inside one GPU (flash-decoding remark of the paper's
// complexity section):   u = sum_r w_r u_r,   w_r = 2^(lse_r - max) / sum_r' 2^(lse_r' - max),
// followed by the per-head projection of Eq. 7 (Option 2).
//
//   slim_partial_out_kernel   joins this GPU's own unit partials of (sequence, head) into (lse_r, u_r)
//   slim_rank_combine_kernel  joins the gathered (lse_r, u_r) of all ranks and leaves the result as a
//                             single-unit partial, so that the ordinary combine + projection tail
//                             finishes the step
#include "slim_internal.h"
#include "slim_sched.cuh"
#include "slim_combine.cuh"

namespace {

__global__ void __launch_bounds__(256)
slim_partial_out_kernel(const SlimDecodeParams p, float* __restrict__ lse_out, float* __restrict__ u_out) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* s_w = reinterpret_cast<float*>(smem_raw);                 // [workers]
  int* s_info = reinterpret_cast<int*>(s_w + p.workers);           // wlo, wn
  int* s_prefix = s_info + 2;                                      // [batch+1]
  const int tid = threadIdx.x, lane = tid & 31;
  const int h = blockIdx.x, b = blockIdx.y;
  const int d = p.d, H = p.H;
  slim_pdl_trigger();
  slim_pdl_wait();
  if (blockIdx.x == 0 && blockIdx.y == 0 && tid == 0) *p.any_flag = 0;   // the redo kernel has consumed it
  const SlimSched sc = slim_sched_build(p.lengths, p.batch, p.t_cap, p.workers, p.min_tiles, s_prefix, p.status, p.unit_cost);
  if (tid < 32) {
    int wlo = 0, wn = 0;
    float lse = -INFINITY;                                         // an empty slice weighs nothing
    if (s_prefix[b + 1] > s_prefix[b]) {
      wlo = slim_worker_of_tile(sc, s_prefix[b]);
      wn = slim_worker_of_tile(sc, s_prefix[b + 1] - 1) - wlo + 1;
      lse = slim_comb::weights_warp(p.part_m, p.part_l, wlo + b, wn, H, h, s_w, lane);
    }
    if (lane == 0) { s_info[0] = wlo; s_info[1] = wn; lse_out[(size_t)b * H + h] = lse; }
  }
  __syncthreads();
  const int wlo = s_info[0], wn = s_info[1];
  const size_t ustride = (size_t)H * d;
  for (int j = tid; j < d; j += blockDim.x) {
    const float* U = p.part_u + ((size_t)(wlo + b) * H + h) * d + j;
    float a = 0.f;
    for (int i = 0; i < wn; ++i) a = fmaf(s_w[i], U[(size_t)i * ustride], a);
    u_out[((size_t)b * H + h) * d + j] = a;
  }
}

// part_u[b][h][:] = sum_r w_r u_all[r][b][h][:], part_m = 0, part_l = 1: one finished unit per sequence
__global__ void __launch_bounds__(256)
slim_rank_combine_kernel(const SlimDecodeParams p, const float* __restrict__ lse_all, const float* __restrict__ u_all, int ranks) {
  __shared__ float s_w[64];
  const int tid = threadIdx.x;
  const int h = blockIdx.x, b = blockIdx.y;
  const int d = p.d, H = p.H;
  slim_pdl_trigger();
  slim_pdl_wait();
  if (tid == 0) {
    float M = -INFINITY;
    for (int r = 0; r < ranks; ++r) M = fmaxf(M, lse_all[((size_t)r * p.batch + b) * H + h]);
    float L = 0.f;
    for (int r = 0; r < ranks; ++r) {
      const float lse = lse_all[((size_t)r * p.batch + b) * H + h];
      const float wg = lse == -INFINITY ? 0.f : exp2f(lse - M);
      s_w[r] = wg;
      L += wg;
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
    for (int r = 0; r < ranks; ++r) s_w[r] *= inv;
    p.part_m[(size_t)b * H + h] = 0.f;
    p.part_l[(size_t)b * H + h] = 1.f;
  }
  __syncthreads();
  const size_t rstride = (size_t)p.batch * H * d;
  for (int j = tid; j < d; j += blockDim.x) {
    const float* U = u_all + ((size_t)b * H + h) * d + j;
    float a = 0.f;
    for (int r = 0; r < ranks; ++r)
      if (s_w[r] != 0.f) a = fmaf(s_w[r], U[(size_t)r * rstride], a);      // a rank without rows may hold anything
    p.part_u[((size_t)b * H + h) * d + j] = a;
  }
}

}  // namespace

cudaError_t slim_launch_partial_out(const slim_ctx* ctx, const SlimDecodeParams& p, float* lse_out, float* u_out, cudaStream_t st) {
  const size_t smem = sizeof(float) * p.workers + sizeof(int) * (2 + p.batch + 1) + 16;
  return slim_launch_pdl(slim_partial_out_kernel, dim3(p.H, p.batch), dim3(256), smem, st, p, lse_out, u_out);
}

cudaError_t slim_launch_rank_combine(const slim_ctx* ctx, const SlimDecodeParams& p, const float* lse_all, const float* u_all,
                                     int ranks, cudaStream_t st) {
  return slim_launch_pdl(slim_rank_combine_kernel, dim3(p.H, p.batch), dim3(256), 0, st, p, lse_all, u_all, ranks);
}
