// Pieces of the log-sum-exp combine kernels (slim_proj.cu): the weights of a sequence's units, the
// store of eight combined values as a bf16 (hi, lo) pair in the operand layout of the projection
// MMA, and the exact recomputation of one head of a sequence whose tensor-core partials cannot be
// used (a softmax argument ran far above a unit's reference exponent).
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

#include "slim_internal.h"
#include "slim_sched.cuh"

namespace slim_comb {

constexpr int PJ_BG = 16;                      // sequences per projection MMA (N = 32 per head: hi and lo)

// K-major 8x8 core matrices of the projection's B operand, N = 32 columns (16 sequences x {hi, lo})
__device__ __forceinline__ uint32_t u_offset(int n, int k) {
  return (uint32_t)((n & 7) * 16 + (n >> 3) * 256 + (k >> 3) * 128 + (k & 7) * 2);
}

// One warp forms the weights of the wn units (unit0, unit0 + 1, ...) of a sequence for head h:
//   w_i = 2^(m_i - M) / sum_j 2^(m_j - M) l_j,   M = max_j (m_j + log2 l_j),
// so that u = sum_i w_i U_i.  The partials may have been written by other SMs of the same grid:
// they are read from L2.
// Returns M + log2(sum_j 2^(m_j - M) l_j): the log2 of the sum of 2^argument over the sequence's rows.
__device__ __forceinline__ float weights_warp(const float* part_m, const float* part_l, int unit0, int wn, int H, int h,
                                              float* s_w, int lane) {
  float M = -INFINITY;
  for (int i = lane; i < wn; i += 32) {
    const size_t ui = (size_t)(unit0 + i) * H + h;
    M = fmaxf(M, __ldcg(part_m + ui) + log2f(__ldcg(part_l + ui)));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  float L = 0.f;
  for (int i = lane; i < wn; i += 32) {
    const size_t ui = (size_t)(unit0 + i) * H + h;
    const float wg = exp2f(__ldcg(part_m + ui) - M);
    s_w[i] = wg;
    L += wg * __ldcg(part_l + ui);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
  const float inv = 1.f / L;
  __syncwarp();
  for (int i = lane; i < wn; i += 32) s_w[i] *= inv;
  return M + log2f(L);
}

// u[b][h][j0 .. j0+8) as hi = bf16(u), lo = bf16(u - hi) into the operand tiles
__device__ __forceinline__ void store_u8(unsigned char* u_tiled, int d, int H, int hp, int b, int h, int j0, const float (&acc)[8]) {
  uint32_t hi[4], lo[4];
#pragma unroll
  for (int x = 0; x < 4; ++x) {
    const __nv_bfloat16 h0 = __float2bfloat16_rn(acc[2 * x]), h1 = __float2bfloat16_rn(acc[2 * x + 1]);
    const __nv_bfloat16 l0 = __float2bfloat16_rn(acc[2 * x] - __bfloat162float(h0));
    const __nv_bfloat16 l1 = __float2bfloat16_rn(acc[2 * x + 1] - __bfloat162float(h1));
    hi[x] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
    lo[x] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
  }
  const int bg = b / PJ_BG, n = b % PJ_BG;
  const size_t tile_bytes = (size_t)1024 * hp;
  unsigned char* t = u_tiled + ((size_t)(bg * (H / hp) + h / hp) * (d / 16) + j0 / 16) * tile_bytes + (size_t)(h % hp) * 1024;
  *reinterpret_cast<uint4*>(t + u_offset(n, j0 & 15)) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
  *reinterpret_cast<uint4*>(t + u_offset(PJ_BG + n, j0 & 15)) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
}

// acc[0..8) += wg * (eight floats at U)
__device__ __forceinline__ void fma8(float (&acc)[8], float wg, const float4& a, const float4& c) {
  acc[0] = fmaf(wg, a.x, acc[0]); acc[1] = fmaf(wg, a.y, acc[1]); acc[2] = fmaf(wg, a.z, acc[2]); acc[3] = fmaf(wg, a.w, acc[3]);
  acc[4] = fmaf(wg, c.x, acc[4]); acc[5] = fmaf(wg, c.y, acc[5]); acc[6] = fmaf(wg, c.z, acc[6]); acc[7] = fmaf(wg, c.w, acc[7]);
}

// Exact u[b][h][8 jg .. 8 jg + 8) for the column groups jg = jg0 .. jg0 + ngroups - 1 (ngroups <= blockDim.x):
// one plain pass over all rows of sequence b, fp32 online softmax with the true running maximum
// (Eq. 2; Eq. 7 Option 2: weighted sum of the full-width raw keys; RoPE appendix Option 1: keys
// rotated after the read, written as the query rotated against the key).  Slow by design: it only
// runs for a sequence one of whose units was flagged.  Called by all threads of the CTA (bf16 cache).
// s_x: d_k + 2 SLIM_TT + 4 floats of shared memory.
static __device__ __noinline__ void exact_groups(const SlimDecodeParams& p, unsigned char* u_tiled, int hp, int b, int h, int jg0,
                                          int ngroups, float* s_x) {
  const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
  const int d = p.d, dk = p.d_k, half = p.half;
  const int len = min(max(p.lengths[b], 0), p.t_cap);
  float* s_q = s_x;                 // [d_k] query of the head at its own position, scaled
  float* s_S = s_q + dk;            // [16]  arguments of a tile
  float* s_P = s_S + SLIM_TT;       // [16]  probabilities of a tile
  float* s_sc = s_P + SLIM_TT;      // alpha, m, l
  const __nv_bfloat16* __restrict__ Kc = reinterpret_cast<const __nv_bfloat16*>(p.k);
  const __nv_bfloat16* __restrict__ Q = reinterpret_cast<const __nv_bfloat16*>(p.q) + (size_t)b * d;
  __syncthreads();
  {
    const int m = slim_query_pos(p, b, len), mt = m / SLIM_TT, mi = m % SLIM_TT;
    for (int jj = tid; jj < dk; jj += nthr) {
      float v;
      if (p.rope) {
        const int j = jj < half ? jj : jj - half;
        const float2 cb = p.rope_base[(size_t)mt * half + j], co = p.rope_off[mi * half + j];
        const float c = cb.x * co.x - cb.y * co.y, sn = cb.y * co.x + cb.x * co.y;
        const float q1 = __bfloat162float(Q[h * dk + j]), q2 = __bfloat162float(Q[h * dk + j + half]);
        v = jj < half ? (q1 * c + q2 * sn) : (-q1 * sn + q2 * c);
      } else {
        v = __bfloat162float(Q[h * dk + jj]);
      }
      s_q[jj] = v * p.qscale;
    }
    if (tid == 0) { s_sc[1] = -INFINITY; s_sc[2] = 0.f; }
  }
  const bool mine = tid < ngroups;
  const int j0 = (jg0 + tid) * 8;
  float acc[8];
#pragma unroll
  for (int x = 0; x < 8; ++x) acc[x] = 0.f;
  __syncthreads();
  for (int t0 = 0; t0 < len; t0 += SLIM_TT) {
    const __nv_bfloat16* __restrict__ Kt = Kc + (size_t)slim_cache_row(p, b, t0) * d;
    for (int t = warp; t < SLIM_TT; t += nwarp) {
      float a = -INFINITY;
      if (t0 + t < len) {
        a = 0.f;
        const __nv_bfloat16* kr = Kt + (size_t)t * d + h * dk;
        for (int j = lane; j < half; j += 32) {
          const float k1 = __bfloat162float(kr[j]), k2 = __bfloat162float(kr[j + half]);
          const float q1 = s_q[j], q2 = s_q[j + half];
          if (p.rope) {
            const float2 cb = p.rope_base[(size_t)(t0 / SLIM_TT + slim_tile_offset(p, b)) * half + j], co = p.rope_off[t * half + j];
            const float c = cb.x * co.x - cb.y * co.y, sn = cb.y * co.x + cb.x * co.y;
            a += c * (q1 * k1 + q2 * k2) + sn * (q1 * k2 - q2 * k1);
          } else {
            a += q1 * k1 + q2 * k2;
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
      }
      if (lane == 0) s_S[t] = a;
    }
    __syncthreads();
    if (warp == 0) {
      const float sv = lane < SLIM_TT ? s_S[lane] : -INFINITY;
      float mx = sv;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float m_old = s_sc[1], m_new = fmaxf(m_old, mx);
      const float pr = (sv == -INFINITY) ? 0.f : exp2f(sv - m_new);
      float ps = pr;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
      const float alpha = exp2f(m_old - m_new);          // 0 on the first tile
      __syncwarp();
      if (lane < SLIM_TT) s_P[lane] = pr;
      if (lane == 0) { s_sc[0] = alpha; s_sc[1] = m_new; s_sc[2] = s_sc[2] * alpha + ps; }
    }
    __syncthreads();
    if (mine) {
      const float alpha = s_sc[0];
#pragma unroll
      for (int x = 0; x < 8; ++x) acc[x] *= alpha;
      for (int t = 0; t < SLIM_TT && t0 + t < len; ++t) {
        const uint4 kw = __ldg(reinterpret_cast<const uint4*>(Kt + (size_t)t * d + j0));
        const uint32_t w4[4] = {kw.x, kw.y, kw.z, kw.w};
        const float pr = s_P[t];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          acc[2 * x] = fmaf(pr, __uint_as_float(w4[x] << 16), acc[2 * x]);
          acc[2 * x + 1] = fmaf(pr, __uint_as_float(w4[x] & 0xffff0000u), acc[2 * x + 1]);
        }
      }
    }
  }
  if (mine) {
    const float inv = 1.f / s_sc[2];
#pragma unroll
    for (int x = 0; x < 8; ++x) acc[x] *= inv;
    store_u8(u_tiled, d, p.H, hp, b, h, j0, acc);
  }
  __syncthreads();
}

}  // namespace slim_comb
