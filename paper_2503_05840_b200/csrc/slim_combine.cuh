// Pieces of the log-sum-exp combine kernels (slim_proj.cu): the weights of a sequence's units, the
// store of combined values as a scaled float16 (hi, lo) pair in the operand layout of the projection
// MMA, and the exact recomputation of one head of a sequence whose tensor-core partials cannot be
// used (a softmax argument ran far above a unit's reference exponent).
//
// Operand format.  The projection multiplies float16 operands (11-bit mantissas; bf16 weights alone
// cost about 1e-2 of the output RMS).  float16 has a narrow exponent range, so every row u[b][h][:]
// is divided by 2^e, e = exponent of the row's largest magnitude (row values end up in (-1, 1)), and
// stored as hi = f16(v), lo = f16(v - hi); 2^e goes to su[b][h] and is multiplied back in the
// projection's epilogue.  Entries far below the row maximum lose relative precision, but their
// absolute error stays below 2^-24 of the row maximum.
#include <cuda_fp16.h>
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

// u[b][h][j0 .. j0+8) * inv as hi = f16(v), lo = f16(v - hi) into the operand tiles
__device__ __forceinline__ void store_u8_h(unsigned char* u_tiled, int d, int H, int hp, int b, int h, int j0, const float (&acc)[8],
                                           float inv) {
  uint32_t hi[4], lo[4];
#pragma unroll
  for (int x = 0; x < 4; ++x) {
    const float v0 = acc[2 * x] * inv, v1 = acc[2 * x + 1] * inv;
    const __half h0 = __float2half_rn(v0), h1 = __float2half_rn(v1);
    const __half l0 = __float2half_rn(v0 - __half2float(h0)), l1 = __float2half_rn(v1 - __half2float(h1));
    hi[x] = (uint32_t)__half_as_ushort(h0) | ((uint32_t)__half_as_ushort(h1) << 16);
    lo[x] = (uint32_t)__half_as_ushort(l0) | ((uint32_t)__half_as_ushort(l1) << 16);
  }
  const int bg = b / PJ_BG, n = b % PJ_BG;
  const size_t tile_bytes = (size_t)1024 * hp;
  unsigned char* t = u_tiled + ((size_t)(bg * (H / hp) + h / hp) * (d / 16) + j0 / 16) * tile_bytes + (size_t)(h % hp) * 1024;
  *reinterpret_cast<uint4*>(t + u_offset(n, j0 & 15)) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
  *reinterpret_cast<uint4*>(t + u_offset(PJ_BG + n, j0 & 15)) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
}
// the same eight values as plain floats into the row scratch u32[b][h][:]
__device__ __forceinline__ void store_u8_f32(float* u32, int d, int H, int b, int h, int j0, const float (&acc)[8]) {
  float4* t = reinterpret_cast<float4*>(u32 + ((size_t)b * H + h) * d + j0);
  t[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
  t[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
}
// largest |v| over the CTA (all threads call it; s_red: 33 floats of shared memory)
__device__ __forceinline__ float block_absmax(float v, float* s_red) {
  v = fabsf(v);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  __syncthreads();
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
  __syncthreads();
  if (threadIdx.x < 32) {
    float w = threadIdx.x < (blockDim.x >> 5) ? s_red[threadIdx.x] : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) w = fmaxf(w, __shfl_xor_sync(0xffffffffu, w, o));
    if (threadIdx.x == 0) s_red[32] = w;
  }
  __syncthreads();
  return s_red[32];
}
// 2^-e and 2^e for a row whose largest magnitude is mx: mx 2^-e in [0.5, 1); (1, 1) for a zero or non-finite row
__device__ __forceinline__ void row_scale(float mx, float& inv, float& scale) {
  inv = 1.f; scale = 1.f;
  if (mx > 0.f && mx <= 3.0e38f) {
    int x;
    frexpf(mx, &x);
    x = max(-120, min(120, x));
    inv = exp2f((float)-x); scale = exp2f((float)x);
  }
}
// The CTA turns the finished float row u32[b][h][:] into operand tiles and records its scale.
__device__ __forceinline__ void convert_row(const float* u32, unsigned char* u_tiled, float* su, int d, int H, int hp, int b, int h,
                                            float* s_red) {
  const float* row = u32 + ((size_t)b * H + h) * d;
  float mx = 0.f;
  for (int j = threadIdx.x * 4; j < d; j += blockDim.x * 4) {
    const float4 v = *reinterpret_cast<const float4*>(row + j);
    mx = fmaxf(fmaxf(mx, fmaxf(fabsf(v.x), fabsf(v.y))), fmaxf(fabsf(v.z), fabsf(v.w)));
  }
  mx = block_absmax(mx, s_red);
  float inv, scale;
  row_scale(mx, inv, scale);
  for (int j0 = threadIdx.x * 8; j0 < d; j0 += blockDim.x * 8) {
    const float4 a = *reinterpret_cast<const float4*>(row + j0), c = *reinterpret_cast<const float4*>(row + j0 + 4);
    const float acc[8] = {a.x, a.y, a.z, a.w, c.x, c.y, c.z, c.w};
    store_u8_h(u_tiled, d, H, hp, b, h, j0, acc, inv);
  }
  if (threadIdx.x == 0) su[(size_t)b * H + h] = scale;
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
// The result goes to the float row scratch u32[b][h][:].
static __device__ __noinline__ void exact_groups(const SlimDecodeParams& p, float* u32, int b, int h, int jg0,
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
    store_u8_f32(u32, d, p.H, b, h, j0, acc);
  }
  __syncthreads();
}

}  // namespace slim_comb
