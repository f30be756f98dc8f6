// Generic CUDA-core decode kernels (any supported shape, f32 or bf16 cache).
//
// Two passes over the keys:
//   slim_scores_kernel  softmax arguments s[b][h][t] (log2 domain) of every
//                       head for every cached row (Eq. 2, keys rotated after
//                       the read, RoPE appendix Option 1), 16-byte coalesced
//                       row reads, written to a scratch array;
//   slim_accum_kernel   CTA = (worker, d-slice): online softmax per head over
//                       its context tiles and U[h][col] += p[h][t] K[t][col]
//                       for the columns it owns (Eq. 7 Option 2: weighted sum
//                       of the full-width raw keys); writes the partial
//                       (m, l, U) of each unit for the combine.
// The keys are read twice here; the tensor-core path reads them once.
//
// slim_exact_kernel is the single-pass variant (scores recomputed per
// d-slice).  It is only used to redo, exactly, the rare units the tensor-core
// kernel flags because a softmax argument ran away from its reference.
#include <cuda_fp8.h>

#include "slim_internal.h"
#include "slim_sched.cuh"

namespace {

// 8-bit cache (SLIM_FP8): elements are OCP E4M3 codes; the stored key is code * 2^exponent with one
// exponent per (cache row, head).  ld_k returns the bare code value; k_scale the power of two.
typedef unsigned char fp8code;
__device__ __forceinline__ float fp8_value(fp8code c) {
  return __half2float(__half(__nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)c, __NV_E4M3)));
}
__device__ __forceinline__ float ld_k(const float* p) { return __ldg(p); }
__device__ __forceinline__ float ld_k(const __nv_bfloat16* p) {
  return __bfloat162float(__ldg(reinterpret_cast<const __nv_bfloat16*>(p)));
}
__device__ __forceinline__ float ld_k(const fp8code* p) { return fp8_value(__ldg(p)); }
// 2^exponent of (row, head) of an fp8 cache; 1 for the other cache types
__device__ __forceinline__ float k_scale(const SlimDecodeParams& p, long long row, int h) {
  if (!p.k_exp) return 1.f;
  return __int_as_float(((int)__ldg(p.k_exp + (size_t)row * p.H + h) + 127) << 23);
}
// query / weight element type that goes with a cache element type
template <typename KT> struct QueryOf { typedef KT type; };
template <> struct QueryOf<fp8code> { typedef __nv_bfloat16 type; };

constexpr int GEN_THREADS = 256;

template <typename KT, int HP, int COLS>
__global__ void __launch_bounds__(GEN_THREADS)
slim_exact_kernel(SlimDecodeParams p, int only_flagged) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* s_q = reinterpret_cast<float*>(smem_raw);                 // [d]
  float* s_S = s_q + p.d;                                           // [HP][TT]
  float* s_P = s_S + HP * SLIM_TT;                                  // [HP][TT]
  float* s_alpha = s_P + HP * SLIM_TT;                              // [HP]
  float* s_m = s_alpha + HP;                                        // [HP]
  float* s_l = s_m + HP;                                            // [HP]
  int* s_prefix = reinterpret_cast<int*>(s_l + HP);                 // [batch+1]

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int w = blockIdx.y;
  slim_pdl_trigger();
  slim_pdl_wait();
  if (only_flagged && *p.any_flag == 0) return;         // nothing was flagged in this decode
  const int col0 = blockIdx.x * (GEN_THREADS * COLS);
  const KT* __restrict__ Kc = reinterpret_cast<const KT*>(p.k);
  const KT* __restrict__ Q = reinterpret_cast<const KT*>(p.q);
  const int d = p.d, H = p.H, dk = p.d_k, half = p.half;

  const SlimSched sc = slim_sched_build(p.lengths, p.batch, p.t_cap, p.workers, p.min_tiles, s_prefix, p.status, p.unit_cost);
  if (sc.total_tiles == 0 || w >= sc.workers_eff) return;
  const int g_begin = slim_worker_start(sc, w), g_end = slim_worker_start(sc, w + 1);

  float acc[HP][COLS];

  int g = g_begin;
  while (g < g_end) {
    const int b = slim_seq_of_tile(s_prefix, p.batch, g);
    const int seg_end = min(g_end, s_prefix[b + 1]);
    const int tile0 = g - s_prefix[b], tile1 = seg_end - s_prefix[b];
    const int unit = w + b;
    if (only_flagged && (p.unit_flags[2 * unit] | p.unit_flags[2 * unit + 1]) == 0) { g = seg_end; continue; }
    int len = p.lengths[b];
    len = min(max(len, 0), p.t_cap);

    // ---- a2: rotate and scale the query of this sequence --------------------
    __syncthreads();
    {
      const int m = slim_query_pos(p, b, len), mt = m / SLIM_TT, mi = m % SLIM_TT;
      for (int e = tid; e < d; e += GEN_THREADS) {
        const int h = e / dk, jj = e - h * dk;
        float v;
        if (p.rope) {
          const int j = jj < half ? jj : jj - half;
          const float2 cb = p.rope_base[(size_t)mt * half + j], co = p.rope_off[mi * half + j];
          const float c = cb.x * co.x - cb.y * co.y, s = cb.y * co.x + cb.x * co.y;
          const float q1 = ld_k(Q + (size_t)b * d + h * dk + j);
          const float q2 = ld_k(Q + (size_t)b * d + h * dk + j + half);
          v = jj < half ? (q1 * c + q2 * s) : (-q1 * s + q2 * c);
        } else {
          v = ld_k(Q + (size_t)b * d + e);
        }
        s_q[e] = v * p.qscale;
      }
      if (tid < HP) { s_m[tid] = -INFINITY; s_l[tid] = 0.f; }
#pragma unroll
      for (int h = 0; h < HP; ++h)
#pragma unroll
        for (int c = 0; c < COLS; ++c) acc[h][c] = 0.f;
    }
    __syncthreads();

    for (int tile = tile0; tile < tile1; ++tile) {
      const int t0 = tile * SLIM_TT;
      const KT* __restrict__ Kt = Kc + (size_t)slim_cache_row(p, b, t0) * d;

      // ---- A: softmax arguments for all heads, rows of this tile ------------
      for (int pi = wid; pi < H * SLIM_TT; pi += GEN_THREADS / 32) {
        const int h = pi / SLIM_TT, t = pi - h * SLIM_TT;
        float a = 0.f;
        if (t0 + t < len) {
          const KT* kr = Kt + (size_t)t * d + h * dk;
          const float* qh = s_q + h * dk;
          for (int j = lane; j < half; j += 32) {
            const float k1 = ld_k(kr + j), k2 = ld_k(kr + j + half);
            const float q1 = qh[j], q2 = qh[j + half];
            if (p.rope) {
              const float2 cb = p.rope_base[(size_t)(tile + slim_tile_offset(p, b)) * half + j], co = p.rope_off[t * half + j];
              const float c = cb.x * co.x - cb.y * co.y, s = cb.y * co.x + cb.x * co.y;
              a += c * (q1 * k1 + q2 * k2) + s * (q1 * k2 - q2 * k1);
            } else {
              a += q1 * k1 + q2 * k2;
            }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        } else {
          a = -INFINITY;
        }
        if (lane == 0) s_S[h * SLIM_TT + t] = a;
      }
      __syncthreads();

      // ---- B: online softmax per head ---------------------------------------
      for (int h = wid; h < H; h += GEN_THREADS / 32) {
        const float s = lane < SLIM_TT ? s_S[h * SLIM_TT + lane] : -INFINITY;
        float mx = s;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        const float m_old = s_m[h];
        const float m_new = fmaxf(m_old, mx);
        const float pr = (s == -INFINITY) ? 0.f : exp2f(s - m_new);
        float ps = pr;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
        const float alpha = exp2f(m_old - m_new);      // 0 on the first tile
        if (lane < SLIM_TT) s_P[h * SLIM_TT + lane] = pr;
        if (lane == 0) { s_alpha[h] = alpha; s_m[h] = m_new; s_l[h] = s_l[h] * alpha + ps; }
      }
      __syncthreads();

      // ---- C: U[h][col] = alpha U[h][col] + sum_t p[h][t] K[t][col] ----------
      float kv[COLS][SLIM_TT];
#pragma unroll
      for (int c = 0; c < COLS; ++c) {
        const int col = col0 + tid + c * GEN_THREADS;
#pragma unroll
        for (int t = 0; t < SLIM_TT; ++t)
          kv[c][t] = (col < d && t0 + t < len) ? ld_k(Kt + (size_t)t * d + col) : 0.f;
      }
#pragma unroll
      for (int h = 0; h < HP; ++h) {
        if (h < H) {
          const float al = s_alpha[h];
          const float4* P4 = reinterpret_cast<const float4*>(s_P + h * SLIM_TT);
          float pv[SLIM_TT];
#pragma unroll
          for (int i = 0; i < SLIM_TT / 4; ++i) {
            const float4 v = P4[i];
            pv[4 * i] = v.x; pv[4 * i + 1] = v.y; pv[4 * i + 2] = v.z; pv[4 * i + 3] = v.w;
          }
#pragma unroll
          for (int c = 0; c < COLS; ++c) {
            float a = acc[h][c] * al;
#pragma unroll
            for (int t = 0; t < SLIM_TT; ++t) a = fmaf(pv[t], kv[c][t], a);
            acc[h][c] = a;
          }
        }
      }
      __syncthreads();
    }

    // ---- partial of this unit -------------------------------------------------
#pragma unroll
    for (int h = 0; h < HP; ++h) {
      if (h < H) {
#pragma unroll
        for (int c = 0; c < COLS; ++c) {
          const int col = col0 + tid + c * GEN_THREADS;
          if (col < d) p.part_u[((size_t)unit * H + h) * d + col] = acc[h][c];
        }
      }
    }
    if (blockIdx.x == 0 && tid < H) {
      p.part_m[(size_t)unit * H + tid] = s_m[tid];
      p.part_l[(size_t)unit * H + tid] = s_l[tid];
    }
    g = seg_end;
  }
}

// ---------------------------------------------------------------------------
// pass 1: softmax arguments
// ---------------------------------------------------------------------------
template <typename KT> struct Vec;
template <> struct Vec<float> {
  static constexpr int N = 4;
  __device__ static void load(const float* p, float (&v)[4]) {
    const float4 x = __ldg(reinterpret_cast<const float4*>(p));
    v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
  }
};
template <> struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void load(const __nv_bfloat16* p, float (&v)[8]) {
    const uint4 x = __ldg(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
};

template <> struct Vec<fp8code> {
  static constexpr int N = 8;
  __device__ static void load(const fp8code* p, float (&v)[8]) {
    const uint2 x = __ldg(reinterpret_cast<const uint2*>(p));
    const uint32_t w[2] = {x.x, x.y};
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = fp8_value((fp8code)((w[i >> 2] >> (8 * (i & 3))) & 0xffu));
  }
};

// One CTA walks tiles g = blockIdx.x, blockIdx.x + gridDim.x, ...  A warp owns
// rows of the tile; a lane owns "pair vectors": VEC consecutive elements j of
// the first half of a head together with their partners j + d_k/2.
template <typename KT>
__global__ void __launch_bounds__(GEN_THREADS)
slim_scores_kernel(SlimDecodeParams p, float* __restrict__ scores) {
  constexpr int VEC = Vec<KT>::N;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* s_q = reinterpret_cast<float*>(smem_raw);                         // [d] rotated, scaled query
  float* s_part = s_q + p.d;                                                // [TT][d / (2 VEC)]
  int* s_prefix = reinterpret_cast<int*>(s_part + SLIM_TT * (p.d / (2 * VEC)));
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int d = p.d, H = p.H, dk = p.d_k, half = p.half;
  const int npv = d / (2 * VEC), pv_per_head = half / VEC;
  typedef typename QueryOf<KT>::type QT;
  const KT* __restrict__ Kc = reinterpret_cast<const KT*>(p.k);
  const QT* __restrict__ Q = reinterpret_cast<const QT*>(p.q);

  const SlimSched sc = slim_sched_build(p.lengths, p.batch, p.t_cap, p.workers, p.min_tiles, s_prefix, p.status, p.unit_cost);
  int cur_b = -1;
  for (int g = blockIdx.x; g < sc.total_tiles; g += gridDim.x) {
    const int b = slim_seq_of_tile(s_prefix, p.batch, g);
    const int tile = g - s_prefix[b], t0 = tile * SLIM_TT;
    const int len = min(max(p.lengths[b], 0), p.t_cap);
    __syncthreads();
    if (b != cur_b) {                       // a2: rotate + scale the query of sequence b
      cur_b = b;
      const int m = slim_query_pos(p, b, len), mt = m / SLIM_TT, mi = m % SLIM_TT;
      for (int e = tid; e < d; e += GEN_THREADS) {
        const int h = e / dk, jj = e - h * dk;
        float v;
        if (p.rope) {
          const int j = jj < half ? jj : jj - half;
          const float2 cb = p.rope_base[(size_t)mt * half + j], co = p.rope_off[mi * half + j];
          const float c = cb.x * co.x - cb.y * co.y, s = cb.y * co.x + cb.x * co.y;
          const float q1 = ld_k(Q + (size_t)b * d + h * dk + j), q2 = ld_k(Q + (size_t)b * d + h * dk + j + half);
          v = jj < half ? (q1 * c + q2 * s) : (-q1 * s + q2 * c);
        } else {
          v = ld_k(Q + (size_t)b * d + e);
        }
        s_q[e] = v * p.qscale;
      }
      __syncthreads();
    }
    if (half % VEC != 0) {
      // head widths whose half is not a multiple of the vector width (e.g. d_k = 100): element loads,
      // one warp per row, the lanes share the pairs of a head
      for (int t = wid; t < SLIM_TT; t += GEN_THREADS / 32) {
        if (t0 + t >= len) continue;
        const long long row = slim_cache_row(p, b, t0) + t;
        const KT* kr = Kc + (size_t)row * d;
        for (int h = 0; h < H; ++h) {
          const float* q1 = s_q + h * dk;
          float a = 0.f;
          for (int j = lane; j < half; j += 32) {
            const float k1 = ld_k(kr + h * dk + j), k2 = ld_k(kr + h * dk + j + half);
            if (p.rope) {
              const float2 cb = __ldg(p.rope_base + (size_t)(tile + slim_tile_offset(p, b)) * half + j), co = __ldg(p.rope_off + t * half + j);
              const float c = cb.x * co.x - cb.y * co.y, s = cb.y * co.x + cb.x * co.y;
              a += c * (q1[j] * k1 + q1[j + half] * k2) + s * (q1[j] * k2 - q1[j + half] * k1);
            } else {
              a += q1[j] * k1 + q1[j + half] * k2;
            }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
          if (lane == 0) scores[((size_t)b * H + h) * p.t_cap + t0 + t] = a * k_scale(p, row, h);
        }
      }
      continue;
    }
    for (int t = wid; t < SLIM_TT; t += GEN_THREADS / 32) {
      if (t0 + t >= len) continue;
      const KT* kr = Kc + (size_t)(slim_cache_row(p, b, t0) + t) * d;
      for (int pv = lane; pv < npv; pv += 32) {
        const int h = pv / pv_per_head, j0 = (pv - h * pv_per_head) * VEC;
        float k1[VEC], k2[VEC];
        Vec<KT>::load(kr + h * dk + j0, k1);
        Vec<KT>::load(kr + h * dk + half + j0, k2);
        const float* q1 = s_q + h * dk + j0;
        const float* q2 = q1 + half;
        float a = 0.f;
        if (p.rope) {
          const float2* cbp = p.rope_base + (size_t)(tile + slim_tile_offset(p, b)) * half + j0;
          const float2* cop = p.rope_off + t * half + j0;
#pragma unroll
          for (int x = 0; x < VEC; ++x) {
            const float2 cb = __ldg(cbp + x), co = __ldg(cop + x);
            const float c = cb.x * co.x - cb.y * co.y, s = cb.y * co.x + cb.x * co.y;
            a += c * (q1[x] * k1[x] + q2[x] * k2[x]) + s * (q1[x] * k2[x] - q2[x] * k1[x]);
          }
        } else {
#pragma unroll
          for (int x = 0; x < VEC; ++x) a += q1[x] * k1[x] + q2[x] * k2[x];
        }
        s_part[t * npv + pv] = a;
      }
    }
    __syncthreads();
    for (int e = tid; e < H * SLIM_TT; e += GEN_THREADS) {
      const int h = e / SLIM_TT, t = e - h * SLIM_TT;
      if (t0 + t < len) {
        float a = 0.f;
        for (int x = 0; x < pv_per_head; ++x) a += s_part[t * npv + h * pv_per_head + x];
        scores[((size_t)b * H + h) * p.t_cap + t0 + t] = a * k_scale(p, slim_cache_row(p, b, t0) + t, h);
      }
    }
  }
}

// ---------------------------------------------------------------------------
// pass 2: online softmax + weighted sum of the raw keys
// ---------------------------------------------------------------------------
template <typename KT, int HP>
__global__ void __launch_bounds__(GEN_THREADS, 2)
slim_accum_kernel(SlimDecodeParams p, const float* __restrict__ scores, int only_if_flagged) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* s_P = reinterpret_cast<float*>(smem_raw);                  // [HP][TT]
  float* s_alpha = s_P + HP * SLIM_TT;                              // [HP]
  float* s_m = s_alpha + HP;                                        // [HP]
  float* s_l = s_m + HP;                                            // [HP]
  int* s_prefix = reinterpret_cast<int*>(s_l + HP);                 // [batch+1]
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int w = blockIdx.y;
  if (only_if_flagged) {
    slim_pdl_wait();
    if (*p.any_flag == 0) return;                     // nothing overflowed its reference exponent
  }
  const int col = blockIdx.x * GEN_THREADS + tid;
  const KT* __restrict__ Kc = reinterpret_cast<const KT*>(p.k);
  const int d = p.d, H = p.H;

  const SlimSched sc = slim_sched_build(p.lengths, p.batch, p.t_cap, p.workers, p.min_tiles, s_prefix, p.status, p.unit_cost);
  if (sc.total_tiles == 0 || w >= sc.workers_eff) return;
  const int g_begin = slim_worker_start(sc, w), g_end = slim_worker_start(sc, w + 1);
  float acc[HP];
  int g = g_begin;
  while (g < g_end) {
    const int b = slim_seq_of_tile(s_prefix, p.batch, g);
    const int seg_end = min(g_end, s_prefix[b + 1]);
    const int tile0 = g - s_prefix[b], tile1 = seg_end - s_prefix[b];
    const int unit = w + b;
    const int len = min(max(p.lengths[b], 0), p.t_cap);
    __syncthreads();
    if (tid < HP) { s_m[tid] = -INFINITY; s_l[tid] = 0.f; }
#pragma unroll
    for (int h = 0; h < HP; ++h) acc[h] = 0.f;
    __syncthreads();
    for (int tile = tile0; tile < tile1; ++tile) {
      const int t0 = tile * SLIM_TT;
      const KT* __restrict__ Kt = Kc + (size_t)slim_cache_row(p, b, t0) * d;
      float kv[SLIM_TT];
      const long long row0 = slim_cache_row(p, b, t0);
#pragma unroll
      for (int t = 0; t < SLIM_TT; ++t)
        kv[t] = (col < d && t0 + t < len) ? ld_k(Kt + (size_t)t * d + col) * k_scale(p, row0 + t, col / p.d_k) : 0.f;
      // ---- a5: online softmax, one warp per head ----
      for (int h = wid; h < H; h += GEN_THREADS / 32) {
        const float s = (lane < SLIM_TT && t0 + lane < len)
                            ? __ldg(scores + ((size_t)b * H + h) * p.t_cap + t0 + lane) : -INFINITY;
        float mx = s;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        const float m_old = s_m[h], m_new = fmaxf(m_old, mx);
        const float pr = (s == -INFINITY) ? 0.f : exp2f(s - m_new);
        float ps = pr;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
        const float alpha = exp2f(m_old - m_new);
        if (lane < SLIM_TT) s_P[h * SLIM_TT + lane] = pr;
        if (lane == 0) { s_alpha[h] = alpha; s_m[h] = m_new; s_l[h] = s_l[h] * alpha + ps; }
      }
      __syncthreads();
      // ---- a6: U[h][col] = alpha U[h][col] + sum_t p[h][t] K[t][col] ----
#pragma unroll
      for (int h = 0; h < HP; ++h) {
        if (h < H) {
          const float4* P4 = reinterpret_cast<const float4*>(s_P + h * SLIM_TT);
          float a = acc[h] * s_alpha[h];
#pragma unroll
          for (int i = 0; i < SLIM_TT / 4; ++i) {
            const float4 v = P4[i];
            a = fmaf(v.x, kv[4 * i], a); a = fmaf(v.y, kv[4 * i + 1], a);
            a = fmaf(v.z, kv[4 * i + 2], a); a = fmaf(v.w, kv[4 * i + 3], a);
          }
          acc[h] = a;
        }
      }
      __syncthreads();
    }
    if (col < d) {
#pragma unroll
      for (int h = 0; h < HP; ++h)
        if (h < H) p.part_u[((size_t)unit * H + h) * d + col] = acc[h];
    }
    if (blockIdx.x == 0 && tid < H) {
      p.part_m[(size_t)unit * H + tid] = s_m[tid];
      p.part_l[(size_t)unit * H + tid] = s_l[tid];
    }
    g = seg_end;
  }
}


// ---------------------------------------------------------------------------
// X-cache / E-cache scheme (non-square Option 2, encoder-decoder Option 2): the cache
// holds the layer inputs X and the softmax arguments come from a dense d-wide query per
// head, A_i = ((x_n W_Q,i + b) W_K,i^T) X^T.
// ---------------------------------------------------------------------------
// q~[b][h][j] = qscale * sum_c q[b][h d_k + c] W_K[j][h d_k + c]      (one warp per j)
template <typename KT>
__global__ void __launch_bounds__(GEN_THREADS)
slim_xq_kernel(SlimDecodeParams p, const float* __restrict__ W_K, float* __restrict__ qt) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* s_q = reinterpret_cast<float*>(smem_raw);                   // [d_k]
  const int h = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int d = p.d, dk = p.d_k;
  const KT* Q = reinterpret_cast<const KT*>(p.q) + (size_t)b * p.e + h * dk;
  for (int c = tid; c < dk; c += GEN_THREADS) s_q[c] = ld_k(Q + c) * p.qscale;
  __syncthreads();
  for (int j = wid; j < d; j += GEN_THREADS / 32) {
    const float* w = W_K + (size_t)j * p.e + h * dk;
    float a = 0.f;
    for (int c = lane; c < dk; c += 32) a = fmaf(s_q[c], __ldg(w + c), a);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
    if (lane == 0) qt[((size_t)b * p.H + h) * d + j] = a;
  }
}

// scores[b][h][t] = q~[b][h][:] . X[b][t][:]   CTA = (32-row tile, sequence); thread = (row, head group)
constexpr int XS_ROWS = 32, XS_DC = 128;
template <typename KT>
__global__ void __launch_bounds__(GEN_THREADS)
slim_xscores_kernel(SlimDecodeParams p, const float* __restrict__ qt, float* __restrict__ scores) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* s_x = reinterpret_cast<float*>(smem_raw);                   // [32][XS_DC + 1]
  float* s_qt = s_x + XS_ROWS * (XS_DC + 1) + 3;                     // [H][XS_DC], 16-byte aligned below
  s_qt = reinterpret_cast<float*>((reinterpret_cast<uintptr_t>(s_qt) + 15) & ~(uintptr_t)15);
  const int b = blockIdx.y, t0 = blockIdx.x * XS_ROWS, tid = threadIdx.x, tx = tid & 31, ty = tid >> 5;
  const int d = p.d, H = p.H;
  const int len = min(max(p.lengths[b], 0), p.t_cap);
  if (t0 >= len) return;
  const KT* __restrict__ X = reinterpret_cast<const KT*>(p.k) + ((size_t)b * p.t_cap + t0) * d;
  const float* __restrict__ Qb = qt + (size_t)b * H * d;
  float acc[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = 0.f;
  for (int j0 = 0; j0 < d; j0 += XS_DC) {
    const int dc = min(XS_DC, d - j0);
    for (int e = tid; e < XS_ROWS * XS_DC; e += GEN_THREADS) {
      const int r = e / XS_DC, k = e % XS_DC;
      s_x[r * (XS_DC + 1) + k] = (k < dc && t0 + r < len) ? ld_k(X + (size_t)r * d + j0 + k) : 0.f;   // rows past the end may hold anything
    }
    for (int e = tid; e < H * XS_DC; e += GEN_THREADS) {
      const int hh = e / XS_DC, k = e % XS_DC;
      s_qt[e] = k < dc ? __ldg(Qb + (size_t)hh * d + j0 + k) : 0.f;
    }
    __syncthreads();
    const float* xr = s_x + tx * (XS_DC + 1);
    for (int k = 0; k < XS_DC; k += 4) {
      const float x0 = xr[k], x1 = xr[k + 1], x2 = xr[k + 2], x3 = xr[k + 3];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int hh = ty + 8 * i;
        if (hh < H) {
          const float4 q4 = *reinterpret_cast<const float4*>(s_qt + hh * XS_DC + k);
          acc[i] = fmaf(x0, q4.x, acc[i]); acc[i] = fmaf(x1, q4.y, acc[i]);
          acc[i] = fmaf(x2, q4.z, acc[i]); acc[i] = fmaf(x3, q4.w, acc[i]);
        }
      }
    }
    __syncthreads();
  }
  if (t0 + tx < len) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int hh = ty + 8 * i;
      if (hh < H) scores[((size_t)b * H + hh) * p.t_cap + t0 + tx] = acc[i];
    }
  }
}

template <typename KT, int HP, int COLS>
cudaError_t launch_exact(const SlimDecodeParams& p, int only_flagged, cudaStream_t st) {
  const int dsplit = (p.d + GEN_THREADS * COLS - 1) / (GEN_THREADS * COLS);
  const size_t smem = sizeof(float) * (p.d + 2 * HP * SLIM_TT + 3 * HP) + sizeof(int) * (p.batch + 1);
  auto kern = slim_exact_kernel<KT, HP, COLS>;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  dim3 grid(dsplit, p.workers);
  return slim_launch_pdl(kern, grid, dim3(GEN_THREADS), smem, st, p, only_flagged);
}

template <typename KT>
cudaError_t launch_scores(const slim_ctx* ctx, const SlimDecodeParams& p, float* scores, cudaStream_t st) {
  constexpr int VEC = Vec<KT>::N;
  const size_t smem = sizeof(float) * (p.d + SLIM_TT * (p.d / (2 * VEC))) + sizeof(int) * (p.batch + 1);
  auto kern = slim_scores_kernel<KT>;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  kern<<<4 * ctx->num_sms, GEN_THREADS, smem, st>>>(p, scores);
  return cudaGetLastError();
}

template <typename KT>
cudaError_t launch_xscores(const SlimDecodeParams& p, float* scores, const float* xc_wk, float* xc_qt, cudaStream_t st) {
  slim_xq_kernel<KT><<<dim3(p.H, p.batch), GEN_THREADS, sizeof(float) * p.d_k, st>>>(p, xc_wk, xc_qt);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const size_t smem = sizeof(float) * (XS_ROWS * (XS_DC + 1) + 8 + (size_t)p.H * XS_DC);
  auto kern = slim_xscores_kernel<KT>;
  e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kern<<<dim3((p.t_cap + XS_ROWS - 1) / XS_ROWS, p.batch), GEN_THREADS, smem, st>>>(p, xc_qt, scores);
  return cudaGetLastError();
}

template <typename KT>
cudaError_t launch_accum(const SlimDecodeParams& p, const float* scores, int only_if_flagged, cudaStream_t st) {
  const int dsplit = (p.d + GEN_THREADS - 1) / GEN_THREADS;
  dim3 grid(dsplit, p.workers);
  if (p.H <= 8) {
    const size_t smem = sizeof(float) * (8 * SLIM_TT + 3 * 8) + sizeof(int) * (p.batch + 1);
    slim_accum_kernel<KT, 8><<<grid, GEN_THREADS, smem, st>>>(p, scores, only_if_flagged);
  } else if (p.H <= 32) {
    const size_t smem = sizeof(float) * (32 * SLIM_TT + 3 * 32) + sizeof(int) * (p.batch + 1);
    slim_accum_kernel<KT, 32><<<grid, GEN_THREADS, smem, st>>>(p, scores, only_if_flagged);
  } else {
    const size_t smem = sizeof(float) * (64 * SLIM_TT + 3 * 64) + sizeof(int) * (p.batch + 1);
    slim_accum_kernel<KT, 64><<<grid, GEN_THREADS, smem, st>>>(p, scores, only_if_flagged);
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t slim_launch_xcache_scores(const slim_ctx* ctx, const SlimDecodeParams& p, float* scores, const float* W_K,
                                      float* qt, cudaStream_t st) {
  return p.dtype == SLIM_BF16 ? launch_xscores<__nv_bfloat16>(p, scores, W_K, qt, st)
                              : launch_xscores<float>(p, scores, W_K, qt, st);
}

cudaError_t slim_launch_accum(const slim_ctx* ctx, const SlimDecodeParams& p, const float* scores, int whole, cudaStream_t st) {
  if (p.kdtype == SLIM_FP8) return launch_accum<fp8code>(p, scores, whole ? 0 : 1, st);
  return p.dtype == SLIM_BF16 ? launch_accum<__nv_bfloat16>(p, scores, whole ? 0 : 1, st)
                              : launch_accum<float>(p, scores, whole ? 0 : 1, st);
}

int slim_generic_dsplit(const slim_ctx* ctx) { return (ctx->d + GEN_THREADS - 1) / GEN_THREADS; }

int slim_generic_workers(const slim_ctx* ctx) {
  // about three CTAs per SM in flight, shared between the d-slices of a worker
  int w = (3 * ctx->num_sms) / slim_generic_dsplit(ctx);
  if (w < 1) w = 1;
  if (w > ctx->num_sms) w = ctx->num_sms;
  return w;
}

cudaError_t slim_launch_generic(const slim_ctx* ctx, const SlimDecodeParams& p, float* scores, cudaStream_t st) {
  cudaError_t e = p.kdtype == SLIM_FP8 ? launch_scores<fp8code>(ctx, p, scores, st)
                  : p.dtype == SLIM_BF16 ? launch_scores<__nv_bfloat16>(ctx, p, scores, st) : launch_scores<float>(ctx, p, scores, st);
  if (e != cudaSuccess) return e;
  return slim_launch_accum(ctx, p, scores, 1, st);
}

// Redo exactly the units whose flag is set (schedule taken from p.workers / p.min_tiles).
cudaError_t slim_launch_exact_flagged(const slim_ctx* ctx, const SlimDecodeParams& p, cudaStream_t st) {
  const bool bf = p.dtype == SLIM_BF16;
  if (p.H <= 8) return bf ? launch_exact<__nv_bfloat16, 8, 2>(p, 1, st) : launch_exact<float, 8, 2>(p, 1, st);
  if (p.H <= 32) return bf ? launch_exact<__nv_bfloat16, 32, 2>(p, 1, st) : launch_exact<float, 32, 2>(p, 1, st);
  return bf ? launch_exact<__nv_bfloat16, 64, 1>(p, 1, st) : launch_exact<float, 64, 1>(p, 1, st);
}
