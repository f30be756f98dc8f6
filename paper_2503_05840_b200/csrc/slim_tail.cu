// Tail of the decode step: log-sum-exp combine of the context-split partials
// fused with the per-head projection o_h = u_h W_KV,h (Eq. 7 Option 2), and the
// K-cache append.
//
//   tail1: CTA (head h, j-slice js).  For a tile of sequences it rebuilds
//          u[b][h][j] = sum_s w_s U_s[h][j] / sum_s w_s l_s over the units of b
//          (w_s = 2^(m_s - M)), keeps it in shared memory, and multiplies by
//          W_KV[h][j][0..d_k): a partial sum over its j-slice, written to
//          o_part[js][b][h*d_k + c].
//   tail2: o[b][:] = sum_js o_part[js][b][:]   (fixed order => deterministic)
#include <cuda_fp8.h>

#include "slim_internal.h"
#include "slim_sched.cuh"

namespace {

constexpr int JR = 256;        // rows of W_KV,h (= columns of u) per tail1 CTA
constexpr int BT_MAX = 32;     // sequences per pass
constexpr int BPT = 8;         // sequences per thread

__device__ __forceinline__ float ld_w(const float* p) { return __ldg(p); }
__device__ __forceinline__ float ld_w(const __nv_bfloat16* p) { return __bfloat162float(__ldg(p)); }

template <typename WT>
__global__ void __launch_bounds__(256) slim_tail1_kernel(SlimDecodeParams p, int bg_count, float* o_part) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* s_u = reinterpret_cast<float*>(smem_raw);              // [BT][JR]
  float* s_wgt = s_u + BT_MAX * JR;                             // [BT][workers]
  int* s_wlo = reinterpret_cast<int*>(s_wgt + BT_MAX * p.workers);   // [BT]
  int* s_wn = s_wlo + BT_MAX;                                   // [BT]
  int* s_prefix = s_wn + BT_MAX;                                // [batch+1]

  slim_pdl_trigger();
  slim_pdl_wait();
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nwarp = blockDim.x >> 5;
  const int h = blockIdx.x, js = blockIdx.y;
  if (h == 0 && js == 0 && tid == 0) *p.any_flag = 0;       // the redo kernel before this one has consumed it
  const int d = p.d, H = p.H, dk = p.d_k;
  const int j0 = js * JR, jn = min(JR, d - j0);
  const int BT = bg_count * BPT;
  const WT* __restrict__ W = reinterpret_cast<const WT*>(p.wkv) + ((size_t)h * d + j0) * dk;

  const SlimSched sc = slim_sched_build(p.lengths, p.batch, p.t_cap, p.workers, p.min_tiles, s_prefix, p.status, p.unit_cost);
  const int c = tid % dk, bg = tid / dk;          // blockDim.x == dk * bg_count

  for (int b0 = 0; b0 < p.batch; b0 += BT) {
    const int nb = min(BT, p.batch - b0);
    __syncthreads();
    // ---- combine weights per sequence (one warp per sequence) ----------------
    for (int bi = wid; bi < nb; bi += nwarp) {
      const int b = b0 + bi;
      const int g_lo = s_prefix[b], g_hi = s_prefix[b + 1];
      int wlo = 0, wn = 0;
      if (g_hi > g_lo) {
        wlo = slim_worker_of_tile(sc, g_lo);
        wn = slim_worker_of_tile(sc, g_hi - 1) - wlo + 1;
        float M = -INFINITY;
        for (int i = lane; i < wn; i += 32) {
          const size_t ui = (size_t)(wlo + i + b) * H + h;
          M = fmaxf(M, p.part_m[ui] + log2f(p.part_l[ui]));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
        float L = 0.f;
        for (int i = lane; i < wn; i += 32) {
          const size_t ui = (size_t)(wlo + i + b) * H + h;
          const float wg = exp2f(p.part_m[ui] - M);
          s_wgt[bi * p.workers + i] = wg;
          L += wg * p.part_l[ui];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
        const float inv = 1.f / L;
        __syncwarp();
        for (int i = lane; i < wn; i += 32) s_wgt[bi * p.workers + i] *= inv;
      }
      if (lane == 0) { s_wlo[bi] = wlo; s_wn[bi] = wn; }
    }
    __syncthreads();
    // ---- a7: u tile = weighted sum of the partials --------------------------
    for (int e = tid; e < nb * JR; e += blockDim.x) {
      const int bi = e / JR, j = e - bi * JR;
      float v = 0.f;
      if (j < jn) {
        const int b = b0 + bi, wlo = s_wlo[bi], wn = s_wn[bi];
        const float* wg = s_wgt + bi * p.workers;
        for (int i = 0; i < wn; ++i)
          v = fmaf(wg[i], __ldg(p.part_u + ((size_t)(wlo + i + b) * H + h) * d + j0 + j), v);
      }
      s_u[bi * JR + j] = v;
    }
    __syncthreads();
    // ---- a8: partial projection over this j-slice ------------------------------
    if (bg < bg_count) {
      float acc[BPT];
#pragma unroll
      for (int i = 0; i < BPT; ++i) acc[i] = 0.f;
      const float* ub = s_u + (bg * BPT) * JR;
      int j = 0;
      for (; j + 4 <= jn; j += 4) {
        const float w0 = ld_w(W + (size_t)(j + 0) * dk + c), w1 = ld_w(W + (size_t)(j + 1) * dk + c);
        const float w2 = ld_w(W + (size_t)(j + 2) * dk + c), w3 = ld_w(W + (size_t)(j + 3) * dk + c);
#pragma unroll
        for (int i = 0; i < BPT; ++i) {
          const float4 uv = *reinterpret_cast<const float4*>(ub + i * JR + j);
          acc[i] = fmaf(uv.x, w0, acc[i]); acc[i] = fmaf(uv.y, w1, acc[i]);
          acc[i] = fmaf(uv.z, w2, acc[i]); acc[i] = fmaf(uv.w, w3, acc[i]);
        }
      }
      for (; j < jn; ++j) {
        const float w0 = ld_w(W + (size_t)j * dk + c);
#pragma unroll
        for (int i = 0; i < BPT; ++i) acc[i] = fmaf(ub[i * JR + j], w0, acc[i]);
      }
#pragma unroll
      for (int i = 0; i < BPT; ++i) {
        const int bi = bg * BPT + i;
        if (bi < nb) o_part[((size_t)js * p.batch + b0 + bi) * p.e + h * dk + c] = acc[i];
      }
    }
  }
}

__global__ void __launch_bounds__(256) slim_tail2_kernel(const float* __restrict__ o_part, float* __restrict__ o,
                                                         int n, int nsplit) {
  slim_pdl_trigger();
  slim_pdl_wait();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float a = 0.f;
  for (int s = 0; s < nsplit; ++s) a += o_part[(size_t)s * n + i];
  o[i] = a;
}

template <typename KT>
__global__ void slim_append_kernel(KT* __restrict__ cache, const KT* __restrict__ k_new,
                                   const int32_t* __restrict__ positions, int d, int t_cap, int n_new,
                                   int* status, const int32_t* __restrict__ block_table, int page_rows, int max_pages,
                                   int num_pages, int pos_is_length) {
  slim_pdl_trigger();
  slim_pdl_wait();
  const int b = blockIdx.x, r = blockIdx.y;
  int pos = positions[b];
  if (pos_is_length) {                       // positions[] holds the lengths after the append
    if (pos <= 0) return;                    // an empty sequence receives no row
    pos -= 1;
  }
  if (pos < 0 || pos > t_cap - n_new) {            // (n_new <= t_cap is checked on the host; no overflow for any pos)
    if (threadIdx.x == 0) atomicMax(status, (int)SLIM_ERR_CAPACITY);
    return;
  }
  const KT* src = k_new + ((size_t)b * n_new + r) * d;
  size_t row = (size_t)b * t_cap + pos + r;
  if (block_table) {                                // paged storage
    const int pg = block_table[(size_t)b * max_pages + (pos + r) / page_rows];
    if (pg < 0 || pg >= num_pages) {
      if (threadIdx.x == 0) atomicMax(status, (int)SLIM_ERR_CAPACITY);
      return;
    }
    row = (size_t)pg * page_rows + (pos + r) % page_rows;
  }
  KT* dst = cache + row * d;
  // rows are 16-byte aligned when d * sizeof(KT) is a multiple of 16 and the buffers are
  const size_t bytes = (size_t)d * sizeof(KT);
  if ((bytes & 15) == 0 && (((uintptr_t)src | (uintptr_t)dst) & 15) == 0) {
    const uint4* s4 = reinterpret_cast<const uint4*>(src);
    uint4* d4 = reinterpret_cast<uint4*>(dst);
    for (int e = threadIdx.x; e < (int)(bytes >> 4); e += blockDim.x) d4[e] = __ldg(s4 + e);
  } else {
    for (int e = threadIdx.x; e < d; e += blockDim.x) dst[e] = src[e];
  }
}

// 8-bit cache: quantise the new bf16 rows.  Per (row, head): exponent e = the smallest integer with
// max|k| * 2^-e <= 448 (the E4M3 range), code = E4M3(k * 2^-e) rounded to nearest even; the scaling by
// a power of two is exact, so the codes depend on the input bits only.  One warp per head.
__global__ void __launch_bounds__(256)
slim_append_fp8_kernel(unsigned char* __restrict__ codes, signed char* __restrict__ exps, const __nv_bfloat16* __restrict__ k_new,
                       const int32_t* __restrict__ positions, int d, int H, int d_k, int t_cap, int n_new, int* status,
                       int pos_is_length) {
  slim_pdl_trigger();
  slim_pdl_wait();
  const int b = blockIdx.x, r = blockIdx.y, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int pos = positions[b];
  if (pos_is_length) {
    if (pos <= 0) return;
    pos -= 1;
  }
  if (pos < 0 || pos > t_cap - n_new) {
    if (threadIdx.x == 0) atomicMax(status, (int)SLIM_ERR_CAPACITY);
    return;
  }
  const __nv_bfloat16* src = k_new + ((size_t)b * n_new + r) * d;
  const size_t row = (size_t)b * t_cap + pos + r;
  for (int h = warp; h < H; h += blockDim.x >> 5) {
    float amax = 0.f;
    for (int c = lane; c < d_k; c += 32) amax = fmaxf(amax, fabsf(__bfloat162float(src[h * d_k + c])));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    int e = 0;
    if (amax > 0.f && amax <= 3.0e38f) {
      int x;
      const float m = frexpf(amax, &x);                 // amax = m 2^x, 0.5 <= m < 1; 448 = 0.875 * 2^9
      e = m <= 0.875f ? x - 9 : x - 8;
      e = max(-126, min(127, e));
    }
    const float inv = __int_as_float((127 - e) << 23);  // 2^-e (e >= -126 keeps it finite: 2^126 at most)
    for (int c = lane; c < d_k; c += 32)
      codes[row * d + h * d_k + c] = (unsigned char)__nv_cvt_float_to_fp8(__bfloat162float(src[h * d_k + c]) * inv, __NV_SATFINITE, __NV_E4M3);
    if (lane == 0) exps[row * H + h] = (signed char)e;
  }
}

// 8-bit cache -> bf16 rows for the tensor-core kernels: stored key = code * 2^exponent, one exponent per (row,
// head).  An E4M3 code has four significant bits, so the product is exact in bf16 (as long as the sum of the two
// exponents stays in bf16's range, which the quantiser's clamp of the exponent together with the code's own range
// leaves a wide margin for).  A thread decodes 16 codes of one head (d_k is a multiple of 16); a CTA takes
// DQ_ROWS rows of one sequence; rows at or beyond lengths[b] are left as they are (the decode kernel masks them).
constexpr int DQ_ROWS = 8;
__global__ void __launch_bounds__(256)
slim_dequant_kernel(const unsigned char* __restrict__ codes, const signed char* __restrict__ exps, __nv_bfloat16* __restrict__ out,
                    const int32_t* __restrict__ lengths, int d, int H, int d_k, int t_cap) {
  slim_pdl_trigger();
  slim_pdl_wait();
  const int b = blockIdx.y, t0 = blockIdx.x * DQ_ROWS;
  const int len = min(max(lengths[b], 0), t_cap);
  if (t0 >= len) return;
  const int vec_per_row = d / 16;
  const int n = min(DQ_ROWS, len - t0) * vec_per_row;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const int r = i / vec_per_row, v = i - r * vec_per_row;
    const size_t row = (size_t)b * t_cap + t0 + r;
    const uint4 c = __ldcs(reinterpret_cast<const uint4*>(codes + row * d) + v);
    const float scale = __int_as_float(((int)__ldg(exps + row * H + (v * 16) / d_k) + 127) << 23);
    const uint32_t w[4] = {c.x, c.y, c.z, c.w};
    uint32_t o[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const uint32_t pair = (w[k >> 1] >> (16 * (k & 1))) & 0xffffu;                  // two codes
      const __half2_raw h2 = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)pair, __NV_E4M3);
      const float2 f = __half22float2(__half2(h2));
      const __nv_bfloat162 bb = __floats2bfloat162_rn(f.x * scale, f.y * scale);
      o[k] = *reinterpret_cast<const uint32_t*>(&bb);
    }
    uint4* dst = reinterpret_cast<uint4*>(out + row * d) + 2 * v;
    dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
    dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
  }
}

}  // namespace

cudaError_t slim_launch_dequant(const slim_ctx* ctx, const slim_cache* c, const int32_t* lengths, void* scratch, cudaStream_t st) {
  return slim_launch_pdl(slim_dequant_kernel, dim3((c->t_cap + DQ_ROWS - 1) / DQ_ROWS, c->batch), dim3(256), 0, st,
                         (const unsigned char*)c->k, (const signed char*)c->k_exp, (__nv_bfloat16*)scratch, lengths, ctx->d, ctx->H,
                         ctx->d_k, c->t_cap);
}

size_t slim_tail_opart_floats(int d, int e, int batch) {
  const int slices = (d + JR - 1) / JR;
  return (size_t)(slices > 8 ? slices : 8) * batch * e;
}

cudaError_t slim_launch_sum_slices(const float* o_part, float* o, int n, int nsplit, cudaStream_t st) {
  return slim_launch_pdl(slim_tail2_kernel, dim3((n + 255) / 256), dim3(256), 0, st, o_part, o, n, nsplit);
}

cudaError_t slim_launch_tail(const slim_ctx* ctx, const SlimDecodeParams& p, cudaStream_t st) {
  const int nsplit = (p.d + JR - 1) / JR;
  int bg_count = 256 / p.d_k;
  if (bg_count < 1) bg_count = 1;
  if (bg_count > BT_MAX / BPT) bg_count = BT_MAX / BPT;
  const int threads = ((p.d_k * bg_count + 31) / 32) * 32;
  // o_part lives behind u in the workspace
  float* o_part = p.u;
  const size_t smem = sizeof(float) * ((size_t)BT_MAX * JR + (size_t)BT_MAX * p.workers) +
                      sizeof(int) * (2 * BT_MAX + p.batch + 1);
  cudaError_t e;
  dim3 grid(p.H, nsplit);
  if (p.dtype == SLIM_BF16) {
    auto kern = slim_tail1_kernel<__nv_bfloat16>;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, threads, smem, st>>>(p, bg_count, o_part);
  } else {
    auto kern = slim_tail1_kernel<float>;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, threads, smem, st>>>(p, bg_count, o_part);
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const int n = p.batch * p.e;
  slim_tail2_kernel<<<(n + 255) / 256, 256, 0, st>>>(o_part, p.o, n, nsplit);
  return cudaGetLastError();
}

cudaError_t slim_launch_append(const slim_ctx* ctx, const slim_cache* c, const void* k_new,
                               const int32_t* positions, int n_new, int pos_is_length, cudaStream_t st) {
  dim3 grid(c->batch, n_new);
  if (ctx->kdtype == SLIM_FP8)
    return slim_launch_pdl(slim_append_fp8_kernel, grid, dim3(256), 0, st, (unsigned char*)c->k, c->k_exp,
                           (const __nv_bfloat16*)k_new, positions, ctx->d, ctx->H, ctx->d_k, c->t_cap, n_new, ctx->status,
                           pos_is_length);
  if (ctx->dtype == SLIM_BF16)
    return slim_launch_pdl(slim_append_kernel<__nv_bfloat16>, grid, dim3(256), 0, st, (__nv_bfloat16*)c->k,
                           (const __nv_bfloat16*)k_new, positions, ctx->d, c->t_cap, n_new, ctx->status, c->block_table,
                           c->page_rows, c->max_pages, c->num_pages, pos_is_length);
  return slim_launch_pdl(slim_append_kernel<float>, grid, dim3(256), 0, st, (float*)c->k, (const float*)k_new, positions,
                         ctx->d, c->t_cap, n_new, ctx->status, c->block_table, c->page_rows, c->max_pages, c->num_pages, pos_is_length);
}
