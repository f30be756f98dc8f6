// X-cache / E-cache scheme: dense softmax arguments on the tensor cores.
//   A_i[t] = q~_i . X[t][:]   with   q~_i = (x_n W_Q,i + b) W_K,i^T  (a d-vector per head)
// for all heads at once: S[128 rows x N] += X_tile[128 x 16] Q~^T[16 x N] over d in steps of 16,
// one tcgen05.mma per step.  A = rows of the cache, K-major with 128-byte swizzle exactly as TMA
// delivers them; B = the per-sequence query tiles, written by slim_xq_tiled_kernel as a bf16
// hi/lo pair (N = 64: heads 0..31 hi, 32..63 lo) in the K-major core-matrix layout; D in tensor
// memory.  A CTA owns 128 rows of one sequence.  Every mbarrier wait is bounded in time.
#include <cstring>

#include "slim_internal.h"
#include "slim_ptx.cuh"

namespace {
using namespace slim_ptx;

constexpr int XT_ROWS = 128;                      // cache rows per CTA (MMA M)
constexpr int XT_COLS = 64;                       // cache columns per stage (4 k-steps)
constexpr int XT_A_BYTES = XT_ROWS * XT_COLS * 2; // 16 KB
constexpr int XT_B_BYTES = (XT_COLS / 16) * 2048; // 4 k-steps x [64 x 16] bf16
constexpr int XT_NS = 4;

__device__ __forceinline__ uint32_t qt_offset(int n, int k) {     // K-major 8x8 core matrices, N = 64
  return (uint32_t)((n & 7) * 16 + (n >> 3) * 256 + (k >> 3) * 128 + (k & 7) * 2);
}
// q~[b][h][j] = qscale sum_c q[b][h d_k + c] W_K[j][h d_k + c], written as bf16 hi / lo rows h and 32 + h
// of the [64 x 16] tile of k-step j / 16.  CTA = (head, 64 rows j of W_K): the weight tile is read once
// and used for every sequence of the batch.
constexpr int XQ_J = 64, XQ_B = 64;             // rows of W_K per CTA; sequences per pass (one pass up to batch 64)
__global__ void __launch_bounds__(256)
slim_xq_tiled_kernel(SlimDecodeParams p, const float* __restrict__ W_K, unsigned char* __restrict__ qt_tiled) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int dk = p.d_k, d = p.d;
  float* s_w = reinterpret_cast<float*>(smem_raw);                   // [XQ_J][dk + 1]
  float* s_q = s_w + XQ_J * (dk + 1);                                // [dk][XQ_B]
  slim_pdl_wait();
  const int h = blockIdx.x, j0 = blockIdx.y * XQ_J, tid = threadIdx.x;
  for (int e = tid; e < XQ_J * dk; e += 256) {
    const int j = e / dk, c = e % dk;
    s_w[j * (dk + 1) + c] = (j0 + j < d) ? __ldg(W_K + (size_t)(j0 + j) * p.e + h * dk + c) : 0.f;
  }
  constexpr int XQ_S = XQ_B / 4;                                     // sequences per thread and pass
  const int j = tid & (XQ_J - 1), bq = tid >> 6;                     // a thread: row j, sequences XQ_S bq .. XQ_S bq + XQ_S - 1 of a pass
  for (int b0 = 0; b0 < p.batch; b0 += XQ_B) {
    __syncthreads();
    for (int e = tid; e < XQ_B * dk; e += 256) {                     // s_q[c][bb]: the sequences of one c side by side
      const int bb = e / dk, c = e % dk;
      s_q[c * XQ_B + bb] = (b0 + bb < p.batch)
                               ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.q)[(size_t)(b0 + bb) * p.e + h * dk + c]) * p.qscale : 0.f;
    }
    __syncthreads();
    if (j0 + j >= d || b0 + XQ_S * bq >= p.batch) continue;
    const float* w = s_w + j * (dk + 1);
    float a[XQ_S];
#pragma unroll
    for (int x = 0; x < XQ_S; ++x) a[x] = 0.f;
#pragma unroll 4
    for (int c = 0; c < dk; ++c) {
      const float wc = w[c];
#pragma unroll
      for (int x4 = 0; x4 < XQ_S / 4; ++x4) {
        const float4 qv = *reinterpret_cast<const float4*>(s_q + c * XQ_B + XQ_S * bq + 4 * x4);
        a[4 * x4] = fmaf(qv.x, wc, a[4 * x4]); a[4 * x4 + 1] = fmaf(qv.y, wc, a[4 * x4 + 1]);
        a[4 * x4 + 2] = fmaf(qv.z, wc, a[4 * x4 + 2]); a[4 * x4 + 3] = fmaf(qv.w, wc, a[4 * x4 + 3]);
      }
    }
#pragma unroll
    for (int x = 0; x < XQ_S; ++x) {
      const int b = b0 + XQ_S * bq + x;
      if (b >= p.batch) continue;
      const __nv_bfloat16 hi = __float2bfloat16_rn(a[x]), lo = __float2bfloat16_rn(a[x] - __bfloat162float(hi));
      unsigned char* t = qt_tiled + ((size_t)b * (d / 16) + (j0 + j) / 16) * 2048;
      *reinterpret_cast<__nv_bfloat16*>(t + qt_offset(h, (j0 + j) & 15)) = hi;
      *reinterpret_cast<__nv_bfloat16*>(t + qt_offset(32 + h, (j0 + j) & 15)) = lo;
    }
  }
}

__global__ void __launch_bounds__(128)
slim_xscores_tc_kernel(const __grid_constant__ CUtensorMap xmap, const SlimDecodeParams p,
                       const unsigned char* __restrict__ qt_tiled, float* __restrict__ scores) {
  const int b = blockIdx.y, t0 = blockIdx.x * XT_ROWS;
  const int len = min(max(p.lengths[b], 0), p.t_cap);
  if (t0 >= len) return;                                       // whole CTA: nothing allocated yet

  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw_u32 = smem_u32(smem_raw);
  const uint32_t base = (raw_u32 + 1023u) & ~1023u;
  unsigned char* sm = smem_raw + (base - raw_u32);
  constexpr uint32_t stage_bytes = XT_A_BYTES + XT_B_BYTES;
  const uint32_t bars = base + XT_NS * stage_bytes;
  const uint32_t bar_full = bars, bar_empty = bars + 8 * XT_NS, bar_done = bars + 16 * XT_NS;
  unsigned char* misc = sm + (bar_done + 8 - base);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(misc);
  volatile int* s_abort = reinterpret_cast<volatile int*>(misc + 4);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nst = p.d / XT_COLS;

  if (tid == 0) {
    prefetch_tensormap(&xmap);
    for (int i = 0; i < XT_NS; ++i) { mbar_init(bar_full + 8 * i, 1); mbar_init(bar_empty + 8 * i, 1); }
    mbar_init(bar_done, 1);
    *s_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) tmem_alloc(smem_u32(s_tmem), 64);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  slim_pdl_wait();                                             // the query tiles come from the kernel before

  if (warp == 0 && lane == 0) {
    const unsigned char* qsrc = qt_tiled + (size_t)b * (p.d / 16) * 2048;
    int s = 0;
    bool ok = true;
    for (; s < nst; ++s) {
      const int st = s % XT_NS;
      ok = mbar_wait<false>(bar_empty + 8 * st, ((s / XT_NS) & 1) ^ 1, s_abort, p.status);
      if (!ok) break;
      const uint32_t dst = base + (uint32_t)st * stage_bytes;
      mbar_arrive_expect_tx(bar_full + 8 * st, stage_bytes);
      tma_load_3d(dst, &xmap, bar_full + 8 * st, s * XT_COLS, b * p.t_cap + t0, 0);
      bulk_load(dst + XT_A_BYTES, qsrc + (size_t)s * XT_B_BYTES, XT_B_BYTES, bar_full + 8 * st);
    }
    if (!ok) {
      const int issued = s < XT_NS ? s : XT_NS;
      for (int k = 0; k < issued; ++k) {
        const int j = s - 1 - k, st = j % XT_NS;
        const unsigned long long tt = globaltimer();
        while (!mbar_try_wait(bar_full + 8 * st, (j / XT_NS) & 1) && globaltimer() - tt < SLIM_WAIT_NS) {}
      }
    }
  } else if (warp == 1 && lane == 0) {
    bool ok = true;
    for (int s = 0; s < nst && ok; ++s) {
      const int st = s % XT_NS;
      ok = mbar_wait<false>(bar_full + 8 * st, (s / XT_NS) & 1, s_abort, p.status);
      if (!ok) break;
      tc_fence_after();
      const uint32_t abase = base + (uint32_t)st * stage_bytes, bbase = abase + XT_A_BYTES;
#pragma unroll
      for (int kk = 0; kk < XT_COLS / 16; ++kk)
        umma_bf16(tmem_base, desc_kmajor_sw128(abase + (uint32_t)kk * 32u), desc_b(bbase + (uint32_t)kk * 2048u), umma_idesc_major(64, 0, 0),
                  (s | kk) ? 1u : 0u);
      umma_commit(bar_empty + 8 * st);
      if (s == nst - 1) umma_commit(bar_done);
    }
  }
  __syncwarp();
  {
    bool ok = mbar_wait<false>(bar_done, 0, s_abort, p.status);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tc_fence_after();
      const int row = warp * 32 + lane;                        // accumulator row = cache row of the tile
      uint32_t hi[32], lo[32];
      tmem_ld32_issue(tmem_base + ((uint32_t)(warp * 32) << 16), hi);
      tmem_ld32_issue(tmem_base + ((uint32_t)(warp * 32) << 16) + 32u, lo);
      tmem_ld_wait();
      if (t0 + row < len) {
#pragma unroll
        for (int h = 0; h < 32; ++h)
          if (h < p.H) scores[((size_t)b * p.H + h) * p.t_cap + t0 + row] = __uint_as_float(hi[h]) + __uint_as_float(lo[h]);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 64);
  }
}

constexpr size_t XT_SMEM = 1024 + (size_t)XT_NS * (XT_A_BYTES + XT_B_BYTES) + 16 * XT_NS + 8 + 16 + 64;

}  // namespace

int slim_xscores_tc_ok(const slim_ctx* ctx) {
  return ctx->dtype == SLIM_BF16 && ctx->d % XT_COLS == 0 && ctx->H <= 32 && ctx->rope_theta == 0.0;
}

size_t slim_xscores_qt_bytes(int d, int batch) { return (size_t)batch * (d / 16) * 2048; }

cudaError_t slim_xscores_make_tmap(const slim_ctx* ctx, slim_cache* c) {
  // (d columns, batch * t_cap rows); box 64 columns x 128 rows; rows past the end read as zeros
  const unsigned long long dims[3] = {(unsigned long long)ctx->d, (unsigned long long)c->batch * c->t_cap, 1};
  const unsigned long long strides[2] = {(unsigned long long)ctx->d * 2, (unsigned long long)ctx->d * 2 * c->batch * c->t_cap};
  const unsigned int box[3] = {XT_COLS, XT_ROWS, 1};
  cudaError_t e = slim_tmap_encode_3d(c->xmap, c->k, dims, strides, box);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute((const void*)slim_xscores_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)XT_SMEM);
}

cudaError_t slim_launch_xscores_tc(const slim_ctx* ctx, const slim_cache* c, const SlimDecodeParams& p, const float* W_K,
                                   unsigned char* qt_tiled, float* scores, cudaStream_t st) {
  const size_t xq_smem = sizeof(float) * (XQ_J * (p.d_k + 1) + XQ_B * p.d_k);
  if (xq_smem > 48 * 1024) {                         // function attributes are kept per device: opt in once on each
    static bool attr_set[64] = {};
    if (ctx->device < 0 || ctx->device >= 64 || !attr_set[ctx->device]) {
      cudaError_t ea = cudaFuncSetAttribute((const void*)slim_xq_tiled_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
      if (ea != cudaSuccess) return ea;
      if (ctx->device >= 0 && ctx->device < 64) attr_set[ctx->device] = true;
    }
  }
  // (a plain launch: letting this kernel start under the one before it was measured slower, 5.16 -> 5.44 ms per step)
  slim_xq_tiled_kernel<<<dim3(p.H, (p.d + XQ_J - 1) / XQ_J), 256, xq_smem, st>>>(p, W_K, qt_tiled);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  CUtensorMap map;
  memcpy(&map, c->xmap, sizeof(map));
  return slim_launch_pdl(slim_xscores_tc_kernel, dim3((p.t_cap + XT_ROWS - 1) / XT_ROWS, p.batch), dim3(128), XT_SMEM, st, map, p,
                         (const unsigned char*)qt_tiled, scores);
}
