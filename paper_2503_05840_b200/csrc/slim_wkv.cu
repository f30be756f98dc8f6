// Eq. 6 on the device in float64:  solve W_K X = W_V  (X = W_KV) by blocked LU
// with partial pivoting on the augmented matrix M = [W_K | W_V] (n x 2n),
// followed by a blocked back substitution.  Offline set-up work; written for
// clarity and a few seconds at n = 4096, not for peak FP64 rate.  The right-hand
// side may have any number of columns m (M is n x (n + m)): the non-square case
// (section "Support for non-square weight matrices", Option 1) solves
// (W_K W_K^T) Y = W_V with n = d_model and m = e.
#include <cuda_fp16.h>

#include "slim_internal.h"

namespace {

constexpr int NB = 32;          // panel width

// --- panel factorisation: columns [k0, k0+kb) of rows [k0, n) ---------------
// One CTA.  Row swaps are applied to the panel columns only; piv[k0+j] records
// the row exchanged with row k0+j.  info[0] = 1 if a pivot is too small.
__global__ void __launch_bounds__(1024) lu_panel_kernel(double* __restrict__ M, int ld, int n, int k0, int kb,
                                                        int* __restrict__ piv, int* info, double tiny) {
  __shared__ double s_val[32];
  __shared__ int s_idx[32];
  __shared__ double s_row[NB];
  __shared__ int s_p;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nw = blockDim.x >> 5;
  for (int j = 0; j < kb; ++j) {
    const int col = k0 + j;
    // arg max |M[i][col]| over i >= col
    double best = -1.0; int bi = col;
    for (int i = col + tid; i < n; i += blockDim.x) {
      const double v = fabs(M[(size_t)i * ld + col]);
      if (v > best) { best = v; bi = i; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const double ov = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
    }
    if (lane == 0) { s_val[wid] = best; s_idx[wid] = bi; }
    __syncthreads();
    if (wid == 0) {
      best = lane < nw ? s_val[lane] : -1.0; bi = lane < nw ? s_idx[lane] : 0x7fffffff;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const double ov = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
      }
      if (lane == 0) {
        s_p = bi; piv[col] = bi;
        if (!(best > tiny)) info[0] = 1;
      }
    }
    __syncthreads();
    const int prow = s_p;
    // swap rows col <-> prow inside the panel, keep the pivot row in smem
    if (tid < kb) {
      const double a = M[(size_t)col * ld + k0 + tid], b = M[(size_t)prow * ld + k0 + tid];
      M[(size_t)col * ld + k0 + tid] = b;
      M[(size_t)prow * ld + k0 + tid] = a;
      s_row[tid] = b;
    }
    __syncthreads();
    const double pv = s_row[j];
    const double rinv = (pv != 0.0) ? 1.0 / pv : 0.0;
    for (int i = col + 1 + tid; i < n; i += blockDim.x) {
      double* r = M + (size_t)i * ld + k0;
      const double l = r[j] * rinv;
      r[j] = l;
      for (int jj = j + 1; jj < kb; ++jj) r[jj] -= l * s_row[jj];
    }
    __syncthreads();
  }
}

// --- apply the panel's row exchanges to every column outside the panel --------
__global__ void lu_swap_kernel(double* __restrict__ M, int ld, int ncols, int k0, int kb,
                               const int* __restrict__ piv) {
  int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= ncols - kb) return;
  if (c >= k0) c += kb;                       // skip the panel columns
  for (int j = 0; j < kb; ++j) {
    const int r0 = k0 + j, r1 = piv[r0];
    if (r1 != r0) {
      const double a = M[(size_t)r0 * ld + c], b = M[(size_t)r1 * ld + c];
      M[(size_t)r0 * ld + c] = b; M[(size_t)r1 * ld + c] = a;
    }
  }
}

// --- U12 = L11^{-1} A12 (unit lower), one thread per column -----------------
__global__ void lu_trsm_lower_kernel(double* __restrict__ M, int ld, int ncols, int k0, int kb) {
  __shared__ double s_L[NB][NB + 1];
  for (int e = threadIdx.x; e < kb * kb; e += blockDim.x)
    s_L[e / kb][e % kb] = M[(size_t)(k0 + e / kb) * ld + k0 + e % kb];
  __syncthreads();
  const int c = k0 + kb + blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= ncols) return;
  double x[NB];
#pragma unroll
  for (int r = 0; r < NB; ++r) {
    if (r < kb) {
      double v = M[(size_t)(k0 + r) * ld + c];
#pragma unroll
      for (int s = 0; s < NB; ++s) if (s < r) v -= s_L[r][s] * x[s];
      x[r] = v;
      M[(size_t)(k0 + r) * ld + c] = v;
    }
  }
}

// --- C[r0:r1, c0:c1] -= A[r0:r1, k0:k0+kb] * B[k0:k0+kb, c0:c1]   (all inside M)
// 64x64 tile per CTA, 16x16 threads, 4x4 outputs per thread.
__global__ void __launch_bounds__(256) lu_gemm_kernel(double* __restrict__ M, int ld, int r0, int r1, int c0, int c1,
                                                      int k0, int kb) {
  __shared__ double s_A[64][NB + 1];
  __shared__ double s_B[NB][64 + 1];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int rb = r0 + blockIdx.y * 64, cb = c0 + blockIdx.x * 64;
  for (int e = threadIdx.x; e < 64 * NB; e += 256) {
    const int r = e / NB, k = e % NB;
    s_A[r][k] = (rb + r < r1 && k < kb) ? M[(size_t)(rb + r) * ld + k0 + k] : 0.0;
  }
  for (int e = threadIdx.x; e < NB * 64; e += 256) {
    const int k = e / 64, c = e % 64;
    s_B[k][c] = (cb + c < c1 && k < kb) ? M[(size_t)(k0 + k) * ld + cb + c] : 0.0;
  }
  __syncthreads();
  double acc[4][4] = {};
#pragma unroll 8
  for (int k = 0; k < NB; ++k) {
    double a[4], b[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) { a[i] = s_A[ty + 16 * i][k]; b[i] = s_B[k][tx + 16 * i]; }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = fma(a[i], b[j], acc[i][j]);
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int r = rb + ty + 16 * i, c = cb + tx + 16 * j;
      if (r < r1 && c < c1) M[(size_t)r * ld + c] -= acc[i][j];
    }
}

// --- X[k0:k0+kb, :] = U11^{-1} Y[k0:k0+kb, :] (upper, non-unit), thread per column of the right half
__global__ void lu_trsm_upper_kernel(double* __restrict__ M, int ld, int n, int k0, int kb) {   // rhs columns [n, ld)
  __shared__ double s_U[NB][NB + 1];
  for (int e = threadIdx.x; e < kb * kb; e += blockDim.x)
    s_U[e / kb][e % kb] = M[(size_t)(k0 + e / kb) * ld + k0 + e % kb];
  __syncthreads();
  const int c = n + blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= ld) return;
  double x[NB];
#pragma unroll
  for (int rr = 0; rr < NB; ++rr) {
    const int r = NB - 1 - rr;
    if (r < kb) {
      double v = M[(size_t)(k0 + r) * ld + c];
#pragma unroll
      for (int s = 0; s < NB; ++s) if (s > r && s < kb) v -= s_U[r][s] * x[s];
      v /= s_U[r][r];
      x[r] = v;
      M[(size_t)(k0 + r) * ld + c] = v;
    }
  }
}

// M = [A | B]: A is n x n, B is n x m
__global__ void pack_aug_kernel(const double* __restrict__ A, const double* __restrict__ B, double* __restrict__ M, int n, int m) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t ld = (size_t)n + m;
  if (i >= (size_t)n * ld) return;
  const size_t r = i / ld, c = i % ld;
  M[i] = c < (size_t)n ? A[r * n + c] : B[r * m + (c - n)];
}

__global__ void unpack_x_kernel(const double* __restrict__ M, double* __restrict__ X, int n, int m) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (size_t)n * m) return;
  const size_t r = i / m, c = i % m;
  X[i] = M[r * ((size_t)n + m) + n + c];
}

// C[M x N] = op(A) op(B), float64, 64 x 64 tiles.  op(A) is M x K: A is [M][K] (ta = 0) or [K][M]
// (ta = 1); op(B) is K x N: B is [K][N] (tb = 0) or [N][K] (tb = 1).  Row-major, dense.
__global__ void __launch_bounds__(256) dgemm_kernel(const double* __restrict__ A, const double* __restrict__ B,
                                                    double* __restrict__ C, int Mr, int Nc, int Kd, int ta, int tb) {
  __shared__ double s_A[64][NB + 1];
  __shared__ double s_B[NB][64 + 1];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int rb = blockIdx.y * 64, cb = blockIdx.x * 64;
  double acc[4][4] = {};
  for (int k0 = 0; k0 < Kd; k0 += NB) {
    for (int e = threadIdx.x; e < 64 * NB; e += 256) {
      const int r = e / NB, k = e % NB;
      double v = 0.0;
      if (rb + r < Mr && k0 + k < Kd) v = ta ? A[(size_t)(k0 + k) * Mr + rb + r] : A[(size_t)(rb + r) * Kd + k0 + k];
      s_A[r][k] = v;
    }
    for (int e = threadIdx.x; e < NB * 64; e += 256) {
      const int k = e / 64, c = e % 64;
      double v = 0.0;
      if (cb + c < Nc && k0 + k < Kd) v = tb ? B[(size_t)(cb + c) * Kd + k0 + k] : B[(size_t)(k0 + k) * Nc + cb + c];
      s_B[k][c] = v;
    }
    __syncthreads();
#pragma unroll 4
    for (int k = 0; k < NB; ++k) {
      double a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = s_A[ty * 4 + i][k]; b[i] = s_B[k][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fma(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int r = rb + ty * 4 + i, c = cb + tx * 4 + j;
      if (r < Mr && c < Nc) C[(size_t)r * Nc + c] = acc[i][j];
    }
}

__global__ void absdiff_max_kernel(const double* __restrict__ A, const double* __restrict__ B, size_t n, double* out) {
  double m = 0.0;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    m = fmax(m, fabs(A[i] - B[i]));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0)
    atomicMax(reinterpret_cast<unsigned long long*>(out), (unsigned long long)__double_as_longlong(m));
}

__global__ void absmax_kernel(const double* __restrict__ A, size_t n, double* out) {
  double m = 0.0;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    m = fmax(m, fabs(A[i]));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0)   // non-negative doubles order like their bit patterns
    atomicMax(reinterpret_cast<unsigned long long*>(out), (unsigned long long)__double_as_longlong(m));
}

// residual: max | Wk X - Wv |, 64x64 tiles
__global__ void __launch_bounds__(256) residual_kernel(const double* __restrict__ Wk, const double* __restrict__ X,
                                                       const double* __restrict__ Wv, int n, double* out) {
  __shared__ double s_A[64][NB + 1];
  __shared__ double s_B[NB][64 + 1];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int rb = blockIdx.y * 64, cb = blockIdx.x * 64;
  double acc[4][4] = {};
  for (int k0 = 0; k0 < n; k0 += NB) {
    for (int e = threadIdx.x; e < 64 * NB; e += 256) {
      const int r = e / NB, k = e % NB;
      s_A[r][k] = (rb + r < n && k0 + k < n) ? Wk[(size_t)(rb + r) * n + k0 + k] : 0.0;
    }
    for (int e = threadIdx.x; e < NB * 64; e += 256) {
      const int k = e / 64, c = e % 64;
      s_B[k][c] = (cb + c < n && k0 + k < n) ? X[(size_t)(k0 + k) * n + cb + c] : 0.0;
    }
    __syncthreads();
#pragma unroll 8
    for (int k = 0; k < NB; ++k) {
      double a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = s_A[ty + 16 * i][k]; b[i] = s_B[k][tx + 16 * i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fma(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
  double m = 0.0;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int r = rb + ty + 16 * i, c = cb + tx + 16 * j;
      if (r < n && c < n) m = fmax(m, fabs(acc[i][j] - Wv[(size_t)r * n + c]));
    }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0)
    atomicMax(reinterpret_cast<unsigned long long*>(out), (unsigned long long)__double_as_longlong(m));
}

template <typename WT>
__global__ void store_wkv_kernel(const double* __restrict__ X, WT* __restrict__ dst, __half* __restrict__ dst_h,
                                 const float* __restrict__ hscale, int d, int H, int dk) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (size_t)d * H * dk) return;
  const int c = (int)(i % dk);
  const size_t rest = i / dk;
  const int j = (int)(rest % d), h = (int)(rest / d);
  const double v = X[(size_t)j * H * dk + h * dk + c];
  if constexpr (sizeof(WT) == 2) {
    dst[i] = __double2bfloat16(v);
    if (dst_h) dst_h[i] = __double2half(v / (double)hscale[h]);      // power-of-two scale: exact
  } else {
    dst[i] = (float)v;
  }
}

// hscale[h] = 2^-a with max |W_KV,h| * 2^a in [2^14, 2^15) (1 for an all-zero head): one CTA per head
__global__ void head_scale_kernel(const double* __restrict__ X, float* __restrict__ hscale, int d, int dk, int e) {
  __shared__ double s_max[256];
  const int h = blockIdx.x;
  double m = 0.0;
  for (size_t i = threadIdx.x; i < (size_t)d * dk; i += blockDim.x) {
    const double v = fabs(X[(i / dk) * e + (size_t)h * dk + i % dk]);
    m = v > m ? v : m;
  }
  s_max[threadIdx.x] = m;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) s_max[threadIdx.x] = fmax(s_max[threadIdx.x], s_max[threadIdx.x + o]);
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    float sc = 1.f;
    const double mx = s_max[0];
    if (mx > 0.0 && mx < 1e300) {
      int x;
      frexp(mx, &x);                                   // mx = m 2^x, 0.5 <= m < 1  =>  mx 2^(15 - x) in [2^14, 2^15)
      int a = 15 - x;
      a = a < -100 ? -100 : (a > 100 ? 100 : a);
      sc = exp2f((float)-a);
    }
    hscale[h] = sc;
  }
}

#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { cudaFree(M); cudaFree(piv); cudaFree(scal); return e_; } } while (0)

}  // namespace

cudaError_t slim_wkv_solve(double* A, double* B, int n, int* info_host) { return slim_wkv_solve_rhs(A, B, n, n, info_host); }

cudaError_t slim_wkv_solve_rhs(double* A, double* B, int n, int m, int* info_host) {
  double* M = nullptr; int* piv = nullptr; double* scal = nullptr;   // scal: [0] = max|A| bits, [1] = info
  const int ld = n + m;
  CK(cudaMalloc(&M, sizeof(double) * (size_t)n * ld));
  CK(cudaMalloc(&piv, sizeof(int) * n));
  CK(cudaMalloc(&scal, 16));
  CK(cudaMemset(scal, 0, 16));
  const size_t nn = (size_t)n * n;
  pack_aug_kernel<<<(unsigned)(((size_t)n * ld + 255) / 256), 256>>>(A, B, M, n, m);
  absmax_kernel<<<256, 256>>>(A, nn, scal);
  double amax = 0.0;
  CK(cudaMemcpy(&amax, scal, sizeof(double), cudaMemcpyDeviceToHost));
  const double tiny = 1e-13 * amax * n;
  int* info = reinterpret_cast<int*>(scal + 1);
  for (int k0 = 0; k0 < n; k0 += NB) {
    const int kb = (n - k0 < NB) ? n - k0 : NB;
    lu_panel_kernel<<<1, 1024>>>(M, ld, n, k0, kb, piv, info, tiny);
    lu_swap_kernel<<<(ld - kb + 255) / 256, 256>>>(M, ld, ld, k0, kb, piv);
    const int rest_c = ld - (k0 + kb);
    lu_trsm_lower_kernel<<<(rest_c + 127) / 128, 128>>>(M, ld, ld, k0, kb);
    const int rest_r = n - (k0 + kb);
    if (rest_r > 0) {
      dim3 g((rest_c + 63) / 64, (rest_r + 63) / 64);
      lu_gemm_kernel<<<g, 256>>>(M, ld, k0 + kb, n, k0 + kb, ld, k0, kb);
    }
  }
  // back substitution on the right half: U X = Y
  const int nblk = (n + NB - 1) / NB;
  for (int blk = nblk - 1; blk >= 0; --blk) {
    const int k0 = blk * NB, kb = (n - k0 < NB) ? n - k0 : NB;
    lu_trsm_upper_kernel<<<(m + 127) / 128, 128>>>(M, ld, n, k0, kb);
    if (k0 > 0) {
      dim3 g((m + 63) / 64, (k0 + 63) / 64);
      lu_gemm_kernel<<<g, 256>>>(M, ld, 0, k0, n, ld, k0, kb);
    }
  }
  unpack_x_kernel<<<(unsigned)(((size_t)n * m + 255) / 256), 256>>>(M, B, n, m);
  CK(cudaGetLastError());
  CK(cudaMemcpy(info_host, info, sizeof(int), cudaMemcpyDeviceToHost));
  cudaFree(M); cudaFree(piv); cudaFree(scal);
  return cudaSuccess;
}

cudaError_t slim_wkv_residual(const double* Wk, const double* X, const double* Wv, int n, double* res_host) {
  double* out = nullptr;
  cudaError_t e = cudaMalloc(&out, sizeof(double));
  if (e != cudaSuccess) return e;
  cudaMemset(out, 0, sizeof(double));
  dim3 g((n + 63) / 64, (n + 63) / 64);
  residual_kernel<<<g, 256>>>(Wk, X, Wv, n, out);
  e = cudaMemcpy(res_host, out, sizeof(double), cudaMemcpyDeviceToHost);
  cudaFree(out);
  return e;
}

cudaError_t slim_wkv_store(const double* X, int d, int H, int d_k, int dtype, void* dst, void* dst_h, float* hscale) {
  const size_t nn = (size_t)d * H * d_k;
  if (dtype == SLIM_BF16) {
    if (dst_h) head_scale_kernel<<<H, 256>>>(X, hscale, d, d_k, H * d_k);
    store_wkv_kernel<__nv_bfloat16><<<(unsigned)((nn + 255) / 256), 256>>>(X, (__nv_bfloat16*)dst, (__half*)dst_h, hscale, d, H, d_k);
  } else {
    store_wkv_kernel<float><<<(unsigned)((nn + 255) / 256), 256>>>(X, (float*)dst, nullptr, nullptr, d, H, d_k);
  }
  return cudaGetLastError();
}

cudaError_t slim_dgemm(const double* A, const double* B, double* C, int M, int N, int K, int ta, int tb) {
  dim3 g((N + 63) / 64, (M + 63) / 64);
  dgemm_kernel<<<g, 256>>>(A, B, C, M, N, K, ta, tb);
  return cudaGetLastError();
}

cudaError_t slim_absdiff_max(const double* A, const double* B, size_t n, double* res_host) {
  double* out = nullptr;
  cudaError_t e = cudaMalloc(&out, sizeof(double));
  if (e != cudaSuccess) return e;
  cudaMemset(out, 0, sizeof(double));
  absdiff_max_kernel<<<256, 256>>>(A, B, n, out);
  e = cudaMemcpy(res_host, out, sizeof(double), cudaMemcpyDeviceToHost);
  cudaFree(out);
  return e;
}
