// C-ABI entry points of libslim (argument checks, ownership, launch order).
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "slim_internal.h"

size_t slim_tail_opart_floats(int d, int e, int batch);

// Built-in scratch for slim_decode_static_ws: device memory that exists from the moment
// the library is loaded on a GPU until the process exits, so that entry point never has
// to ask an allocator for anything.  In host code this name is only a handle for
// cudaGetSymbolAddress; the real device address is looked up once per device below.
#define SLIM_STATIC_WS_BYTES (16u << 20)
static __device__ __align__(256) unsigned char slim_static_ws[SLIM_STATIC_WS_BYTES];

namespace {

inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }
inline size_t esize(int dtype) { return dtype == SLIM_BF16 ? 2 : 4; }

struct WsLayout {
  size_t part_u, part_m, part_l, flags, o_part, scores, u_tiled, u32, su, kscratch, total;
  int units;
};

WsLayout ws_layout(const slim_ctx* ctx, int batch, int t_cap) {
  WsLayout L;
  L.units = ctx->num_sms + batch;
  size_t off = 0;
  L.part_u = off; off = align256(off + sizeof(float) * (size_t)L.units * ctx->H * ctx->d);
  L.part_m = off; off = align256(off + sizeof(float) * (size_t)L.units * ctx->H);
  L.part_l = off; off = align256(off + sizeof(float) * (size_t)L.units * ctx->H);
  L.flags = off;  off = align256(off + sizeof(int) * 2 * (size_t)L.units);
  L.o_part = off; off = align256(off + sizeof(float) * slim_tail_opart_floats(ctx->d, ctx->e, batch));
  L.scores = off; off = align256(off + sizeof(float) * (size_t)batch * ctx->H * t_cap);   // generic path only
  L.u_tiled = off; off = align256(off + (ctx->proj_ok ? slim_proj_u_bytes(ctx->d, ctx->H, batch) : 0));   // tensor-core tail only
  L.u32 = off; off = align256(off + (ctx->proj_ok ? sizeof(float) * (size_t)batch * ctx->H * ctx->d : 0));
  L.su = off; off = align256(off + (ctx->proj_ok ? sizeof(float) * (size_t)((batch + 15) / 16) * 16 * ctx->H : 0));
  // 8-bit cache on the tensor-core path: one layer's keys as bf16 (the cache itself stays in 8 bits)
  L.kscratch = off; off = align256(off + ((ctx->kdtype == SLIM_FP8 && ctx->tc_ok) ? 2 * (size_t)batch * t_cap * ctx->d : 0));
  L.total = off;
  return L;
}

int path_in_use(const slim_ctx* ctx) {
  if (ctx->path_req == SLIM_PATH_GENERIC) return SLIM_PATH_GENERIC;
  if (ctx->path_req == SLIM_PATH_TC) return ctx->tc_ok ? SLIM_PATH_TC : -1;
  return ctx->tc_ok ? SLIM_PATH_TC : SLIM_PATH_GENERIC;
}

int min_tiles_for(const slim_ctx* ctx) {
  int v = ctx->H / (2 * (int)esize(ctx->dtype));
  return v < 2 ? 2 : v;
}

slim_status grow_rope_base(slim_ctx* ctx, int t_cap) {
  if (ctx->rope_theta == 0.0) return SLIM_OK;
  const int tiles = (t_cap + SLIM_TT - 1) / SLIM_TT + 1;
  if (tiles <= ctx->rope_base_tiles) return SLIM_OK;
  const int half = ctx->d_k / 2;
  std::vector<float2> tab((size_t)tiles * half);
  for (int j = 0; j < half; ++j) {
    const double th = std::pow(ctx->rope_theta, -2.0 * j / ctx->d_k);
    for (int t = 0; t < tiles; ++t) {
      const double a = (double)t * SLIM_TT * th;
      tab[(size_t)t * half + j] = make_float2((float)std::cos(a), (float)std::sin(a));
    }
  }
  float2* dev = nullptr;
  if (cudaMalloc(&dev, sizeof(float2) * tab.size()) != cudaSuccess) return SLIM_ERR_OOM;
  if (cudaMemcpy(dev, tab.data(), sizeof(float2) * tab.size(), cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaFree(dev);
    return SLIM_ERR_CUDA;
  }
  // the old table may still be referenced by enqueued work
  cudaDeviceSynchronize();
  cudaFree(ctx->rope_base);
  ctx->rope_base = dev;
  ctx->rope_base_tiles = tiles;
  return SLIM_OK;
}

slim_status upload_f64(const void* src, int host_dtype, size_t n, double** dev_out) {
  std::vector<double> tmp;
  const double* h = nullptr;
  if (host_dtype == SLIM_HOST_F64) {
    h = static_cast<const double*>(src);
  } else {
    tmp.resize(n);
    const float* f = static_cast<const float*>(src);
    for (size_t i = 0; i < n; ++i) tmp[i] = (double)f[i];
    h = tmp.data();
  }
  double* dev = nullptr;
  if (cudaMalloc(&dev, sizeof(double) * n) != cudaSuccess) return SLIM_ERR_OOM;
  if (cudaMemcpy(dev, h, sizeof(double) * n, cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaFree(dev);
    return SLIM_ERR_CUDA;
  }
  *dev_out = dev;
  return SLIM_OK;
}

// Device address of slim_static_ws on `device` (which must be the current device).
// Looked up on the first call per device and remembered.
constexpr int kMaxDevices = 64;
void* g_static_ws_ptr[kMaxDevices] = {};
std::mutex g_static_ws_mutex;

slim_status static_ws_address(int device, void** out) {
  if (device < 0 || device >= kMaxDevices) return SLIM_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_ws_mutex);
  if (!g_static_ws_ptr[device]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, slim_static_ws) != cudaSuccess || !ptr) {
      cudaGetLastError();
      return SLIM_ERR_CUDA;
    }
    g_static_ws_ptr[device] = ptr;
  }
  *out = g_static_ws_ptr[device];
  return SLIM_OK;
}

}  // namespace

extern "C" {

const char* slim_strerror(int status) {
  switch (status) {
    case SLIM_OK: return "ok";
    case SLIM_ERR_INVALID_ARG: return "invalid argument";
    case SLIM_ERR_UNSUPPORTED: return "unsupported shape or option";
    case SLIM_ERR_SINGULAR: return "W_K is singular to working precision";
    case SLIM_ERR_CAPACITY: return "K-cache capacity exceeded";
    case SLIM_ERR_OOM: return "out of device memory";
    case SLIM_ERR_CUDA: return "CUDA error or no CUDA device";
    case SLIM_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case SLIM_ERR_NO_WEIGHTS: return "W_KV has not been set";
    case SLIM_ERR_STATIC_WS: return "this batch / capacity needs more scratch than the built-in static workspace holds";
    default: return "unknown status";
  }
}

namespace {
// d: width of a cache row.  For the K-cache scheme d == H * d_k (square projections); an X-cache
// context may have d != e = H * d_k (xcache_only).
slim_status create_impl(slim_ctx** out, int d, int H, int d_k, double rope_theta, int dtype, bool xcache_only);
}

slim_status slim_create(slim_ctx** out, int d, int H, int d_k, double rope_theta, int dtype) {
  return create_impl(out, d, H, d_k, rope_theta, dtype, false);
}

slim_status slim_xcache_create(slim_ctx** out, int d_model, int H, int d_k, int dtype) {
  return create_impl(out, d_model, H, d_k, 0.0, dtype, true);
}

namespace {
slim_status create_impl(slim_ctx** out, int d, int H, int d_k, double rope_theta, int dtype, bool xcache_only) {
  if (!out) return SLIM_ERR_INVALID_ARG;
  *out = nullptr;
  if (d <= 0 || H <= 0 || d_k <= 0 || !(rope_theta >= 0.0) || (dtype != SLIM_F32 && dtype != SLIM_BF16 && dtype != SLIM_FP8))
    return SLIM_ERR_INVALID_ARG;
  const int kdtype = dtype;
  if (dtype == SLIM_FP8) dtype = SLIM_BF16;            // 8-bit cache; queries, new rows and W_KV are bf16
  if ((long long)H * d_k != d && !xcache_only) return SLIM_ERR_UNSUPPORTED;       // Eq. 6 needs a square W_K
  if (xcache_only && dtype == SLIM_FP8) return SLIM_ERR_UNSUPPORTED;
  if (H > SLIM_MAX_H || d_k > 256 || (d_k % 2) != 0 || d > 16384 || (long long)H * d_k > 16384) return SLIM_ERR_UNSUPPORTED;      // rotation pairs need an even width
  const int e = H * d_k;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SLIM_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return SLIM_ERR_CUDA;
  slim_ctx* c = new (std::nothrow) slim_ctx();
  if (!c) return SLIM_ERR_OOM;
  std::memset(c, 0, sizeof(*c));
  c->d = d; c->e = e; c->H = H; c->d_k = d_k; c->dtype = dtype; c->kdtype = kdtype; c->rope_theta = rope_theta;
  c->device = dev; c->num_sms = prop.multiProcessorCount;
  c->path_req = SLIM_PATH_AUTO;
  {
    // tuning switches for sweeps and tests: the environment is read here, once per context, never on
    // the decode path
    const char* e;
    c->opt_tc_sets1 = ((e = getenv("SLIM_TC_SETS")) && atoi(e) == 1) ? 1 : 0;
    c->opt_tc_rt = (e = getenv("SLIM_TC_RT")) ? atoi(e) : 0;
    c->opt_unit_cost = ((e = getenv("SLIM_TC_UNIT_COST")) && atoi(e) >= 0 && atoi(e) <= 64) ? atoi(e) : -1;
    c->opt_xscores_cuda = getenv("SLIM_XSCORES_CUDA") ? 1 : 0;
    c->opt_legacy_flow = getenv("SLIM_TC_LEGACY") ? 1 : 0;
    c->opt_proj_ns = (e = getenv("SLIM_PROJ_NS")) ? atoi(e) : 0;
    c->opt_tail_fused = (e = getenv("SLIM_TAIL_FUSED")) ? atoi(e) : 1;
    c->opt_prompt_pair = ((e = getenv("SLIM_PROMPT_PAIR")) && atoi(e) == 0) ? 0 : 1;
    c->opt_k_evict = (e = getenv("SLIM_TC_K_EVICT")) ? atoi(e) : 1;      // measured side by side: ~1 % per step
  }
  if (cudaMalloc(&c->status, sizeof(int)) != cudaSuccess) { delete c; return SLIM_ERR_OOM; }
  cudaMemset(c->status, 0, sizeof(int));
  if (cudaMalloc(&c->any_flag, sizeof(int)) != cudaSuccess) { slim_destroy(c); return SLIM_ERR_OOM; }
  cudaMemset(c->any_flag, 0, sizeof(int));
  if (cudaMalloc(&c->wkv, esize(dtype) * (size_t)d * e + 256) != cudaSuccess) { slim_destroy(c); return SLIM_ERR_OOM; }
  if (dtype == SLIM_BF16) {
    if (cudaMalloc(&c->wkv_h, 2 * (size_t)d * e + 256) != cudaSuccess) { slim_destroy(c); return SLIM_ERR_OOM; }
    cudaMemset(c->wkv_h, 0, 2 * (size_t)d * e + 256);
    if (cudaMalloc(&c->wkv_hscale, sizeof(float) * SLIM_MAX_H) != cudaSuccess) { slim_destroy(c); return SLIM_ERR_OOM; }
    cudaMemset(c->wkv_hscale, 0, sizeof(float) * SLIM_MAX_H);
  }
  if (rope_theta != 0.0) {
    const int half = d_k / 2;
    std::vector<float2> off((size_t)SLIM_TT * half);
    for (int j = 0; j < half; ++j) {
      const double th = std::pow(rope_theta, -2.0 * j / d_k);
      for (int i = 0; i < SLIM_TT; ++i)
        off[(size_t)i * half + j] = make_float2((float)std::cos(i * th), (float)std::sin(i * th));
    }
    if (cudaMalloc(&c->rope_off, sizeof(float2) * off.size()) != cudaSuccess) { slim_destroy(c); return SLIM_ERR_OOM; }
    if (cudaMemcpy(c->rope_off, off.data(), sizeof(float2) * off.size(), cudaMemcpyHostToDevice) != cudaSuccess) {
      slim_destroy(c);
      return SLIM_ERR_CUDA;
    }
  }
  cudaMemset(c->wkv, 0, esize(dtype) * (size_t)d * e + 256);
  c->proj_ok = prop.major == 10 ? slim_proj_shape_ok(d, H, d_k, dtype) : 0;
  if (c->proj_ok && slim_proj_make_wmap(c) != cudaSuccess) { cudaGetLastError(); c->proj_ok = 0; }
  {
    const char* e = getenv("SLIM_TAIL");                 // "cuda" forces the CUDA-core tail (sweeps, tests)
    if (e && !strcmp(e, "cuda")) c->proj_ok = 0;
  }
  c->tc_ok = 0;
  for (int cl = 1; cl <= 2; ++cl) {
    c->tc_workers[cl - 1] = (prop.major == 10 && slim_tc_shape_ok(d, H, d_k, dtype, rope_theta != 0.0, cl)) ? slim_tc_workers(c, cl) : 0;
    if (c->tc_workers[cl - 1] < 0) c->tc_workers[cl - 1] = 0;
    if (c->tc_workers[cl - 1] > 0) c->tc_ok = 1;
  }
  c->gen_workers = slim_generic_workers(c);
  *out = c;
  return SLIM_OK;
}
}  // namespace

void slim_destroy(slim_ctx* ctx) {
  if (!ctx) return;
  cudaFree(ctx->wkv);
  cudaFree(ctx->wkv_h);
  cudaFree(ctx->wkv_hscale);
  cudaFree(ctx->rope_off);
  cudaFree(ctx->rope_base);
  cudaFree(ctx->status);
  cudaFree(ctx->any_flag);
  cudaFree(ctx->xc_wk);
  for (int i = 0; i < 3; ++i)
    if (ctx->prof_ev[i]) cudaEventDestroy(ctx->prof_ev[i]);
  delete ctx;
}

slim_status slim_set_weights(slim_ctx* ctx, const void* W_K, const void* W_V, int host_dtype,
                             double* wkv_out, double* residual_out) {
  if (!ctx || !W_K || !W_V || (host_dtype != SLIM_HOST_F32 && host_dtype != SLIM_HOST_F64))
    return SLIM_ERR_INVALID_ARG;
  if (ctx->e != ctx->d) return SLIM_ERR_UNSUPPORTED;              // an X-cache context with non-square projections
  const int n = ctx->d;
  const size_t nn = (size_t)n * n;
  double *A = nullptr, *B = nullptr, *A0 = nullptr, *B0 = nullptr;
  slim_status st = upload_f64(W_K, host_dtype, nn, &A);
  if (st == SLIM_OK) st = upload_f64(W_V, host_dtype, nn, &B);
  if (st == SLIM_OK && residual_out) {
    if (cudaMalloc(&A0, sizeof(double) * nn) != cudaSuccess || cudaMalloc(&B0, sizeof(double) * nn) != cudaSuccess)
      st = SLIM_ERR_OOM;
    else if (cudaMemcpy(A0, A, sizeof(double) * nn, cudaMemcpyDeviceToDevice) != cudaSuccess ||
             cudaMemcpy(B0, B, sizeof(double) * nn, cudaMemcpyDeviceToDevice) != cudaSuccess)
      st = SLIM_ERR_CUDA;
  }
  int info = 0;
  if (st == SLIM_OK) {
    cudaError_t e = slim_wkv_solve(A, B, n, &info);
    if (e == cudaErrorMemoryAllocation) st = SLIM_ERR_OOM;
    else if (e != cudaSuccess) st = SLIM_ERR_CUDA;
    else if (info != 0) st = SLIM_ERR_SINGULAR;
  }
  if (st == SLIM_OK && residual_out) {
    if (slim_wkv_residual(A0, B, B0, n, residual_out) != cudaSuccess) st = SLIM_ERR_CUDA;
  }
  if (st == SLIM_OK && wkv_out) {
    if (cudaMemcpy(wkv_out, B, sizeof(double) * nn, cudaMemcpyDeviceToHost) != cudaSuccess) st = SLIM_ERR_CUDA;
  }
  if (st == SLIM_OK) {
    if (slim_wkv_store(B, ctx->d, ctx->H, ctx->d_k, ctx->dtype, ctx->wkv, ctx->wkv_h, ctx->wkv_hscale) != cudaSuccess ||
        cudaDeviceSynchronize() != cudaSuccess)
      st = SLIM_ERR_CUDA;
    else
      ctx->has_weights = 1;
  }
  cudaFree(A); cudaFree(B); cudaFree(A0); cudaFree(B0);
  if (st != SLIM_OK) cudaGetLastError();
  return st;
}

slim_status slim_set_weights_nonsquare(slim_ctx* ctx, const void* W_K, const void* W_V, int d_model, int host_dtype,
                                       double* wkv_out, double* residual_out) {
  if (!ctx || !W_K || !W_V || (host_dtype != SLIM_HOST_F32 && host_dtype != SLIM_HOST_F64)) return SLIM_ERR_INVALID_ARG;
  if (ctx->e != ctx->d) return SLIM_ERR_UNSUPPORTED;
  const int e = ctx->d;                                  // width of K and V: e = H d_k
  if (d_model <= 0 || d_model > e) return SLIM_ERR_INVALID_ARG;
  const size_t de = (size_t)d_model * e, ee = (size_t)e * e, dd = (size_t)d_model * d_model;
  double *Wk = nullptr, *Wv = nullptr, *G = nullptr, *Y = nullptr, *X = nullptr, *R = nullptr;
  slim_status st = upload_f64(W_K, host_dtype, de, &Wk);
  if (st == SLIM_OK) st = upload_f64(W_V, host_dtype, de, &Wv);
  if (st == SLIM_OK && (cudaMalloc(&G, sizeof(double) * dd) != cudaSuccess || cudaMalloc(&Y, sizeof(double) * de) != cudaSuccess ||
                        cudaMalloc(&X, sizeof(double) * ee) != cudaSuccess))
    st = SLIM_ERR_OOM;
  int info = 0;
  if (st == SLIM_OK) {
    // right inverse: W_K^{-1} = W_K^T (W_K W_K^T)^{-1};  W_KV = W_K^{-1} W_V = W_K^T [ (W_K W_K^T)^{-1} W_V ]
    cudaError_t ce = slim_dgemm(Wk, Wk, G, d_model, d_model, e, 0, 1);                       // G = W_K W_K^T
    if (ce == cudaSuccess) ce = cudaMemcpy(Y, Wv, sizeof(double) * de, cudaMemcpyDeviceToDevice);
    if (ce == cudaSuccess) ce = slim_wkv_solve_rhs(G, Y, d_model, e, &info);                  // G Y = W_V
    if (ce == cudaSuccess && info == 0) ce = slim_dgemm(Wk, Y, X, e, e, d_model, 1, 0);       // W_KV = W_K^T Y
    if (ce == cudaErrorMemoryAllocation) st = SLIM_ERR_OOM;
    else if (ce != cudaSuccess) st = SLIM_ERR_CUDA;
    else if (info != 0) st = SLIM_ERR_SINGULAR;
  }
  if (st == SLIM_OK && residual_out) {                   // max | W_K W_KV - W_V |
    if (cudaMalloc(&R, sizeof(double) * de) != cudaSuccess) st = SLIM_ERR_OOM;
    else if (slim_dgemm(Wk, X, R, d_model, e, e, 0, 0) != cudaSuccess || slim_absdiff_max(R, Wv, de, residual_out) != cudaSuccess)
      st = SLIM_ERR_CUDA;
  }
  if (st == SLIM_OK && wkv_out && cudaMemcpy(wkv_out, X, sizeof(double) * ee, cudaMemcpyDeviceToHost) != cudaSuccess) st = SLIM_ERR_CUDA;
  if (st == SLIM_OK) {
    if (slim_wkv_store(X, ctx->d, ctx->H, ctx->d_k, ctx->dtype, ctx->wkv, ctx->wkv_h, ctx->wkv_hscale) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess)
      st = SLIM_ERR_CUDA;
    else
      ctx->has_weights = 1;
  }
  cudaFree(Wk); cudaFree(Wv); cudaFree(G); cudaFree(Y); cudaFree(X); cudaFree(R);
  if (st != SLIM_OK) cudaGetLastError();
  return st;
}

slim_status slim_xcache_set_weights(slim_ctx* ctx, const void* W_K, const void* W_V, int host_dtype) {
  if (!ctx || !W_K || !W_V || (host_dtype != SLIM_HOST_F32 && host_dtype != SLIM_HOST_F64)) return SLIM_ERR_INVALID_ARG;
  if (ctx->rope_theta != 0.0) return SLIM_ERR_UNSUPPORTED;          // the scheme has no place for RoPE
  if (ctx->kdtype == SLIM_FP8) return SLIM_ERR_UNSUPPORTED;
  const size_t nn = (size_t)ctx->d * ctx->e;              // W_K, W_V: [d][e]
  std::vector<float> wk(nn);
  if (host_dtype == SLIM_HOST_F64) { const double* s = static_cast<const double*>(W_K); for (size_t i = 0; i < nn; ++i) wk[i] = (float)s[i]; }
  else std::memcpy(wk.data(), W_K, sizeof(float) * nn);
  if (!ctx->xc_wk && cudaMalloc(&ctx->xc_wk, sizeof(float) * nn) != cudaSuccess) { ctx->xc_wk = nullptr; cudaGetLastError(); return SLIM_ERR_OOM; }
  if (cudaMemcpy(ctx->xc_wk, wk.data(), sizeof(float) * nn, cudaMemcpyHostToDevice) != cudaSuccess) return SLIM_ERR_CUDA;
  return slim_set_wkv(ctx, W_V, host_dtype);                        // the projection uses W_V,i in place of W_KV,i
}

size_t slim_xcache_workspace_bytes(const slim_ctx* ctx, int batch, int t_cap) {
  const size_t base = slim_workspace_bytes(ctx, batch, t_cap);
  return base ? base + align256(sizeof(float) * (size_t)batch * ctx->H * ctx->d) + align256(slim_xscores_qt_bytes(ctx->d, batch)) : 0;
}

slim_status slim_set_wkv(slim_ctx* ctx, const void* W_KV, int host_dtype) {
  if (!ctx || !W_KV || (host_dtype != SLIM_HOST_F32 && host_dtype != SLIM_HOST_F64)) return SLIM_ERR_INVALID_ARG;
  double* X = nullptr;
  slim_status st = upload_f64(W_KV, host_dtype, (size_t)ctx->d * ctx->e, &X);
  if (st != SLIM_OK) return st;
  if (slim_wkv_store(X, ctx->d, ctx->H, ctx->d_k, ctx->dtype, ctx->wkv, ctx->wkv_h, ctx->wkv_hscale) != cudaSuccess ||
      cudaDeviceSynchronize() != cudaSuccess)
    st = SLIM_ERR_CUDA;
  else
    ctx->has_weights = 1;
  cudaFree(X);
  return st;
}

size_t slim_cache_bytes(const slim_ctx* ctx, int batch, int t_cap) {
  if (!ctx || batch <= 0 || t_cap <= 0) return 0;
  if (ctx->kdtype == SLIM_FP8)                             // codes, then one exponent per (row, head)
    return ((((size_t)batch * t_cap * ctx->d) + 15) & ~(size_t)15) + (size_t)batch * t_cap * ctx->H;
  return esize(ctx->dtype) * (size_t)batch * t_cap * ctx->d;
}

size_t slim_workspace_bytes(const slim_ctx* ctx, int batch, int t_cap) {
  if (!ctx || batch <= 0 || t_cap <= 0 || batch > SLIM_MAX_BATCH) return 0;
  return ws_layout(ctx, batch, t_cap).total;
}

slim_status slim_cache_create(slim_ctx* ctx, slim_cache** out, void* k_storage, int batch, int t_cap) {
  if (!out) return SLIM_ERR_INVALID_ARG;
  *out = nullptr;
  if (!ctx || !k_storage || batch <= 0 || t_cap <= 0) return SLIM_ERR_INVALID_ARG;
  if (batch > SLIM_MAX_BATCH || ((uintptr_t)k_storage & 15)) return SLIM_ERR_UNSUPPORTED;
  if ((long long)batch * t_cap > 0x7fffffffLL - 64) return SLIM_ERR_UNSUPPORTED;
  slim_status st = grow_rope_base(ctx, t_cap);
  if (st != SLIM_OK) return st;
  slim_cache* c = new (std::nothrow) slim_cache();
  if (!c) return SLIM_ERR_OOM;
  c->ctx = ctx; c->k = k_storage; c->batch = batch; c->t_cap = t_cap;
  c->k_exp = ctx->kdtype == SLIM_FP8
                 ? reinterpret_cast<signed char*>(k_storage) + ((((size_t)batch * t_cap * ctx->d) + 15) & ~(size_t)15) : nullptr;
  c->block_table = nullptr; c->page_rows = 0; c->max_pages = 0; c->num_pages = 0;
  c->total_rows = (long long)batch * t_cap;
  for (int cl = 1; cl <= 2; ++cl) {
    c->has_tmap[cl - 1] = 0;
    if (ctx->tc_workers[cl - 1] > 0 && ctx->kdtype != SLIM_FP8) {       // (an 8-bit cache is read through a bf16 scratch)
      if (slim_tc_make_tmap(ctx, c, cl) == cudaSuccess) c->has_tmap[cl - 1] = 1;
      else cudaGetLastError();
    }
  }
  c->has_xmap = 0;
  if (ctx->proj_ok && ctx->kdtype != SLIM_FP8 && slim_xscores_tc_ok(ctx)) {
    if (slim_xscores_make_tmap(ctx, c) == cudaSuccess) c->has_xmap = 1;
    else cudaGetLastError();
  }
  *out = c;
  return SLIM_OK;
}

slim_status slim_cache_create_paged(slim_ctx* ctx, slim_cache** out, void* pool, int num_pages, int page_rows,
                                    const int32_t* block_table, int batch, int max_pages) {
  if (!out) return SLIM_ERR_INVALID_ARG;
  *out = nullptr;
  if (!ctx || !pool || !block_table || num_pages <= 0 || page_rows <= 0 || batch <= 0 || max_pages <= 0) return SLIM_ERR_INVALID_ARG;
  if (page_rows % SLIM_TT != 0 || batch > SLIM_MAX_BATCH || ((uintptr_t)pool & 15)) return SLIM_ERR_UNSUPPORTED;
  if (ctx->kdtype == SLIM_FP8) return SLIM_ERR_UNSUPPORTED;
  if ((long long)num_pages * page_rows > 0x7fffffffLL - 64 || (long long)batch * max_pages * page_rows > 0x7fffffffLL - 64)
    return SLIM_ERR_UNSUPPORTED;
  const int t_cap = max_pages * page_rows;
  slim_status st = grow_rope_base(ctx, t_cap);
  if (st != SLIM_OK) return st;
  slim_cache* c = new (std::nothrow) slim_cache();
  if (!c) return SLIM_ERR_OOM;
  c->ctx = ctx; c->k = pool; c->k_exp = nullptr; c->batch = batch; c->t_cap = t_cap;
  c->block_table = block_table; c->page_rows = page_rows; c->max_pages = max_pages; c->num_pages = num_pages;
  c->total_rows = (long long)num_pages * page_rows;
  for (int cl = 1; cl <= 2; ++cl) {
    c->has_tmap[cl - 1] = 0;
    if (ctx->tc_workers[cl - 1] > 0) {
      if (slim_tc_make_tmap(ctx, c, cl) == cudaSuccess) c->has_tmap[cl - 1] = 1;
      else cudaGetLastError();
    }
  }
  c->has_xmap = 0;                                     // the X-cache scheme takes contiguous caches only
  *out = c;
  return SLIM_OK;
}

void slim_cache_destroy(slim_cache* cache) { delete cache; }

slim_status slim_append_k(slim_ctx* ctx, slim_cache* cache, const void* k_new, const int32_t* positions,
                          int n_new, void* stream) {
  if (!ctx || !cache || !k_new || !positions || cache->ctx != ctx) return SLIM_ERR_INVALID_ARG;
  if (n_new <= 0 || n_new > 65535) return SLIM_ERR_INVALID_ARG;
  if (n_new > cache->t_cap) return SLIM_ERR_CAPACITY;
  if (slim_launch_append(ctx, cache, k_new, positions, n_new, 0, (cudaStream_t)stream) != cudaSuccess)
    return SLIM_ERR_CUDA;
  return SLIM_OK;
}

namespace {
// What a context-split rank asks for instead of the projected output: the slice's (lse, u) per (sequence, head).
struct PartialOut {
  const int32_t* first_tile;     // device [batch]: absolute tile of the cache's first row
  const int32_t* q_pos;          // device [batch]: absolute position of the query
  float* lse;                    // device [batch][H]
  float* u;                      // device [batch][H][d]
};

// k_new != NULL: the generate-phase step (newest key rows written at lengths[b] - 1 first)
slim_status decode_impl(slim_ctx* ctx, const void* q, const slim_cache* cache, const int32_t* lengths, float* o,
                        void* workspace, void* stream, bool xcache, const void* k_new = nullptr, const PartialOut* part = nullptr) {
  if (!ctx || !q || !cache || !lengths || (!o && !part) || !workspace || cache->ctx != ctx) return SLIM_ERR_INVALID_ARG;
  if (((uintptr_t)workspace & 255) || ((uintptr_t)q & 15) || ((uintptr_t)o & 15)) return SLIM_ERR_INVALID_ARG;
  if (!ctx->has_weights) return SLIM_ERR_NO_WEIGHTS;
  int path = path_in_use(ctx);
  if (xcache && !ctx->xc_wk) return SLIM_ERR_NO_WEIGHTS;
  if (!xcache && ctx->e != ctx->d) return SLIM_ERR_UNSUPPORTED;   // the K-cache scheme needs square projections
  if (xcache && cache->block_table) return SLIM_ERR_UNSUPPORTED;
  if (path < 0) return SLIM_ERR_UNSUPPORTED;
  // CTAs per worker: the pair when the kernel computes the scores, the lone CTA with external scores
  int cl = 0;
  const bool fp8_tc = path == SLIM_PATH_TC && ctx->kdtype == SLIM_FP8;      // decoded into a bf16 scratch first
  if (path == SLIM_PATH_TC) {
    const int pref = xcache ? 1 : 2, other = 3 - pref;
    if (ctx->tc_workers[pref - 1] > 0 && (fp8_tc || cache->has_tmap[pref - 1])) cl = pref;
    else if (ctx->tc_workers[other - 1] > 0 && (fp8_tc || cache->has_tmap[other - 1])) cl = other;
  }
  if (path == SLIM_PATH_TC && cl == 0) {
    if (ctx->path_req == SLIM_PATH_TC) return SLIM_ERR_UNSUPPORTED;
    path = SLIM_PATH_GENERIC;
  }
  const WsLayout L = ws_layout(ctx, cache->batch, cache->t_cap);
  char* ws = static_cast<char*>(workspace);
  SlimDecodeParams p;
  p.d = ctx->d; p.e = ctx->e; p.H = ctx->H; p.d_k = ctx->d_k; p.half = ctx->d_k / 2;
  p.batch = cache->batch; p.t_cap = cache->t_cap;
  p.rope = ctx->rope_theta != 0.0; p.dtype = ctx->dtype; p.kdtype = ctx->kdtype; p.k_exp = cache->k_exp;
  p.workers = path == SLIM_PATH_TC ? ctx->tc_workers[cl - 1] : ctx->gen_workers;
  p.cl = cl;
  p.min_tiles = min_tiles_for(ctx);
  // measured: closing a unit (accumulator drain + pipeline restart) costs a worker about H/4 + 4 tiles
  p.unit_cost = path == SLIM_PATH_TC ? (ctx->H + 3) / 4 + 4 : 0;
  if (path == SLIM_PATH_TC && ctx->opt_unit_cost >= 0) p.unit_cost = ctx->opt_unit_cost;      // override for sweeps
  p.qscale = (float)(1.4426950408889634 / std::sqrt((double)ctx->d_k));
  p.q = q; p.k = cache->k; p.lengths = lengths;
  p.rope_base = ctx->rope_base; p.rope_off = ctx->rope_off; p.wkv = ctx->wkv;
  p.part_u = reinterpret_cast<float*>(ws + L.part_u);
  p.part_m = reinterpret_cast<float*>(ws + L.part_m);
  p.part_l = reinterpret_cast<float*>(ws + L.part_l);
  p.unit_flags = reinterpret_cast<int*>(ws + L.flags);
  p.u = reinterpret_cast<float*>(ws + L.o_part);
  p.o = o; p.status = ctx->status; p.any_flag = ctx->any_flag;
  p.ext_scores = nullptr;
  p.block_table = cache->block_table; p.page_rows = cache->page_rows; p.max_pages = cache->max_pages;
  p.num_pages = cache->num_pages;
  // K-cache path on the tensor cores: the decode kernel writes the newest key rows itself, and a sequence
  // with a flagged unit is recomputed by the combine kernel (no append kernel, no redo kernel)
  const bool tc_kcache = !xcache && path == SLIM_PATH_TC && !ctx->opt_legacy_flow;
  p.k_new = (tc_kcache && !fp8_tc) ? k_new : nullptr;        // (new rows of an 8-bit cache go through the quantising append)
  p.redo_in_combine = (tc_kcache && ctx->proj_ok && !part) ? 1 : 0;
  p.pos_tiles = part ? part->first_tile : nullptr;
  p.q_pos = part ? part->q_pos : nullptr;
  p.rope_tiles = ctx->rope_base_tiles;
  p.k_evict_first = ctx->opt_k_evict;
  p.trace = ctx->trace;
  cudaStream_t st = (cudaStream_t)stream;
  int launches = 0;
  if (k_new && !p.k_new) {                           // no fused update on this path: the append kernel first
    if (slim_launch_append(ctx, cache, k_new, lengths, 1, 1, st) != cudaSuccess) { cudaGetLastError(); return SLIM_ERR_CUDA; }
    ++launches;
  }
  if (ctx->prof_on) cudaEventRecord(ctx->prof_ev[0], st);
  cudaError_t e;
  slim_cache view;                                   // what the tensor-core kernel reads when the cache is 8-bit
  const slim_cache* tc_cache = cache;
  if (fp8_tc) {
    // 8-bit cache on the tensor cores: decode the live rows into the bf16 scratch of the workspace and run the
    // bf16 kernels on that (contiguous) copy; codes x 2^exponent are exact in bf16, so the result is the one
    // the CUDA-core kernels get from the codes, up to the rounding of P
    void* scratch = ws + L.kscratch;
    if (slim_launch_dequant(ctx, cache, lengths, scratch, st) != cudaSuccess) { cudaGetLastError(); return SLIM_ERR_CUDA; }
    ++launches;
    view = *cache;
    view.k = scratch; view.k_exp = nullptr; view.block_table = nullptr;
    view.total_rows = (long long)cache->batch * cache->t_cap;
    view.has_tmap[0] = view.has_tmap[1] = 0;
    if (slim_tc_make_tmap(ctx, &view, cl) != cudaSuccess) { cudaGetLastError(); return SLIM_ERR_CUDA; }
    view.has_tmap[cl - 1] = 1;
    tc_cache = &view;
    p.k = scratch; p.kdtype = SLIM_BF16; p.k_exp = nullptr;
  }
  float* scores = reinterpret_cast<float*>(ws + L.scores);
  if (xcache) {
    // dense scores first; then P.X on the tensor cores where the shape allows it (an argument that
    // overflows its reference exponent triggers the CUDA-core accumulation as the exact redo)
    launches += 2;                                   // query transform + dense scores
    if (cache->has_xmap && !ctx->opt_xscores_cuda)
      e = slim_launch_xscores_tc(ctx, cache, p, ctx->xc_wk,
                                 reinterpret_cast<unsigned char*>(ws + L.total + align256(sizeof(float) * (size_t)p.batch * p.H * p.d)), scores, st);
    else
      e = slim_launch_xcache_scores(ctx, p, scores, ctx->xc_wk, reinterpret_cast<float*>(ws + L.total), st);
    if (e == cudaSuccess) {
      if (path == SLIM_PATH_TC) {
        p.ext_scores = scores;
        e = slim_launch_tc(ctx, cache, p, st);
        if (e == cudaSuccess) e = slim_launch_accum(ctx, p, scores, 0, st);
        launches += 2;
      } else {
        e = slim_launch_accum(ctx, p, scores, 1, st);
        launches += 1;
      }
    }
  } else if (path == SLIM_PATH_TC) {
    e = slim_launch_tc(ctx, tc_cache, p, st);
    ++launches;
    if (e == cudaSuccess && !p.redo_in_combine) { e = slim_launch_exact_flagged(ctx, p, st); ++launches; }
  } else {
    e = slim_launch_generic(ctx, p, scores, st);
    launches += 2;                                   // scores, accumulation
  }
  if (ctx->prof_on) cudaEventRecord(ctx->prof_ev[1], st);
  if (e == cudaSuccess && part) {                    // a rank of a split context: (lse, u) of its slice, no projection
    e = slim_launch_partial_out(ctx, p, part->lse, part->u, st);
    ++launches;
  } else if (e == cudaSuccess) {
    if (ctx->proj_ok) {
      e = slim_launch_proj(ctx, p, reinterpret_cast<unsigned char*>(ws + L.u_tiled), reinterpret_cast<float*>(ws + L.u32),
                           reinterpret_cast<float*>(ws + L.su), st);
      launches += slim_proj_launch_count(ctx, p);                 // combine (, operand conversion), projection -- or the fused kernel
    } else {
      e = slim_launch_tail(ctx, p, st);
      launches += 2;                                 // combine + projection slices, slice sum
    }
  }
  ctx->launches_last = launches;
  if (ctx->prof_on) { cudaEventRecord(ctx->prof_ev[2], st); ctx->prof_valid = 1; }
  if (e != cudaSuccess) { cudaGetLastError(); return SLIM_ERR_CUDA; }
  return SLIM_OK;
}
}  // namespace

slim_status slim_decode(slim_ctx* ctx, const void* q, const slim_cache* cache, const int32_t* lengths,
                        float* o, void* workspace, void* stream) {
  return decode_impl(ctx, q, cache, lengths, o, workspace, stream, false);
}

slim_status slim_decode_step(slim_ctx* ctx, const void* q, const void* k_new, slim_cache* cache, const int32_t* lengths,
                             float* o, void* workspace, void* stream) {
  if (!k_new || ((uintptr_t)k_new & 15)) return SLIM_ERR_INVALID_ARG;
  return decode_impl(ctx, q, cache, lengths, o, workspace, stream, false, k_new);
}

slim_status slim_reserve_positions(slim_ctx* ctx, int max_position) {
  if (!ctx || max_position <= 0) return SLIM_ERR_INVALID_ARG;
  return grow_rope_base(ctx, max_position);
}

slim_status slim_decode_partial(slim_ctx* ctx, const void* q, const slim_cache* cache, const int32_t* lengths,
                                const int32_t* first_tile, const int32_t* q_pos, float* lse_out, float* u_out,
                                void* workspace, void* stream) {
  if (!first_tile || !q_pos || !lse_out || !u_out) return SLIM_ERR_INVALID_ARG;
  if (ctx && ctx->kdtype == SLIM_FP8) return SLIM_ERR_UNSUPPORTED;
  const PartialOut part = {first_tile, q_pos, lse_out, u_out};
  return decode_impl(ctx, q, cache, lengths, nullptr, workspace, stream, false, nullptr, &part);
}

slim_status slim_combine_project(slim_ctx* ctx, const float* lse_all, const float* u_all, int ranks, const int32_t* total_lengths,
                                 int batch, float* o, void* workspace, void* stream) {
  if (!ctx || !lse_all || !u_all || !total_lengths || !o || !workspace) return SLIM_ERR_INVALID_ARG;
  if (ranks <= 0 || ranks > 64 || batch <= 0 || batch > SLIM_MAX_BATCH) return SLIM_ERR_INVALID_ARG;
  if (((uintptr_t)workspace & 255) || ((uintptr_t)o & 15)) return SLIM_ERR_INVALID_ARG;
  if (!ctx->has_weights) return SLIM_ERR_NO_WEIGHTS;
  // the joined result is laid down as one finished unit per sequence (worker 0 owns every tile of the
  // schedule below), and the ordinary combine + projection tail completes the step
  const WsLayout L = ws_layout(ctx, batch, SLIM_TT);
  char* ws = static_cast<char*>(workspace);
  SlimDecodeParams p;
  std::memset(&p, 0, sizeof(p));
  p.d = ctx->d; p.e = ctx->e; p.H = ctx->H; p.d_k = ctx->d_k; p.half = ctx->d_k / 2;
  p.batch = batch; p.t_cap = 0x3fffffff;
  p.dtype = ctx->dtype; p.kdtype = ctx->kdtype;
  p.workers = 1; p.cl = 0; p.min_tiles = 1; p.unit_cost = 0;
  p.lengths = total_lengths; p.wkv = ctx->wkv;
  p.part_u = reinterpret_cast<float*>(ws + L.part_u);
  p.part_m = reinterpret_cast<float*>(ws + L.part_m);
  p.part_l = reinterpret_cast<float*>(ws + L.part_l);
  p.unit_flags = reinterpret_cast<int*>(ws + L.flags);
  p.u = reinterpret_cast<float*>(ws + L.o_part);
  p.o = o; p.status = ctx->status; p.any_flag = ctx->any_flag;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = slim_launch_rank_combine(ctx, p, lse_all, u_all, ranks, st);
  if (e == cudaSuccess) {
    if (ctx->proj_ok) e = slim_launch_proj(ctx, p, reinterpret_cast<unsigned char*>(ws + L.u_tiled), reinterpret_cast<float*>(ws + L.u32),
                                           reinterpret_cast<float*>(ws + L.su), st);
    else e = slim_launch_tail(ctx, p, st);
  }
  ctx->launches_last = 1 + (ctx->proj_ok ? slim_proj_launch_count(ctx, p) : 2);      // join, then the tail's kernels
  if (e != cudaSuccess) { cudaGetLastError(); return SLIM_ERR_CUDA; }
  return SLIM_OK;
}

slim_status slim_xcache_decode(slim_ctx* ctx, const void* q, const slim_cache* cache, const int32_t* lengths,
                               float* o, void* workspace, void* stream) {
  return decode_impl(ctx, q, cache, lengths, o, workspace, stream, true);
}

slim_status slim_values_from_keys(slim_ctx* ctx, const void* K, int n, float* V, void* stream) {
  if (!ctx || !K || !V || n <= 0) return SLIM_ERR_INVALID_ARG;
  if (ctx->e != ctx->d) return SLIM_ERR_UNSUPPORTED;
  if (!ctx->has_weights) return SLIM_ERR_NO_WEIGHTS;
  if (slim_launch_values(ctx, K, n, V, (cudaStream_t)stream) != cudaSuccess) { cudaGetLastError(); return SLIM_ERR_CUDA; }
  return SLIM_OK;
}

slim_status slim_prefill(slim_ctx* ctx, slim_cache* cache, const void* k_new, const int32_t* positions, int n_new,
                         float* V, void* stream) {
  if (!ctx || !cache || !k_new || !positions || !V || cache->ctx != ctx) return SLIM_ERR_INVALID_ARG;
  if (n_new <= 0 || n_new > 65535) return SLIM_ERR_INVALID_ARG;
  if (n_new > cache->t_cap) return SLIM_ERR_CAPACITY;
  if ((long long)cache->batch * n_new > 0x7fffffffLL || ctx->e != ctx->d) return SLIM_ERR_UNSUPPORTED;
  if (!ctx->has_weights) return SLIM_ERR_NO_WEIGHTS;
  if (slim_launch_values(ctx, k_new, cache->batch * n_new, V, (cudaStream_t)stream, cache, positions, n_new) != cudaSuccess) {
    cudaGetLastError();
    return SLIM_ERR_CUDA;
  }
  return SLIM_OK;
}

size_t slim_static_workspace_max(void) { return SLIM_STATIC_WS_BYTES; }

slim_status slim_decode_static_ws(slim_ctx* ctx, const void* q, const slim_cache* cache, const int32_t* lengths,
                                  float* o, void* stream) {
  if (!ctx || !q || !cache || !lengths || !o || cache->ctx != ctx) return SLIM_ERR_INVALID_ARG;
  const size_t need = ws_layout(ctx, cache->batch, cache->t_cap).total;
  if (need > (size_t)SLIM_STATIC_WS_BYTES) return SLIM_ERR_STATIC_WS;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return SLIM_ERR_CUDA; }
  if (dev != ctx->device) return SLIM_ERR_INVALID_ARG;          // the ctx's device must be current
  void* ws = nullptr;
  const slim_status st = static_ws_address(dev, &ws);
  if (st != SLIM_OK) return st;
  // Nothing in the scratch has to start at zero: every word that reaches a stored output was
  // written earlier in the same call (partials, redo flags, projection operand tiles).
  return slim_decode(ctx, q, cache, lengths, o, ws, stream);
}

slim_status slim_device_status(slim_ctx* ctx, void* stream) {
  if (!ctx) return SLIM_ERR_INVALID_ARG;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) { cudaGetLastError(); return SLIM_ERR_CUDA; }
  int v = 0;
  if (cudaMemcpy(&v, ctx->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return SLIM_ERR_CUDA;
  if (v != 0) cudaMemset(ctx->status, 0, sizeof(int));
  return (slim_status)v;
}

slim_status slim_selftest_bounded_wait(slim_ctx* ctx, void* stream) {
  if (!ctx) return SLIM_ERR_INVALID_ARG;
  // any_flag doubles as the kernel's "gave up" word; it is 0 between decodes
  cudaStream_t st = (cudaStream_t)stream;
  if (slim_launch_wait_selftest(ctx->status, ctx->any_flag, st) != cudaSuccess) { cudaGetLastError(); return SLIM_ERR_CUDA; }
  if (cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return SLIM_ERR_CUDA; }
  int gave_up = 0;
  if (cudaMemcpy(&gave_up, ctx->any_flag, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return SLIM_ERR_CUDA;
  cudaMemset(ctx->any_flag, 0, sizeof(int));
  return gave_up ? SLIM_OK : SLIM_ERR_CUDA;
}

slim_status slim_profile_enable(slim_ctx* ctx, int enable) {
  if (!ctx) return SLIM_ERR_INVALID_ARG;
  if (enable && !ctx->prof_ev[0]) {
    for (int i = 0; i < 3; ++i)
      if (cudaEventCreate(&ctx->prof_ev[i]) != cudaSuccess) return SLIM_ERR_CUDA;
  }
  ctx->prof_on = enable ? 1 : 0;
  ctx->prof_valid = 0;
  return SLIM_OK;
}

slim_status slim_profile_read(slim_ctx* ctx, float* main_ms, float* tail_ms) {
  if (!ctx || !main_ms || !tail_ms) return SLIM_ERR_INVALID_ARG;
  if (!ctx->prof_on || !ctx->prof_valid) return SLIM_ERR_INVALID_ARG;
  if (cudaEventSynchronize(ctx->prof_ev[2]) != cudaSuccess) return SLIM_ERR_CUDA;
  if (cudaEventElapsedTime(main_ms, ctx->prof_ev[0], ctx->prof_ev[1]) != cudaSuccess ||
      cudaEventElapsedTime(tail_ms, ctx->prof_ev[1], ctx->prof_ev[2]) != cudaSuccess)
    return SLIM_ERR_CUDA;
  return SLIM_OK;
}

slim_status slim_set_trace(slim_ctx* ctx, void* device_buffer) {
  if (!ctx) return SLIM_ERR_INVALID_ARG;
#ifdef SLIM_TC_TRACE
  ctx->trace = static_cast<long long*>(device_buffer);
  return SLIM_OK;
#else
  (void)device_buffer;
  return SLIM_ERR_UNSUPPORTED;                    // this build of the library carries no instrumentation
#endif
}

slim_status slim_set_path(slim_ctx* ctx, int path) {
  if (!ctx || path < SLIM_PATH_AUTO || path > SLIM_PATH_TC) return SLIM_ERR_INVALID_ARG;
  if (path == SLIM_PATH_TC && !ctx->tc_ok) return SLIM_ERR_UNSUPPORTED;
  ctx->path_req = path;
  return SLIM_OK;
}

long long slim_query(const slim_ctx* ctx, int key) {
  if (!ctx) return -1;
  const int path = path_in_use(ctx);
  switch (key) {
    case SLIM_Q_PATH_IN_USE: return path;
    case SLIM_Q_LAUNCHES_PER_DECODE:              // counted by the last decode call of this ctx (0 before the first)
      return ctx->launches_last;
    case SLIM_Q_MAX_UNITS: return ctx->num_sms;   // + batch, known only per cache
    case SLIM_Q_NUM_SMS: return ctx->num_sms;
    case SLIM_Q_WORKERS: return path == SLIM_PATH_TC ? (ctx->tc_workers[1] > 0 ? ctx->tc_workers[1] : ctx->tc_workers[0]) : ctx->gen_workers;
    default: return -1;
  }
}

}  // extern "C"
