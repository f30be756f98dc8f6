// Internal declarations shared by the translation units of libslim.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/slim.h"

// Context tile: every kernel walks the context in tiles of SLIM_TT rows that
// start at absolute positions that are multiples of SLIM_TT.  The RoPE base
// table has one entry per tile and the offset table one per row of a tile.
#define SLIM_TT 16
#define SLIM_MAX_H 64
#define SLIM_MAX_BATCH 2048
#define SLIM_TRACE_TILES 192      // tiles per CTA that a trace build records

// Parameters every decode kernel receives (passed by value).
struct SlimDecodeParams {
  int d, H, d_k, half;           // d: width of a cache row (and of u); half = d_k / 2
  int e;                         // width of q and o: H * d_k (= d except for a non-square X-cache)
  int batch, t_cap;
  int rope;                      // 0 / 1
  int dtype;                     // slim_dtype of q and W_KV (f32 or bf16)
  int kdtype;                    // slim_dtype of the cache elements (f32, bf16 or fp8 codes)
  const signed char* k_exp;      // fp8 cache: [batch][t_cap][H] exponents (stored key = code * 2^exponent), else NULL
  int workers;                   // context-split workers (W)
  int cl;                        // tensor-core path: CTAs per worker (1 or 2)
  int min_tiles;                 // a worker gets at least this many tiles if it gets any
  int unit_cost;                 // tiles of time that closing a unit costs a worker (schedule)
  float qscale;                  // log2(e) / sqrt(d_k)
  const void* q;                 // [batch][d]
  const void* k;                 // [batch][t_cap][d]
  const int32_t* lengths;        // [batch]
  const float2* rope_base;       // [ceil(t_cap/TT)+1][half]  (cos, sin) of TT*tile*theta_j
  const float2* rope_off;        // [TT][half]                (cos, sin) of i*theta_j
  const void* wkv;               // [H][d][d_k] ctx dtype
  float* part_u;                 // [units][H][d]
  float* part_m;                 // [units][H]   reference exponent (log2 domain)
  float* part_l;                 // [units][H]   sum of 2^(s - m)
  int* unit_flags;               // [units][2]   1 = unit must be redone exactly (one word per CTA of the pair)
  float* u;                      // [batch][H][d] combined
  float* o;                      // [batch][d]
  int* status;                   // sticky device status word
  int* any_flag;                 // set to 1 by a kernel that flags a unit
  const float* ext_scores;       // X-cache scheme: precomputed softmax arguments [batch][H][t_cap] (else NULL)
  const int32_t* block_table;    // paged cache: [batch][max_pages] page ids (NULL = contiguous [batch][t_cap][d])
  int page_rows, max_pages, num_pages;
  // a cache that holds a slice of a longer context (context split over several GPUs): its rows start at absolute
  // position SLIM_TT * pos_tiles[b] and the query sits at absolute position q_pos[b] (both NULL otherwise)
  const int32_t* pos_tiles;
  const int32_t* q_pos;
  int k_evict_first;             // tensor-core path: key tiles are loaded with the L2 evict-first hint
  int rope_tiles;                // entries of rope_base (positions < SLIM_TT * rope_tiles are covered)
  long long* trace;              // builds with SLIM_TC_TRACE only: [CTAs][SLIM_TRACE_TILES][8] SM clocks (else NULL, unused)
  const void* k_new;             // tensor-core path: [batch][d] newest key rows, written at row lengths[b]-1 before the read (or NULL)
  int redo_in_combine;           // 1: the combine kernel recomputes the sequences that have a flagged unit (no redo kernel runs)
};

struct slim_ctx {
  int d, H, d_k, dtype;          // d: width of a cache row; dtype: q and W_KV (f32 or bf16)
  int e;                         // width of q and o: H * d_k; differs from d only for an X-cache context with non-square projections
  int kdtype;                    // cache elements: dtype, or SLIM_FP8
  double rope_theta;
  int device;
  int num_sms;
  int path_req;                  // slim_path requested
  int has_weights;
  void* wkv;                     // device [H][d][d_k] ctx dtype
  void* wkv_h;                   // bf16 contexts: device [H][d][d_k] float16, W_KV,h * 2^a_h (head maximum in [2^14, 2^15)): the
                                 // operand of the tensor-core projection (11-bit mantissa instead of bf16's 8)
  float* wkv_hscale;             // device [H]: 2^-a_h
  float2* rope_off;              // device [TT][half]
  float2* rope_base;             // device table, grown by slim_cache_create
  int rope_base_tiles;
  int* status;                   // device status word
  int tc_ok;                     // shape fits the tensor-core path with some cluster size
  int tc_workers[2];             // workers of the tensor-core kernel with 1 / 2 CTAs per worker (0 = not usable)
  int gen_workers;
  int prof_on, prof_valid;
  cudaEvent_t prof_ev[3];
  int proj_ok;                   // tensor-core combine + projection usable for this shape
  float* xc_wk;                  // X-cache scheme: device fp32 W_K [d][d] (NULL until slim_xcache_set_weights)
  int* any_flag;                 // device: 1 while some unit of the current decode is flagged for the exact redo
  int launches_last;             // kernels the last decode call enqueued
  // tuning switches, read from the environment once, by slim_create (sweeps and tests only)
  int opt_tc_sets1;              // SLIM_TC_SETS=1: never use two score-warp sets
  int opt_tc_rt;                 // SLIM_TC_RT: rows per thread and tile (0 = default)
  int opt_unit_cost;             // SLIM_TC_UNIT_COST: boundary cost of the schedule in tiles (-1 = default)
  int opt_xscores_cuda;          // SLIM_XSCORES_CUDA: dense X-cache scores on CUDA cores
  int opt_k_evict;               // SLIM_TC_K_EVICT (0/1): L2 evict-first hint on the key loads (default on)
  long long* trace;              // device buffer set by slim_set_trace (trace builds)
  int opt_tail_fused;            // SLIM_TAIL_FUSED: combine + projection in one kernel: 0 never, 1 where it pays (default), 2 wherever possible
  int opt_prompt_pair;           // SLIM_PROMPT_PAIR=0: the prompt GEMM never runs on CTA pairs (for comparisons)
  int opt_proj_ns;               // SLIM_PROJ_NS: stages of the projection kernel (0 = default)
  int opt_legacy_flow;           // SLIM_TC_LEGACY: append and exact redo as kernels of their own (for side-by-side timing)
  alignas(64) unsigned char wmap[128];   // CUtensorMap over W_KV for the projection kernel
  alignas(64) unsigned char wmap_h[128];    // the same over wkv_h
};

struct slim_cache {
  slim_ctx* ctx;
  void* k;
  signed char* k_exp;            // fp8 cache: exponents behind the codes, else NULL
  int batch, t_cap;              // paged: t_cap = max_pages * page_rows
  const int32_t* block_table;    // paged: device [batch][max_pages]; NULL for a contiguous cache
  int page_rows, max_pages, num_pages;
  long long total_rows;          // rows of the storage: batch * t_cap, or num_pages * page_rows
  alignas(64) unsigned char tmap[2][128];   // CUtensorMaps of the tensor-core path for 1 / 2 CTAs per worker
  int has_tmap[2];
  alignas(64) unsigned char xmap[128];   // CUtensorMap for the dense X-cache scores (rows x 64 columns)
  int has_xmap;
};

// ---- launchers implemented in the kernel translation units -----------------
int  slim_generic_workers(const slim_ctx* ctx);
int  slim_generic_dsplit(const slim_ctx* ctx);
cudaError_t slim_launch_generic(const slim_ctx* ctx, const SlimDecodeParams& p, float* scores, cudaStream_t st);
// X-cache scheme: dense query transform + dense scores into `scores`; then either the CUDA-core
// accumulation (whole = 1) or, after the tensor-core kernel, the same accumulation as an exact
// redo that runs only if a unit was flagged (whole = 0)
cudaError_t slim_launch_xcache_scores(const slim_ctx* ctx, const SlimDecodeParams& p, float* scores, const float* W_K,
                                      float* qt, cudaStream_t st);
cudaError_t slim_launch_accum(const slim_ctx* ctx, const SlimDecodeParams& p, const float* scores, int whole, cudaStream_t st);
cudaError_t slim_launch_exact_flagged(const slim_ctx* ctx, const SlimDecodeParams& p, cudaStream_t st);
cudaError_t slim_launch_tail(const slim_ctx* ctx, const SlimDecodeParams& p, cudaStream_t st);
// pos_is_length = 1: positions[b] holds the length AFTER the append (row positions[b]-1 is written; 0 writes nothing)
// 8-bit cache on the tensor-core path: rows [0, lengths[b]) of every sequence are decoded (code * 2^exponent,
// exact in bf16) into `scratch`, a contiguous bf16 cache [batch][t_cap][d] that the bf16 kernels then read
cudaError_t slim_launch_dequant(const slim_ctx* ctx, const slim_cache* c, const int32_t* lengths, void* scratch, cudaStream_t st);
cudaError_t slim_launch_append(const slim_ctx* ctx, const slim_cache* c, const void* k_new,
                               const int32_t* positions, int n_new, int pos_is_length, cudaStream_t st);
// fp64 solve W_K X = W_V on the device; A and B are device row-major [n][n]
// float64, both overwritten; X is returned in B.  info: 0 ok, 1 singular.
cudaError_t slim_wkv_solve(double* A, double* B, int n, int* info_host);
// same with an n x m right-hand side B (row-major), X returned in B
cudaError_t slim_wkv_solve_rhs(double* A, double* B, int n, int m, int* info_host);
// C[M x N] = op(A) op(B) in float64 on the device (row-major, t* = 1 transposes); max |A - B|
cudaError_t slim_dgemm(const double* A, const double* B, double* C, int M, int N, int K, int ta, int tb);
cudaError_t slim_absdiff_max(const double* A, const double* B, size_t n, double* res_host);
cudaError_t slim_wkv_residual(const double* Wk, const double* X, const double* Wv, int n, double* res_host);
// X: [d][H * d_k] row-major (d rows: the contraction index of the projection)
cudaError_t slim_wkv_store(const double* X, int d, int H, int d_k, int dtype, void* dst, void* dst_h, float* hscale);

// tensor-core path (slim_tc.cu)
int  slim_tc_shape_ok(int d, int H, int d_k, int dtype, int rope, int cl);
int  slim_tc_workers(const slim_ctx* ctx, int cl);
cudaError_t slim_tc_make_tmap(const slim_ctx* ctx, slim_cache* c, int cl);
cudaError_t slim_launch_wait_selftest(int* status, int* gave_up, cudaStream_t st);
cudaError_t slim_launch_tc(const slim_ctx* ctx, const slim_cache* c, const SlimDecodeParams& p, cudaStream_t st);

// 3-D tiled tensor map with 128-byte swizzle over bf16 data (driver entry point looked up once)
cudaError_t slim_tmap_encode_3d(void* out_map, void* base, const unsigned long long dims[3],
                                const unsigned long long strides[2], const unsigned int box[3]);

// tensor-core combine + projection (slim_proj.cu)
int    slim_proj_shape_ok(int d, int H, int d_k, int dtype);
int    slim_proj_jsplit(int d);
int    slim_proj_needs_convert(const slim_ctx* ctx, int batch);      // 1: the combine writes float rows and a conversion kernel follows
int    slim_proj_launch_count(const slim_ctx* ctx, const SlimDecodeParams& p);   // kernels slim_launch_proj enqueues
size_t slim_proj_u_bytes(int d, int H, int batch);
cudaError_t slim_proj_make_wmap(slim_ctx* ctx);
// u32: [batch][H][d] float scratch, su: [16 ceil(batch / 16)][H] float scales of the operand rows
cudaError_t slim_launch_proj(const slim_ctx* ctx, const SlimDecodeParams& p, unsigned char* u_tiled, float* u32, float* su,
                             cudaStream_t st);
cudaError_t slim_launch_sum_slices(const float* o_part, float* o, int n, int nsplit, cudaStream_t st);

// ---- programmatic dependent launch ---------------------------------------------
// The kernels of one decode step run back to back on one stream.  Launched with
// slim_launch_pdl, a kernel may be scheduled while its predecessor is still
// finishing; it must execute slim_pdl_wait() before it touches anything a
// predecessor wrote (the wait returns once the predecessor grid has completed and
// its memory is visible).  slim_pdl_trigger() lets the successor's launch begin.
#ifdef __CUDACC__
__device__ __forceinline__ void slim_pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void slim_pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t slim_launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                   Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}
#endif

// X-cache scheme: dense scores on the tensor cores (slim_xscores.cu)
int    slim_xscores_tc_ok(const slim_ctx* ctx);
size_t slim_xscores_qt_bytes(int d, int batch);
cudaError_t slim_xscores_make_tmap(const slim_ctx* ctx, slim_cache* c);
cudaError_t slim_launch_xscores_tc(const slim_ctx* ctx, const slim_cache* c, const SlimDecodeParams& p, const float* W_K,
                                   unsigned char* qt_tiled, float* scores, cudaStream_t st);

// context split over several GPUs (slim_split.cu)
cudaError_t slim_launch_partial_out(const slim_ctx* ctx, const SlimDecodeParams& p, float* lse_out, float* u_out, cudaStream_t st);
cudaError_t slim_launch_rank_combine(const slim_ctx* ctx, const SlimDecodeParams& p, const float* lse_all, const float* u_all,
                                     int ranks, cudaStream_t st);

// prompt phase: V = K W_KV for n rows (slim_prompt.cu)
cudaError_t slim_launch_values(const slim_ctx* ctx, const void* K, int n, float* V, cudaStream_t st,
                               const slim_cache* cache = nullptr, const int32_t* positions = nullptr, int n_new = 0);
