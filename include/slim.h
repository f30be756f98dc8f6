/*
 * slim.h -- C ABI of the K-cache-only ("slim") multi-head decode-attention
 * library for NVIDIA B200 (sm_100a).
 *
 * The library implements one attention layer's generate-phase step of slim
 * attention (arxiv 2503.05840): only keys are cached; values are recovered
 * from keys through W_KV = W_K^{-1} W_V (Eq. 6) and the attention output is
 * computed as   head_i = [ softmax(q_i K_i^T / sqrt(d_k)) K ] W_KV,i
 * (Eq. 7, Option 2), with RoPE applied to the keys after they are read from
 * the cache (appendix "Support for RoPE", Option 1).
 *
 * Conventions
 *   - Row vectors, K = X W_K; every weight matrix is row-major [d_in][d_out];
 *     head i owns columns i*d_k .. (i+1)*d_k-1.  Square MHA only: d = H*d_k.
 *   - "device" pointers are CUDA device memory of the current device, "host"
 *     pointers are ordinary host memory.  The caller owns every buffer it
 *     passes; the library owns only what slim_create / slim_set_weights /
 *     slim_cache_create allocate (W_KV, RoPE tables, tensor maps, a status word).
 *   - Every call returns a slim_status; nothing throws across the ABI.
 *   - Calls taking `stream` (a cudaStream_t passed as void*, NULL = default
 *     stream) only enqueue work and return; device-side problems are reported
 *     by slim_device_status.
 *   - No call falls back to the CPU.  Without a usable CUDA device every
 *     compute call returns SLIM_ERR_CUDA.
 *   - A context is not re-entrant on the device: decode calls of one context
 *     share its status word and redo flag, and calls given the same workspace
 *     share its partials.  Enqueue the calls of one context (and of contexts
 *     that share a workspace) on one stream, or order them with events; host
 *     threads must not call into one context at the same time.
 */
#ifndef SLIM_H_
#define SLIM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SLIM_OK = 0,
  SLIM_ERR_INVALID_ARG = 1,  /* NULL pointer, non-positive size, bad enum          */
  SLIM_ERR_UNSUPPORTED = 2,  /* d != H*d_k, odd d_k, H > 64, ...                       */
  SLIM_ERR_SINGULAR = 3,     /* W_K has a (numerically) zero pivot                  */
  SLIM_ERR_CAPACITY = 4,     /* append beyond t_cap / length beyond t_cap (device)  */
  SLIM_ERR_OOM = 5,          /* a library-owned allocation failed                   */
  SLIM_ERR_CUDA = 6,         /* CUDA runtime/driver error, or no device             */
  SLIM_ERR_TIMEOUT = 7,      /* a bounded device-side wait ran out (device)         */
  SLIM_ERR_NO_WEIGHTS = 8,   /* slim_decode before slim_set_weights / slim_set_wkv  */
  SLIM_ERR_STATIC_WS = 9     /* slim_decode_static_ws: scratch need above the built-in maximum */
} slim_status;

/* cache / query dtype.  SLIM_FP8: the cache holds 8-bit keys (1 byte per value, the paper's own byte
 * accounting in its introduction), queries, new key rows and W_KV are bf16 -- see slim_cache_bytes. */
typedef enum { SLIM_F32 = 0, SLIM_BF16 = 1, SLIM_FP8 = 2 } slim_dtype;
typedef enum { SLIM_HOST_F32 = 0, SLIM_HOST_F64 = 1 } slim_host_dtype;

/* Kernel selection for slim_decode (slim_set_path). */
typedef enum {
  SLIM_PATH_AUTO = 0,     /* tensor-core path when the shape allows it, else generic */
  SLIM_PATH_GENERIC = 1,  /* CUDA-core kernels (any supported shape, f32 or bf16)    */
  SLIM_PATH_TC = 2        /* TMA + tcgen05 kernels (bf16; UNSUPPORTED if shape unfit) */
} slim_path;

/* Keys for slim_query. */
typedef enum {
  SLIM_Q_PATH_IN_USE = 0,        /* slim_path that slim_decode will take             */
  SLIM_Q_LAUNCHES_PER_DECODE = 1,/* kernels the last decode call of this ctx enqueued (counted) */
  SLIM_Q_MAX_UNITS = 2,          /* upper bound of (sequence, context-split) units   */
  SLIM_Q_NUM_SMS = 3,
  SLIM_Q_WORKERS = 4             /* context-split workers of the path in use         */
} slim_query_key;

typedef struct slim_ctx slim_ctx;     /* one attention layer: shape, W_KV, RoPE tables  */
typedef struct slim_cache slim_cache; /* view of caller-owned key storage [B][t_cap][d] */

/* One layer of shape (d, H, d_k); rope_theta = 0 disables RoPE; dtype is the
 * type of the K-cache and of q.  Requires d == H*d_k (Eq. 6 needs a square
 * W_K), H <= 64, d_k even and <= 256 (the tensor-core kernels take d_k = 64, 96, 128; other
 * widths, e.g. d_k = 100, run on the CUDA-core kernels).  Uses the current CUDA device. */
slim_status slim_create(slim_ctx** out, int d, int H, int d_k, double rope_theta, int dtype);
void        slim_destroy(slim_ctx* ctx);

/* Eq. 6 with the appendix-A recipe: forms W_KV = W_K^{-1} W_V in float64 (LU
 * with partial pivoting on the device, solving W_K W_KV = W_V) and stores it,
 * rounded to the ctx dtype, as H column blocks [d][d_k].
 *   W_K, W_V      host, row-major [d][d], host_dtype = SLIM_HOST_F32 | _F64
 *   wkv_out       host [d][d] float64, receives the unrounded W_KV (may be NULL)
 *   residual_out  receives max |W_K W_KV - W_V| (may be NULL)
 * Synchronous.  SLIM_ERR_SINGULAR if a pivot is below 1e-13 * max|W_K| * d.   */
slim_status slim_set_weights(slim_ctx* ctx, const void* W_K, const void* W_V, int host_dtype,
                             double* wkv_out, double* residual_out);

/* Non-square projections (section "Support for non-square weight matrices", Option 1):
 * the model width d_model is smaller than e = H*d_k, W_K and W_V are [d_model][e] (host,
 * row-major) and K = X W_K is e wide.  Forms the right inverse
 * W_K^{-1} = W_K^T (W_K W_K^T)^{-1} in float64 (LU solve of the d_model x d_model system)
 * and stores W_KV = W_K^{-1} W_V, an [e][e] matrix, so that K W_KV = V for every K in the
 * row space of W_K.  The ctx must have been created with d = e; caches, slim_append_k and
 * slim_decode are used unchanged.  wkv_out (may be NULL) receives the [e][e] float64
 * W_KV, residual_out (may be NULL) max |W_K W_KV - W_V|.  SLIM_ERR_SINGULAR if W_K does
 * not have full row rank.  Synchronous.                                              */
slim_status slim_set_weights_nonsquare(slim_ctx* ctx, const void* W_K, const void* W_V, int d_model,
                                       int host_dtype, double* wkv_out, double* residual_out);

/* Load a precomputed W_KV (the paper stores it in the parameter file in place
 * of W_V, Eq. 6).  W_KV: host, row-major [d][d].  Synchronous.                 */
slim_status slim_set_wkv(slim_ctx* ctx, const void* W_KV, int host_dtype);

/* Bytes of key storage for `batch` sequences of capacity t_cap, and of the
 * scratch workspace slim_decode needs for such a cache (0 on bad arguments).
 * SLIM_FP8 caches: the storage holds the codes [batch][t_cap][d] (OCP FP8 E4M3, one byte per
 * value) followed, at the next multiple of 16 bytes, by one int8 exponent per (row, head)
 * [batch][t_cap][H]: the stored key is code * 2^exponent, the exponent being the smallest one
 * for which the head slice of the row fits the E4M3 range (|value| <= 448), codes rounded to
 * nearest even.  Such a cache is filled only through slim_append_k / slim_decode_step /
 * slim_prefill (which quantise bf16 rows); it is contiguous (no paged variant) and has no X-cache
 * mode.  Where the shape fits the tensor-core kernels, slim_decode first decodes the live rows
 * exactly into a bf16 copy inside the workspace (slim_workspace_bytes then includes
 * 2 * batch * t_cap * d bytes for it) and runs the bf16 kernels on the copy; otherwise, and with
 * SLIM_PATH_GENERIC, the CUDA-core kernels read the codes directly.                       */
size_t slim_cache_bytes(const slim_ctx* ctx, int batch, int t_cap);
size_t slim_workspace_bytes(const slim_ctx* ctx, int batch, int t_cap);

/* Wrap caller-owned device storage k_storage (layout [batch][t_cap][d], ctx
 * dtype, 16-byte aligned; 1024-byte alignment recommended) as a K-cache of
 * UN-ROTATED keys.  Builds the RoPE tables for positions < t_cap.  The storage
 * must outlive the cache object; its contents are not touched.                */
slim_status slim_cache_create(slim_ctx* ctx, slim_cache** out, void* k_storage, int batch, int t_cap);
/* Paged K-cache: the keys live in a caller-owned pool of num_pages pages of page_rows rows each
 * (device, [num_pages][page_rows][d], ctx dtype, 16-byte aligned; page_rows a multiple of 16), and
 * context row t of sequence b is row t % page_rows of page block_table[b][t / page_rows].
 * block_table: device int32 [batch][max_pages], read by the kernels at every call (the caller may
 * update it between calls); capacity per sequence t_cap = max_pages * page_rows.  A page id
 * outside the pool raises SLIM_ERR_CAPACITY on the device.  slim_append_k and slim_decode take
 * such a cache like a contiguous one (workspace: slim_workspace_bytes(ctx, batch, t_cap)); the
 * X-cache calls do not.                                                               */
slim_status slim_cache_create_paged(slim_ctx* ctx, slim_cache** out, void* pool, int num_pages, int page_rows,
                                    const int32_t* block_table, int batch, int max_pages);
void        slim_cache_destroy(slim_cache* cache);

/* Prompt phase (Fig. 3(a)): the values of the n prompt tokens are formed once from their keys,
 * V = K W_KV (Eq. 6), so that the prompt can be processed like vanilla attention while only K is
 * kept.  K: device [n][d], ctx dtype, un-rotated keys; V: device [n][d] float32.  bf16 with
 * d_k in {64, 96, 128} runs on the tensor cores (16-byte aligned K and V), else on CUDA cores. */
slim_status slim_values_from_keys(slim_ctx* ctx, const void* K, int n, float* V, void* stream);

/* Prompt phase in one call (Fig. 3(a)): the prompt's keys are stored in the K-cache AND their values
 * V = K W_KV (Eq. 6) are returned, from one pass over the keys.
 *   k_new      device [batch][n_new][d], ctx dtype, un-rotated keys of the prompt tokens
 *   positions  device int32 [batch]: first cache row of sequence b (0 for a fresh prompt)
 *   V          device [batch][n_new][d] float32
 * Equivalent to slim_append_k(k_new, positions, n_new) + slim_values_from_keys on the same rows; a
 * sequence whose rows would pass t_cap is left unwritten (device status SLIM_ERR_CAPACITY), its
 * values are still returned.  On the tensor-core path (bf16, d_k in {64, 96, 128}, 16-byte aligned
 * buffers) both happen in one kernel: otherwise idle warps of the GEMM CTAs store the rows while the
 * same CTAs stream them, so the keys are read from HBM once.  Contiguous and paged caches.      */
slim_status slim_prefill(slim_ctx* ctx, slim_cache* cache, const void* k_new, const int32_t* positions,
                         int n_new, float* V, void* stream);

/* Generate-phase cache update: for every sequence b write the n_new rows
 * k_new[b][0..n_new) (device, [batch][n_new][d], ctx dtype, un-rotated keys
 * k = x W_K) at rows positions[b] .. positions[b]+n_new-1 (device int32).
 * A sequence whose rows would pass t_cap is left unwritten and the device
 * status becomes SLIM_ERR_CAPACITY.                                            */
slim_status slim_append_k(slim_ctx* ctx, slim_cache* cache, const void* k_new,
                          const int32_t* positions, int n_new, void* stream);

/* Eq. 7 Option 2 for one decode token per sequence.
 *   q        device [batch][d], ctx dtype, un-rotated, bias (if any) included
 *   lengths  device int32 [batch]; sequence b attends over cache rows
 *            0 .. lengths[b]-1; the query sits at position lengths[b]-1;
 *            lengths[b] == 0 gives a zero output row; lengths[b] > t_cap is
 *            clamped and reported as SLIM_ERR_CAPACITY
 *   o        device float32 [batch][d] = concat(head_1 .. head_H), no W_O
 *   workspace device, >= slim_workspace_bytes(ctx, batch, t_cap), 256-byte
 *            aligned; contents are scratch                                    */
slim_status slim_decode(slim_ctx* ctx, const void* q, const slim_cache* cache,
                        const int32_t* lengths, float* o, void* workspace, void* stream);

/* One generate-phase step of a layer in a single call: the cache update and the attention
 * (introduction, "one new K-vector per iteration": the newest key is appended, then the token
 * attends over all cached keys, itself included; Eq. 7 Option 2).
 *   k_new    device [batch][d], ctx dtype, un-rotated key row x_n W_K of every sequence, 16-byte
 *            aligned; it is written to cache row lengths[b]-1 before that row is read
 *   lengths  device int32 [batch]: the context lengths AFTER the update.  lengths[b] == 0 writes
 *            nothing and gives a zero output row; lengths[b] > t_cap writes nothing, is clamped
 *            and reported as SLIM_ERR_CAPACITY
 *   other arguments and the result as for slim_decode.
 * Equivalent to slim_append_k(k_new, positions = lengths-1, n_new = 1) followed by slim_decode.
 * On the tensor-core path the row is written by the decode kernel itself (by the CTA pair that
 * reads the sequence's last tile, ahead of its first load), so no append kernel runs; other
 * paths launch the append kernel first.                                                 */
slim_status slim_decode_step(slim_ctx* ctx, const void* q, const void* k_new, slim_cache* cache,
                             const int32_t* lengths, float* o, void* workspace, void* stream);

/* slim_decode for callers that cannot allocate device memory.  (The paper has no
 * counterpart; this is a convenience of the library.)  Some hosts of this code must
 * not call cudaMalloc or any allocator while they run: a serving loop whose memory
 * pool is frozen after start-up, a plug-in that is handed a device it does not own,
 * code running where an allocation would synchronise the whole device.  For them the
 * scratch that slim_decode takes as `workspace` lives in a fixed array inside the
 * library: slim_static_workspace_max() bytes (16 MiB) of device memory that every
 * GPU which loads the library keeps until the process exits.  Same arguments and
 * result as slim_decode, minus `workspace`; no device or host memory is allocated or
 * freed by the call.
 *   - If slim_workspace_bytes(ctx, batch, t_cap) of the cache exceeds the maximum,
 *     nothing is launched and SLIM_ERR_STATIC_WS is returned (use slim_decode with
 *     your own workspace for such sizes; the need grows with batch, H*d and the SM count).
 *   - The ctx's device must be the current device.  The first call on a device looks
 *     up the array's device address (once per device); make that first call before
 *     starting any stream capture.
 *   - All calls on a device share the one array, and it keeps whatever the previous
 *     call left.  Nothing needs clearing: every word that can reach a stored output is
 *     written earlier in the same call (words of padding sequences of a 16-sequence
 *     group may be read unwritten, but only feed outputs that are never stored).  Two
 *     calls whose kernels overlap on the GPU (different streams, different ctx objects)
 *     race on it: run them one after another.                                      */
size_t      slim_static_workspace_max(void);
slim_status slim_decode_static_ws(slim_ctx* ctx, const void* q, const slim_cache* cache,
                                  const int32_t* lengths, float* o, void* stream);

/* X-cache / E-cache scheme (section "Support for non-square weight matrices", Option 2, and
 * section "Support for encoder-decoder transformers", Option 2): the cache holds the layer
 * inputs X (or the encoder output E, which all decoder layers may share: wrap the same
 * storage with slim_cache_create for every layer's ctx) instead of keys.  Per head
 *   A_i = ((x_n W_Q,i + b) W_K,i^T) X^T,   head_i = [softmax(A_i / sqrt(d_k)) X] W_V,i.
 * No RoPE (the ctx must have rope_theta = 0).  Projections need not be square here: with
 * slim_xcache_create the model width d (cache rows, the inner index of W_K and W_V) and the
 * projection width e = H*d_k (queries, outputs) are independent, W_K, W_V in R^{d x e}
 * (section "Support for non-square weight matrices", Option 2: e > d as in T5-style models, or
 * e < d).  A context from slim_create (d = e) works as well.
 *   slim_xcache_create        d_model = width of a cache row; H <= 64, even d_k <= 256,
 *                             d_model, H*d_k <= 16384; SLIM_F32 or SLIM_BF16.  Such a context
 *                             serves the slim_xcache_* calls and slim_cache_create only (the K-cache
 *                             calls return SLIM_ERR_UNSUPPORTED unless d_model = H*d_k)
 *   slim_xcache_set_weights   W_K, W_V host row-major [d][e]; W_K is kept in float32 for the
 *                             per-token query transform, W_V replaces W_KV in the projection
 *   slim_xcache_decode        as slim_decode: q = x_n W_Q (+ bias) [batch][e], `cache` holds
 *                             X rows [batch][t_cap][d], o is [batch][e];
 *                             workspace >= slim_xcache_workspace_bytes
 * bf16 caches with d % 64 == 0 and H <= 32 run on the tensor cores (dense scores: cache rows
 * as a K-major TMA operand against bf16 hi/lo query tiles; weighted sum and projection: the
 * kernels of slim_decode); other shapes use the CUDA-core kernels.  The cache is read twice
 * per layer (scores, then the weighted sum).                                            */
slim_status slim_xcache_create(slim_ctx** out, int d_model, int H, int d_k, int dtype);
slim_status slim_xcache_set_weights(slim_ctx* ctx, const void* W_K, const void* W_V, int host_dtype);
size_t      slim_xcache_workspace_bytes(const slim_ctx* ctx, int batch, int t_cap);
slim_status slim_xcache_decode(slim_ctx* ctx, const void* q, const slim_cache* cache, const int32_t* lengths,
                               float* o, void* workspace, void* stream);

/* One context split over several GPUs (the complexity section's remark that the scheme works with
 * flash-style splitting; Eq. 2 and Eq. 7 Option 2 evaluated slice by slice).  Every rank caches a
 * slice of the rows of each sequence, starting at a multiple of 16 rows, and calls
 * slim_decode_partial on it; the ranks exchange the results (an all-gather of H (d + 1) floats per
 * sequence -- the caller's job, e.g. with NCCL) and slim_combine_project joins them.
 *   slim_reserve_positions  grows the RoPE tables to cover absolute positions < max_position
 *                           (a slice's cache only covers its own t_cap rows).  Synchronous; call
 *                           it at set-up.  Positions outside the tables are clamped and reported as
 *                           SLIM_ERR_CAPACITY by the device status.
 *   slim_decode_partial     q, cache, lengths as for slim_decode, lengths[b] = rows of the slice;
 *                           first_tile  device int32 [batch]: absolute row of the slice's row 0, / 16
 *                           q_pos       device int32 [batch]: absolute position of the query
 *                           lse_out     device float [batch][H]: log2 of the slice's softmax
 *                                       denominator (arguments in log2 units); -inf for an empty slice
 *                           u_out       device float [batch][H][d]: the slice's weighted sum of keys
 *                                       divided by that denominator
 *                           bf16 and f32 caches (not SLIM_FP8)
 *   slim_combine_project    lse_all [ranks][batch][H], u_all [ranks][batch][H][d] (device, rank
 *                           order free), total_lengths device int32 [batch] (0 gives a zero row):
 *                           u = sum_r w_r u_r with w_r = 2^(lse_r - max) / sum_r' 2^(lse_r' - max),
 *                           then the per-head projection with W_KV; o device float [batch][d];
 *                           workspace >= slim_workspace_bytes(ctx, batch, 16); ranks <= 64.      */
slim_status slim_reserve_positions(slim_ctx* ctx, int max_position);
slim_status slim_decode_partial(slim_ctx* ctx, const void* q, const slim_cache* cache, const int32_t* lengths,
                                const int32_t* first_tile, const int32_t* q_pos, float* lse_out, float* u_out,
                                void* workspace, void* stream);
slim_status slim_combine_project(slim_ctx* ctx, const float* lse_all, const float* u_all, int ranks,
                                 const int32_t* total_lengths, int batch, float* o, void* workspace, void* stream);

/* Synchronises `stream`, returns the sticky device status (SLIM_OK,
 * SLIM_ERR_CAPACITY or SLIM_ERR_TIMEOUT) and clears it.                        */
slim_status slim_device_status(slim_ctx* ctx, void* stream);

/* Self-test of the bounded device-side waits every TMA / tcgen05 kernel relies on: runs
 * a one-CTA kernel that waits on a barrier nothing completes.  The wait must give up after
 * its limit (about two seconds), the kernel must return normally, and the sticky device
 * status must read SLIM_ERR_TIMEOUT afterwards.  Returns SLIM_OK if the kernel gave up as
 * designed (the caller then reads and clears the status with slim_device_status); the CUDA
 * context stays usable.  Synchronises `stream`.                                       */
slim_status slim_selftest_bounded_wait(slim_ctx* ctx, void* stream);

/* Kernel timing for roofline reports.  While enabled, slim_decode records CUDA
 * events on its stream before the main (K-reading) kernel, after it, and after
 * the combine/projection tail.  slim_profile_read waits for the last decode of
 * this ctx to finish and returns the two durations in milliseconds.           */
slim_status slim_profile_enable(slim_ctx* ctx, int enable);
slim_status slim_profile_read(slim_ctx* ctx, float* main_ms, float* tail_ms);

/* Per-tile timing of the tensor-core decode kernel, for builds of the library compiled with
 * -DSLIM_TC_TRACE (python -m paper_2503_05840_b200.trace builds one and prints the statistics; the
 * default build returns SLIM_ERR_UNSUPPORTED).  device_buffer: device int64 [CTAs][192][8], zeroed by
 * the caller; while set, every slim_decode of this ctx records, for the first 192 tiles of each CTA,
 * the SM clock at eight points of the producer, score-warp and MMA loops.  NULL switches it off.  */
slim_status slim_set_trace(slim_ctx* ctx, void* device_buffer);

slim_status slim_set_path(slim_ctx* ctx, int path);
long long   slim_query(const slim_ctx* ctx, int key);
const char* slim_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* SLIM_H_ */
