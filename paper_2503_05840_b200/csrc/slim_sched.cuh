// Device-side work schedule shared by all decode kernels.
//
// The context of sequence b is cut into tiles of SLIM_TT rows.  All tiles of
// the batch are laid end to end (sequence 0 first) and cut into W_eff equal
// contiguous ranges, one per worker ("stream-K" over the ragged batch).  The
// part of a worker's range that falls into one sequence is a *unit*: it
// produces one partial (m, l, U[H][d]) for the log-sum-exp combine.  Because
// (worker, sequence) pairs are monotone along the tile line, unit id =
// worker + sequence is unique and < workers + batch.  The schedule is a pure
// function of `lengths`, so every CTA (and the combine kernel) recomputes it
// and the result is deterministic.
//
// Closing a unit costs a worker about `unit_cost` tiles of time (draining the
// accumulator, restarting the pipeline), so the cut is made on a *virtual*
// line in which every boundary between two sequences is unit_cost slots wide:
// a worker whose range crosses a boundary gets that many tiles fewer.
#pragma once
#include "slim_internal.h"

struct SlimSched {
  int total_tiles;   // NT
  int workers_eff;   // W_eff <= workers
  int unit_cost;     // E: width of a sequence boundary on the virtual line, in tiles
  int virt_total;    // NT + E (batch - 1)
  int batch;
  const int* prefix; // shared memory, batch + 1 entries
};

// Exclusive prefix of per-sequence tile counts into s_prefix[0..batch]
// (shared memory, batch+1 ints).  Must be called by all threads of the CTA
// (uses __syncthreads).  Lengths are clamped to [0, t_cap]; a length above
// t_cap also raises SLIM_ERR_CAPACITY in *status.
__device__ __forceinline__ SlimSched slim_sched_build(const int32_t* __restrict__ lengths, int batch,
                                                      int t_cap, int workers, int min_tiles,
                                                      int* s_prefix, int* status, int unit_cost = 0) {
  const int tid = threadIdx.x + threadIdx.y * blockDim.x;
  const int nthr = blockDim.x * blockDim.y;
  for (int b = tid; b < batch; b += nthr) {
    int len = lengths[b];
    if (len > t_cap) { len = t_cap; atomicMax(status, (int)SLIM_ERR_CAPACITY); }
    if (len < 0) len = 0;
    s_prefix[b + 1] = (len + SLIM_TT - 1) / SLIM_TT;
  }
  if (tid == 0) s_prefix[0] = 0;
  __syncthreads();
  if (tid < 32) {
    // warp 0: each lane scans a contiguous chunk, then the chunk sums are scanned.
    const int chunk = (batch + 31) / 32;
    const int lo = tid * chunk, hi = min(batch, lo + chunk);
    int sum = 0;
    for (int b = lo; b < hi; ++b) sum += s_prefix[b + 1];
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (tid >= o) incl += v;
    }
    int run = incl - sum;
    for (int b = lo; b < hi; ++b) { run += s_prefix[b + 1]; s_prefix[b + 1] = run; }
  }
  __syncthreads();
  SlimSched s;
  s.total_tiles = s_prefix[batch];
  int we = s.total_tiles / (min_tiles > 0 ? min_tiles : 1);
  if (we < 1) we = 1;
  s.workers_eff = we < workers ? we : workers;
  s.unit_cost = unit_cost;
  s.virt_total = s.total_tiles + unit_cost * (batch - 1);
  s.batch = batch;
  s.prefix = s_prefix;
  return s;
}

// First tile of worker w (w = workers_eff gives total_tiles).  A worker's range
// [start(w), start(w+1)) may be empty.
__device__ __forceinline__ int slim_worker_start(const SlimSched& s, int w) {
  const int v = (int)(((long long)w * s.virt_total) / s.workers_eff);
  // sequence whose virtual span [prefix[b] + E b, prefix[b+1] + E (b+1)) holds v
  int lo = 0, hi = s.batch;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (s.prefix[mid] + s.unit_cost * mid <= v) lo = mid; else hi = mid;
  }
  const int t = v - s.unit_cost * lo;
  return t < s.prefix[lo + 1] ? t : s.prefix[lo + 1];
}

// Sequence that owns global tile g: prefix[b] <= g < prefix[b+1].
__device__ __forceinline__ int slim_seq_of_tile(const int* s_prefix, int batch, int g) {
  int lo = 0, hi = batch;            // invariant: prefix[lo] <= g < prefix[hi]
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (s_prefix[mid] <= g) lo = mid; else hi = mid;
  }
  return lo;
}

// Worker that owns global tile g (0 <= g < total_tiles): the largest w with start(w) <= g.
__device__ __forceinline__ int slim_worker_of_tile(const SlimSched& s, int g) {
  const int b = slim_seq_of_tile(s.prefix, s.batch, g);
  const long long v = (long long)g + (long long)s.unit_cost * b;
  return (int)(((v + 1) * s.workers_eff - 1) / s.virt_total);
}

// Row of the key storage that holds context row t0 of sequence b (t0 a multiple of SLIM_TT; a tile
// never straddles pages because page_rows is a multiple of SLIM_TT).  A page id outside the pool
// raises SLIM_ERR_CAPACITY and reads page 0.
__device__ __forceinline__ long long slim_cache_row(const SlimDecodeParams& p, int b, int t0) {
  if (p.block_table) {
    int pg = p.block_table[(size_t)b * p.max_pages + t0 / p.page_rows];
    if (pg < 0 || pg >= p.num_pages) { atomicMax(p.status, (int)SLIM_ERR_CAPACITY); pg = 0; }
    return (long long)pg * p.page_rows + t0 % p.page_rows;
  }
  return (long long)b * p.t_cap + t0;
}

// A cache may hold a slice of a longer context (context split over several GPUs): then its row t sits at
// absolute position SLIM_TT * pos_tiles[b] + t and the query at q_pos[b].  Otherwise row t is position t and
// the query sits at the newest row.
// Positions beyond the RoPE table (slim_reserve_positions) are clamped into it and reported as SLIM_ERR_CAPACITY.
__device__ __forceinline__ int slim_query_pos(const SlimDecodeParams& p, int b, int len) {
  if (!p.q_pos) return len - 1;
  int q = p.q_pos[b];
  const int top = p.rope_tiles * SLIM_TT - 1;
  if (q < 0 || q > top) { atomicMax(p.status, (int)SLIM_ERR_CAPACITY); q = q < 0 ? 0 : top; }
  return q;
}
__device__ __forceinline__ int slim_tile_offset(const SlimDecodeParams& p, int b) {
  if (!p.pos_tiles) return 0;
  int off = p.pos_tiles[b];
  const int top = p.rope_tiles - 1 - (p.t_cap + SLIM_TT - 1) / SLIM_TT;      // the slice's last tile must stay inside the table
  if (off < 0 || off > top) { atomicMax(p.status, (int)SLIM_ERR_CAPACITY); off = off < 0 || top < 0 ? 0 : top; }
  return off;
}
