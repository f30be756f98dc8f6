// Tail of the decode step on the tensor cores (bf16 caches, d_k = 64, 96 or 128):
//
//   slim_combine_kernel   log-sum-exp combine of the context-split partials:
//                         u[b][h][:] = sum_s w_s U_s[h][:] / sum_s w_s l_s over the
//                         units s of sequence b.  u is written as a scaled float16
//                         pair (row divided by 2^e, hi = f16(v), lo = f16(v - hi);
//                         see slim_combine.cuh) directly in the shared-memory
//                         operand layout of the projection MMA, so the projection
//                         kernel fetches it with plain bulk copies.
//   slim_proj_tc_kernel   the per-head projection o_h = u_h W_KV,h of Eq. 7
//                         (Option 2) for 16 sequences at a time:
//                         O^T[128 x N] += W_tile^T[128 x 16] u^T[16 x N] with one
//                         tcgen05.mma per 16 rows of W_KV,h; A = the TMA-staged
//                         float16 weights (scaled per head) used MN-major, B = the u tiles, D in tensor
//                         memory.  N = 32 per head (16 sequences x {hi, lo}); for
//                         d_k = 64 two heads share an instruction (M = 2 x 64,
//                         N = 2 x 32) and the off-diagonal quadrants are ignored; for
//                         d_k = 96 the accumulator rows 96..127 are ignored.
//                         A CTA owns (head group, slice of the d rows of W_KV,h,
//                         16-sequence group); the CTAs of the row slices form a
//                         cluster, leave their slice results in shared memory and
//                         each adds, in slice order, a share of the output rows
//                         through distributed shared memory (bitwise repeatable).
//
//   slim_tail_fused_kernel  both of the above in one kernel: the projection CTA forms its own columns of u
//                         from the partials (used where a CTA has few partial bytes to pull; see tail_fused).
//
// Every mbarrier wait is bounded in time; a wait that runs out sets the device
// status to SLIM_ERR_TIMEOUT and the CTA drains and exits.
#include <cstring>

#include "slim_internal.h"
#include "slim_sched.cuh"
#include "slim_ptx.cuh"
#include "slim_combine.cuh"

namespace {
using namespace slim_ptx;
using slim_comb::PJ_BG;

constexpr int PJ_ROWS = 64;                    // rows of W_KV,h per stage (4 MMA k-steps)
constexpr int PJ_W_BYTES = PJ_ROWS * 128 * 2;  // two 64-column atoms x 64 rows x 128 B
constexpr int PJ_NS = 4;                       // stages (at most; a CTA uses g.ns of them)
constexpr int COMBINE_SMEM_ROW = 8192;         // widest row u[b][h][:] the combine kernel collects in shared memory

struct ProjGeom {
  int hp;        // heads per MMA: 1 (d_k = 96, 128) or 2 (d_k = 64)
  int hg;        // head groups = H / hp
  int jsplit;    // slices of the d rows of W_KV,h
  int nst;       // stages per CTA = d / 64 / jsplit
  int nbg;       // 16-sequence groups
  int u_bytes;   // bytes of u per stage = 4 k-steps x hp x 1 KB
  int ns;        // stages in use: as many as keep two CTAs on an SM
};

// weights [workers], info [4], prefix [batch + 1]; behind them, 16-byte aligned, the scratch of the exact path
__device__ __forceinline__ size_t exact_scratch_offset(const SlimDecodeParams& p) {
  return (sizeof(float) * p.workers + sizeof(int) * (4 + p.batch + 1) + 15) & ~(size_t)15;
}

// Units of sequence b and their weights for head h (warp 0 of the CTA):
// s_info = (first worker, unit count, 1 if a unit of the sequence is flagged for the exact recomputation)
__device__ __forceinline__ void combine_prologue(const SlimDecodeParams& p, const SlimSched& sc, const int* s_prefix, int b, int h,
                                                 float* s_w, int* s_info, int lane) {
  int wlo = 0, wn = 0, flagged = 0;
  if (b < p.batch && s_prefix[b + 1] > s_prefix[b]) {
    wlo = slim_worker_of_tile(sc, s_prefix[b]);
    wn = slim_worker_of_tile(sc, s_prefix[b + 1] - 1) - wlo + 1;
    if (p.redo_in_combine) {
      for (int i = lane; i < 2 * wn; i += 32) flagged |= p.unit_flags[2 * (wlo + b) + i];
      flagged = __any_sync(0xffffffffu, flagged != 0) ? 1 : 0;
    }
    if (!flagged) slim_comb::weights_warp(p.part_m, p.part_l, wlo + b, wn, p.H, h, s_w, lane);
  }
  if (lane == 0) { s_info[0] = wlo; s_info[1] = wn; s_info[2] = flagged; }
}

// (launch bounds: the register budget of the hot loop; the exact path, a call, may spill under it)
__global__ void __launch_bounds__(256, 4)
slim_combine_kernel(const __grid_constant__ SlimDecodeParams p, unsigned char* __restrict__ u_tiled, float* __restrict__ u32,
                    float* __restrict__ su, const int hp) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* s_w = reinterpret_cast<float*>(smem_raw);                 // [workers]
  int* s_info = reinterpret_cast<int*>(s_w + p.workers);           // wlo, wn, flagged
  int* s_prefix = s_info + 4;                                      // [batch+1]
  const int tid = threadIdx.x, lane = tid & 31;
  const int h = blockIdx.x, b = blockIdx.y;
  const int d = p.d, H = p.H;
  slim_pdl_trigger();
  slim_pdl_wait();
  if (blockIdx.x == 0 && blockIdx.y == 0 && tid == 0) *p.any_flag = 0;   // the redo kernel has consumed it

  const SlimSched sc = slim_sched_build(p.lengths, p.batch, p.t_cap, p.workers, p.min_tiles, s_prefix, p.status, p.unit_cost);
  if (tid < 32) combine_prologue(p, sc, s_prefix, b, h, s_w, s_info, lane);
  __syncthreads();
  const int wlo = s_info[0], wn = s_info[1];
  float* s_x = reinterpret_cast<float*>(smem_raw + exact_scratch_offset(p));     // d_k + 36 floats (>= the 33 of a reduction)
  const int ngroups = d / 8;
  if (b >= p.batch) {                            // padding sequence of a 16-sequence group: zero operand columns
    const float zero[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int jg = tid; jg < ngroups; jg += blockDim.x) slim_comb::store_u8_h(u_tiled, d, H, hp, b, h, jg * 8, zero, 1.f);
    return;
  }
  if (s_info[2]) {                               // a flagged unit: this (head, sequence) is recomputed exactly
    for (int jg0 = 0; jg0 < ngroups; jg0 += blockDim.x)
      slim_comb::exact_groups(p, u32, b, h, jg0, min((int)blockDim.x, ngroups - jg0), s_x);
    slim_comb::convert_row(u32, u_tiled, su, d, H, hp, b, h, s_x);
    return;
  }
  // The row is first collected as floats -- in shared memory when it fits (d <= 8192), else in the global
  // scratch -- so that its scale is known before anything is stored as float16.
  const size_t ustride = (size_t)H * d;
  const bool in_smem = d <= COMBINE_SMEM_ROW;
  float* s_row = s_x + p.d_k + 2 * SLIM_TT + 4 + 36;
  float mx = 0.f;
  for (int jg = tid; jg < ngroups; jg += blockDim.x) {
    const int j0 = jg * 8;
    float acc[8];
#pragma unroll
    for (int x = 0; x < 8; ++x) acc[x] = 0.f;
    const float* Ub = p.part_u + ((size_t)(wlo + b) * H + h) * d + j0;        // unit i lives H*d floats further
    int i = 0;
    for (; i + 4 <= wn; i += 4) {                // four units' loads in flight
      float4 a[4], c[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float4* U = reinterpret_cast<const float4*>(Ub + (size_t)(i + k) * ustride);
        a[k] = __ldcs(U); c[k] = __ldcs(U + 1);
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) slim_comb::fma8(acc, s_w[i + k], a[k], c[k]);
    }
    for (; i < wn; ++i) {
      const float4* U = reinterpret_cast<const float4*>(Ub + (size_t)i * ustride);
      slim_comb::fma8(acc, s_w[i], __ldcs(U), __ldcs(U + 1));
    }
    if (in_smem) {
#pragma unroll
      for (int x = 0; x < 8; ++x) mx = fmaxf(mx, fabsf(acc[x]));
      float4* t = reinterpret_cast<float4*>(s_row + j0);
      t[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
      t[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
    } else {
      slim_comb::store_u8_f32(u32, d, H, b, h, j0, acc);
    }
  }
  if (!in_smem) {                                // wide rows: through the float scratch
    __syncthreads();
    slim_comb::convert_row(u32, u_tiled, su, d, H, hp, b, h, s_x);
    return;
  }
  mx = slim_comb::block_absmax(mx, s_x);         // (its barriers also order the row stores before the reads below)
  float inv, scale;
  slim_comb::row_scale(mx, inv, scale);
  for (int jg = tid; jg < ngroups; jg += blockDim.x) {       // each thread converts what it wrote itself
    const float4 a = *reinterpret_cast<const float4*>(s_row + jg * 8), c = *reinterpret_cast<const float4*>(s_row + jg * 8 + 4);
    const float acc[8] = {a.x, a.y, a.z, a.w, c.x, c.y, c.z, c.w};
    slim_comb::store_u8_h(u_tiled, d, H, hp, b, h, jg * 8, acc, inv);
  }
  if (tid == 0) su[(size_t)b * H + h] = scale;
}

// The same for small batches, where a sequence has many units and few (head, sequence) pairs exist:
// grid.z CTAs share the d / 8 column groups of a pair, a CTA takes G of them per pass and spreads the
// units over UL = 256 / G thread rows, whose sums meet in shared memory.  No CTA sees a whole row here,
// so the rows are left as floats in u32 and slim_convert_kernel turns them into operand tiles.
__global__ void __launch_bounds__(256, 4)
slim_combine_split_kernel(const __grid_constant__ SlimDecodeParams p, float* __restrict__ u32, const int G) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* s_w = reinterpret_cast<float*>(smem_raw);                 // [workers]
  int* s_info = reinterpret_cast<int*>(s_w + p.workers);           // wlo, wn, flagged
  int* s_prefix = s_info + 4;                                      // [batch+1]
  // [UL - 1][G][8] floats (7 KB at most) behind the prefix, 16-byte aligned (the exact path uses the same room)
  float* s_red = reinterpret_cast<float*>(smem_raw + exact_scratch_offset(p));
  const int tid = threadIdx.x, lane = tid & 31;
  const int h = blockIdx.x, b = blockIdx.y;
  const int d = p.d, H = p.H;
  slim_pdl_trigger();
  slim_pdl_wait();
  if (blockIdx.x == 0 && blockIdx.y == 0 && tid == 0) *p.any_flag = 0;   // the redo kernel has consumed it

  const SlimSched sc = slim_sched_build(p.lengths, p.batch, p.t_cap, p.workers, p.min_tiles, s_prefix, p.status, p.unit_cost);
  if (tid < 32) combine_prologue(p, sc, s_prefix, b, h, s_w, s_info, lane);
  __syncthreads();
  const int wlo = s_info[0], wn = s_info[1];
  if (s_info[2]) {                               // a flagged unit: this CTA's column groups are recomputed exactly
    for (int jg0 = blockIdx.z * G; jg0 < d / 8; jg0 += gridDim.z * G)
      slim_comb::exact_groups(p, u32, b, h, jg0, min(G, d / 8 - jg0), s_red);
    return;
  }
  const int UL = 256 / G, gi = tid % G, ul = tid / G;
  const size_t ustride = (size_t)H * d;                                       // unit i lives H*d floats further
  for (int jg0 = blockIdx.z * G; jg0 < d / 8; jg0 += gridDim.z * G) {
    const int jg = jg0 + gi, j0 = jg * 8;
    const bool live = jg < d / 8;
    float acc[8];
#pragma unroll
    for (int x = 0; x < 8; ++x) acc[x] = 0.f;
    const float* Ub = p.part_u + ((size_t)(wlo + b) * H + h) * d + j0;
    int i = ul;
    if (live) {
      for (; i + 3 * UL < wn; i += 4 * UL) {      // four units' loads in flight
        float4 a[4], c[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float4* U = reinterpret_cast<const float4*>(Ub + (size_t)(i + k * UL) * ustride);
          a[k] = __ldcs(U); c[k] = __ldcs(U + 1);
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float wg = s_w[i + k * UL];
          acc[0] = fmaf(wg, a[k].x, acc[0]); acc[1] = fmaf(wg, a[k].y, acc[1]); acc[2] = fmaf(wg, a[k].z, acc[2]); acc[3] = fmaf(wg, a[k].w, acc[3]);
          acc[4] = fmaf(wg, c[k].x, acc[4]); acc[5] = fmaf(wg, c[k].y, acc[5]); acc[6] = fmaf(wg, c[k].z, acc[6]); acc[7] = fmaf(wg, c[k].w, acc[7]);
        }
      }
      for (; i < wn; i += UL) {
        const float wg = s_w[i];
        const float4* U = reinterpret_cast<const float4*>(Ub + (size_t)i * ustride);
        const float4 a = __ldcs(U), c = __ldcs(U + 1);
        acc[0] = fmaf(wg, a.x, acc[0]); acc[1] = fmaf(wg, a.y, acc[1]); acc[2] = fmaf(wg, a.z, acc[2]); acc[3] = fmaf(wg, a.w, acc[3]);
        acc[4] = fmaf(wg, c.x, acc[4]); acc[5] = fmaf(wg, c.y, acc[5]); acc[6] = fmaf(wg, c.z, acc[6]); acc[7] = fmaf(wg, c.w, acc[7]);
      }
    }
    if (UL > 1) {                        // thread row 0 adds the other rows' sums in row order
      __syncthreads();                            // the last pass has been read
      if (ul > 0) {
        float4* r = reinterpret_cast<float4*>(s_red + ((size_t)(ul - 1) * G + gi) * 8);
        r[0] = make_float4(acc[0], acc[1], acc[2], acc[3]); r[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
      }
      __syncthreads();
      if (ul == 0) {
        for (int u2 = 1; u2 < UL; ++u2) {
          const float4* r = reinterpret_cast<const float4*>(s_red + ((size_t)(u2 - 1) * G + gi) * 8);
          const float4 a = r[0], c = r[1];
          acc[0] += a.x; acc[1] += a.y; acc[2] += a.z; acc[3] += a.w; acc[4] += c.x; acc[5] += c.y; acc[6] += c.z; acc[7] += c.w;
        }
      }
    }
    if (ul != 0 || !live) continue;
    slim_comb::store_u8_f32(u32, d, H, b, h, j0, acc);
  }
}

// operand tiles and row scales from the float rows (one CTA per (head, sequence))
__global__ void __launch_bounds__(256)
slim_convert_kernel(const float* __restrict__ u32, unsigned char* __restrict__ u_tiled, float* __restrict__ su, const int d,
                    const int H, const int hp) {
  __shared__ float s_red[33];
  slim_pdl_trigger();
  slim_pdl_wait();
  slim_comb::convert_row(u32, u_tiled, su, d, H, hp, blockIdx.y, blockIdx.x, s_red);
}

__global__ void __launch_bounds__(128)
slim_proj_tc_kernel(const __grid_constant__ CUtensorMap wmap, const float* __restrict__ hscale, const float* __restrict__ su,
                    const unsigned char* __restrict__ u_tiled,
                    float* __restrict__ o, const ProjGeom g, const int d, const int d_k, const int batch,
                    int* status, const int32_t* __restrict__ lengths, const int e) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw_u32 = smem_u32(smem_raw);
  const uint32_t base = (raw_u32 + 1023u) & ~1023u;
  unsigned char* sm = smem_raw + (base - raw_u32);
  const uint32_t stage_bytes = (uint32_t)(PJ_W_BYTES + g.u_bytes);
  const int NS = g.ns;
  const uint32_t bars = base + (uint32_t)NS * stage_bytes;
  const uint32_t bar_full = bars, bar_empty = bars + 8 * PJ_NS, bar_done = bars + 16 * PJ_NS;
  unsigned char* misc = sm + (bar_done + 8 - base);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(misc);
  volatile int* s_abort = reinterpret_cast<volatile int*>(misc + 4);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int hg = blockIdx.x, js = blockIdx.y, bg = blockIdx.z;
  const uint32_t tmem_cols = (uint32_t)(32 * g.hp);

  if (tid == 0) {
    prefetch_tensormap(&wmap);
    for (int i = 0; i < NS; ++i) { mbar_init(bar_full + 8 * i, 1); mbar_init(bar_empty + 8 * i, 1); }
    mbar_init(bar_done, 1);
    *s_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) tmem_alloc(smem_u32(s_tmem), tmem_cols);
  slim_pdl_trigger();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  const int row0 = js * g.nst * PJ_ROWS;                      // first row of W_KV,h of this CTA
  // The weights do not depend on the kernels before this one: the producer starts the W_KV tiles
  // of the first stages before the dependency wait, so they stream in while the combine kernel
  // still runs; the u tiles of those stages follow after the wait (same barrier, one byte count).
  const int npre = g.nst < NS ? g.nst : NS;
  // the weight tile of stage s (rows row0 + s * PJ_ROWS ..) into the stage at dst
  auto load_w = [&](uint32_t dst, uint32_t bar, int s) {
    if (g.hp == 1) tma_load_3d(dst, &wmap, bar, 0, hg * d + row0 + s * PJ_ROWS, 0);
    else           tma_load_3d(dst, &wmap, bar, 0, row0 + s * PJ_ROWS, 2 * hg);
  };
  if (warp == 0 && lane == 0) {
    for (int s = 0; s < npre; ++s) {
      mbar_arrive_expect_tx(bar_full + 8 * s, stage_bytes);
      load_w(base + (uint32_t)s * stage_bytes, bar_full + 8 * s, s);
    }
  }
  slim_pdl_wait();                                             // u tiles come from the combine kernel

  if (warp == 0 && lane == 0) {
    // =========================== producer ===========================
    const unsigned char* usrc = u_tiled + ((size_t)(bg * g.hg + hg) * (d / 16) + row0 / 16) * ((size_t)1024 * g.hp);
    int s = 0;
    bool ok = true;
    for (; s < npre; ++s)
      bulk_load(base + (uint32_t)s * stage_bytes + PJ_W_BYTES, usrc + (size_t)s * g.u_bytes, (uint32_t)g.u_bytes, bar_full + 8 * s);
    for (; s < g.nst; ++s) {
      const int st = s % NS;
      ok = mbar_wait<false>(bar_empty + 8 * st, ((s / NS) & 1) ^ 1, s_abort, status);
      if (!ok) break;
      const uint32_t dst = base + (uint32_t)st * stage_bytes;
      mbar_arrive_expect_tx(bar_full + 8 * st, stage_bytes);
      load_w(dst, bar_full + 8 * st, s);
      bulk_load(dst + PJ_W_BYTES, usrc + (size_t)s * g.u_bytes, (uint32_t)g.u_bytes, bar_full + 8 * st);
    }
    if (!ok) {
      // gave up: let the copies that were issued land before the CTA goes away
      const int issued = s < NS ? s : NS;
      for (int k = 0; k < issued; ++k) {
        const int j = s - 1 - k, st = j % NS;
        const unsigned long long t0 = globaltimer();
        while (!mbar_try_wait(bar_full + 8 * st, (j / NS) & 1) && globaltimer() - t0 < SLIM_WAIT_NS) {}
      }
    }
  } else if (warp == 1 && lane == 0) {
    // =========================== MMA issuer ===========================
    const uint32_t idesc = umma_idesc_f16((uint32_t)(32 * g.hp));      // both operands float16
    bool ok = true;
    for (int s = 0; s < g.nst && ok; ++s) {
      const int st = s % NS;
      ok = mbar_wait<false>(bar_full + 8 * st, (s / NS) & 1, s_abort, status);
      if (!ok) break;
      tc_fence_after();
      const uint32_t wbase = base + (uint32_t)st * stage_bytes, ubase = wbase + PJ_W_BYTES;
#pragma unroll
      for (int kk = 0; kk < PJ_ROWS / 16; ++kk)
        umma_bf16(tmem_base, desc_a(wbase + (uint32_t)kk * 2048u, PJ_ROWS * 128), desc_b(ubase + (uint32_t)(kk * 1024 * g.hp)),
                  idesc, (s | kk) ? 1u : 0u);
      umma_commit(bar_empty + 8 * st);
      if (s == g.nst - 1) umma_commit(bar_done);
    }
  }
  __syncwarp();
  // =========================== epilogue: all four warps ===========================
  // This CTA's slice result [16 sequences][128 accumulator rows] goes to shared memory (the stage
  // area is free once bar_done has completed); after a cluster barrier CTA r of the jsplit slices
  // adds sequences [16 r / jsplit, 16 (r + 1) / jsplit) over all slices in slice order.
  const int m = warp * 32 + lane;                             // accumulator row = TMEM lane
  const int upper = g.hp == 2 ? (warp >> 1) : 0;              // d_k = 64: lanes 64..127 hold the second head
  const int head = hg * g.hp + upper;
  const int c = g.hp == 2 ? (m & 63) : m;
  // the scales taken out of the operands, fetched while the MMAs run: 2^e of the rows u[b][head][:] and 2^-a of
  // the head's weights
  float sc[PJ_BG];
  {
    const float hs = hscale[head];
#pragma unroll
    for (int n = 0; n < PJ_BG; ++n) {
      const int b = bg * PJ_BG + n;
      sc[n] = b < batch ? __ldg(su + (size_t)b * (g.hg * g.hp) + head) * hs : 0.f;
    }
  }
  {
    bool ok = mbar_wait<false>(bar_done, 0, s_abort, status);
    ok = __all_sync(0xffffffffu, ok);
    uint32_t r[32];
#pragma unroll
    for (int n = 0; n < 32; ++n) r[n] = 0u;
    if (ok) {
      tc_fence_after();
      tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(32 * upper), r);
    }
    // (hi + lo) columns of a sequence, times the scales
    float* tile = reinterpret_cast<float*>(sm);
#pragma unroll
    for (int n = 0; n < PJ_BG; ++n) tile[n * 128 + m] = (__uint_as_float(r[n]) + __uint_as_float(r[PJ_BG + n])) * sc[n];
  }
  cluster_sync_all();
  {
    const int n_lo = (js * PJ_BG) / g.jsplit, n_hi = ((js + 1) * PJ_BG) / g.jsplit;
    for (int n = n_lo; n < n_hi; ++n) {
      const int b = bg * PJ_BG + n;
      float a = 0.f;
      for (int sl = 0; sl < g.jsplit; ++sl) a += ld_cluster_f32(mapa(base + (uint32_t)(n * 128 + m) * 4u, (uint32_t)sl));
      // an empty sequence has no partials: its operand columns hold whatever an earlier call left
      if (b < batch && c < d_k) o[(size_t)b * e + head * d_k + c] = lengths[b] > 0 ? a : 0.f;
    }
  }
  cluster_sync_all();                                          // nobody leaves while its tile may still be read
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, tmem_cols);
  }
}

// Combine and projection in one kernel.  The CTA of (head group, row slice js of W_KV,h, 16-sequence group)
// needs exactly the columns [row0, row0 + ncols) of u[b][h][:] for its 16 sequences, and no other CTA needs
// them: it forms them itself from the context-split partials (the weights, the sums, the scaled float16
// (hi, lo) pair written straight into the operand layout in shared memory) while the first stages of its
// weight tiles, requested before the dependency wait, stream in.  The scale is per (sequence, head, slice) --
// each slice's result is multiplied back before the slices are summed -- so nothing has to know a whole row.
// Against the two kernels this saves a launch boundary, the trip of u through global memory, and the combine
// kernel's own prologue.  A sequence with a flagged unit is recomputed exactly for the CTA's columns first.
// PF_MAXR rounds of 256 (item, column group) pairs per CTA keep the combined values in registers between the
// pass that finds the scales and the pass that stores the operands.
constexpr int PF_THREADS = 256;
constexpr int PF_MAXR = 8;                 // (the kernel is instantiated for 4 and 8 rounds)

struct FusedSmem {              // offsets (bytes) behind the barriers; all 16-byte aligned
  uint32_t prefix, info, amax, x, w, total;
};
__host__ __device__ inline FusedSmem fused_smem(const ProjGeom& g, int batch, int workers, int d_k) {
  const uint32_t items = (uint32_t)(PJ_BG * g.hp);
  FusedSmem f;
  uint32_t off = 0;
  f.prefix = off; off += (uint32_t)((sizeof(int) * (batch + 1) + 15) & ~15u);
  f.info = off;   off += 16u * items;
  f.amax = off;   off += (uint32_t)((4u * items + 15) & ~15u);
  f.x = off;      off += (uint32_t)((sizeof(float) * (d_k + 2 * SLIM_TT + 4 + 36) + 15) & ~15u);
  f.w = off;      off += (uint32_t)((sizeof(float) * items * workers + 15) & ~15u);
  f.total = off;
  return f;
}

template <int MAXR>
__global__ void __launch_bounds__(PF_THREADS, 2)
slim_tail_fused_kernel(const __grid_constant__ CUtensorMap wmap, const __grid_constant__ SlimDecodeParams p,
                       const float* __restrict__ hscale, float* __restrict__ u32, const ProjGeom g, const int from_u32) {
  // from_u32: the rows u[b][h][:] are already combined (float rows in u32, written by the column-split combine of
  // small batches); the CTA only turns its columns into operand tiles, which saves the conversion kernel.
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw_u32 = smem_u32(smem_raw);
  const uint32_t base = (raw_u32 + 1023u) & ~1023u;
  unsigned char* sm = smem_raw + (base - raw_u32);
  const int NS = g.ns;
  const uint32_t u_region = base + (uint32_t)NS * PJ_W_BYTES;              // all nst stages of u operand tiles
  const uint32_t bars = u_region + (uint32_t)(g.nst * g.u_bytes);
  const uint32_t bar_full = bars, bar_empty = bars + 8 * PJ_NS, bar_done = bars + 16 * PJ_NS;
  unsigned char* misc = sm + (bar_done + 8 - base);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(misc);
  volatile int* s_abort = reinterpret_cast<volatile int*>(misc + 4);
  const FusedSmem fs = fused_smem(g, p.batch, p.workers, p.d_k);
  unsigned char* area = misc + 24;                            // (16-byte aligned: the barriers end 8 bytes short of it)
  int* s_prefix = reinterpret_cast<int*>(area + fs.prefix);
  int* s_info = reinterpret_cast<int*>(area + fs.info);                    // per item: first worker, unit count, flagged
  int* s_amax = reinterpret_cast<int*>(area + fs.amax);                    // per item: bits of the largest magnitude
  float* s_x = reinterpret_cast<float*>(area + fs.x);
  float* s_w = reinterpret_cast<float*>(area + fs.w);                      // per item: [workers] weights

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int hg = blockIdx.x, js = blockIdx.y, bg = blockIdx.z;
  const int d = p.d, H = p.H, hp = g.hp;
  const uint32_t tmem_cols = (uint32_t)(32 * hp);
  const int items = PJ_BG * hp;                               // (sequence, head of the group) pairs of this CTA

  if (tid == 0) {
    prefetch_tensormap(&wmap);
    for (int i = 0; i < NS; ++i) { mbar_init(bar_full + 8 * i, 1); mbar_init(bar_empty + 8 * i, 1); }
    mbar_init(bar_done, 1);
    *s_abort = 0;
    fence_mbar_init();
  }
  if (tid < items) s_amax[tid] = 0;
  if (warp == 1) tmem_alloc(smem_u32(s_tmem), tmem_cols);
  slim_pdl_trigger();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  const int row0 = js * g.nst * PJ_ROWS;                      // first row of W_KV,h = first column of u of this CTA
  const int ncols = g.nst * PJ_ROWS;
  const int npre = g.nst < NS ? g.nst : NS;
  auto load_w = [&](uint32_t dst, uint32_t bar, int s) {
    if (hp == 1) tma_load_3d(dst, &wmap, bar, 0, hg * d + row0 + s * PJ_ROWS, 0);
    else         tma_load_3d(dst, &wmap, bar, 0, row0 + s * PJ_ROWS, 2 * hg);
  };
  // the weights do not depend on the kernels before this one: the first stages are requested now
  if (warp == 0 && lane == 0) {
    for (int s = 0; s < npre; ++s) {
      mbar_arrive_expect_tx(bar_full + 8 * s, PJ_W_BYTES);
      load_w(base + (uint32_t)s * PJ_W_BYTES, bar_full + 8 * s, s);
    }
  }
  slim_pdl_wait();                                             // the partials come from the decode kernel
  if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && tid == 0 && !from_u32) *p.any_flag = 0;

  // ---- combine: units and weights of the CTA's (sequence, head) items ----
  if (!from_u32) {
  const SlimSched sc = slim_sched_build(p.lengths, p.batch, p.t_cap, p.workers, p.min_tiles, s_prefix, p.status, p.unit_cost);
  {
    // All items at once: LPI = 256 / items lanes (16 or 8, a power of two within a warp) share an item and take its
    // units i = sub, sub + LPI, ...:  w_i = 2^(m_i - M) / sum_j 2^(m_j - M) l_j,  M = max_j (m_j + log2 l_j).
    const int LPI = PF_THREADS / items, item = tid / LPI, sub = tid % LPI;
    const int b = bg * PJ_BG + item / hp, h = hg * hp + item % hp;
    float* sw = s_w + (size_t)item * p.workers;
    int wlo = 0, wn = 0, flagged = 0;
    if (b < p.batch && s_prefix[b + 1] > s_prefix[b]) {
      wlo = slim_worker_of_tile(sc, s_prefix[b]);
      wn = slim_worker_of_tile(sc, s_prefix[b + 1] - 1) - wlo + 1;
      if (p.redo_in_combine)
        for (int i = sub; i < 2 * wn; i += LPI) flagged |= p.unit_flags[2 * (wlo + b) + i];
    }
    float M = -INFINITY, m0 = 0.f, l0 = 0.f;                  // (m, l) of this lane's first unit stay in registers
    for (int i = sub; i < wn; i += LPI) {
      const size_t ui = (size_t)(wlo + b + i) * H + h;
      const float mi = __ldcg(p.part_m + ui), li = __ldcg(p.part_l + ui);
      if (i == sub) { m0 = mi; l0 = li; }
      M = fmaxf(M, mi + log2f(li));
    }
    for (int o = LPI >> 1; o > 0; o >>= 1) {
      M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
      flagged |= __shfl_xor_sync(0xffffffffu, flagged, o);
    }
    float L = 0.f;
    for (int i = sub; i < wn; i += LPI) {
      const size_t ui = (size_t)(wlo + b + i) * H + h;
      const float mi = i == sub ? m0 : __ldcg(p.part_m + ui), li = i == sub ? l0 : __ldcg(p.part_l + ui);
      const float wg = exp2f(mi - M);
      sw[i] = wg;
      L += wg * li;
    }
    for (int o = LPI >> 1; o > 0; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
    const float inv = 1.f / L;
    __syncwarp();
    for (int i = sub; i < wn; i += LPI) sw[i] *= inv;
    if (sub == 0) { s_info[4 * item] = wlo; s_info[4 * item + 1] = wn; s_info[4 * item + 2] = flagged != 0; }
  }
  __syncthreads();
  // a sequence with a flagged unit: its columns are recomputed exactly into the float scratch first (rare)
  for (int item = 0; item < items; ++item)
    if (s_info[4 * item + 2]) slim_comb::exact_groups(p, u32, bg * PJ_BG + item / hp, hg * hp + item % hp, row0 / 8, ncols / 8, s_x);
  } else if (tid < items) {
    s_info[4 * tid] = 0; s_info[4 * tid + 1] = 0; s_info[4 * tid + 2] = 1;         // every row comes from the float scratch
  }
  __syncthreads();
  const int gpi = ncols / 8;                                  // column groups per item
  const int total = items * gpi, rounds = (total + PF_THREADS - 1) / PF_THREADS;
  const size_t ustride = (size_t)H * d;
  constexpr int UB = MAXR <= 4 ? 8 : 4;                       // units whose loads are in flight together
  float acc[MAXR][8];
#pragma unroll
  for (int r = 0; r < MAXR; ++r) {
#pragma unroll
    for (int x = 0; x < 8; ++x) acc[r][x] = 0.f;
    const int idx = r * PF_THREADS + tid;
    if (r < rounds && idx < total) {
      const int item = idx / gpi, jg = idx - item * gpi;
      const int b = bg * PJ_BG + item / hp, h = hg * hp + item % hp, j0 = row0 + jg * 8;
      const int wlo = s_info[4 * item], wn = s_info[4 * item + 1];
      if (b < p.batch) {
        if (s_info[4 * item + 2]) {
          const float4* U = reinterpret_cast<const float4*>(u32 + ((size_t)b * H + h) * d + j0);
          const float4 a = U[0], c = U[1];
          acc[r][0] = a.x; acc[r][1] = a.y; acc[r][2] = a.z; acc[r][3] = a.w; acc[r][4] = c.x; acc[r][5] = c.y; acc[r][6] = c.z; acc[r][7] = c.w;
        } else {
          const float* sw = s_w + (size_t)item * p.workers;
          const float* Ub = p.part_u + ((size_t)(wlo + b) * H + h) * d + j0;        // unit i lives H*d floats further
          for (int i = 0; i < wn; i += UB) {         // UB units' loads in flight (a short last batch repeats its last unit with weight 0)
            float4 a[UB], c[UB];
#pragma unroll
            for (int k = 0; k < UB; ++k) {
              const float4* U = reinterpret_cast<const float4*>(Ub + (size_t)min(i + k, wn - 1) * ustride);
              a[k] = __ldcs(U); c[k] = __ldcs(U + 1);
            }
#pragma unroll
            for (int k = 0; k < UB; ++k) slim_comb::fma8(acc[r], i + k < wn ? sw[i + k] : 0.f, a[k], c[k]);
          }
        }
        float mx = 0.f;
#pragma unroll
        for (int x = 0; x < 8; ++x) mx = fmaxf(mx, fabsf(acc[r][x]));
        if (!(mx <= 3.0e38f)) mx = 3.4e38f;          // a NaN or an infinity: the row keeps scale 1 (row_scale)
        atomicMax(s_amax + item, __float_as_int(mx));
      }
    }
  }
  __syncthreads();
#pragma unroll
  for (int r = 0; r < MAXR; ++r) {
    const int idx = r * PF_THREADS + tid;
    if (r < rounds && idx < total) {
      const int item = idx / gpi, jg = idx - item * gpi;
      float inv, scale;
      slim_comb::row_scale(__int_as_float(s_amax[item]), inv, scale);
      uint32_t hi[4], lo[4];
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        const float v0 = acc[r][2 * x] * inv, v1 = acc[r][2 * x + 1] * inv;
        const __half h0 = __float2half_rn(v0), h1 = __float2half_rn(v1);
        const __half l0 = __float2half_rn(v0 - __half2float(h0)), l1 = __float2half_rn(v1 - __half2float(h1));
        hi[x] = (uint32_t)__half_as_ushort(h0) | ((uint32_t)__half_as_ushort(h1) << 16);
        lo[x] = (uint32_t)__half_as_ushort(l0) | ((uint32_t)__half_as_ushort(l1) << 16);
      }
      const int n = item / hp, jl = jg * 8;                   // column within the CTA's slice
      const uint32_t t = u_region + (uint32_t)(jl / 16) * (uint32_t)(1024 * hp) + (uint32_t)(item % hp) * 1024u;
      sts128(t + slim_comb::u_offset(n, jl & 15), make_uint4(hi[0], hi[1], hi[2], hi[3]));
      sts128(t + slim_comb::u_offset(PJ_BG + n, jl & 15), make_uint4(lo[0], lo[1], lo[2], lo[3]));
    }
  }
  fence_proxy_async_smem();                                    // operand tiles: generic-proxy stores -> tensor-core reads
  __syncthreads();

  if (warp == 0 && lane == 0) {
    // =========================== producer: the remaining weight stages ===========================
    int s = npre;
    bool ok = true;
    for (; s < g.nst; ++s) {
      const int st = s % NS;
      ok = mbar_wait<false>(bar_empty + 8 * st, ((s / NS) & 1) ^ 1, s_abort, p.status);
      if (!ok) break;
      mbar_arrive_expect_tx(bar_full + 8 * st, PJ_W_BYTES);
      load_w(base + (uint32_t)st * PJ_W_BYTES, bar_full + 8 * st, s);
    }
    if (!ok) {
      // gave up: let the copies that were issued land before the CTA goes away
      const int issued = s < NS ? s : NS;
      for (int k = 0; k < issued; ++k) {
        const int j = s - 1 - k, st = j % NS;
        const unsigned long long t0 = globaltimer();
        while (!mbar_try_wait(bar_full + 8 * st, (j / NS) & 1) && globaltimer() - t0 < SLIM_WAIT_NS) {}
      }
    }
  } else if (warp == 1 && lane == 0) {
    // =========================== MMA issuer ===========================
    const uint32_t idesc = umma_idesc_f16((uint32_t)(32 * hp));        // both operands float16
    bool ok = true;
    for (int s = 0; s < g.nst && ok; ++s) {
      const int st = s % NS;
      ok = mbar_wait<false>(bar_full + 8 * st, (s / NS) & 1, s_abort, p.status);
      if (!ok) break;
      tc_fence_after();
      const uint32_t wbase = base + (uint32_t)st * PJ_W_BYTES, ubase = u_region + (uint32_t)(s * g.u_bytes);
#pragma unroll
      for (int kk = 0; kk < PJ_ROWS / 16; ++kk)
        umma_bf16(tmem_base, desc_a(wbase + (uint32_t)kk * 2048u, PJ_ROWS * 128), desc_b(ubase + (uint32_t)(kk * 1024 * hp)),
                  idesc, (s | kk) ? 1u : 0u);
      umma_commit(bar_empty + 8 * st);
      if (s == g.nst - 1) umma_commit(bar_done);
    }
  }
  __syncwarp();
  // =========================== epilogue (warps 0-3 hold the 128 accumulator rows) ===========================
  const int m = (warp & 3) * 32 + lane;                       // accumulator row = TMEM lane
  const int upper = hp == 2 ? ((warp & 3) >> 1) : 0;          // d_k = 64: lanes 64..127 hold the second head
  const int head = hg * hp + upper;
  const int c = hp == 2 ? (m & 63) : m;
  if (warp < 4) {
    bool ok = mbar_wait<false>(bar_done, 0, s_abort, p.status);
    ok = __all_sync(0xffffffffu, ok);
    uint32_t r[32];
#pragma unroll
    for (int n = 0; n < 32; ++n) r[n] = 0u;
    if (ok) {
      tc_fence_after();
      tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(32 * upper), r);
    }
    // (hi + lo) columns of a sequence, times the scales taken out of the operands: 2^e of the item's slice and
    // 2^-a of the head's weights
    const float hs = hscale[head];
    float* tile = reinterpret_cast<float*>(sm);
#pragma unroll
    for (int n = 0; n < PJ_BG; ++n) {
      float inv, scale;
      slim_comb::row_scale(__int_as_float(s_amax[n * hp + upper]), inv, scale);
      tile[n * 128 + m] = (__uint_as_float(r[n]) + __uint_as_float(r[PJ_BG + n])) * (scale * hs);
    }
  }
  cluster_sync_all();
  if (warp < 4) {
    const int n_lo = (js * PJ_BG) / g.jsplit, n_hi = ((js + 1) * PJ_BG) / g.jsplit;
    for (int n = n_lo; n < n_hi; ++n) {
      const int b = bg * PJ_BG + n;
      float a = 0.f;
      for (int sl = 0; sl < g.jsplit; ++sl) a += ld_cluster_f32(mapa(base + (uint32_t)(n * 128 + m) * 4u, (uint32_t)sl));
      if (b < p.batch && c < p.d_k) p.o[(size_t)b * p.e + head * p.d_k + c] = p.lengths[b] > 0 ? a : 0.f;
    }
  }
  cluster_sync_all();                                          // nobody leaves while its tile may still be read
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, tmem_cols);
  }
}

ProjGeom make_proj_geom(int d, int H, int d_k, int batch, int ns_opt = 0) {
  ProjGeom g;
  g.hp = d_k == 64 ? 2 : 1;
  g.hg = H / g.hp;
  const int stages = d / PJ_ROWS;
  int js = 1;
  for (int c = 1; c <= 8; ++c)
    if (stages % c == 0) js = c;
  g.jsplit = js;
  g.nst = stages / js;
  g.nbg = (batch + PJ_BG - 1) / PJ_BG;
  g.u_bytes = (PJ_ROWS / 16) * 1024 * g.hp;
  g.ns = PJ_NS;
  if (ns_opt >= 2 && ns_opt <= PJ_NS) g.ns = ns_opt;          // sweeps
  return g;
}

size_t proj_smem_bytes(const ProjGeom& g) { return 1024 + (size_t)g.ns * (PJ_W_BYTES + g.u_bytes) + 16 * PJ_NS + 8 + 16 + 64; }
size_t fused_smem_bytes(const ProjGeom& g, int batch, int workers, int d_k) {
  return 1024 + (size_t)g.ns * PJ_W_BYTES + (size_t)g.nst * g.u_bytes + 16 * PJ_NS + 8 + 24 + fused_smem(g, batch, workers, d_k).total + 64;
}

}  // namespace

int slim_proj_shape_ok(int d, int H, int d_k, int dtype) {
  if (dtype != SLIM_BF16) return 0;
  if (d_k != 64 && d_k != 96 && d_k != 128) return 0;
  if (d % PJ_ROWS != 0 || (d_k == 64 && (H & 1))) return 0;
  return 1;
}

int slim_proj_jsplit(int d) { return make_proj_geom(d, 2, 64, 1).jsplit; }

size_t slim_proj_u_bytes(int d, int H, int batch) {
  return (size_t)((batch + PJ_BG - 1) / PJ_BG) * PJ_BG * H * d * sizeof(float);
}

cudaError_t slim_proj_make_wmap(slim_ctx* ctx) {
  const int d = ctx->d, d_k = ctx->d_k, H = ctx->H;
  unsigned long long dims[3], strides[2];
  unsigned int box[3] = {64, PJ_ROWS, 2};
  if (d_k != 64) {           // (64 columns, H*d rows, 2 column halves).  With d_k = 96 the second half runs
                             // 32 columns into the next row: finite weights that land in ignored accumulator
                             // rows (the W_KV allocation is padded so the very last row stays in bounds).
    dims[0] = 64; dims[1] = (unsigned long long)H * d; dims[2] = 2;
    strides[0] = (unsigned long long)d_k * 2; strides[1] = 128;
  } else {                   // d_k = 64: (64 columns, d rows, H heads)
    dims[0] = 64; dims[1] = d; dims[2] = H;
    strides[0] = 128; strides[1] = (unsigned long long)d * 128;
  }
  // (the float16 copy is described as a 16-bit type of the same size: the copy engine only moves bits)
  cudaError_t e = slim_tmap_encode_3d(ctx->wmap, ctx->wkv, dims, strides, box);
  if (e == cudaSuccess) e = slim_tmap_encode_3d(ctx->wmap_h, ctx->wkv_h, dims, strides, box);
  if (e != cudaSuccess) return e;
  const ProjGeom g = make_proj_geom(d, H, d_k, 1, PJ_NS);      // the largest stage count a sweep may ask for
  return cudaFuncSetAttribute((const void*)slim_proj_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)proj_smem_bytes(g));
}

// Small batches (fewer than two (head, sequence) pairs per SM): the combine is split over column slices
// (grid.z) so that ~2 CTAs per SM exist; returns the slice count (1 = the one-CTA-per-row kernel).
static int combine_slices(const slim_ctx* ctx, int H, int batch, int d) {
  const int ngroups = d / 8;
  int nslice = 1;
  while (nslice < 16 && (long long)H * batch * nslice < 2 * ctx->num_sms && ngroups / (2 * nslice) >= 32) nslice <<= 1;
  return nslice;
}

int slim_proj_needs_convert(const slim_ctx* ctx, int batch) { return combine_slices(ctx, ctx->H, batch, ctx->d) > 1 ? 1 : 0; }

// Combine and projection in one kernel?  (see slim_tail_fused_kernel)  Measured: where the tail is a chain of
// latencies over little data (many short sequences: 64 x 1500 rows at d = 1280: step 2.53 -> 2.40 ms) the fused
// kernel wins; where a CTA has a lot of partials to pull out of L2 (16 long sequences at d = 4096: 184 KB per
// CTA) the separate combine kernel with four times the threads per SM is faster (step 10.47 against 10.70 ms).
// In between (the same 64 sequences with lone-CTA workers, 148 of them: 108 KB) the separate kernels still win
// (X-cache scheme: 5.21 against 5.69 ms).  The partial bytes per CTA are estimated from the unit count a
// sequence has on average.
static bool fused_possible(const slim_ctx* ctx, const SlimDecodeParams& p, const ProjGeom& g) {
  return ctx->opt_tail_fused && g.hp * (g.nst * PJ_ROWS) <= 128 * PF_MAXR &&
         fused_smem_bytes(g, p.batch, p.workers, p.d_k) <= (size_t)227 * 1024;
}
static bool tail_fused(const slim_ctx* ctx, const SlimDecodeParams& p, const ProjGeom& g) {
  if (!fused_possible(ctx, p, g) || combine_slices(ctx, p.H, p.batch, p.d) != 1) return false;
  if (ctx->opt_tail_fused >= 2) return true;                  // forced (sweeps)
  const double units_per_seq = (double)(p.workers + p.batch) / p.batch;
  return 4.0 * PJ_BG * g.hp * (g.nst * PJ_ROWS) * units_per_seq <= 80.0 * 1024;
}
// Small batches (column-split combine into float rows): the fused kernel takes the rows from there and makes
// the operand tiles itself, so no conversion kernel runs.
static bool convert_fused(const slim_ctx* ctx, const SlimDecodeParams& p, const ProjGeom& g) {
  return fused_possible(ctx, p, g) && combine_slices(ctx, p.H, p.batch, p.d) > 1;
}
int slim_proj_launch_count(const slim_ctx* ctx, const SlimDecodeParams& p) {
  const ProjGeom g = make_proj_geom(p.d, p.H, p.d_k, p.batch, ctx->opt_proj_ns);
  if (tail_fused(ctx, p, g)) return 1;
  if (convert_fused(ctx, p, g)) return 2;
  return 2 + slim_proj_needs_convert(ctx, p.batch);
}

static cudaError_t launch_fused(const slim_ctx* ctx, const SlimDecodeParams& p, const ProjGeom& g, float* u32, int from_u32,
                                cudaStream_t st) {
  const size_t smem = fused_smem_bytes(g, p.batch, p.workers, p.d_k);
  const bool r4 = g.hp * (g.nst * PJ_ROWS) <= 128 * 4;      // rounds of 256 (item, column group) pairs per CTA
  void (*kern)(const CUtensorMap, const SlimDecodeParams, const float*, float*, const ProjGeom, const int) =
      r4 ? slim_tail_fused_kernel<4> : slim_tail_fused_kernel<8>;
  static size_t attr_set[64][2] = {};              // function attributes are kept per device
  if (ctx->device < 0 || ctx->device >= 64 || attr_set[ctx->device][r4] < smem) {
    cudaError_t e = cudaFuncSetAttribute((const void*)kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if (ctx->device >= 0 && ctx->device < 64) attr_set[ctx->device][r4] = smem;
  }
  CUtensorMap map;
  memcpy(&map, ctx->wmap_h, sizeof(map));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(g.hg, g.jsplit, g.nbg);
  cfg.blockDim = dim3(PF_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;            // the row slices of one output tile
  attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = g.jsplit; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, kern, map, p, (const float*)ctx->wkv_hscale, u32, g, from_u32);
}

cudaError_t slim_launch_proj(const slim_ctx* ctx, const SlimDecodeParams& p, unsigned char* u_tiled, float* u32, float* su,
                             cudaStream_t st) {
  const ProjGeom g = make_proj_geom(p.d, p.H, p.d_k, p.batch, ctx->opt_proj_ns);
  // One kernel for combine and projection where every (head, sequence) row has a CTA of its own anyway (no
  // column-split combine) and a CTA's share of the combined values fits its registers.
  if (tail_fused(ctx, p, g)) return launch_fused(ctx, p, g, u32, 0, st);
  {
    // No CTAs for the padding sequences of a 16-sequence group in the split variant (their columns of the
    // projection's B operand stay unwritten and only feed outputs that are never stored).
    const int ngroups = p.d / 8;
    const int nslice = combine_slices(ctx, p.H, p.batch, p.d);
    cudaError_t e;
    if (nslice > 1) {
      int G = 256;
      while (G > 32 && G / 2 * nslice >= ngroups) G >>= 1;
      const size_t smem = sizeof(float) * p.workers + sizeof(int) * (4 + p.batch + 1) + 16 + sizeof(float) * 7 * 256;
      e = slim_launch_pdl(slim_combine_split_kernel, dim3(p.H, p.batch, nslice), dim3(256), smem, st, p, u32, G);
      if (e == cudaSuccess && convert_fused(ctx, p, g)) return launch_fused(ctx, p, g, u32, 1, st);
      if (e == cudaSuccess)
        e = slim_launch_pdl(slim_convert_kernel, dim3(p.H, p.batch), dim3(256), 0, st, (const float*)u32, u_tiled, su, p.d, p.H, g.hp);
    } else {
      dim3 grid(p.H, g.nbg * PJ_BG);
      // weights, info, prefix | exact path / reduction scratch | the float row
      const size_t smem = sizeof(float) * p.workers + sizeof(int) * (4 + p.batch + 1) + 16 + sizeof(float) * (p.d_k + 2 * SLIM_TT + 4 + 36) +
                          sizeof(float) * (p.d <= COMBINE_SMEM_ROW ? p.d : 0) + 16;
      if (smem > 48 * 1024) {
        e = cudaFuncSetAttribute((const void*)slim_combine_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
      }
      e = slim_launch_pdl(slim_combine_kernel, grid, dim3(256), smem, st, p, u_tiled, u32, su, g.hp);
    }
    if (e != cudaSuccess) return e;
  }
  CUtensorMap map;
  memcpy(&map, ctx->wmap_h, sizeof(map));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(g.hg, g.jsplit, g.nbg);
  cfg.blockDim = dim3(128);
  cfg.dynamicSmemBytes = proj_smem_bytes(g);
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;            // the row slices of one output tile
  attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = g.jsplit; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, slim_proj_tc_kernel, map, (const float*)ctx->wkv_hscale, (const float*)su, (const unsigned char*)u_tiled,
                            p.o, g, p.d, p.d_k, p.batch, p.status, p.lengths, p.e);
}
