// Tensor-core decode path for sm_100a: TMA-staged K tiles, CUDA-core scores
// with RoPE in registers, tcgen05 (UMMA) weighted sum of the raw keys with the
// accumulator in tensor memory.
//
// Work split.  A *worker* is a cluster of two CTAs; CTA r of the pair owns the
// key columns [r d/2, (r+1) d/2) and therefore the heads that live in those
// columns.  Both CTAs walk the same context tiles (16 rows) of the worker's
// units.  Per tile and CTA:
//   producer warp   one TMA load brings the [16 x d/2] slice of the tile into a
//                   128-byte-swizzled shared-memory stage (each key byte is
//                   staged exactly once in the whole GPU);
//   score warps     (two heads each) read the stage and form the softmax
//                   arguments of their heads (Eq. 2).  A thread owns one head,
//                   eight rotation pairs and every RP-th row of the tile.  The
//                   rotation of the RoPE appendix (Option 1: keys are rotated
//                   after the read) is moved onto the query: with q^ the query
//                   at its own position, q^ . RoPE_t(k) = Q(t) . k where
//                   Q(t) = q^ e^{i t theta} per pair, and Q is stepped from row
//                   to row by one packed complex multiplication in registers
//                   (re-seeded from the tables every TC_RESEED tiles).  The
//                   arguments become p = 2^(s - m_ref); the bf16 probabilities
//                   are shipped into the P tile of BOTH CTAs with st.async
//                   (distributed shared memory; the bytes complete on the
//                   receiver's p_full barrier, so no thread waits on a remote
//                   fence), because every head weights the full key row;
//   MMA warp        U^T[128 cols x 32 heads] += K_tile^T[128 x 16] P^T[16 x 32]
//                   for every 128-column chunk of the slice: one tcgen05.mma
//                   per chunk, A = the staged keys (MN-major, straight from
//                   the TMA layout), B = the P tile, D in tensor memory
//                   (Eq. 7 Option 2: the weighted sum of the full-width keys).
// At the end of a unit warps 0-3 read U from tensor memory and write the
// partial (m_ref, l, U) for the log-sum-exp combine.
//
// Narrow shapes (d_k = 64 without RoPE, d <= 2048: the Whisper-like ones) run with one CTA per
// worker (CL = 1): the whole key row and all heads live in one SM, the P exchange stays local and
// twice as many workers share the context.
//
// Two score-warp sets (SETS = 2, the narrow d_k = 64 shapes).  There a tile is so small that a score
// warp's chain of dependent steps per tile (wait, shared-memory reads, dot products, shuffles,
// exponent, staging, shipping), not its instruction count, sets the pace.  With two sets of score
// warps, set s forms the probabilities of the worker's tiles number s, s + 2, ... (counted through all
// its units), so two tiles are in the chain at once and a set only ever meets the stages of its own
// parity.  The set that has a unit's first tile fixes m_ref and hands it to the other through shared
// memory (barrier xm); the other hands its share of l back at the unit's end (barrier xl).  Both
// sets wait on both barriers in every unit, which orders the re-use of the two slots.
//
// Softmax reference.  m_ref of a (unit, head) is the maximum argument of the
// unit's first tile and is never changed, so the accumulator is never rescaled.
// 2^(s - m_ref) is exact in relative terms for any exponent below 2^127; a later
// argument more than 96 (log2 units) above m_ref sets the unit's flag and the
// unit is redone by the exact CUDA-core kernel afterwards.  l is accumulated
// from the bf16-rounded p, so U / l stays an exact weighted mean of key rows.
//
// With k_new set, the worker that owns a sequence's last tile first writes the newest key row
// (position lengths[b] - 1, each CTA its own column half) and orders the write before its TMA reads:
// the cache update of the generate phase needs no kernel of its own.
//
// Every wait on an mbarrier is bounded in time; a wait that runs out sets the
// device status to SLIM_ERR_TIMEOUT, all roles leave their loops, and the CTA
// frees its tensor memory and exits.
#include <cuda.h>
#include <cstring>

#include "slim_internal.h"
#include "slim_sched.cuh"
#include "slim_ptx.cuh"

namespace {
using namespace slim_ptx;

// Compile-time instrumentation, off by default (-DSLIM_TC_TRACE, see build.py and trace.py): for the first
// SLIM_TRACE_TILES tiles of every CTA one thread of each role stores the SM clock at fixed points of its
// per-tile loop.  Slots: 0 producer at the top of its loop, 1 producer when the stage is free (load issued),
// 2 score warp 0 when the keys have landed, 3 when its probabilities are computed, 4 when the P stage is
// free, 5 when it has shipped and released, 6 MMA thread when the tile's probabilities are complete,
// 7 when its MMAs and the commit are issued.  The last tile index (SLIM_TRACE_TILES - 1, beyond any worker's
// tile count at the traced shapes) holds whole-kernel marks of thread 0: slot 0 kernel entry, 1 set-up done,
// 2 / 3 begin / end of the drain of its last unit's accumulator, 4 kernel exit.
#ifdef SLIM_TC_TRACE
#define TC_TRACE(slot, tile_no)                                                                              \
  do {                                                                                                       \
    if (p.trace && (tile_no) < SLIM_TRACE_TILES)                                                             \
      p.trace[((size_t)blockIdx.x * SLIM_TRACE_TILES + (tile_no)) * 8 + (slot)] = clock64();                 \
  } while (0)
#else
#define TC_TRACE(slot, tile_no) do {} while (0)
#endif
// the score warp whose per-tile points are recorded (-DSLIM_TC_TRACE_WARP=n to look at another one)
#ifndef SLIM_TC_TRACE_WARP
#define SLIM_TC_TRACE_WARP 0
#endif
#define TC_TRACE_MARK(slot) do { if (threadIdx.x == 0) TC_TRACE(slot, SLIM_TRACE_TILES - 1); } while (0)

constexpr int TC_P_BYTES = 1024;         // [32 heads][16 rows] bf16
constexpr int TC_MAX_NS = 8;             // K stages
constexpr int TC_MAX_SW = 16;            // score warps
constexpr float TC_XMAX = 96.f;          // largest exponent accepted above m_ref
constexpr int TC_RESEED = 64;            // tiles between exact re-seeds of the stepped query rotation

struct TcGeom {
  int cl;           // CTAs per worker
  int dsl;          // key columns per CTA (d / cl)
  int nch;          // 128-column chunks per CTA
  int nc64;         // 64-column TMA chunks per CTA
  int hl;           // heads per CTA
  int nsw;          // score warps of one set (tc_heads_per_warp heads each)
  int sets;         // score-warp sets
  int nswl;         // launched score/epilogue warps = max(4, nsw * sets)
  int ns;           // K stages
  int stage_bytes;  // 16 * dsl * 2
  int tmem_cols;    // power of two >= 32 * nch
};

// Lane mapping of the score warps: JL lanes share a (head, row set); a thread
// owns RT rows of the tile; 16 / RT row sets and JL lanes make one head.
__host__ __device__ constexpr int tc_jl(int dk) { return dk / 16 <= 4 ? 4 : 8; }
__host__ __device__ constexpr int tc_heads_per_warp(int dk, int rt) { return 32 / (tc_jl(dk) * (SLIM_TT / rt)); }
constexpr int TC_SETS2_WARPS = 10;       // score warps of a two-set launch (both sets together), at most
__host__ __device__ constexpr int tc_threads(int dk, int rt, int cl, int sets) {
  // up to 32 / cl heads per CTA, at least four score/epilogue warps, plus the producer and MMA warps
  return sets == 2 ? 32 * (TC_SETS2_WARPS + 2)
                   : 32 * (((32 / cl) / tc_heads_per_warp(dk, rt) < 4 ? 4 : (32 / cl) / tc_heads_per_warp(dk, rt)) + 2);
}

// ------------------------------------------------------------------ the kernel
// EXT: the softmax arguments are read from p.ext_scores (X-cache scheme) instead of being
// formed from the staged rows; the rest of the pipeline is the same.
// CL: CTAs per worker (cluster size), 2 or 1.  SETS: score-warp sets, 1 or 2.
template <int DK, bool ROPE, int RT, bool EXT, int CL, int SETS>
__global__ void __launch_bounds__(tc_threads(DK, RT, CL, SETS), 1)
slim_tc_kernel(const __grid_constant__ CUtensorMap tmap, const SlimDecodeParams p, const TcGeom g) {
  constexpr int PAIRS = DK / 2;                   // rotation pairs (j, j + DK/2) per head
  constexpr int OCT = PAIRS / 8;                  // 8-pair groups per head
  constexpr int JL = tc_jl(DK);                   // lanes along j (lanes >= OCT idle)
  constexpr int RP = SLIM_TT / RT;                // a thread owns the RT rows rp, rp + RP, ...
  constexpr int DUP = JL / RT;                    // lanes that end up with the same row's sum
  constexpr int HL = JL * RP;                     // lanes per head
  constexpr int HW = 32 / HL;                     // heads per warp
  // PAIR (with the two score-warp sets, stage count even): stages 2k and 2k + 1 are freed together by
  // one commit on p_empty[k]; the MMA thread then takes two tiles per turn of its loop where it can,
  // which halves its waits, fences, commits and loop bookkeeping per tile.
  constexpr bool PAIR = SETS == 2;
  static_assert(RT <= JL && HL <= 32 && HW == tc_heads_per_warp(DK, RT), "lane mapping");

  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw_u32 = smem_u32(smem_raw);
  const uint32_t base = (raw_u32 + 1023u) & ~1023u;
  unsigned char* sm = smem_raw + (base - raw_u32);
  const uint32_t k_stage0 = base;
  const uint32_t p_stage0 = base + (uint32_t)g.ns * g.stage_bytes;
  const uint32_t stg0 = p_stage0 + TC_MAX_NS * TC_P_BYTES;            // per-warp P staging: 2 x 64 B
  const uint32_t bars = stg0 + TC_MAX_SW * 128;
  const uint32_t bar_k_full = bars, bar_k_empty = bars + 8 * TC_MAX_NS;
  const uint32_t bar_p_full = bars + 16 * TC_MAX_NS, bar_p_empty = bar_p_full + 8 * TC_MAX_NS;
  const uint32_t bar_u_full = bar_p_empty + 8 * TC_MAX_NS, bar_u_empty = bar_u_full + 8;
  const uint32_t bar_xm = bar_u_empty + 8, bar_xl = bar_xm + 8;
  unsigned char* misc = sm + (bar_xl + 8 - base);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(misc);
  volatile int* s_abort = reinterpret_cast<volatile int*>(misc + 4);
  float* s_xm = reinterpret_cast<float*>(misc + 8);          // m_ref per local head, set 0 -> set 1
  float* s_xl = s_xm + 32;                                   // l per local head, set 1 -> set 0
  int* s_prefix = reinterpret_cast<int*>(misc + 8 + 256);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t rank = cluster_ctarank();
  const int w = blockIdx.x / CL;                  // worker = cluster index
  const int producer_warp = g.nswl, mma_warp = g.nswl + 1;
  TC_TRACE_MARK(0);

  // ---- set-up -------------------------------------------------------------------
  const int nepi = (g.nswl / 4) * 4;              // warps that drain the accumulator at a unit's end
  if (tid == 0) {
    prefetch_tensormap(&tmap);
    // Stage i holds the keys AND the probabilities of the tiles it, it + ns, ...: one commit of the
    // MMA thread (p_empty, to both CTAs) frees both.  k_empty counts the score warps that are done
    // reading the keys; p_full counts the local score warps, each of which also announces the bytes
    // that it and its twin in the other CTA ship into this CTA's P tile.
    for (int i = 0; i < g.ns; ++i) {
      mbar_init(bar_k_full + 8 * i, 1); mbar_init(bar_k_empty + 8 * i, g.nsw);
      mbar_init(bar_p_full + 8 * i, g.nsw); mbar_init(bar_p_empty + 8 * i, CL);
    }
    mbar_init(bar_u_full, 1);
    mbar_init(bar_u_empty, nepi);
    mbar_init(bar_xm, g.nsw);
    mbar_init(bar_xl, g.nsw);
    *s_abort = 0;
    fence_mbar_init();
  }
  for (int i = tid; i < TC_MAX_NS * TC_P_BYTES / 16; i += blockDim.x) sts128_zero(p_stage0 + 16 * i);
  if (warp == mma_warp) tmem_alloc(smem_u32(s_tmem), (uint32_t)g.tmem_cols);
  // Cluster-wide rendezvous first, while nothing is in flight (a cluster barrier that has
  // to wait behind outstanding TMA loads costs several microseconds): after it the peer's
  // barriers and P tiles may be written.
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  slim_pdl_wait();          // lengths, q and the newest key rows may come from the kernels before this one
  const SlimSched sc = slim_sched_build(p.lengths, p.batch, p.t_cap, p.workers, p.min_tiles, s_prefix, p.status, p.unit_cost);
  const bool in_range = sc.total_tiles > 0 && w < sc.workers_eff;
  const int g_begin = in_range ? slim_worker_start(sc, w) : 0;
  const int g_end = in_range ? slim_worker_start(sc, w + 1) : 0;
  const bool have_work = g_end > g_begin;
  TC_TRACE_MARK(1);

  if (have_work) {
    if (warp < g.nswl) {
      // =========================== score / epilogue warps ===========================
      const bool scorer = warp < g.nsw * SETS;
      const int wset = (SETS == 2 && warp >= g.nsw) ? 1 : 0;     // this warp's set
      const int wis = warp - wset * g.nsw;                       // warp within the set
      const int jl = lane % JL, rp = (lane / JL) % RP, hw = lane / HL;
      const int hl = HW * wis + hw;                              // head within this CTA
      const bool head_valid = scorer && hl < g.hl;
      const bool active = head_valid && jl < OCT;
      const int my_n = (int)rank * g.hl + hl;                    // global head
      // Row i of this thread's RT rows.  Without RoPE nothing ties a thread to equidistant rows, and for
      // d_k = 64 (a head's half is 64 bytes, half a swizzled line) the rows read by one load instruction
      // are then chosen two swizzle phases apart, so that the 32 lanes cover all banks (no conflicts).
      constexpr bool SPREAD = !ROPE && DK == 64 && RT == 4;
      auto row_of = [&](const int i) { return SPREAD ? 2 * rp + (i & 1) + 8 * (i >> 1) : rp + RP * i; };
      const int my_row = row_of(jl / DUP);                       // row whose argument this lane ends up with
      // byte offsets of this thread's two 16-byte key units (first / second half of the head)
      uint32_t koff[2], kunit[2];
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        const int col = hl * DK + hf * PAIRS + 8 * jl;
        koff[hf] = (uint32_t)(col >> 6) * 2048u;
        kunit[hf] = (uint32_t)((col & 63) >> 3);
      }
      // bytes that this warp and its twin in the other CTA(s) ship into one P tile: 32 per head
      const int nvalid = min(HW, max(g.hl - HW * wis, 0));
      const uint32_t p_bytes_w = (uint32_t)(CL * 32 * nvalid);
      // e^{i RP theta}: one step of this thread's rows
      f32x2 stc[4], sts[4], stn[4];
      // Three-term form of the same step, Q(n+1) = 2 cos(RP theta) Q(n) - Q(n-1), used for a tile's rows from
      // the third on: one packed FMA per register instead of two packed operations.  The subtraction is
      // folded into the signs: Z(n) = sg(n) Q(n) with sg = + + - - + + ..., Z(n+1) = a(n) Z(n) + Z(n-1),
      // a(n) = -/+ 2 cos alternating; a row's sum takes sg(n) back, and sg(RT) = + (RT a multiple of 4).
      constexpr bool CHEB = ROPE && RT % 4 == 0;
      f32x2 tcp[4], tcn[4];
      if (ROPE && active) {
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const float2 a = p.rope_off[RP * PAIRS + 8 * jl + 2 * x], b = p.rope_off[RP * PAIRS + 8 * jl + 2 * x + 1];
          stc[x] = pack2(a.x, b.x); sts[x] = pack2(a.y, b.y); stn[x] = pack2(-a.y, -b.y);
          if (CHEB) { tcp[x] = pack2(2.f * a.x, 2.f * b.x); tcn[x] = pack2(-2.f * a.x, -2.f * b.x); }
        }
      }

      // Tile number `it` of the worker (counted through all its units) belongs to set it mod SETS, so
      // a set meets only the stages of its own parity (ns is even then) and sees each of their
      // barrier phases in order.  (st, kph): stage and phase parity of this set's next tile it_own,
      // stepped instead of divided.
      int it_base = 0, it_own = wset, uc = 0, st = wset;
      uint32_t kph = 0;
      bool ok = true;
      for (int gg = g_begin; gg < g_end && ok; ++uc) {
        const int b = slim_seq_of_tile(s_prefix, p.batch, gg);
        const int seg_end = min(g_end, s_prefix[b + 1]);
        const int tile0 = gg - s_prefix[b], ntile = seg_end - gg;
        const int unit = w + b;
        const int len = min(max(p.lengths[b], 0), p.t_cap);
        const int toff = ROPE ? slim_tile_offset(p, b) : 0;       // absolute tile of the cache's first row
        // ---- a2: this thread's slice of the query at its own position, scaled ----
        float qh1[8], qh2[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) { qh1[x] = 0.f; qh2[x] = 0.f; }
        if (active && !EXT) {         // (with external scores the query is not needed here, and its rows are H d_k wide, not d)
          const __nv_bfloat16* Q = reinterpret_cast<const __nv_bfloat16*>(p.q) + (size_t)b * p.d + my_n * DK + 8 * jl;
          float a[8], c[8];
          unpack8(__ldg(reinterpret_cast<const uint4*>(Q)), a);
          unpack8(__ldg(reinterpret_cast<const uint4*>(Q + PAIRS)), c);
          if (ROPE) {
            const int m = slim_query_pos(p, b, len), mt = m / SLIM_TT, mi = m % SLIM_TT;
#pragma unroll
            for (int x = 0; x < 8; ++x) {
              const float2 cb = p.rope_base[(size_t)mt * PAIRS + 8 * jl + x], co = p.rope_off[mi * PAIRS + 8 * jl + x];
              const float cm = cb.x * co.x - cb.y * co.y, sn = cb.y * co.x + cb.x * co.y;
              qh1[x] = (a[x] * cm + c[x] * sn) * p.qscale;
              qh2[x] = (-a[x] * sn + c[x] * cm) * p.qscale;
            }
          } else {
#pragma unroll
            for (int x = 0; x < 8; ++x) { qh1[x] = a[x] * p.qscale; qh2[x] = c[x] * p.qscale; }
          }
        }
        // Q(t) = q^ e^{i t theta}: (Qa, Qb) weight the first / second half of the head
        f32x2 Qa[4], Qb[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) { Qa[x] = pack2(qh1[2 * x], qh1[2 * x + 1]); Qb[x] = pack2(qh2[2 * x], qh2[2 * x + 1]); }
        float mref = 0.f, lsum = 0.f;
        // this set's first tile of the unit; the set that has the unit's first tile owns m_ref
        const int kt0 = SETS == 1 ? 0 : it_own - it_base;
        const bool owner = kt0 == 0;

        for (int kt = kt0; kt < ntile && ok; kt += SETS, it_own += SETS, st += SETS) {
          if (st >= g.ns) { st -= g.ns; kph ^= 1u; }
          const int tile = tile0 + kt, t0 = tile * SLIM_TT;
          const uint32_t kbase = k_stage0 + (uint32_t)st * g.stage_bytes;
          float sv = 0.f;
          if (scorer) {
            if (ROPE && active && ((kt >> (SETS - 1)) % (TC_RESEED / SETS)) == 0) {
              // exact Q at this thread's first row of the tile (position t0 + rp)
#pragma unroll
              for (int x = 0; x < 4; ++x) {
                const float4 cb = __ldg(reinterpret_cast<const float4*>(p.rope_base + (size_t)(tile + toff) * PAIRS + 8 * jl + 2 * x));
                const float4 co = __ldg(reinterpret_cast<const float4*>(p.rope_off + rp * PAIRS + 8 * jl + 2 * x));
                const float c0 = cb.x * co.x - cb.y * co.y, s0 = cb.y * co.x + cb.x * co.y;
                const float c1 = cb.z * co.z - cb.w * co.w, s1 = cb.w * co.z + cb.z * co.w;
                Qa[x] = pack2(qh1[2 * x] * c0 - qh2[2 * x] * s0, qh1[2 * x + 1] * c1 - qh2[2 * x + 1] * s1);
                Qb[x] = pack2(qh1[2 * x] * s0 + qh2[2 * x] * c0, qh1[2 * x + 1] * s1 + qh2[2 * x + 1] * c1);
              }
            }
            // a wait that ran out is acted on after the vote below (until then the lanes only
            // touch their own registers and this CTA's shared memory)
            ok = mbar_wait<false>(bar_k_full + 8 * st, kph, s_abort, p.status);
            if (warp == SLIM_TC_TRACE_WARP && lane == 0) TC_TRACE(2, it_own);
            // rows at or beyond the sequence end must not reach the tensor core (0 x NaN)
            if (t0 + SLIM_TT > len) {
              const int nz = len - t0;
              for (int c64 = wis; c64 < g.nc64; c64 += g.nsw)
                for (int e = lane; e < (SLIM_TT - nz) * 8; e += 32)
                  sts128_zero(kbase + (uint32_t)c64 * 2048u + (uint32_t)(nz + (e >> 3)) * 128u + (uint32_t)(e & 7) * 16u);
            }
            // ---- a4: softmax arguments ----
            if (EXT) {
              // X-cache scheme: the arguments were computed by the dense-score kernel (log2 domain)
              if (head_valid && t0 + my_row < len)
                sv = __ldg(p.ext_scores + ((size_t)b * p.H + my_n) * p.t_cap + t0 + my_row);
            } else {
            // this thread's partial sums for its RT rows
            float v[RT];
#pragma unroll
            for (int i = 0; i < RT; ++i) v[i] = 0.f;
            if (active) {
              f32x2 Pa[4], Pb[4];                        // Z(n-1) of the three-term step
#pragma unroll
              for (int i = 0; i < RT; ++i) {
                const int row = row_of(i);
                const uint32_t rbase = kbase + (uint32_t)row * 128u;
                const uint32_t sw = (uint32_t)(row & 7);
                const uint4 ka = lds128(rbase + koff[0] + ((kunit[0] ^ sw) << 4));
                const uint4 kb = lds128(rbase + koff[1] + ((kunit[1] ^ sw) << 4));
                f32x2 acc0 = mul2(unpack2(ka.x), Qa[0]);
                f32x2 acc1 = mul2(unpack2(kb.x), Qb[0]);
                acc0 = fma2(unpack2(ka.y), Qa[1], acc0); acc1 = fma2(unpack2(kb.y), Qb[1], acc1);
                acc0 = fma2(unpack2(ka.z), Qa[2], acc0); acc1 = fma2(unpack2(kb.z), Qb[2], acc1);
                acc0 = fma2(unpack2(ka.w), Qa[3], acc0); acc1 = fma2(unpack2(kb.w), Qb[3], acc1);
                v[i] = (CHEB && (i & 2)) ? -sum2(add2(acc0, acc1)) : sum2(add2(acc0, acc1));
                if (ROPE) {
                  if (!CHEB || i == 0) {
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                      if (CHEB) { Pa[x] = Qa[x]; Pb[x] = Qb[x]; }
                      const f32x2 na = fma2(Qb[x], stn[x], mul2(Qa[x], stc[x]));
                      Qb[x] = fma2(Qa[x], sts[x], mul2(Qb[x], stc[x]));
                      Qa[x] = na;
                    }
                  } else {
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                      const f32x2 tw = (i & 1) ? tcn[x] : tcp[x];
                      const f32x2 na = fma2(tw, Qa[x], Pa[x]), nb = fma2(tw, Qb[x], Pb[x]);
                      Pa[x] = Qa[x]; Pb[x] = Qb[x];
                      Qa[x] = na; Qb[x] = nb;
                    }
                  }
                }
              }
            }
            // sum over the JL lanes of a (head, row set); lane jl keeps row rp + RP (jl / DUP)
            {
              int n = RT;
#pragma unroll
              for (int o = JL / 2; o >= 1; o >>= 1) {
                if (n > 1) {
                  const int half = n / 2;
                  const bool up = (jl & o) != 0;
#pragma unroll
                  for (int i = 0; i < half; ++i) {
                    const float send = up ? v[i] : v[i + half];
                    const float keep = up ? v[i + half] : v[i];
                    v[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
                  }
                  n = half;
                } else {
                  v[0] += __shfl_xor_sync(0xffffffffu, v[0], o);
                }
              }
              sv = v[0];
            }
            }
            const bool valid = head_valid && (t0 + my_row < len);
            // ---- a5: probabilities against the fixed reference of this unit ----
            if (kt == 0) {
              float mx = valid ? sv : -INFINITY;
#pragma unroll
              for (int o = 1; o < HL; o <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
              mref = mx;
              lsum = 0.f;
              if (SETS == 2) {
                if (head_valid && (lane % HL) == 0) s_xm[hl] = mref;
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_xm);
              }
            } else if (SETS == 2 && kt == 1) {
              ok = mbar_wait<false>(bar_xm, uc & 1, s_abort, p.status) && ok;
              mref = head_valid ? s_xm[hl] : 0.f;
              lsum = 0.f;
            }
            float x = sv - mref;
            if (valid && x > TC_XMAX) { p.unit_flags[2 * unit + (int)rank] = 1; if (EXT || !p.redo_in_combine) *p.any_flag = 1; x = TC_XMAX; }
            const float pf = valid ? ex2_approx(x) : 0.f;
            const __nv_bfloat16 pb = __float2bfloat16_rn(pf);
            if ((jl % DUP) == 0) lsum += __bfloat162float(pb);
            if (warp == SLIM_TC_TRACE_WARP && lane == 0) TC_TRACE(3, it_own);
            // the P stage is free once the MMAs of tile it - ns are done in both CTAs
            ok = mbar_wait<false>(bar_p_empty + 8 * (PAIR ? st >> 1 : st), kph ^ 1, s_abort, p.status) && ok;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (warp == SLIM_TC_TRACE_WARP && lane == 0) TC_TRACE(4, it_own);
            {
              // stage this warp's probabilities in the K-major order of the P tile, then ship
              // them in 16-byte pieces (8 rows of one head) to both CTAs
              const uint32_t stg = stg0 + (uint32_t)warp * 128u + (uint32_t)((kt >> (SETS - 1)) & 1) * 64u;
              if ((jl % DUP) == 0) sts_u16(stg + (uint32_t)(hw * 16 + my_row) * 2u, __bfloat16_as_ushort(pb));
              __syncwarp();
              if (lane < 4 * HW) {
                const int hsel = lane >> 2, half = (lane >> 1) & 1, dest = lane & 1;
                const int hl_s = HW * wis + hsel;
                if (hl_s < g.hl && dest < CL) {
                  const uint4 pv = lds128(stg + (uint32_t)(hsel * 16 + half * 8) * 2u);
                  const int n_s = (int)rank * g.hl + hl_s;
                  const uint32_t dst = p_stage0 + (uint32_t)st * TC_P_BYTES + p_offset(n_s & 31, half * 8);
                  st_async_v4(mapa(dst, dest), pv, mapa(bar_p_full + 8 * st, dest));
                }
              }
            }
            // The local arrival releases this warp's zero-fill of the K stage (if any) to the
            // MMA thread, whose proxy fence orders it before the tensor-core reads.
            __syncwarp();
            if (lane == 0) {
              mbar_arrive_expect_tx(bar_p_full + 8 * st, p_bytes_w);
              mbar_arrive(bar_k_empty + 8 * st);
              if (warp == SLIM_TC_TRACE_WARP) TC_TRACE(5, it_own);
            }
            if (ROPE && active && SETS == 2) {
              // the other set's tile: RT row steps of RP rows keep the stepped rotation in step
#pragma unroll
              for (int i = 0; i < RT; ++i)
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                  const f32x2 na = fma2(Qb[x], stn[x], mul2(Qa[x], stc[x]));
                  Qb[x] = fma2(Qa[x], sts[x], mul2(Qb[x], stc[x]));
                  Qa[x] = na;
                }
            }
          }
        }
        if (!ok) break;
        // ---- partial of this unit: (m_ref, l) per head, then U from tensor memory ----
        if (scorer) {
#pragma unroll
          for (int o = 1; o < HL; o <<= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
          if (SETS == 2) {
            // Both sets wait on both hand-over barriers in every unit, so each warp sees every
            // phase of them, whichever role its set had.
            if (!owner) {
              if (kt0 >= ntile) ok = mbar_wait<false>(bar_xm, uc & 1, s_abort, p.status);   // no tile of this unit
              if (head_valid && (lane % HL) == 0) s_xl[hl] = lsum;
              __syncwarp();
              if (lane == 0) mbar_arrive(bar_xl);
            }
            ok = mbar_wait<false>(bar_xl, uc & 1, s_abort, p.status) && ok;
            if (owner) {
              ok = mbar_wait<false>(bar_xm, uc & 1, s_abort, p.status) && ok;
              if (head_valid) lsum += s_xl[hl];
            }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
          }
          if (owner && head_valid && (lane % HL) == 0) {
            p.part_m[(size_t)unit * p.H + my_n] = mref;
            p.part_l[(size_t)unit * p.H + my_n] = lsum;
          }
        }
        if (warp < nepi) {
          // Warp w drains TMEM lanes 32 (w & 3) .. +31 (the only ones it can reach) for the
          // chunks w >> 2, w >> 2 + nepi / 4, ...; the next chunk is fetched while this one
          // is stored.
          ok = mbar_wait<false>(bar_u_full, uc & 1, s_abort, p.status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          TC_TRACE_MARK(2);
          tc_fence_after();
          const int q = warp & 3, cstep = nepi >> 2;
          const uint32_t tlane = tmem_base + ((uint32_t)(q * 32) << 16);
          float* dst = p.part_u + (size_t)unit * p.H * p.d + (size_t)rank * g.dsl + q * 32 + lane;
          uint32_t ra[32], rb[32];
          int c = warp >> 2;
          if (c < g.nch) tmem_ld32_issue(tlane + (uint32_t)(c * 32), ra);
          while (c < g.nch) {
            tmem_ld_wait();
            if (c + cstep < g.nch) tmem_ld32_issue(tlane + (uint32_t)((c + cstep) * 32), rb);
#pragma unroll
            for (int n = 0; n < 32; ++n)
              if (n < p.H) dst[(size_t)n * p.d + c * 128] = __uint_as_float(ra[n]);
            c += cstep;
            if (c >= g.nch) break;
            tmem_ld_wait();
            if (c + cstep < g.nch) tmem_ld32_issue(tlane + (uint32_t)((c + cstep) * 32), ra);
#pragma unroll
            for (int n = 0; n < 32; ++n)
              if (n < p.H) dst[(size_t)n * p.d + c * 128] = __uint_as_float(rb[n]);
            c += cstep;
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_u_empty);
          TC_TRACE_MARK(3);
        }
        gg = seg_end;
        it_base += ntile;
      }
    } else if (warp == producer_warp) {
      // =========================== TMA producer ===========================
      if (!EXT && p.k_new != nullptr) {
        // Generate-phase cache update: the newest key row of every sequence whose last tile this worker
        // reads goes to row lengths[b] - 1 (this CTA's column half), by the whole warp, before the first
        // load.  Each lane orders its own stores before the TMA reads (generic -> async proxy).
        const int b_lo = slim_seq_of_tile(s_prefix, p.batch, g_begin), b_hi = slim_seq_of_tile(s_prefix, p.batch, g_end - 1);
        for (int b = b_lo; b <= b_hi; ++b) {
          const int last = s_prefix[b + 1] - 1;
          const int len = p.lengths[b];
          if (s_prefix[b + 1] == s_prefix[b] || last < g_begin || last >= g_end || len > p.t_cap) continue;
          const long long row = slim_cache_row(p, b, ((len - 1) / SLIM_TT) * SLIM_TT) + (len - 1) % SLIM_TT;
          const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.k_new) + (size_t)b * p.d + (size_t)rank * g.dsl);
          uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(const_cast<void*>(p.k)) + (size_t)row * p.d + (size_t)rank * g.dsl);
          for (int e = lane; e < g.dsl / 8; e += 32) dst[e] = __ldg(src + e);
        }
        fence_proxy_async_global();
        __syncwarp();
      }
      if (lane == 0) {
        int it = 0, st = 0;
        uint32_t kph = 0;
        bool ok = true;
        const uint64_t l2pol = l2_policy_evict_first();
        {
          // Clear this CTA's redo flags of the worker's units.  A score warp can only raise one after
          // it has seen a k_full phase, which takes this thread's arming arrival (a release) below:
          // the clears are ordered before any such store.
          const int b_lo = slim_seq_of_tile(s_prefix, p.batch, g_begin), b_hi = slim_seq_of_tile(s_prefix, p.batch, g_end - 1);
          for (int b = b_lo; b <= b_hi; ++b) {
            p.unit_flags[2 * (w + b) + (int)rank] = 0;
            if (CL == 1) p.unit_flags[2 * (w + b) + 1] = 0;        // a lone CTA owns both words of its units
          }
          __threadfence_block();
        }
        for (int gg = g_begin; gg < g_end && ok;) {
          const int b = slim_seq_of_tile(s_prefix, p.batch, gg);
          const int seg_end = min(g_end, s_prefix[b + 1]);
          const int tile0 = gg - s_prefix[b], ntile = seg_end - gg;
          for (int kt = 0; kt < ntile; ++kt, ++it, st = (st + 1 == g.ns ? 0 : st + 1), kph ^= (st == 0)) {
            // free once the score warps have read the keys and the tensor core has consumed them
            TC_TRACE(0, it);
            ok = mbar_wait<false>(bar_k_empty + 8 * st, kph ^ 1, s_abort, p.status) &&
                 mbar_wait<false>(bar_p_empty + 8 * (PAIR ? st >> 1 : st), kph ^ 1, s_abort, p.status);
            if (!ok) break;
            TC_TRACE(1, it);
            mbar_arrive_expect_tx(bar_k_full + 8 * st, (uint32_t)g.stage_bytes);
            if (p.k_evict_first)
              tma_load_3d_hint(k_stage0 + (uint32_t)st * g.stage_bytes, &tmap, bar_k_full + 8 * st, 0,
                               (int)slim_cache_row(p, b, (tile0 + kt) * SLIM_TT), (int)rank * g.nc64, l2pol);
            else
              tma_load_3d(k_stage0 + (uint32_t)st * g.stage_bytes, &tmap, bar_k_full + 8 * st, 0,
                          (int)slim_cache_row(p, b, (tile0 + kt) * SLIM_TT), (int)rank * g.nc64);
          }
          gg = seg_end;
        }
        if (!ok) {
          // gave up: let the loads that were issued land before the CTA goes away
          const int issued = it < g.ns ? it : g.ns;
          for (int k = 0; k < issued; ++k) {
            const int j = it - 1 - k, st = j % g.ns;
            const unsigned long long t0 = globaltimer();
            while (!mbar_try_wait(bar_k_full + 8 * st, (j / g.ns) & 1) && globaltimer() - t0 < SLIM_WAIT_NS) {}
          }
        }
      }
    } else if (warp == mma_warp) {
      // =========================== MMA issuer ===========================
      if (lane == 0) {
        int it = 0, uc = 0, st = 0;
        uint32_t kph = 0;
        bool ok = true;
        // p_full of a tile completes on the local score warps' arrivals + the 32 bytes per head
        // shipped by the score warps of both CTAs (announced by the local ones)
        // operand descriptors of stage 0 as (low, high) words; a stage or a chunk further on only
        // moves the start-address field (all of shared memory stays below its 18-bit range)
        const uint64_t ad0 = desc_a(k_stage0), bd0 = desc_b(p_stage0);
        const uint32_t a_lo = (uint32_t)ad0, a_hi = (uint32_t)(ad0 >> 32), b_lo = (uint32_t)bd0, b_hi = (uint32_t)(bd0 >> 32);
        const uint32_t a_step = (uint32_t)g.stage_bytes >> 4;
        for (int gg = g_begin; gg < g_end && ok; ++uc) {
          const int b = slim_seq_of_tile(s_prefix, p.batch, gg);
          const int seg_end = min(g_end, s_prefix[b + 1]);
          const int ntile = seg_end - gg;
          for (int kt = 0; kt < ntile;) {
            // two tiles in one turn: the even stage of a pair with the odd one behind it, same unit
            const bool two = PAIR && (st & 1) == 0 && kt + 1 < ntile;
            // p_full alone is enough: every local score warp arrives on it after it has seen
            // k_full of this stage, so the keys have landed (and are ordered before this wait).
            ok = mbar_wait<true>(bar_p_full + 8 * st, kph, s_abort, p.status);
            if (ok && two) ok = mbar_wait<true>(bar_p_full + 8 * (st + 1), kph, s_abort, p.status);
            if (ok && kt == 0 && uc > 0) ok = mbar_wait<false>(bar_u_empty, (uc - 1) & 1, s_abort, p.status);
            if (!ok) break;
            TC_TRACE(6, it);
            fence_proxy_async_smem();        // P pieces and zero-filled key rows -> tensor-core reads
            tc_fence_after();
            // One instruction per 128-column chunk.  The tensor core takes one of these every ~65
            // clocks; this thread's own instructions between two of them must stay below that, so
            // the descriptors are stepped as 32-bit words instead of being rebuilt.
            {
              const uint32_t acc = kt > 0 ? 1u : 0u;
              uint32_t al = a_lo + (uint32_t)st * a_step, dcol = tmem_base;
              const uint32_t bl = b_lo + (uint32_t)st * (TC_P_BYTES >> 4);
              for (int c = 0; c < g.nch; ++c, al += 4096u >> 4, dcol += 32u)
                umma_bf16_words(dcol, al, a_hi, bl, b_hi, umma_idesc(32), acc);
              if (two) {
                al = a_lo + (uint32_t)(st + 1) * a_step; dcol = tmem_base;
                for (int c = 0; c < g.nch; ++c, al += 4096u >> 4, dcol += 32u)
                  umma_bf16_words(dcol, al, a_hi, bl + (TC_P_BYTES >> 4), b_hi, umma_idesc(32), 1u);
              }
            }
            const int last = two ? st + 1 : st;
            if (!PAIR) {
              if (CL == 2) umma_commit_pair(bar_p_empty + 8 * st); else umma_commit(bar_p_empty + 8 * st);
            } else if (last & 1) {               // the odd stage closes the pair (the even one is older)
              if (CL == 2) umma_commit_pair(bar_p_empty + 8 * (last >> 1)); else umma_commit(bar_p_empty + 8 * (last >> 1));
            }
            TC_TRACE(7, it);
            const int adv = two ? 2 : 1;
            kt += adv; it += adv; st += adv;
            if (st >= g.ns) { st -= g.ns; kph ^= 1u; }
            if (kt == ntile) umma_commit(bar_u_full);
          }
          gg = seg_end;
        }
        // Every tile of this CTA is with the tensor core: from here on the kernels behind this one may
        // take their places on the SMs (they still wait for this grid to finish before they read its
        // results).  Letting them in at the start of this kernel was measured ~1 % slower per step.
        slim_pdl_trigger();
      }
    }
  }
  slim_pdl_trigger();

  // ---- teardown: nobody may still write into a CTA that has left ------------------
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == mma_warp) {
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)g.tmem_cols);
  }
  TC_TRACE_MARK(4);
}

// ------------------------------------------------------------------ host side
TcGeom make_geom(int d, int H, int d_k, int rt, int cl, int sets, int smem_limit) {
  TcGeom g;
  g.cl = cl;
  g.sets = sets;
  g.dsl = d / cl;
  g.nch = g.dsl / 128;
  g.nc64 = g.dsl / 64;
  g.hl = H / cl;
  const int hw = tc_heads_per_warp(d_k, rt);
  g.nsw = (g.hl + hw - 1) / hw;
  g.nswl = g.nsw * sets < 4 ? 4 : g.nsw * sets;
  g.stage_bytes = SLIM_TT * g.dsl * 2;
  int ns = (smem_limit - 16 * 1024) / g.stage_bytes;
  g.ns = ns > TC_MAX_NS ? TC_MAX_NS : ns;
  if (sets == 2) g.ns &= ~1;                     // each set keeps to the stages of its own parity
  int cols = 32;
  while (cols < 32 * g.nch) cols <<= 1;
  g.tmem_cols = cols;
  return g;
}

size_t tc_smem_bytes(const TcGeom& g, int batch) {
  size_t need = 1024 + (size_t)g.ns * g.stage_bytes + TC_MAX_NS * TC_P_BYTES + TC_MAX_SW * 128 + 32 * TC_MAX_NS + 32 + 8 + 256 +
                sizeof(int) * (batch + 1) + 64;
  const size_t floor_bytes = 120 * 1024;         // one CTA per SM: tensor memory is not shared
  return need < floor_bytes ? floor_bytes : need;
}

typedef void (*tc_kernel_t)(const CUtensorMap, const SlimDecodeParams, const TcGeom);

// Two score-warp sets where a tile is small (d_k = 64, scores formed in the kernel, CTA pair) and both
// sets fit the block.  ctx->opt_tc_sets1 switches them off for comparisons.
int tc_sets(const slim_ctx* ctx, int H, int d_k, int rt, bool ext, int cl) {
  if (ctx->opt_tc_sets1) return 1;
  if (d_k != 64 || rt != 4 || ext || cl != 2) return 1;
  const int hw = tc_heads_per_warp(d_k, rt), nsw = (H / cl + hw - 1) / hw;
  return 2 * nsw <= TC_SETS2_WARPS ? 2 : 1;
}

// Rows per thread and tile.  Measured on the d = 4096 / 32-head shape: 8 rows per
// thread (8 score warps) beats 4 rows (16 warps); the stepped query rotation is
// re-used over more rows and fewer warps contend for the issue slots.
// ctx->opt_tc_rt overrides the choice for sweeps.
int tc_rows_per_thread(const slim_ctx* ctx) {
  const int d_k = ctx->d_k, want = ctx->opt_tc_rt;
  if (d_k == 64) return want == 2 ? 2 : 4;
  return want == 4 ? 4 : 8;
}

// One CTA per worker (cl = 1) where a whole key row fits one SM's tensor memory and the kernel stays
// under the register budget of its larger block (instantiated for d_k = 64 without RoPE).  Measured on
// the Whisper-large shape: with scores computed in the kernel the CTA pair is faster (the score warps
// of a lone CTA carry all heads); with external scores (X-cache scheme) the lone CTA is faster.
bool tc_cl_ok(int d, int H, int d_k, bool rope, int cl) {
  if (cl == 1) return d_k == 64 && !rope && d % 128 == 0 && d <= 2048 && H >= 1 && H <= 32;
  return !(H & 1) && H <= 32 && H >= 2 && d % 256 == 0 && d <= 4096;   // d/2 in 128-column chunks, <= 512 TMEM columns
}

template <int DK, bool ROPE, int RT>
tc_kernel_t pick_ext_cl(bool ext, int cl, int sets) {
  if (sets == 2) {
    if constexpr (DK == 64 && RT == 4) return (!ext && cl == 2) ? slim_tc_kernel<DK, ROPE, RT, false, 2, 2> : nullptr;
    else return nullptr;
  }
  if (cl == 1) {
    if constexpr (DK == 64 && !ROPE && RT == 4) return ext ? slim_tc_kernel<DK, ROPE, RT, true, 1, 1> : slim_tc_kernel<DK, ROPE, RT, false, 1, 1>;
    else return nullptr;
  }
  if (ext) {
    if constexpr (!ROPE) return slim_tc_kernel<DK, ROPE, RT, true, 2, 1>;
    else return nullptr;
  }
  return slim_tc_kernel<DK, ROPE, RT, false, 2, 1>;
}

tc_kernel_t pick_kernel(int d_k, bool rope, int rt, bool ext, int cl, int sets) {
  switch (d_k * 16 + rt) {
    case 64 * 16 + 2: return rope ? pick_ext_cl<64, true, 2>(ext, cl, sets) : pick_ext_cl<64, false, 2>(ext, cl, sets);
    case 64 * 16 + 4: return rope ? pick_ext_cl<64, true, 4>(ext, cl, sets) : pick_ext_cl<64, false, 4>(ext, cl, sets);
    case 96 * 16 + 4: return rope ? pick_ext_cl<96, true, 4>(ext, cl, sets) : pick_ext_cl<96, false, 4>(ext, cl, sets);
    case 96 * 16 + 8: return rope ? pick_ext_cl<96, true, 8>(ext, cl, sets) : pick_ext_cl<96, false, 8>(ext, cl, sets);
    case 128 * 16 + 4: return rope ? pick_ext_cl<128, true, 4>(ext, cl, sets) : pick_ext_cl<128, false, 4>(ext, cl, sets);
    case 128 * 16 + 8: return rope ? pick_ext_cl<128, true, 8>(ext, cl, sets) : pick_ext_cl<128, false, 8>(ext, cl, sets);
    default: return nullptr;
  }
}

constexpr int TC_SMEM_LIMIT = 227 * 1024;

}  // namespace

namespace {
// A CTA waits on an mbarrier that nothing ever arrives at: the bounded wait has to give up,
// report SLIM_ERR_TIMEOUT through the status word and let the kernel return normally.
__global__ void slim_wait_selftest_kernel(int* status, int* gave_up) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  const uint32_t b = smem_u32(&bar);
  if (threadIdx.x == 0) { mbar_init(b, 1); abort_flag = 0; fence_mbar_init(); }
  __syncthreads();
  const bool ok = mbar_wait<false>(b, 0, &abort_flag, status);
  if (threadIdx.x == 0) *gave_up = ok ? 0 : 1;
}
}  // namespace

cudaError_t slim_launch_wait_selftest(int* status, int* gave_up, cudaStream_t st) {
  slim_wait_selftest_kernel<<<1, 64, 0, st>>>(status, gave_up);
  return cudaGetLastError();
}

int slim_tc_shape_ok(int d, int H, int d_k, int dtype, int rope, int cl) {
  if (dtype != SLIM_BF16) return 0;
  if (d_k != 64 && d_k != 96 && d_k != 128) return 0;
  return tc_cl_ok(d, H, d_k, rope != 0, cl) ? 1 : 0;
}

int slim_tc_workers(const slim_ctx* ctx, int cl) {
  const int rt = tc_rows_per_thread(ctx);
  const bool rope = ctx->rope_theta != 0.0;
  const int sets = tc_sets(ctx, ctx->H, ctx->d_k, rt, false, cl);
  tc_kernel_t kern = pick_kernel(ctx->d_k, rope, rt, false, cl, sets);
  if (!kern) return 0;
  const TcGeom g = make_geom(ctx->d, ctx->H, ctx->d_k, rt, cl, sets, TC_SMEM_LIMIT);
  if (g.ns < 2) return 0;
  const size_t smem = tc_smem_bytes(g, SLIM_MAX_BATCH);
  if (smem > (size_t)TC_SMEM_LIMIT) return 0;
  if (cudaFuncSetAttribute((const void*)kern, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_LIMIT) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(cl * (ctx->num_sms / cl));
  cfg.blockDim = dim3((g.nswl + 2) * 32);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cl; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  int nclusters = 0;
  if (cudaOccupancyMaxActiveClusters(&nclusters, (const void*)kern, &cfg) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  const int cap = ctx->num_sms / cl;
  return nclusters < cap ? nclusters : cap;
}

cudaError_t slim_tmap_encode_3d(void* out_map, void* base, const unsigned long long dims_in[3],
                                const unsigned long long strides_in[2], const unsigned int box_in[3]) {
  typedef CUresult (*encode_t)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                               const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                               CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static encode_t encode = nullptr;
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
    encode = (encode_t)fn;
  }
  const cuuint64_t dims[3] = {dims_in[0], dims_in[1], dims_in[2]};
  const cuuint64_t strides[2] = {strides_in[0], strides_in[1]};
  const cuuint32_t box[3] = {box_in[0], box_in[1], box_in[2]};
  const cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = encode(reinterpret_cast<CUtensorMap*>(out_map), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims,
                      strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

cudaError_t slim_tc_make_tmap(const slim_ctx* ctx, slim_cache* c, int cl) {
  const TcGeom g = make_geom(ctx->d, ctx->H, ctx->d_k, tc_rows_per_thread(ctx), cl, 1, TC_SMEM_LIMIT);
  // dim0: 64 contiguous elements; dim1: cache rows (stride d elements); dim2: 64-column chunks
  const unsigned long long dims[3] = {64, (unsigned long long)c->total_rows, (unsigned long long)(ctx->d / 64)};
  const unsigned long long strides[2] = {(unsigned long long)ctx->d * 2, 128};
  const unsigned int box[3] = {64, SLIM_TT, (unsigned int)g.nc64};
  return slim_tmap_encode_3d(c->tmap[cl - 1], c->k, dims, strides, box);
}

cudaError_t slim_launch_tc(const slim_ctx* ctx, const slim_cache* c, const SlimDecodeParams& p, cudaStream_t st) {
  const int rt = tc_rows_per_thread(ctx);
  const bool ext = p.ext_scores != nullptr;
  const int cl = p.cl;
  const int sets = tc_sets(ctx, ctx->H, ctx->d_k, rt, ext, cl);
  tc_kernel_t kern = pick_kernel(ctx->d_k, ctx->rope_theta != 0.0, rt, ext, cl, sets);
  if (!kern || cl < 1 || cl > 2 || !c->has_tmap[cl - 1]) return cudaErrorNotSupported;
  if (ext) {
    cudaError_t ea = cudaFuncSetAttribute((const void*)kern, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_LIMIT);
    if (ea != cudaSuccess) return ea;
  }
  const TcGeom g = make_geom(ctx->d, ctx->H, ctx->d_k, rt, cl, sets, TC_SMEM_LIMIT);
  const size_t smem = tc_smem_bytes(g, p.batch);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(cl * p.workers);
  cfg.blockDim = dim3((g.nswl + 2) * 32);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cl; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 2;
  CUtensorMap map;
  memcpy(&map, c->tmap[cl - 1], sizeof(map));
  return cudaLaunchKernelEx(&cfg, kern, map, p, g);
}
