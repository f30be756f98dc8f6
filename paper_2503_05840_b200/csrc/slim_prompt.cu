// Prompt phase of slim attention (Fig. 3(a)): the values of a whole prompt are formed once from
// its keys, V = K W_KV (Eq. 6), after which the prompt is processed like vanilla attention.
//
//   slim_values_tc_kernel   bf16, d_k in {64, 96, 128}: CTA = (128 prompt rows, head group);
//                           V[128 x N] += K_tile[128 x 16] W_KV,h[16 x N] per 16 columns of K on
//                           tcgen05: A = key rows, K-major with 128-byte swizzle as TMA delivers
//                           them; B = the W_KV tile, MN-major (the same TMA tiles the decode
//                           projection uses); D in tensor memory (N = 128: one head of d_k = 128 or
//                           96, or two heads of d_k = 64).
//   slim_values_pair_kernel the same on CTA pairs (tcgen05.mma.cta_group::2, 256 x 256 tiles, persistent,
//                           double-buffered accumulator): d_k in {64, 128} with an even number of
//                           128-column groups and more than one row tile.
//   slim_values_kernel      any dtype / shape: CUDA-core tiles.
// With a cache given (slim_prefill) the same launch also stores the prompt's keys: the CTAs that work on
// column group 0 have warps that idle during the MMAs (single-CTA kernel: two of four; pair kernel: the
// epilogue warps); those copy the CTA's 128 key rows into the K-cache (rows positions[b] ..), reading
// them through L2 while the TMA of the same CTA streams them, so the prompt's keys leave HBM once.
// Every mbarrier wait is bounded in time.
#include <cstring>

#include "slim_internal.h"
#include "slim_sched.cuh"
#include "slim_ptx.cuh"

namespace {
using namespace slim_ptx;

constexpr int PV_ROWS = 128;                       // prompt rows per CTA (MMA M)
constexpr int PV_J = 64;                           // columns of K (rows of W_KV) per stage
constexpr int PV_A_BYTES = PV_ROWS * PV_J * 2;     // 16 KB
constexpr int PV_B_BYTES = PV_J * 128 * 2;         // two 64-column atoms x 64 rows x 128 B = 16 KB
constexpr int PV_NS = 3;                          // 97 KB per CTA: two CTAs per SM, one's epilogue under the other's MMAs

// cp (cache side of slim_prefill; cp.k == NULL: values only): the fields of SlimDecodeParams that address
// cache rows, plus q = the prompt's keys [batch][n_new][d], lengths = first row per sequence, workers = n_new.
__global__ void __launch_bounds__(128)
slim_values_tc_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap wmap, float* __restrict__ V,
                      const int n, const int d, const int d_k, const int hp, int* status, const SlimDecodeParams cp) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw_u32 = smem_u32(smem_raw);
  const uint32_t base = (raw_u32 + 1023u) & ~1023u;
  unsigned char* sm = smem_raw + (base - raw_u32);
  constexpr uint32_t stage_bytes = PV_A_BYTES + PV_B_BYTES;
  const uint32_t bars = base + PV_NS * stage_bytes;
  const uint32_t bar_full = bars, bar_empty = bars + 8 * PV_NS, bar_done = bars + 16 * PV_NS;
  unsigned char* misc = sm + (bar_done + 8 - base);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(misc);
  volatile int* s_abort = reinterpret_cast<volatile int*>(misc + 4);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // head groups vary fastest: the CTAs in flight share a few key tiles and all of W_KV (L2-resident)
  const int t0 = blockIdx.y * PV_ROWS, hg = blockIdx.x;
  const int nst = d / PV_J;

  if (tid == 0) {
    prefetch_tensormap(&kmap);
    prefetch_tensormap(&wmap);
    for (int i = 0; i < PV_NS; ++i) { mbar_init(bar_full + 8 * i, 1); mbar_init(bar_empty + 8 * i, 1); }
    mbar_init(bar_done, 1);
    *s_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) tmem_alloc(smem_u32(s_tmem), 128);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  slim_pdl_wait();

  if (warp == 0 && lane == 0) {
    int s = 0;
    bool ok = true;
    for (; s < nst; ++s) {
      const int st = s % PV_NS;
      ok = mbar_wait<false>(bar_empty + 8 * st, ((s / PV_NS) & 1) ^ 1, s_abort, status);
      if (!ok) break;
      const uint32_t dst = base + (uint32_t)st * stage_bytes;
      mbar_arrive_expect_tx(bar_full + 8 * st, stage_bytes);
      tma_load_3d(dst, &kmap, bar_full + 8 * st, s * PV_J, t0, 0);
      if (hp == 1) tma_load_3d(dst + PV_A_BYTES, &wmap, bar_full + 8 * st, 0, hg * d + s * PV_J, 0);
      else         tma_load_3d(dst + PV_A_BYTES, &wmap, bar_full + 8 * st, 0, s * PV_J, 2 * hg);
    }
    if (!ok) {
      const int issued = s < PV_NS ? s : PV_NS;
      for (int k = 0; k < issued; ++k) {
        const int j = s - 1 - k, st = j % PV_NS;
        const unsigned long long tt = globaltimer();
        while (!mbar_try_wait(bar_full + 8 * st, (j / PV_NS) & 1) && globaltimer() - tt < SLIM_WAIT_NS) {}
      }
    }
  } else if (warp >= 2 && hg == 0 && cp.k != nullptr) {
    // bulk append: prompt row r = b * n_new + i goes to cache row (b, positions[b] + i); a sequence whose
    // rows would pass the capacity is left unwritten and reported
    const int n_new = cp.workers, t64 = tid - 64;
    const uint4* src = reinterpret_cast<const uint4*>(cp.q);
    uint4* dst = reinterpret_cast<uint4*>(const_cast<void*>(cp.k));
    const int vec_per_row = d / 8;
    for (int r = t0; r < min(t0 + PV_ROWS, n); ++r) {
      const int b = r / n_new, i = r - b * n_new;
      const int pos = cp.lengths[b];
      if (pos < 0 || pos > cp.t_cap - n_new) { if (t64 == 0) atomicMax(status, (int)SLIM_ERR_CAPACITY); continue; }
      const long long row = slim_cache_row(cp, b, pos + i);
      for (int e = t64; e < vec_per_row; e += 64) dst[(size_t)row * vec_per_row + e] = __ldg(src + (size_t)r * vec_per_row + e);
    }
  } else if (warp == 1 && lane == 0) {
    bool ok = true;
    // descriptors of stage 0 as words; a stage or a k-step only moves the start-address field
    const uint64_t ad0 = desc_kmajor_sw128(base), bd0 = desc_a(base + PV_A_BYTES, PV_J * 128);
    const uint32_t a_lo0 = (uint32_t)ad0, a_hi = (uint32_t)(ad0 >> 32), b_lo0 = (uint32_t)bd0, b_hi = (uint32_t)(bd0 >> 32);
    int st = 0;
    uint32_t ph = 0;
    for (int s = 0; s < nst && ok; ++s, st = (st + 1 == PV_NS ? 0 : st + 1), ph ^= (st == 0)) {
      ok = mbar_wait<false>(bar_full + 8 * st, ph, s_abort, status);
      if (!ok) break;
      tc_fence_after();
      const uint32_t a_lo = a_lo0 + (uint32_t)st * (stage_bytes >> 4), b_lo = b_lo0 + (uint32_t)st * (stage_bytes >> 4);
#pragma unroll
      for (int kk = 0; kk < PV_J / 16; ++kk)
        umma_bf16_words(tmem_base, a_lo + (uint32_t)kk * (32u >> 4), a_hi, b_lo + (uint32_t)kk * (2048u >> 4), b_hi,
                        umma_idesc_major(128, 0, 1), (s | kk) ? 1u : 0u);
      umma_commit(bar_empty + 8 * st);
      if (s == nst - 1) umma_commit(bar_done);
    }
  }
  __syncwarp();
  {
    bool ok = mbar_wait<false>(bar_done, 0, s_abort, status);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tc_fence_after();
      const int row = t0 + warp * 32 + lane;                   // accumulator row = prompt row
      const int ncols = hp == 2 ? 128 : d_k;                   // valid accumulator columns
      float* out = V + (size_t)row * d + (size_t)hg * hp * d_k;
      for (int c0 = 0; c0 < 128; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, r);
        if (row < n) {
#pragma unroll
          for (int c = 0; c < 32; c += 4)
            if (c0 + c < ncols)
              *reinterpret_cast<float4*>(out + c0 + c) = make_float4(__uint_as_float(r[c]), __uint_as_float(r[c + 1]),
                                                                    __uint_as_float(r[c + 2]), __uint_as_float(r[c + 3]));
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 128);
  }
}

// The same product on CTA pairs, persistent.  A pair (cluster of two, one CTA per SM) walks pair tiles of
// 256 prompt rows x 256 output columns; one tcgen05.mma.cta_group::2 with M = 256 covers the 128 rows of each
// CTA, and each CTA stages its own key rows and only HALF of the tile's W_KV columns (its half of B's N), so
// the operand bytes fetched per flop drop to a half of the single-CTA kernel's.  Roles:
//   warp 0      producer: TMA loads into a ring of stages that runs on across tile boundaries.  Both CTAs'
//               loads of a stage count their bytes on the EVEN CTA's barrier (pair form of the TMA load);
//   warp 1      (even CTA) issues the pair's MMAs; one multicast commit frees a stage in both CTAs, another
//               hands a finished accumulator to the epilogue warps of both;
//   warps 2-5   epilogue: tensor memory -> V, and for the first column group the bulk append of the rows.
// The accumulator is double-buffered in tensor memory, so a tile's epilogue runs under the next tile's MMAs.
// The pair tile is 256 x 256 (a CTA stages two 64-column atoms of W_KV, N = 256 per MMA): six 32 KB stages
// and two 256-column accumulators per CTA.  Pair tiles are numbered with the column groups fastest: the pairs
// in flight share a few key tiles and all of W_KV (L2-resident).  Shapes whose 128-column groups do not pair
// up, and prompts of one row tile, take the single-CTA kernel.
constexpr int PV2_B_BYTES = PV_J * 128 * 2;                 // two atoms x 64 rows x 128 B
constexpr int PV2_NS = 6;
constexpr uint32_t PV2_STAGE = PV_A_BYTES + PV2_B_BYTES;
constexpr int PV2_NCOL = 256;                               // accumulator columns = N of the pair's MMA
constexpr size_t PV2_SMEM = 1024 + (size_t)PV2_NS * PV2_STAGE + 16 * PV2_NS + 32 + 16 + 64;
constexpr int PV2_THREADS = 192;

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(PV2_THREADS, 1)
slim_values_pair_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap wmapb, float* __restrict__ V,
                        const int n, const int d, const int d_k, const int hp, int* status, const SlimDecodeParams cp) {
  constexpr int NS = PV2_NS, NCOL = PV2_NCOL;
  constexpr uint32_t STAGE = PV2_STAGE;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw_u32 = smem_u32(smem_raw);
  const uint32_t base = (raw_u32 + 1023u) & ~1023u;
  unsigned char* sm = smem_raw + (base - raw_u32);
  const uint32_t bars = base + NS * STAGE;
  // full: (even CTA's copy only) both CTAs' loads of a stage have landed; empty: the pair's MMAs on the stage
  // are done; acc_full[2]: an accumulator is complete (commit from the even CTA, to both); acc_empty[2]: (even
  // CTA's copy only) the eight epilogue warps of the pair have read an accumulator out
  const uint32_t bar_full = bars, bar_empty = bars + 8 * NS, bar_accf = bars + 16 * NS, bar_acce = bar_accf + 16;
  unsigned char* misc = sm + (bar_acce + 16 - base);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(misc);
  volatile int* s_abort = reinterpret_cast<volatile int*>(misc + 4);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t rank = cluster_ctarank();
  const int groups = d / NCOL;                             // column groups of the output (hp d_k = 128)
  const int ntiles = groups * ((n + 2 * PV_ROWS - 1) / (2 * PV_ROWS));
  const int pair0 = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const int nst = d / PV_J;

  if (tid == 0) {
    prefetch_tensormap(&kmap);
    prefetch_tensormap(&wmapb);
    for (int i = 0; i < NS; ++i) { mbar_init(bar_full + 8 * i, 1); mbar_init(bar_empty + 8 * i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar_accf + 8 * i, 1); mbar_init(bar_acce + 8 * i, 8); }
    *s_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) tmem_alloc2(smem_u32(s_tmem), 2 * NCOL);  // the same warp of both CTAs
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                      // the peer's barriers exist before anything is sent to them
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  slim_pdl_wait();

  if (warp == 0) {
    if (lane == 0) {
      // ---- producer: this CTA's 128 key rows and its half of the tile's W_KV columns, stage after stage ----
      int g = 0;                                           // stages issued so far (all tiles)
      bool ok = true;
      for (int T = pair0; T < ntiles && ok; T += npairs) {
        const int hg = T % groups, t0 = (2 * (T / groups) + (int)rank) * PV_ROWS;
        for (int s = 0; s < nst; ++s, ++g) {
          const int st = g % NS;
          ok = mbar_wait<false>(bar_empty + 8 * st, ((g / NS) & 1) ^ 1, s_abort, status);
          if (!ok) break;
          const uint32_t dst = base + (uint32_t)st * STAGE;
          const uint32_t full0 = mapa(bar_full + 8 * st, 0);
          if (rank == 0) mbar_arrive_expect_tx(bar_full + 8 * st, 2 * STAGE);
          tma_load_3d_pair(dst, &kmap, full0, s * PV_J, t0, 0);
          // the two atoms of head (hp = 1) / head pair (hp = 2) number 2 hg + rank: this CTA's half of the columns
          if (hp == 1) tma_load_3d_pair(dst + PV_A_BYTES, &wmapb, full0, 0, (2 * hg + (int)rank) * d + s * PV_J, 0);
          else         tma_load_3d_pair(dst + PV_A_BYTES, &wmapb, full0, 0, s * PV_J, 2 * (2 * hg + (int)rank));
        }
      }
      if (!ok) {
        // Gave up (a wait ran out two seconds after the last progress): whatever was issued has landed long
        // since; the even CTA still waits, bounded, on the barriers that count both CTAs' bytes, the odd CTA
        // lets a fixed time pass.  Neither leaves before the final cluster barrier.
        if (rank == 0) {
          const int issued = g < NS ? g : NS;
          for (int k = 0; k < issued; ++k) {
            const int j = g - 1 - k, st = j % NS;
            const unsigned long long tt = globaltimer();
            while (!mbar_try_wait(bar_full + 8 * st, (j / NS) & 1) && globaltimer() - tt < SLIM_WAIT_NS) {}
          }
        } else {
          const unsigned long long tt = globaltimer();
          while (globaltimer() - tt < 200000ull) {}
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      // ---- MMA issuer of the pair ----
      bool ok = true;
      int g = 0, i = 0;                                    // stages consumed, tiles started
      const uint64_t ad0 = desc_kmajor_sw128(base), bd0 = desc_a(base + PV_A_BYTES, PV_J * 128);
      const uint32_t a_lo0 = (uint32_t)ad0, a_hi = (uint32_t)(ad0 >> 32), b_lo0 = (uint32_t)bd0, b_hi = (uint32_t)(bd0 >> 32);
      constexpr uint32_t idesc = umma_idesc_mn(256, NCOL, 0, 1);         // A K-major, B MN-major
      for (int T = pair0; T < ntiles && ok; T += npairs, ++i) {
        const int acc = i & 1;
        ok = mbar_wait<true>(bar_acce + 8 * acc, ((i >> 1) & 1) ^ 1, s_abort, status);   // both CTAs have read it out
        if (!ok) break;
        tc_fence_after();
        const uint32_t dcol = tmem_base + (uint32_t)(acc * NCOL);
        for (int s = 0; s < nst; ++s, ++g) {
          const int st = g % NS;
          ok = mbar_wait<true>(bar_full + 8 * st, (g / NS) & 1, s_abort, status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_lo = a_lo0 + (uint32_t)st * (STAGE >> 4), b_lo = b_lo0 + (uint32_t)st * (STAGE >> 4);
#pragma unroll
          for (int kk = 0; kk < PV_J / 16; ++kk)
            umma2_bf16_words(dcol, a_lo + (uint32_t)kk * (32u >> 4), a_hi, b_lo + (uint32_t)kk * (2048u >> 4), b_hi, idesc,
                             (s | kk) ? 1u : 0u);
          umma2_commit_pair(bar_empty + 8 * st);
        }
        if (ok) umma2_commit_pair(bar_accf + 8 * acc);
      }
    }
  } else {
    // ---- epilogue warps: accumulator row = prompt row (this CTA's 128 TMEM lanes; a warp reads the lane
    // quarter of its number modulo four) ----
    const int q = warp & 3;
    bool ok = true;
    int i = 0;
    for (int T = pair0; T < ntiles && ok; T += npairs, ++i) {
      const int hg = T % groups, t0 = (2 * (T / groups) + (int)rank) * PV_ROWS;
      const int acc = i & 1;
      if (hg == 0 && cp.k != nullptr) {
        // bulk append of this CTA's rows (as in the single-CTA kernel), under the tile's MMAs
        const int n_new = cp.workers, t128 = q * 32 + lane;
        const uint4* src = reinterpret_cast<const uint4*>(cp.q);
        uint4* dst = reinterpret_cast<uint4*>(const_cast<void*>(cp.k));
        const int vec_per_row = d / 8;
        for (int r = t0; r < min(t0 + PV_ROWS, n); ++r) {
          const int b = r / n_new, j = r - b * n_new;
          const int pos = cp.lengths[b];
          if (pos < 0 || pos > cp.t_cap - n_new) { if (t128 == 0) atomicMax(status, (int)SLIM_ERR_CAPACITY); continue; }
          const long long row = slim_cache_row(cp, b, pos + j);
          for (int e = t128; e < vec_per_row; e += 128) dst[(size_t)row * vec_per_row + e] = __ldg(src + (size_t)r * vec_per_row + e);
        }
      }
      ok = mbar_wait<false>(bar_accf + 8 * acc, (i >> 1) & 1, s_abort, status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int row = t0 + q * 32 + lane;
      float* out = V + (size_t)row * d + (size_t)hg * NCOL;
      for (int c0 = 0; c0 < NCOL; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * NCOL + c0), r);
        if (row < n) {
#pragma unroll
          for (int c = 0; c < 32; c += 4)
            *reinterpret_cast<float4*>(out + c0 + c) = make_float4(__uint_as_float(r[c]), __uint_as_float(r[c + 1]),
                                                                  __uint_as_float(r[c + 2]), __uint_as_float(r[c + 3]));
        }
      }
      // this warp has read the accumulator out: tell the issuer (the even CTA's barrier, eight arrivals a tile)
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa(bar_acce + 8 * acc, 0));
    }
  }
  // nobody leaves (or frees the pair's tensor memory) while the other CTA may still be reached
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc2(tmem_base, 2 * NCOL);
  }
}

// CUDA-core version: V[t][h d_k + c] = sum_j K[t][j] W[h][j][c]; 16 x 16 output tile per CTA.
template <typename KT>
__global__ void __launch_bounds__(256)
slim_values_kernel(const KT* __restrict__ K, const KT* __restrict__ W, float* __restrict__ V, int n, int d, int d_k) {
  __shared__ float s_k[16][17], s_w[16][17];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int t = blockIdx.y * 16 + ty, col = blockIdx.x * 16 + tx;       // col = h d_k + c
  const int h = col / d_k, c = col % d_k;
  float acc = 0.f;
  for (int j0 = 0; j0 < d; j0 += 16) {
    s_k[ty][tx] = (t < n && j0 + tx < d) ? (float)K[(size_t)t * d + j0 + tx] : 0.f;
    s_w[ty][tx] = (col < d && j0 + ty < d) ? (float)W[((size_t)h * d + j0 + ty) * d_k + c] : 0.f;
    __syncthreads();
#pragma unroll
    for (int j = 0; j < 16; ++j) acc = fmaf(s_k[ty][j], s_w[j][tx], acc);
    __syncthreads();
  }
  if (t < n && col < d) V[(size_t)t * d + col] = acc;
}

constexpr size_t PV_SMEM = 1024 + (size_t)PV_NS * (PV_A_BYTES + PV_B_BYTES) + 16 * PV_NS + 8 + 16 + 64;

// Launch of the pair kernel (its cluster shape (2, 1, 1) is a compile-time property) behind the previous
// kernel's programmatic completion.  Function attributes are kept per device: opt in once on each.
cudaError_t launch_pair(int device, dim3 grid, cudaStream_t st, const CUtensorMap& kmap, const CUtensorMap& wmap, float* V, int n,
                        int d, int d_k, int hp, int* status, const SlimDecodeParams& cp) {
  static bool attr_set[64] = {};
  if (device < 0 || device >= 64 || !attr_set[device]) {
    cudaError_t e = cudaFuncSetAttribute((const void*)slim_values_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)PV2_SMEM);
    if (e != cudaSuccess) return e;
    if (device >= 0 && device < 64) attr_set[device] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(PV2_THREADS);
  cfg.dynamicSmemBytes = PV2_SMEM;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, slim_values_pair_kernel, kmap, wmap, V, n, d, d_k, hp, status, cp);
}

}  // namespace

// cache != NULL (slim_prefill): K is [batch][n_new][d] and its rows are also stored at positions[b] ..
cudaError_t slim_launch_values(const slim_ctx* ctx, const void* K, int n, float* V, cudaStream_t st, const slim_cache* cache,
                               const int32_t* positions, int n_new) {
  const int d = ctx->d, d_k = ctx->d_k, H = ctx->H;
  const bool tc = ctx->proj_ok && ((uintptr_t)K & 15) == 0 && ((uintptr_t)V & 15) == 0;
  SlimDecodeParams cp;
  memset(&cp, 0, sizeof(cp));
  if (cache) {
    if (!tc || ctx->kdtype == SLIM_FP8 || ((uintptr_t)cache->k & 15)) {   // no fused store on this path (an 8-bit cache quantises): the append kernel first
      cudaError_t e = slim_launch_append(ctx, cache, K, positions, n_new, 0, st);
      if (e != cudaSuccess) return e;
    } else {
      cp.k = cache->k; cp.q = K; cp.lengths = positions; cp.workers = n_new; cp.d = d;
      cp.batch = cache->batch; cp.t_cap = cache->t_cap; cp.status = ctx->status;
      cp.block_table = cache->block_table; cp.page_rows = cache->page_rows; cp.max_pages = cache->max_pages;
      cp.num_pages = cache->num_pages;
    }
  }
  if (tc) {
    // function attributes are kept per device: opt in once on each device this is called on
    static bool attr_set[64] = {};
    if (ctx->device < 0 || ctx->device >= 64 || !attr_set[ctx->device]) {
      cudaError_t e = cudaFuncSetAttribute((const void*)slim_values_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PV_SMEM);
      if (e != cudaSuccess) return e;
      if (ctx->device >= 0 && ctx->device < 64) attr_set[ctx->device] = true;
    }
    CUtensorMap kmap, wmap;
    const unsigned long long dims[3] = {(unsigned long long)d, (unsigned long long)n, 1};
    const unsigned long long strides[2] = {(unsigned long long)d * 2, (unsigned long long)d * 2 * (unsigned long long)n};
    const unsigned int box[3] = {PV_J, PV_ROWS, 1};
    cudaError_t e = slim_tmap_encode_3d(&kmap, const_cast<void*>(K), dims, strides, box);
    if (e != cudaSuccess) return e;
    const int hp = d_k == 64 ? 2 : 1;
    memcpy(&wmap, ctx->wmap, sizeof(wmap));
    // CTA pairs with 256-column tiles where a tile is two whole 128-column groups (d_k = 128 or 64), the groups
    // pair up and the prompt has more than one row tile
    if (ctx->opt_prompt_pair && n > PV_ROWS && hp * d_k == 128 && (H / hp) % 2 == 0) {
      const int ntiles = (d / PV2_NCOL) * ((n + 2 * PV_ROWS - 1) / (2 * PV_ROWS)), pairs = ctx->num_sms / 2;
      const dim3 grid(2 * (ntiles < pairs ? ntiles : pairs));           // one pair per SM pair, each walks its tiles
      return launch_pair(ctx->device, grid, st, kmap, wmap, V, n, d, d_k, hp, ctx->status, cp);
    }
    return slim_launch_pdl(slim_values_tc_kernel, dim3(H / hp, (n + PV_ROWS - 1) / PV_ROWS), dim3(128), PV_SMEM, st, kmap, wmap, V, n,
                           d, d_k, hp, ctx->status, cp);
  }
  dim3 grid((d + 15) / 16, (n + 15) / 16);
  if (ctx->dtype == SLIM_BF16)
    slim_values_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)K, (const __nv_bfloat16*)ctx->wkv, V, n, d, d_k);
  else
    slim_values_kernel<float><<<grid, 256, 0, st>>>((const float*)K, (const float*)ctx->wkv, V, n, d, d_k);
  return cudaGetLastError();
}
