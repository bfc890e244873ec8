// Weight-streaming GEMM for launches of at most 64 rows:  C[M,N] (op)= A[M,K] * W[N,K]^T  with the operands' roles
// swapped on the tensor core.
//
// With a handful of rows the product is bound by reading W once from HBM.  The 128-row MMA operand is therefore a
// 128 x 64 tile of W (16 KB per copy, the unit that has to be kept in flight), the rows of A are the MMA's N (MT = 32 or
// 64), and the accumulator in TMEM is a 128 x MT block of C^T.  An output tile is 128 columns of C; the K range of a
// tile is split over several CTAs so that every SM streams a share of W, whatever N.  Each CTA of a split tile writes
// its partial block to a work space; the CTA that arrives last (an arrival counter per tile, no waiting) adds the
// parts in split order -- the order of arrival never shows in the bits -- and runs the same fused epilogue as the
// other tensor-core kernels.
// A CTA issues the weight copies of its first ring round BEFORE the launch's dependency on the preceding kernel is
// resolved (W is constant data), and the kernel is sized for two CTAs per SM, so the weight stream of a launch starts
// while its predecessor is still draining.
// Every mbarrier wait is bounded, as in the other kernels.
#include <stdlib.h>

#include "gemm_epilogue.cuh"

namespace nz {

namespace {

using namespace gemm_detail;

template <int MT> struct SkinnyCfg {
  static constexpr int kTileBytesW = 128 * BK * 2;
  static constexpr int kTileBytesX = MT * BK * 2;
  static constexpr int kStageBytes = kTileBytesW + kTileBytesX;
  static constexpr int kStages = MT == 32 ? 5 : 4;
  static constexpr int kEpiWarps = 4 * (MT / 32);            // one per (TMEM lane quarter, block of 32 rows of A)
  static constexpr int kThreads = 64 + 32 * kEpiWarps;
  static constexpr int kBarBytes = 128;
  // (the epilogue's transpose tiles reuse the ring: a CTA has one tile, and the ring is idle once it is accumulated)
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + kBarBytes;
  static constexpr int kTmemCols = MT;
  // kind::f16 instruction descriptor: D = f32, A = B = bf16, both K-major, N = MT, M = 128.
  static constexpr uint32_t kInstrDesc =
      (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(MT >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
  static_assert(kEpiWarps * 4096 <= kStages * kStageBytes, "transpose tiles do not fit in the ring");
  static_assert(2 * (kSmemBytes + 1024) <= 228 * 1024, "two CTAs per SM");
};

__device__ __forceinline__ void epi_bar_sync(int n_threads) {
  asm volatile("bar.sync 1, %0;" ::"r"(n_threads) : "memory");
}

// grid = tiles x splits (blockIdx.x = tile * splits + split).  Warp 0: TMA producer; warp 1: TMEM owner and MMA issuer;
// warps 2 ..: epilogue, warp w on TMEM lane quarter w % 4 (columns n0 + 32 q ..) and rows 32 c .. of A, c = (w - 2) / 4.
template <int MT, int EPI>
__global__ void __launch_bounds__(SkinnyCfg<MT>::kThreads, 2)
    gemm_skinny_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, GemmArgs a,
                       SkinnyWork work, int splits, int* status) {
  using C = SkinnyCfg<MT>;
  constexpr int STAGES = C::kStages;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bar_base = base + STAGES * C::kStageBytes;
  // barriers: full[STAGES], empty[STAGES], acc_full; then the TMEM slot, the abort flag and the "last arriver" flag
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  const uint32_t acc_full = bar_base + 8u * (2 * STAGES);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen_base + STAGES * C::kStageBytes + 8 * (2 * STAGES + 1));
  volatile uint32_t* abort_flag = tmem_slot + 1;
  volatile uint32_t* last_flag = tmem_slot + 2;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x / splits, split = blockIdx.x - tile * splits;
  const int n0 = tile * 128;
  // this CTA's share of the k-steps: contiguous, the first (k_iters % splits) shares one step longer
  const int k_iters = a.K / BK;
  const int k_base = k_iters / splits, k_rem = k_iters - k_base * splits;
  const int k_begin = split * k_base + min(split, k_rem), k_count = k_base + (split < k_rem ? 1 : 0);
  const int pre = min(STAGES, k_count);          // ring slots filled in the first round

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(acc_full, 1);
    *abort_flag = 0;
    *last_flag = 0;
    mbar_fence_init();
    tma_prefetch_map(&tmW);
    tma_prefetch_map(&tmX);
    // the weight tiles of the first round: constant data, so they may be fetched while the predecessor still runs
    for (int s = 0; s < pre; ++s) {
      mbar_expect_tx(full_bar(s), C::kStageBytes);
      tma_load_2d(base + s * C::kStageBytes, &tmW, (k_begin + s) * BK, n0, full_bar(s));
    }
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)),
                 "r"(C::kTmemCols));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();
  pdl_launch();
  const int M = a.M_dev ? min(a.M, *a.M_dev) : a.M;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      bool ok = true;
      int issued = pre;                          // k-steps whose `full` barrier has been armed
      for (int s = 0; s < pre; ++s)
        tma_load_2d(base + s * C::kStageBytes + C::kTileBytesW, &tmX, (k_begin + s) * BK, 0, full_bar(s));
      int s = 0;
      uint32_t round = 1;                        // parity bit of the round that k-step `pre` belongs to (pre = STAGES here)
      for (int k = pre; k < k_count; ++k, ++issued) {
        if (!mbar_wait_or_abort(empty_bar(s), round ^ 1u, abort_flag)) { ok = false; break; }
        const uint32_t fb = full_bar(s), dst = base + s * C::kStageBytes;
        mbar_expect_tx(fb, C::kStageBytes);
        tma_load_2d(dst, &tmW, (k_begin + k) * BK, n0, fb);
        tma_load_2d(dst + C::kTileBytesW, &tmX, (k_begin + k) * BK, 0, fb);
        if (++s == STAGES) { s = 0; round ^= 1u; }
      }
      if (!ok) {                                 // drain: wait (bounded) for the copies still in flight
        *abort_flag = 1;
        for (int j = max(0, issued - STAGES); j < issued; ++j) mbar_wait(full_bar(j % STAGES), (j / STAGES) & 1);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      bool ok = true;
      const uint64_t dw0 = smem_desc(base), dx0 = smem_desc(base + C::kTileBytesW);
      int s = 0;
      uint32_t round = 0;
      for (int k = 0; k < k_count; ++k) {
        if (!mbar_wait_or_abort(full_bar(s), round, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint64_t so = (uint64_t)(s * (C::kStageBytes >> 4));
        tc_mma_kstep(tmem_base, dw0 + so, dx0 + so, C::kInstrDesc, k > 0 ? 1u : 0u);
        tc_commit(empty_bar(s));
        if (++s == STAGES) { s = 0; round ^= 1u; }
      }
      if (ok) tc_commit(acc_full);
      else *abort_flag = 1;
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int q = warp & 3, c = (warp - 2) >> 2, ew = warp - 2;
    constexpr int kBlocks = 4 * (MT / 32);       // 32 x 32 blocks of a CTA's partial tile
    float4* stg4 = reinterpret_cast<float4*>(gen_base) + ew * (32 * 8);
    float* stg = reinterpret_cast<float*>(stg4);
    const int row0 = c * 32, n_chunk = n0 + q * 32;
    const int rows_here = min(32, M - row0);     // rows of this block that exist (may be <= 0)
    const bool have = rows_here > 0 && n_chunk < a.N;      // warp-uniform
    const EpiRow er = epilogue_row<EPI>(a, row0 + lane, M);   // overlaps the main loop
    bool ok = warp_wait(acc_full, 0, abort_flag, lane);
    tc_fence_after();
    float v[32];                                 // lane = column n_chunk + lane, v[j] = row row0 + j
    if (ok) tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * 32), v);
    if (splits == 1) {
      if (ok && have) {
        // from lane = column to the "8 lanes per row" image: row j's 32 columns are one 128-byte line, chunks swizzled
#pragma unroll
        for (int j = 0; j < 32; ++j)
          stg[(j * 8 + ((lane >> 2) ^ (j & 7))) * 4 + (lane & 3)] = v[j] * __shfl_sync(0xffffffffu, er.rs, j);
        __syncwarp();
        epilogue_block<EPI>(a, stg4, lane, row0, rows_here, n_chunk, er);
      }
    } else {
      // the partial block goes to the work space in the same image (every store of a warp is one 128-byte line)
      if (ok && have) {
        float* img = work.partials + ((size_t)blockIdx.x * kBlocks + (c * 4 + q)) * 1024;
#pragma unroll
        for (int j = 0; j < 32; ++j) __stcg(img + (j * 8 + ((lane >> 2) ^ (j & 7))) * 4 + (lane & 3), v[j]);
        __threadfence();
      }
      if (!ok && lane == 0) *abort_flag = 1;
      epi_bar_sync(32 * C::kEpiWarps);
      if (ew == 0 && lane == 0 && !*abort_flag) {
        __threadfence();                         // the other warps' parts, ordered before this thread by the barrier
        const unsigned old = atomicAdd(work.arrivals + tile, 1u);
        if (old == (unsigned)(splits - 1)) {
          __threadfence();
          work.arrivals[tile] = 0;               // every part has arrived: ready for the next launch
          *last_flag = 1;
        }
      }
      epi_bar_sync(32 * C::kEpiWarps);
      if (*last_flag && have) {
        __threadfence();
        // lane's 8 chunks of the block image, summed over the parts in split order
        const float4* src = reinterpret_cast<const float4*>(work.partials + ((size_t)(tile * splits) * kBlocks + (c * 4 + q)) * 1024);
        float4 acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = __ldcg(src + i * 32 + lane);
        for (int sp = 1; sp < splits; ++sp) {
          const float4* p = src + (size_t)sp * kBlocks * 256;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float4 t = __ldcg(p + i * 32 + lane);
            acc[i].x += t.x; acc[i].y += t.y; acc[i].z += t.z; acc[i].w += t.w;
          }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float rs = __shfl_sync(0xffffffffu, er.rs, i * 4 + (lane >> 3));     // chunk i*32 + lane is of row i*4 + lane/8
          stg4[i * 32 + lane] = make_float4(acc[i].x * rs, acc[i].y * rs, acc[i].z * rs, acc[i].w * rs);
        }
        __syncwarp();
        epilogue_block<EPI>(a, stg4, lane, row0, rows_here, n_chunk, er);
      }
    }
    if (!ok && lane == 0) *abort_flag = 1;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols));
  }
  if (threadIdx.x == 0 && *abort_flag) atomicOr(status, kStInternal);
}

template <int MT, int EPI>
void launch(const GemmArgs& a, int tiles, int splits, cudaStream_t st) {
  using C = SkinnyCfg<MT>;
  CUtensorMap tw, tx;
  if (!tma_map_bf16(a.W, a.N, a.K, a.ldw, 128, &tw) || !tma_map_bf16(a.A, a.M, a.K, a.lda, MT, &tx)) {
    static const int flag = kStInternal;       // cannot happen for shapes gemm_tc_supported accepted; report, do not guess
    cudaMemcpyAsync(a.status, &flag, sizeof(int), cudaMemcpyHostToDevice, st);
    return;
  }
  static PerDeviceOnce configured;
  configured.run([] {
    cudaFuncSetAttribute(gemm_skinny_kernel<MT, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
  });
  launch_pdl(gemm_skinny_kernel<MT, EPI>, dim3(tiles * splits), dim3(C::kThreads), C::kSmemBytes, st, tw, tx, a, *a.skinny,
             splits, a.status);
}

template <int MT>
void launch_mt(const GemmArgs& a, int tiles, int splits, cudaStream_t st) {
  switch (a.epilogue) {
    case kEpiStoreAct: launch<MT, kEpiStoreAct>(a, tiles, splits, st); break;
    case kEpiStoreF32: launch<MT, kEpiStoreF32>(a, tiles, splits, st); break;
    case kEpiAddF32: launch<MT, kEpiAddF32>(a, tiles, splits, st); break;
    case kEpiBiasTanhF32: launch<MT, kEpiBiasTanhF32>(a, tiles, splits, st); break;
    case kEpiSwiGLU: launch<MT, kEpiSwiGLU>(a, tiles, splits, st); break;
    case kEpiAddNorm: launch<MT, kEpiAddNorm>(a, tiles, splits, st); break;
    case kEpiRopeKV: launch<MT, kEpiRopeKV>(a, tiles, splits, st); break;
    default: break;
  }
}

}  // namespace

// Number of CTAs a tile's K range is split over: as many as bring the grid to about `target` CTAs (one per SM unless
// NEZHA_SKINNY_CTAS says otherwise), each with at least four k-steps (64 KB of W per 16 or 32 KB of partial tile).
// A function of N, K and the device only -- never of the row count -- so a product's bits do not depend on its rows.
int gemm_skinny_splits(int N, int K, int n_sm) {
  static const int forced = getenv("NEZHA_SKINNY_CTAS") ? atoi(getenv("NEZHA_SKINNY_CTAS")) : 0;
  const int target = forced > 0 ? forced : n_sm;
  const int tiles = (N + 127) / 128, k_iters = K / BK;
  int s = target / tiles;
  if (s > k_iters / 4) s = k_iters / 4;
  if (s < 1) s = 1;
  while (s > 1 && (long long)tiles * s > kSkinnyMaxCtas) --s;
  return s;
}

bool gemm_skinny_applies(const GemmArgs& a, int n_sm) {
  return a.skinny && a.skinny->partials && a.skinny->arrivals && a.M <= kSkinnyRows && (a.N + 127) / 128 <= kSkinnyMaxTiles &&
         (long long)((a.N + 127) / 128) * gemm_skinny_splits(a.N, a.K, n_sm) <= kSkinnyMaxCtas;
}

void launch_gemm_skinny(const GemmArgs& a, int n_sm, cudaStream_t st) {
  const int tiles = (a.N + 127) / 128, splits = gemm_skinny_splits(a.N, a.K, n_sm);
  if (a.M <= 32) launch_mt<32>(a, tiles, splits, st);      // (the bound, not the expected count: no row may be dropped)
  else launch_mt<64>(a, tiles, splits, st);
}

}  // namespace nz
