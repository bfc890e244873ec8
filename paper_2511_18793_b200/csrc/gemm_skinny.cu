// Weight-streaming GEMM for launches of at most 128 rows:  C[M,N] (op)= A[M,K] * W[N,K]^T  with the operands' roles
// swapped on the tensor core.
//
// With a handful of rows the product is bound by reading W once from HBM.  The 128-row MMA operand is therefore a
// 128 x 64 tile of W (16 KB per copy, the unit that has to be kept in flight), the rows of A are the MMA's N (MT = 32, 64
// or 128), and the accumulator in TMEM is a 128 x MT block of C^T.  An output tile is 128 columns of C; the K range of a
// tile is split over the CTAs of a thread-block cluster (up to 8) so that every SM streams a share of W, whatever N.
// Each CTA leaves its partial block in its own shared memory; after a cluster barrier the 32 x 32 blocks of the tile are
// dealt out to the cluster's CTAs, which add the parts in rank order, reading their peers' shared memory -- the bits
// never depend on timing -- and run the same fused epilogue as the other tensor-core kernels.
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
  static constexpr int kStages = MT == 32 ? 5 : MT == 64 ? 4 : 3;
  static constexpr int kBlocks = 4 * (MT / 32);              // 32 x 32 blocks of the tile: (TMEM lane quarter, 32 rows of A)
  static constexpr int kEpiWarps = MT == 32 ? 4 : 8;         // warp w: lane quarter w % 4, every (kEpiWarps / 4)-th row block
  static constexpr int kBlocksPerWarp = kBlocks / kEpiWarps;
  static constexpr int kThreads = 64 + 32 * kEpiWarps;
  static constexpr int kBarBytes = 128;
  // (the epilogue's transpose tiles reuse the ring: a CTA has one tile, and the ring is idle once it is accumulated)
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + kBarBytes;
  static constexpr int kTmemCols = MT;
  // kind::f16 instruction descriptor: D = f32, A = B = bf16, both K-major, N = MT, M = 128.
  static constexpr uint32_t kInstrDesc =
      (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(MT >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
  static_assert(kBlocks * 4096 <= kStages * kStageBytes, "transpose tiles do not fit in the ring");
  static_assert(2 * (kSmemBytes + 1024) <= 228 * 1024, "two CTAs per SM");
};

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Every thread of every CTA of the cluster executes both halves, on every path.
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// 16 bytes of the shared memory of CTA `rank` of the cluster, at the address that `local` has in this CTA.
__device__ __forceinline__ float4 ld_peer_f4(uint32_t local, uint32_t rank) {
  uint32_t ra;
  float4 v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local), "r"(rank));
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(ra) : "memory");
  return v;
}

// grid = tiles x splits, clusters of `splits` CTAs (blockIdx.x = tile * splits + split, split = rank in the cluster).  Warp 0: TMA producer; warp 1: TMEM owner and MMA issuer;
// warps 2 ..: epilogue, warp w on TMEM lane quarter w % 4 (columns n0 + 32 q ..) and the 32-row blocks c = (w - 2) / 4, + 1 or 2, .. of A.
template <int MT, int EPI>
__global__ void __launch_bounds__(SkinnyCfg<MT>::kThreads, 2)
    gemm_skinny_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, GemmArgs a,
                       int splits, int* status) {
  using C = SkinnyCfg<MT>;
  constexpr int STAGES = C::kStages;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bar_base = base + STAGES * C::kStageBytes;
  // barriers: full[STAGES], empty[STAGES], acc_full; then the TMEM slot and the abort flag
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  const uint32_t acc_full = bar_base + 8u * (2 * STAGES);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen_base + STAGES * C::kStageBytes + 8 * (2 * STAGES + 1));
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x / splits, split = (int)cluster_rank();
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
  constexpr int BPW = C::kBlocksPerWarp, CSTEP = C::kEpiWarps / 4;
  EpiRow er[BPW];                                // of the epilogue warps: the row the lane answers for in each of its blocks
#pragma unroll
  for (int bi = 0; bi < BPW; ++bi) er[bi] = EpiRow{1.f, 0, -1};

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
    // block b = 4 c + q of the tile: columns n0 + 32 q .., rows 32 c .. of A; its transpose tile is slot b of the (idle) ring
    const int q = warp & 3, c0 = (warp - 2) >> 2;
    const int n_chunk = n0 + q * 32;
#pragma unroll
    for (int bi = 0; bi < BPW; ++bi) {             // overlaps the main loop
      const int c = c0 + bi * CSTEP;
      if (splits == 1 || (c * 4 + q) % splits == split) er[bi] = epilogue_row<EPI>(a, c * 32 + lane, M);
    }
    const bool ok = warp_wait(acc_full, 0, abort_flag, lane);
    tc_fence_after();
#pragma unroll 1
    for (int bi = 0; bi < BPW && ok; ++bi) {
      const int c = c0 + bi * CSTEP, blk = c * 4 + q;
      const int row0 = c * 32, rows_here = min(32, M - row0);   // rows of this block that exist (may be <= 0)
      if (rows_here <= 0 || n_chunk >= a.N) continue;        // warp-uniform
      float4* stg4 = reinterpret_cast<float4*>(gen_base) + blk * (32 * 8);
      float* stg = reinterpret_cast<float*>(stg4);
      float v[32];                               // lane = column n_chunk + lane, v[j] = row row0 + j
      tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * 32), v);
      if (splits > 1) {
        // the partial block stays in this CTA's shared memory, in the "8 lanes per row" image; the cluster adds the parts below
#pragma unroll
        for (int j = 0; j < 32; ++j) stg[(j * 8 + ((lane >> 2) ^ (j & 7))) * 4 + (lane & 3)] = v[j];
      } else {
        // from lane = column to the "8 lanes per row" image: row j's 32 columns are one 128-byte line, chunks swizzled
        const float rs_mine = bi == 0 ? er[0].rs : er[BPW - 1].rs;
#pragma unroll
        for (int j = 0; j < 32; ++j)
          stg[(j * 8 + ((lane >> 2) ^ (j & 7))) * 4 + (lane & 3)] = v[j] * __shfl_sync(0xffffffffu, rs_mine, j);
        __syncwarp();
        epilogue_block<EPI>(a, stg4, lane, row0, rows_here, n_chunk, bi == 0 ? er[0] : er[BPW - 1]);
      }
    }
    if (!ok && lane == 0) *abort_flag = 1;
  }
  if (splits > 1) {
    // The cluster's CTAs are the splits of one tile (rank = split).  Block b of the tile is finished by CTA b mod
    // splits: it adds the parts in rank order, reading its peers' shared memory, and runs the epilogue on the sum.
    cluster_sync_all();                          // all parts are in place (or their CTA has raised its abort flag)
    if (warp >= 2 && !*abort_flag) {
      const int q = warp & 3, c0 = (warp - 2) >> 2;
      const int n_chunk = n0 + q * 32;
#pragma unroll 1
      for (int bi = 0; bi < BPW; ++bi) {
        const int c = c0 + bi * CSTEP, blk = c * 4 + q;
        const int row0 = c * 32, rows_here = min(32, M - row0);
        if (rows_here <= 0 || n_chunk >= a.N || blk % splits != split) continue;
        const EpiRow& erb = bi == 0 ? er[0] : er[BPW - 1];
        float4* stg4 = reinterpret_cast<float4*>(gen_base) + blk * (32 * 8);
        const uint32_t img = base + (uint32_t)blk * 4096u + (uint32_t)lane * 16u;
        float4 acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = ld_peer_f4(img + i * 512, 0);
        for (int sp = 1; sp < splits; ++sp) {
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float4 t = ld_peer_f4(img + i * 512, (uint32_t)sp);
            acc[i].x += t.x; acc[i].y += t.y; acc[i].z += t.z; acc[i].w += t.w;
          }
        }
        __syncwarp();                            // (this CTA's own part is one of the sources)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float rs = __shfl_sync(0xffffffffu, erb.rs, i * 4 + (lane >> 3));
          stg4[i * 32 + lane] = make_float4(acc[i].x * rs, acc[i].y * rs, acc[i].z * rs, acc[i].w * rs);
        }
        __syncwarp();
        epilogue_block<EPI>(a, stg4, lane, row0, rows_here, n_chunk, erb);
      }
    }
    cluster_sync_all();                          // no CTA leaves while a peer may still read its part
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
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(tiles * splits); cfg.blockDim = dim3(C::kThreads); cfg.dynamicSmemBytes = C::kSmemBytes; cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = splits; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = pdl_enabled() ? 2 : 1;
  cudaLaunchKernelEx(&cfg, gemm_skinny_kernel<MT, EPI>, tw, tx, a, splits, a.status);
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

// Number of CTAs a tile's K range is split over (= the cluster size): as many as bring the grid to about one CTA per SM
// (NEZHA_SKINNY_CTAS: another target), at most 8, each with at least four k-steps (64 KB of W per partial tile).
// A function of N, K and the device only -- never of the row count -- so a product's bits do not depend on its rows.
int gemm_skinny_splits(int N, int K, int n_sm) {
  static const int forced = getenv("NEZHA_SKINNY_CTAS") ? atoi(getenv("NEZHA_SKINNY_CTAS")) : 0;
  const int target = forced > 0 ? forced : n_sm;
  const int tiles = (N + 127) / 128, k_iters = K / BK;
  int s = target / tiles;
  if (s > k_iters / 4) s = k_iters / 4;
  if (s > 8) s = 8;                              // the portable cluster size
  if (s < 1) s = 1;
  return s;
}

bool gemm_skinny_applies(const GemmArgs& a, int n_sm) {
  (void)n_sm;
  return a.skinny && a.M <= kSkinnyRows && (long long)((a.N + 127) / 128) * 8 <= 0x7fffffff;
}

void launch_gemm_skinny(const GemmArgs& a, int n_sm, cudaStream_t st) {
  const int tiles = (a.N + 127) / 128, splits = gemm_skinny_splits(a.N, a.K, n_sm);
  if (a.M <= 32) launch_mt<32>(a, tiles, splits, st);      // (the bound, not the expected count: no row may be dropped)
  else if (a.M <= 64) launch_mt<64>(a, tiles, splits, st);
  else launch_mt<128>(a, tiles, splits, st);
}

}  // namespace nz
