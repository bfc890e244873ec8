// The tensor-core GEMM for large problems: CTA pairs.  Two CTAs of a cluster compute one 256 x 256 output tile with
// tcgen05.mma.cta_group::2: each CTA holds 128 of the tile's rows (its own A tile, its own 2 x 256-column TMEM
// accumulators) and stages only HALF of the W tile (128 of its 256 rows); the tensor cores of the pair exchange the
// halves.  Per 128 x 256 of output a CTA therefore pulls 32 KB per k-step through L2 instead of 48 KB -- at K of about
// a thousand the single-CTA kernel is bound by exactly that traffic.  Roles per CTA as in gemm_tc.cu (TMA producer,
// MMA issuer, 8 epilogue warps, persistent over tiles, two accumulators so that the epilogue overlaps the next main
// loop); only the leader CTA (cluster rank 0) issues MMAs.  Barriers: `full` lives in the leader and collects the
// bytes of both CTAs' copies; `empty` and `acc_full` live in both CTAs and are signalled by multicast commits;
// `acc_empty` lives in the leader and counts the epilogue warps of both CTAs.  No TMA multicast is used: every copy
// lands in the shared memory of the CTA that issued it.  Every wait is bounded as in gemm_tc.cu.
#include "gemm_epilogue.cuh"

namespace nz {

namespace {

using namespace gemm_detail;

constexpr int kBN2 = 256;                               // columns of the pair's tile (and of each CTA's accumulator)
constexpr int kTileBytesBHalf = (kBN2 / 2) * BK * 2;    // this CTA's half of the W tile
constexpr int kStageBytes2 = kTileBytesA + kTileBytesBHalf;
constexpr int kStages2 = 6;
constexpr int kSmemBytes2 = kStages2 * kStageBytes2 + 1024 + 256 + kTransposeBytes;
constexpr uint32_t kLeaderMask = 0xFEFFFFFFu;           // clears the CTA-rank bit of a shared-window address: same offset in rank 0
// kind::f16 instruction descriptor: D = f32, A = B = bf16, both K-major, N = 256, M = 256 (over the pair).
constexpr uint32_t kInstrDesc2 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBN2 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// A copy of this CTA into its own shared memory whose completion is counted by the LEADER's barrier.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t leader_bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(leader_bar) : "memory");
}
// The four MMAs (K = 16 each) of one 64-deep k-step over the pair, in one statement (see tc_mma_kstep).
__device__ __forceinline__ void tc_mma_pair_kstep(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t accumulate_first) {
  asm volatile(
      "{\n\t.reg .pred p, t;\n\t.reg .b64 a1, b1, a2, b2, a3, b3;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "setp.eq.b32 t, %4, %4;\n\t"
      "add.s64 a1, %1, 2;\n\tadd.s64 b1, %2, 2;\n\t"
      "add.s64 a2, %1, 4;\n\tadd.s64 b2, %2, 4;\n\t"
      "add.s64 a3, %1, 6;\n\tadd.s64 b3, %2, 6;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], a1, b1, %3, t;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], a2, b2, %3, t;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], a3, b3, %3, t;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(kInstrDesc2), "r"(accumulate_first) : "memory");
}
// Arrives (once the MMAs issued so far have completed) on the barrier at this offset in BOTH CTAs of the pair.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  const uint16_t both = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(both) : "memory");
}
__device__ __forceinline__ void mbar_arrive_leader(uint32_t bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar & kLeaderMask) : "memory");
}

template <int EPI>
__global__ void __launch_bounds__(kThreads) gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap tmA,
                                                                const __grid_constant__ CUtensorMap tmB, GemmArgs a,
                                                                int* status) {
  constexpr int STAGES = kStages2;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = base + STAGES * kStageBytes2;
  // barriers: full[STAGES] (leader's is used), empty[STAGES], acc_full[2], acc_empty[2] (leader's is used)
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto acc_full = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
  auto acc_empty = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
  uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot =
      reinterpret_cast<volatile uint32_t*>(gen_base + STAGES * kStageBytes2 + 8 * (2 * STAGES + 4));
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_rank();              // 0 = leader
  const int k_iters = a.K / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), 2 * kEpiWarps); }
    *abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_map(&tmA);
    tma_prefetch_map(&tmB);
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)),
                 "r"(2 * kBN2));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;");
  }
  tc_fence_before();
  cluster_sync_all();                                // both CTAs' barriers and TMEM exist before either signals the other
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // everything above touched no global memory; from here on the preceding kernel's results are needed
  pdl_wait();
  pdl_launch();
  const int M = a.M_dev ? min(a.M, *a.M_dev) : a.M;
  const int tiles_m = (M + 2 * BM - 1) / (2 * BM), tiles_n = (a.N + kBN2 - 1) / kBN2;
  const int n_tiles = tiles_m * tiles_n;             // tiles of the pair; a pair without a tile falls through every loop
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int s = 0;
      uint32_t round = 0;
      bool ok = true;
      for (int tile = pair; tile < n_tiles && ok; tile += n_pairs) {
        const int m0 = (tile % tiles_m) * (2 * BM) + rank * BM;          // this CTA's rows
        const int nb0 = (tile / tiles_m) * kBN2 + rank * (kBN2 / 2);     // this CTA's half of the W tile
        for (int k = 0; k < k_iters; ++k) {
          // (round 0 never waits: the parity before a fresh barrier's first one counts as complete)
          if (!mbar_wait_or_abort(empty_bar(s), round ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t dst = base + s * kStageBytes2, fb = full_bar(s) & kLeaderMask;
          if (rank == 0) mbar_expect_tx(full_bar(s), 2 * kStageBytes2);  // the bytes of both CTAs' copies
          tma_load_2d_pair(dst, &tmA, k * BK, m0, fb);
          tma_load_2d_pair(dst + kTileBytesA, &tmB, k * BK, nb0, fb);
          if (++s == STAGES) { s = 0; round ^= 1u; }
        }
      }
      if (!ok) *abort_flag = 1;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader only)
    if (lane == 0 && rank == 0) {
      int t_local = 0, s = 0;
      uint32_t round = 0;
      bool ok = true;
      const uint64_t da0 = smem_desc(base), db0 = smem_desc(base + kTileBytesA);   // slot 0; later slots add to the address field
      for (int tile = pair; tile < n_tiles && ok; tile += n_pairs, ++t_local) {
        const int b = t_local & 1;
        if (t_local >= 2 && !mbar_wait_or_abort(acc_empty(b), ((t_local >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_acc = tmem_base + (uint32_t)(b * kBN2);
        for (int k = 0; k < k_iters; ++k) {
          if (!mbar_wait_or_abort(full_bar(s), round, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint64_t so = (uint64_t)(s * (kStageBytes2 >> 4));
          tc_mma_pair_kstep(tmem_acc, da0 + so, db0 + so, k > 0 ? 1u : 0u);
          tc_commit_pair(empty_bar(s));          // slot free in both CTAs once these MMAs have read it
          if (++s == STAGES) { s = 0; round ^= 1u; }
        }
        if (ok) tc_commit_pair(acc_full(b));     // accumulator complete, in both CTAs
      }
      if (!ok) *abort_flag = 1;
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9, both CTAs)
    const int q = warp & 3;
    const int half = (warp - 2) >> 2;
    float4* stg4 = reinterpret_cast<float4*>(gen_base + STAGES * kStageBytes2 + 256) + (warp - 2) * (32 * 8);
    int t_local = 0;
    bool ok = true;
    for (int tile = pair; tile < n_tiles && ok; tile += n_pairs, ++t_local) {
      const int m0 = (tile % tiles_m) * (2 * BM) + rank * BM, n0 = (tile / tiles_m) * kBN2;
      const int b = t_local & 1;
      const EpiRow er = epilogue_row<EPI>(a, m0 + q * 32 + lane, M);
      ok = warp_wait(acc_full(b), (t_local >> 1) & 1, abort_flag, lane);
      if (!ok) break;
      tc_fence_after();
      drain_accumulator<kBN2, EPI>(a, tmem_base + (uint32_t)(b * kBN2), q, half, lane, stg4, m0, n0, M, er);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_leader(acc_empty(b));   // hand the accumulator (of this CTA) back to the leader's MMA warp
    }
    if (!ok && lane == 0) *abort_flag = 1;
  }
  tc_fence_before();
  cluster_sync_all();                            // neither CTA leaves (or frees TMEM) while the other may still signal it
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * kBN2));
  }
  if (threadIdx.x == 0 && *abort_flag) atomicOr(status, kStInternal);
}

template <int EPI>
void launch_pair(const GemmArgs& a, int n_sm, cudaStream_t st) {
  CUtensorMap ta, tb;
  if (!tma_map_bf16(a.A, a.M, a.K, a.lda, BM, &ta) || !tma_map_bf16(a.W, a.N, a.K, a.ldw, kBN2 / 2, &tb)) {
    static const int flag = kStInternal;
    cudaMemcpyAsync(a.status, &flag, sizeof(int), cudaMemcpyHostToDevice, st);
    return;
  }
  static PerDeviceOnce configured;
  configured.run([] {
    cudaFuncSetAttribute(gemm_tc_pair_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes2);
  });
  const long long tiles = (long long)((a.M + 2 * BM - 1) / (2 * BM)) * ((a.N + kBN2 - 1) / kBN2);
  const int pairs = (int)(tiles < n_sm / 2 ? tiles : n_sm / 2);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(2 * pairs); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = kSmemBytes2; cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, gemm_tc_pair_kernel<EPI>, ta, tb, a, a.status);
}

}  // namespace

// The caller has checked gemm_tc_supported(a); n_sm = SMs of the device.
void launch_gemm_tc_pair(const GemmArgs& a, int n_sm, cudaStream_t st) {
  switch (a.epilogue) {
    case kEpiStoreAct: launch_pair<kEpiStoreAct>(a, n_sm, st); break;
    case kEpiStoreF32: launch_pair<kEpiStoreF32>(a, n_sm, st); break;
    case kEpiAddF32: launch_pair<kEpiAddF32>(a, n_sm, st); break;
    case kEpiBiasTanhF32: launch_pair<kEpiBiasTanhF32>(a, n_sm, st); break;
    case kEpiSwiGLU: launch_pair<kEpiSwiGLU>(a, n_sm, st); break;
    case kEpiAddNorm: launch_pair<kEpiAddNorm>(a, n_sm, st); break;
    case kEpiRopeKV: launch_pair<kEpiRopeKV>(a, n_sm, st); break;
    default: break;
  }
}

}  // namespace nz
