// Blackwell tensor-core GEMM:  C[M,N] (op)= A[M,K] * W[N,K]^T,  bf16 operands, fp32 accumulation in TMEM.
//
// Persistent kernel: each CTA walks the 128 x BN output tiles assigned to it (BN = 32 ... 256, chosen so that small
// problems still spread over the SMs and large ones use the widest tile).  Warp 0 streams 128x64 (A) and BNx64 (W)
// bf16 tiles into a shared-memory ring with TMA (128-byte swizzle; K-major on both sides, which is exactly how
// activations [tokens, features] and weights [out, in] are stored).  Warp 1 issues tcgen05.mma (M128 N=BN K16, four per
// stage) into one of TWO BN-column TMEM accumulators and releases ring slots with tcgen05.commit.  Warps 2-9 (two per
// TMEM lane quarter) read a finished accumulator back with tcgen05.ld, 32 columns at a time, transpose the 32 x 32
// block through shared memory so that a warp writes whole row segments, and apply the epilogue -- while the MMA warp
// is already filling the other accumulator with the next tile.  Besides plain stores the epilogue can finish the
// surrounding element-wise work of a transformer layer: the RMSNorm row scale of the A operand, SwiGLU, rotary
// embedding + KV-cache append, residual add + next layer's norm input (see GemmFuse).
// Every mbarrier wait is bounded: on expiry the CTA raises an abort flag that ends every role's loop, records an error
// in the status word, drains the copies it has in flight, frees its TMEM and returns.
#include <stdlib.h>

#include "gemm_epilogue.cuh"

namespace nz {

namespace {

using namespace gemm_detail;

template <int BN> struct Cfg {
  static constexpr int kTileBytesB = BN * BK * 2;
  static constexpr int kStageBytes = kTileBytesA + kTileBytesB;
  // as many stages as fit beside the transpose tiles: short-M launches are bound by bytes in flight per CTA
  // (even, so that with two MMA issuers a ring slot always belongs to the same issuer: see the kernel)
  static constexpr int kStages = BN >= 192 ? 4 : BN == 160 ? 5 : BN == 128 ? 6 : 8;
  static constexpr int kSmemBytes =
      kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/ + kTransposeBytes;
  // kind::f16 instruction descriptor: D = f32, A = B = bf16, both K-major, N = BN, M = 128.
  static constexpr uint32_t kInstrDesc =
      (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
};


// ISS = number of MMA-issuing warps.  The tensor pipe takes a tcgen05.mma of M = 128 about every 76 cycles whatever
// its N, and one issuing thread adds its own barrier wait, fence and commit to every k-step, during which the pipe
// idles: the k-loop of a tile of at most 128 columns is bound by that chain, not by data or flops.  With ISS = 2 the
// warps 1 and 2 take the k-steps alternately, each into an accumulator of its own (added up by the epilogue), so one
// issuer's overhead runs under the other's MMAs.
template <int BN, int EPI, int ISS>
__global__ void __launch_bounds__(kThreads + 32 * (ISS - 1)) gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA,
                                                                            const __grid_constant__ CUtensorMap tmB,
                                                                            GemmArgs a, int* status) {
  using C = Cfg<BN>;
  // two accumulators of ISS chains each, in a power-of-two number of TMEM columns
  constexpr int kAccCols = 2 * BN * ISS;
  constexpr int kTmemCols = kAccCols <= 32 ? 32 : kAccCols <= 64 ? 64 : kAccCols <= 128 ? 128 : kAccCols <= 256 ? 256 : 512;
  static_assert(kAccCols <= 512, "accumulator chains do not fit");
  // A slot's `full` barrier must be waited for by ONE thread, phase after phase: a thread that asked for the phase after
  // the one still in flight would be told "complete" (the parity it names is also that of the phase before).  With the
  // k-steps dealt round-robin that holds exactly when the ring length is a multiple of the number of issuers.
  static_assert(C::kStages % ISS == 0, "a ring slot must always be consumed by the same issuer");
  constexpr int kFirstEpiWarp = 1 + ISS;
  constexpr int STAGES = C::kStages;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = base + STAGES * C::kStageBytes;
  // barriers: full[STAGES], empty[STAGES], acc_full[2], acc_empty[2]; then the TMEM slot and the abort flag
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto acc_full = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
  auto acc_empty = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
  uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot =
      reinterpret_cast<volatile uint32_t*>(gen_base + STAGES * C::kStageBytes + 8 * (2 * STAGES + 4));
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int k_iters = a.K / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), ISS); mbar_init(acc_empty(b), kEpiWarps); }
    *abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_map(&tmA);
    tma_prefetch_map(&tmB);
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)),
                 "r"(kTmemCols));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // everything above touched no global memory; from here on the preceding kernel's results are needed
  pdl_wait();
  pdl_launch();
  const int M = a.M_dev ? min(a.M, *a.M_dev) : a.M;
  const int tiles_m = (M + BM - 1) / BM, tiles_n = (a.N + BN - 1) / BN;
  const int n_tiles = tiles_m * tiles_n;     // a CTA without a tile falls through every role loop

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int it = 0;                                // k-iterations issued so far, over all tiles
      int s = 0;                                 // it % STAGES, and the parity of slot s's current round
      uint32_t round = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        const int m0 = (tile % tiles_m) * BM, n0 = (tile / tiles_m) * BN;
        for (int k = 0; k < k_iters; ++k, ++it) {
          // (waiting for the parity before the first one succeeds at once on a fresh barrier: round 0 never waits)
          if (!mbar_wait_or_abort(empty_bar(s), round ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t fb = full_bar(s), dst = base + s * C::kStageBytes;
          mbar_expect_tx(fb, C::kStageBytes);
          tma_load_2d(dst, &tmA, k * BK, m0, fb);
          tma_load_2d(dst + kTileBytesA, &tmB, k * BK, n0, fb);
          if (++s == STAGES) { s = 0; round ^= 1u; }
        }
      }
      if (!ok) {                                 // drain: wait (bounded) for the copies still in flight
        *abort_flag = 1;
        for (int j = max(0, it - STAGES); j < it; ++j) mbar_wait(full_bar(j % STAGES), (j / STAGES) & 1);
      }
    }
  } else if (warp <= ISS) {
    // ------------------------------------------------------------------ MMA issuers (warp i takes k-steps i-1, i-1+ISS, ...)
    if (lane == 0) {
      const int chain = warp - 1;
      int t_local = 0;
      bool ok = true;
      // descriptors of slot 0; a slot further on adds its byte offset / 16 to the address field (shared memory
      // addresses stay below 2^18, so the 14-bit field never carries)
      const uint64_t da0 = smem_desc(base), db0 = smem_desc(base + kTileBytesA);
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++t_local) {
        const int b = t_local & 1;
        if (t_local >= 2 && !mbar_wait_or_abort(acc_empty(b), ((t_local >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_acc = tmem_base + (uint32_t)(b * BN * ISS + chain * BN);
        const int it0 = t_local * k_iters + chain;   // this issuer's first k-step of the tile, counted over the CTA's tiles
        int s = it0 % STAGES;
        uint32_t round = (uint32_t)(it0 / STAGES) & 1u;
        for (int k = chain; k < k_iters; k += ISS) {
          if (!mbar_wait_or_abort(full_bar(s), round, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint64_t so = (uint64_t)(s * (C::kStageBytes >> 4));
          tc_mma_kstep(tmem_acc, da0 + so, db0 + so, C::kInstrDesc, k >= ISS ? 1u : 0u);
          tc_commit(empty_bar(s));               // slot free once these MMAs have read it
          s += ISS;
          if (s >= STAGES) { s -= STAGES; round ^= 1u; }
        }
        if (ok) tc_commit(acc_full(b));          // this issuer's share of the accumulator is complete
      }
      if (!ok) *abort_flag = 1;
    }
  } else {
    // ------------------------------------------------------------------ epilogue (the last 8 warps)
    const int q = warp & 3;                      // TMEM lane quarter this warp may access
    const int half = (warp - kFirstEpiWarp) >> 2;   // which half of the tile's 32-column groups this warp takes
    float4* stg4 = reinterpret_cast<float4*>(gen_base + STAGES * C::kStageBytes + 256) + (warp - kFirstEpiWarp) * (32 * 8);
    int t_local = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++t_local) {
      const int tn = tile / tiles_m;
      const int m0 = (tile % tiles_m) * BM, n0 = tn * BN;
      const int b = t_local & 1;
      const EpiRow er = epilogue_row<EPI>(a, m0 + q * 32 + lane, M);   // overlaps the main loop
      ok = warp_wait(acc_full(b), (t_local >> 1) & 1, abort_flag, lane);
      if (!ok) break;
      tc_fence_after();
      drain_accumulator<BN, EPI, ISS>(a, tmem_base + (uint32_t)(b * BN * ISS), q, half, lane, stg4, m0, n0, M, er);
      // this warp is done reading the accumulator: hand it back to the MMA warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty(b));
    }
    if (!ok && lane == 0) *abort_flag = 1;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols));
  }
  if (threadIdx.x == 0 && *abort_flag) atomicOr(status, kStInternal);
}

// ---------------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------------
int sm_count() {                                  // of the current device
  static std::mutex mu;
  static int n[kMaxDevices] = {};
  std::lock_guard<std::mutex> g(mu);
  const int dev = current_device();
  if (n[dev] == 0) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
    cudaGetLastError();
    n[dev] = v;
  }
  return n[dev];
}

template <int BN, int EPI, int ISS>
void launch(const GemmArgs& a, cudaStream_t st) {
  CUtensorMap ta, tb;
  if (!tma_map_bf16(a.A, a.M, a.K, a.lda, BM, &ta) || !tma_map_bf16(a.W, a.N, a.K, a.ldw, BN, &tb)) {
    static const int flag = kStInternal;       // cannot happen for shapes gemm_tc_supported accepted; report, do not guess
    cudaMemcpyAsync(a.status, &flag, sizeof(int), cudaMemcpyHostToDevice, st);
    return;
  }
  static PerDeviceOnce configured;
  configured.run([] {
    cudaFuncSetAttribute(gemm_tc_kernel<BN, EPI, ISS>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<BN>::kSmemBytes);
  });
  const long long tiles = (long long)((a.M + BM - 1) / BM) * ((a.N + BN - 1) / BN);
  const int grid = (int)(tiles < sm_count() ? tiles : sm_count());
  launch_pdl(gemm_tc_kernel<BN, EPI, ISS>, dim3(grid), dim3(kThreads + 32 * (ISS - 1)), Cfg<BN>::kSmemBytes, st, ta, tb, a, a.status);
}

template <int BN, int ISS>
void launch_bn(const GemmArgs& a, cudaStream_t st) {
  switch (a.epilogue) {
    case kEpiStoreAct: launch<BN, kEpiStoreAct, ISS>(a, st); break;
    case kEpiStoreF32: launch<BN, kEpiStoreF32, ISS>(a, st); break;
    case kEpiAddF32: launch<BN, kEpiAddF32, ISS>(a, st); break;
    case kEpiBiasTanhF32: launch<BN, kEpiBiasTanhF32, ISS>(a, st); break;
    case kEpiSwiGLU: launch<BN, kEpiSwiGLU, ISS>(a, st); break;
    case kEpiAddNorm: launch<BN, kEpiAddNorm, ISS>(a, st); break;
    case kEpiRopeKV: launch<BN, kEpiRopeKV, ISS>(a, st); break;
    default: break;
  }
}

}  // namespace

// Tiling of a launch: 32 ... 256 = output-tile width of the single-CTA kernel, kPlanPairs = 256 x 256 tiles on CTA pairs.
// Cost model: waves of tiles over the SMs (over the SM pairs) times the relative cost of one wave of that tile.  The
// tiling never changes the order in which a product's K range is summed, so it may depend on the row count.
constexpr int kPlanPairs = 512;
// Output-tile widths of the single-CTA kernel and the measured relative cost of one wave of each (a wider tile does more
// per wave but costs less than proportionally more: it moves fewer operand bytes per flop; 256 / 128 / 64 / 32 measured,
// the widths in between interpolated).  The in-between widths exist for passes of a few hundred rows over a wide model:
// 640 rows x 4096 columns are 80 tiles of 256 columns on 148 SMs, but 130 tiles of 160 columns, each a third shorter.
static const int kWidths[7] = {256, 224, 192, 160, 128, 64, 32}, kWaveCost[7] = {512, 484, 456, 428, 400, 300, 250};
int gemm_tc_plan(int M, int N, int K) {
  static const bool no_pairs = getenv("NEZHA_NO_CTA_PAIRS") != nullptr;
  static const int forced = getenv("NEZHA_GEMM_PLAN") ? atoi(getenv("NEZHA_GEMM_PLAN")) : 0;   // experiments: a width, 512 = pairs
  if (forced == 512 && M >= 1 && N >= 256) return kPlanPairs;
  for (int i = 0; i < 7; ++i)
    if (forced == kWidths[i]) return forced;
  const long long tiles_m = (M + BM - 1) / BM;
  long long best = -1; int plan = 32;
  for (int i = 0; i < 7; ++i) {
    const int bn = kWidths[i];
    if (bn > 32 && N < bn) continue;
    const long long tiles = tiles_m * ((N + bn - 1) / bn);
    const long long cost = ((tiles + sm_count() - 1) / sm_count()) * kWaveCost[i];
    if (best < 0 || cost < best) { best = cost; plan = bn; }
  }
  // pairs: a thousand rows or more, or half of that when the k-loop is long enough to outweigh a cluster launch
  if (!no_pairs && (M >= 1024 || (M >= 512 && K >= 2048)) && N >= 512) {
    const long long pairs = sm_count() / 2;
    const long long tiles = ((M + 2 * BM - 1) / (2 * BM)) * (long long)((N + 255) / 256);
    const long long cost = ((tiles + pairs - 1) / pairs) * 480;
    if (cost < best) { best = cost; plan = kPlanPairs; }
  }
  return plan;
}

bool gemm_tc_supported(const GemmArgs& a) {
  if (!a.status || !tma_encode_fn()) return false;
  if (a.K % BK || a.N % 32 || a.M <= 0) return false;
  if ((a.lda * 2) % 16 || (a.ldw * 2) % 16 || ((uintptr_t)a.A & 15) || ((uintptr_t)a.W & 15)) return false;
  if (((uintptr_t)a.C & 15) || (a.ldc & 3)) return false;          // the epilogue stores 8- and 16-byte vectors
  if (a.epilogue == kEpiBiasTanhF32 && ((uintptr_t)a.bias & 15)) return false;
  return a.epilogue >= kEpiStoreAct && a.epilogue <= kEpiRopeKV;
}

void launch_gemm_tc_pair(const GemmArgs& a, int n_sm, cudaStream_t st);
bool gemm_skinny_applies(const GemmArgs& a, int n_sm);
void launch_gemm_skinny(const GemmArgs& a, int n_sm, cudaStream_t st);

void launch_gemm_tc(const GemmArgs& a, cudaStream_t st) {
  LaunchScope ls(kcGemm, st);
  if (gemm_skinny_applies(a, sm_count())) { launch_gemm_skinny(a, sm_count(), st); return; }
  const int m_plan = a.M_expected > 0 && a.M_expected < a.M ? a.M_expected : a.M;
  // Narrow outputs (N <= 1024) never fill a 256-wide tile well and their k-loops are bound by the MMA issue chain:
  // a caller that asks for two partial sums gets tiles of at most 128 columns with two issuers for them.  The rule
  // looks at N and K only, never at M or at the tiling, so such a product keeps its summation order (and its bits)
  // whatever the number of rows of a launch -- what lets two decode modes whose passes differ in size agree exactly.
  static const bool one_issuer = getenv("NEZHA_ONE_MMA_ISSUER") != nullptr;
  // (An even number of k-steps: then every tile starts on ring slot parity 0 for issuer 0 and a slot keeps its issuer
  // from tile to tile, which is what the kernel's one-waiter-per-slot rule needs.)
  if (a.chains == 2 && a.N <= 1024 && a.K >= 2 * BK && (a.K / BK) % 2 == 0 && !one_issuer) {
    const long long tiles_m = (m_plan + BM - 1) / BM;
    static const int widths[3] = {128, 64, 32}, wave_cost[3] = {400, 300, 250};
    long long best = -1; int plan = 32;
    for (int i = 0; i < 3; ++i) {
      if (widths[i] > 32 && a.N < widths[i]) continue;
      const long long tiles = tiles_m * ((a.N + widths[i] - 1) / widths[i]);
      const long long cost = ((tiles + sm_count() - 1) / sm_count()) * wave_cost[i];
      if (best < 0 || cost < best) { best = cost; plan = widths[i]; }
    }
    switch (plan) {
      case 128: launch_bn<128, 2>(a, st); break;
      case 64: launch_bn<64, 2>(a, st); break;
      default: launch_bn<32, 2>(a, st); break;
    }
    return;
  }
  switch (gemm_tc_plan(m_plan, a.N, a.K)) {
    case kPlanPairs: launch_gemm_tc_pair(a, sm_count(), st); break;
    case 256: launch_bn<256, 1>(a, st); break;
    case 224: launch_bn<224, 1>(a, st); break;
    case 192: launch_bn<192, 1>(a, st); break;
    case 160: launch_bn<160, 1>(a, st); break;
    case 128: launch_bn<128, 1>(a, st); break;
    case 64: launch_bn<64, 1>(a, st); break;
    default: launch_bn<32, 1>(a, st); break;
  }
}

}  // namespace nz
