// Blackwell tensor-core GEMM:  C[M,N] (op)= A[M,K] * W[N,K]^T,  bf16 operands, fp32 accumulation in TMEM.
//
// One CTA computes one 128 x 128 output tile.  Warp 0 streams 128x64 (A) and 128x64 (W) bf16 tiles into a
// shared-memory ring with TMA (128-byte swizzle; K-major on both sides, which is exactly how activations
// [tokens, features] and weights [out, in] are stored), warp 1 issues tcgen05.mma (M128 N128 K16, four per
// stage) into a 128-column TMEM accumulator and releases ring slots with tcgen05.commit, warps 2-5 read the
// accumulator back with tcgen05.ld and apply the epilogue (store / residual add / bias+tanh).
// Every mbarrier wait is bounded: on expiry the CTA records an error in the status word, drains what it has
// in flight, frees its TMEM and returns.
#include "tma.cuh"

namespace nz {

namespace {

constexpr int BM = 128, BN = 128, BK = 64, STAGES = 4;
constexpr int kTileBytesA = BM * BK * 2, kTileBytesB = BN * BK * 2;
constexpr int kStageBytes = kTileBytesA + kTileBytesB;
constexpr int kSmemBytes = STAGES * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr int kThreads = 192;
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }

// K-major operand tile, 128-byte swizzle: rows are 128 B apart, 8-row groups 1024 B apart (SBO), LBO unused (1),
// descriptor version 1 (sm_100), layout type 2 (SWIZZLE_128B).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  return (uint64_t)((addr >> 4) & 0x3FFF) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// kind::f16 instruction descriptor: D = f32, A = B = bf16, both K-major, N = 128, M = 128.
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(kInstrDesc), "r"(accumulate) : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

template <int EPI>
__global__ void __launch_bounds__(kThreads) gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA,
                                                           const __grid_constant__ CUtensorMap tmB, GemmArgs a,
                                                           int* status) {
  const int M = a.M_dev ? min(a.M, *a.M_dev) : a.M;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  if (m0 >= M) return;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = base + STAGES * kStageBytes;
  // barriers: full[STAGES], empty[STAGES], accum; then tmem slot and abort flag
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  const uint32_t accum_bar = bar_base + 8u * (2 * STAGES);
  uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen_base + STAGES * kStageBytes + 8 * (2 * STAGES + 1));
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int k_iters = a.K / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(accum_bar, 1);
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)), "r"(BN));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_acc = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int issued = 0;
      for (int k = 0; k < k_iters; ++k) {
        const int s = k % STAGES;
        if (k >= STAGES && !mbar_wait(empty_bar(s), ((k / STAGES) - 1) & 1)) { *abort_flag = 1; break; }
        if (*abort_flag) break;
        mbar_expect_tx(full_bar(s), kStageBytes);
        tma_load_2d(base + s * kStageBytes, &tmA, k * BK, m0, full_bar(s));
        tma_load_2d(base + s * kStageBytes + kTileBytesA, &tmB, k * BK, n0, full_bar(s));
        issued = k + 1;
      }
      if (*abort_flag) {                       // drain: wait (bounded) for the copies still in flight
        for (int k = max(0, issued - STAGES); k < issued; ++k) mbar_wait(full_bar(k % STAGES), (k / STAGES) & 1);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      bool ok = true;
      for (int k = 0; k < k_iters && ok; ++k) {
        const int s = k % STAGES;
        if (!mbar_wait(full_bar(s), (k / STAGES) & 1) || *abort_flag) { *abort_flag = 1; ok = false; break; }
        tc_fence_after();
        const uint32_t sa = base + s * kStageBytes, sb = sa + kTileBytesA;
#pragma unroll
        for (int kk = 0; kk < BK / 16; ++kk)
          tc_mma(tmem_acc, smem_desc(sa + kk * 32), smem_desc(sb + kk * 32), (k > 0 || kk > 0) ? 1u : 0u);
        tc_commit(empty_bar(s));               // slot free once these MMAs have read it
      }
      tc_commit(accum_bar);                    // accumulator complete (also arrives after an abort)
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int q = warp & 3;                    // TMEM lane quarter this warp may access
    const bool ok = __all_sync(0xffffffffu, mbar_wait(accum_bar, 0) && !*abort_flag);   // warp-uniform
    tc_fence_after();
    if (ok) {
      const int row = m0 + q * 32 + lane;
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        float v[32];
        tmem_ld32(tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * 32), v);
        if (row < M) {
          const int n = n0 + c * 32;
          const long long o = (long long)row * a.ldc + n;
          if (EPI == kEpiStoreAct) {
            __nv_bfloat162* dst = reinterpret_cast<__nv_bfloat162*>(reinterpret_cast<__nv_bfloat16*>(a.C) + o);
#pragma unroll
            for (int i = 0; i < 16; ++i) dst[i] = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
          } else if (EPI == kEpiStoreF32) {
            float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(a.C) + o);
#pragma unroll
            for (int i = 0; i < 8; ++i) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
          } else if (EPI == kEpiAddF32) {
            float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(a.C) + o);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              float4 c4 = dst[i];
              c4.x += v[4 * i]; c4.y += v[4 * i + 1]; c4.z += v[4 * i + 2]; c4.w += v[4 * i + 3];
              dst[i] = c4;
            }
          } else if (EPI == kEpiBiasTanhF32) {
            float* dst = reinterpret_cast<float*>(a.C) + o;
#pragma unroll
            for (int i = 0; i < 32; ++i) dst[i] = tanhf(v[i] + a.bias[n + i]);
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(BN));
  }
  if (threadIdx.x == 0 && *abort_flag) atomicOr(status, kStInternal);
}

// ---------------------------------------------------------------------------------------------------
// host side: tensor maps
// ---------------------------------------------------------------------------------------------------
template <int EPI>
void launch(const CUtensorMap* ta, const CUtensorMap* tb, const GemmArgs& a, cudaStream_t st) {
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(gemm_tc_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    configured = true;
  }
  dim3 grid(a.N / BN, (a.M + BM - 1) / BM);
  gemm_tc_kernel<EPI><<<grid, kThreads, kSmemBytes, st>>>(*ta, *tb, a, a.status);
}

}  // namespace

bool gemm_tc_supported(const GemmArgs& a) {
  if (!a.status || !tma_encode_fn()) return false;
  if (a.K % BK || a.N % BN || a.M <= 0) return false;
  if ((a.lda * 2) % 16 || (a.ldw * 2) % 16 || ((uintptr_t)a.A & 15) || ((uintptr_t)a.W & 15)) return false;
  if (a.epilogue == kEpiStoreAct && (((uintptr_t)a.C & 3) || (a.ldc & 1))) return false;
  if ((a.epilogue == kEpiStoreF32 || a.epilogue == kEpiAddF32) && (((uintptr_t)a.C & 15) || (a.ldc & 3))) return false;
  return a.epilogue == kEpiStoreAct || a.epilogue == kEpiStoreF32 || a.epilogue == kEpiAddF32 ||
         a.epilogue == kEpiBiasTanhF32;
}

void launch_gemm_tc(const GemmArgs& a, cudaStream_t st) {
  const CUtensorMap* ta = tma_map_bf16(a.A, a.M, a.K, a.lda, BM);
  const CUtensorMap* tb = tma_map_bf16(a.W, a.N, a.K, a.ldw, BN);
  if (!ta || !tb) { launch_gemm_simt(a, true, st); return; }
  LaunchScope ls(kcGemm, st);
  switch (a.epilogue) {
    case kEpiStoreAct: launch<kEpiStoreAct>(ta, tb, a, st); break;
    case kEpiStoreF32: launch<kEpiStoreF32>(ta, tb, a, st); break;
    case kEpiAddF32: launch<kEpiAddF32>(ta, tb, a, st); break;
    case kEpiBiasTanhF32: launch<kEpiBiasTanhF32>(ta, tb, a, st); break;
    default: break;
  }
}

}  // namespace nz
