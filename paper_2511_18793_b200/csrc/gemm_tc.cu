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
#include "tma.cuh"

namespace nz {

namespace {

constexpr int BM = 128, BK = 64;
constexpr int kTileBytesA = BM * BK * 2;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr int kTransposeBytes = kEpiWarps * 32 * 32 * 4;   // per epilogue warp: a 32 x 32 fp32 block, chunks swizzled
template <int BN> struct Cfg {
  static constexpr int kTileBytesB = BN * BK * 2;
  static constexpr int kStageBytes = kTileBytesA + kTileBytesB;
  // as many stages as fit beside the transpose tiles: short-M launches are bound by bytes in flight per CTA
  static constexpr int kStages = BN == 256 ? 4 : BN == 128 ? 6 : BN == 64 ? 8 : 9;
  static constexpr int kSmemBytes =
      kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/ + kTransposeBytes;
  static constexpr int kTmemCols = 2 * BN < 32 ? 32 : 2 * BN;       // two accumulators; a power of two >= 32
  // kind::f16 instruction descriptor: D = f32, A = B = bf16, both K-major, N = BN, M = 128.
  static constexpr uint32_t kInstrDesc =
      (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
};

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

__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
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

// The epilogue works on 32 x 32 blocks of the accumulator.  tcgen05.ld hands a block out with lane = row; it is
// transposed through shared memory (128-byte rows, 16-byte chunks XOR-swizzled by the row, so both sides are free of
// bank conflicts) into "8 lanes per row, 4 consecutive columns per lane", in which every global access of a warp is
// four contiguous row segments.  The work on a row is split in two so that the loads of several rows are in flight
// before the first dependent store:
//   epi_prefetch  what the lane needs from memory (old C for the accumulating epilogues, cos / sin for the rotary one);
//   epi_apply     x = 4 accumulators (already multiplied by the A operand's RMSNorm row scale where one applies);
//                 returns what kEpiAddNorm sums squares of.
struct EpiAux { float4 a, b; };

// What a lane needs to know about its 4 columns of the current 32-column group; computed once per group so that the
// per-row code has no divisions left.  k = lane & 7 selects columns [4k, 4k + 4) of the group.
struct ChunkCtx {
  float4 col;        // norm gains (kEpiAddNorm) or biases (kEpiBiasTanhF32) of the lane's columns
  int kind;          // kEpiRopeKV: 0 = q (rotate, to C), 1 = k (rotate, to the K cache), 2 = v (copy to the V cache)
  int tab;           // kEpiRopeKV: first of the lane's 4 rotary-pair indices inside the head (cos / sin table column)
  long long off;     // element offset of the lane's first output inside the row (C) or inside the token's cache entry
};

__device__ __forceinline__ uint2 pack_bf16x4(float a, float b, float c, float d) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  return make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
}

template <int EPI>
__device__ __forceinline__ ChunkCtx chunk_ctx(const GemmArgs& g, int n_chunk, int k) {
  ChunkCtx cc{make_float4(0.f, 0.f, 0.f, 0.f), 0, 0, 0};
  const int n = n_chunk + 4 * k;
  if (EPI == kEpiAddNorm) {
    const __nv_bfloat162* gp = reinterpret_cast<const __nv_bfloat162*>(reinterpret_cast<const __nv_bfloat16*>(g.f.gain) + n);
    const float2 g0 = __bfloat1622float2(gp[0]), g1 = __bfloat1622float2(gp[1]);
    cc.col = make_float4(g0.x, g0.y, g1.x, g1.y);
  }
  if (EPI == kEpiBiasTanhF32) cc.col = *reinterpret_cast<const float4*>(g.bias + n);
  if (EPI == kEpiSwiGLU) cc.off = (n_chunk >> 1) + 2 * k;      // the lane's columns are (gate, gate, up, up) of 2 features
  if (EPI == kEpiRopeKV) {
    const GemmFuse& f = g.f;
    const int q_cols = f.Hq * f.hd, k_cols = f.Hkv * f.hd;
    if (n_chunk < q_cols + k_cols) {
      // the lane's columns are (x_i, x_{i+1}, x_{i+hd/2}, x_{i+1+hd/2}), i = 16 * (32-column group inside the head) + 2k
      const int nn = n_chunk < q_cols ? n_chunk : n_chunk - q_cols;
      const int head = nn / f.hd, in_head = nn - head * f.hd;
      cc.tab = ((in_head >> 5) << 4) + 2 * k;
      cc.kind = n_chunk < q_cols ? 0 : 1;
      cc.off = n_chunk < q_cols ? (long long)(n_chunk - in_head) + cc.tab : (long long)head * f.kv_head_stride + cc.tab;
    } else {
      const int nv = n - q_cols - k_cols;
      const int head = nv / f.hd;
      cc.kind = 2;
      cc.off = (long long)head * f.kv_head_stride + (nv - head * f.hd);
    }
  }
  return cc;
}

template <int EPI>
__device__ __forceinline__ EpiAux epi_prefetch(const GemmArgs& g, const ChunkCtx& cc, int row, int n, int pos) {
  EpiAux r;
  r.a = r.b = make_float4(0.f, 0.f, 0.f, 0.f);
  if (EPI == kEpiAddF32 || EPI == kEpiAddNorm) {
    r.a = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(g.C) + (long long)row * g.ldc + n);
  } else if (EPI == kEpiRopeKV) {
    if (cc.kind < 2) {
      const long long t = (long long)pos * (g.f.hd >> 1) + cc.tab;
      const float2 cs = *reinterpret_cast<const float2*>(g.f.cos_tab + t), sn = *reinterpret_cast<const float2*>(g.f.sin_tab + t);
      r.a = make_float4(cs.x, cs.y, sn.x, sn.y);
    }
  }
  return r;
}

// `valid`: the row exists.
template <int EPI>
__device__ __forceinline__ float4 epi_apply(const GemmArgs& g, const ChunkCtx& cc, bool valid, int row, int n, int k, float4 x,
                                           const EpiAux& aux, long long kv_dst) {
  const long long o = (long long)row * g.ldc + n;
  if (EPI == kEpiStoreAct) {
    if (valid) *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(g.C) + o) = pack_bf16x4(x.x, x.y, x.z, x.w);
  } else if (EPI == kEpiStoreF32) {
    if (valid) *reinterpret_cast<float4*>(reinterpret_cast<float*>(g.C) + o) = x;
  } else if (EPI == kEpiAddF32) {
    if (valid)
      *reinterpret_cast<float4*>(reinterpret_cast<float*>(g.C) + o) =
          make_float4(aux.a.x + x.x, aux.a.y + x.y, aux.a.z + x.z, aux.a.w + x.w);
  } else if (EPI == kEpiBiasTanhF32) {
    if (valid)
      *reinterpret_cast<float4*>(reinterpret_cast<float*>(g.C) + o) =
          make_float4(tanhf(x.x + cc.col.x), tanhf(x.y + cc.col.y), tanhf(x.z + cc.col.z), tanhf(x.w + cc.col.w));
  } else if (EPI == kEpiSwiGLU) {
    if (valid) {
      const __nv_bfloat162 y = __floats2bfloat162_rn(__fdividef(x.x, 1.f + __expf(-x.x)) * x.z,
                                                     __fdividef(x.y, 1.f + __expf(-x.y)) * x.w);
      *reinterpret_cast<__nv_bfloat162*>(reinterpret_cast<__nv_bfloat16*>(g.C) + (long long)row * g.ldc + cc.off) = y;
    }
  } else if (EPI == kEpiAddNorm) {
    const float4 cn = make_float4(aux.a.x + x.x, aux.a.y + x.y, aux.a.z + x.z, aux.a.w + x.w);
    if (valid) {
      *reinterpret_cast<float4*>(reinterpret_cast<float*>(g.C) + o) = cn;
      *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(g.f.xg) + (long long)row * g.N + n) =
          pack_bf16x4(cn.x * cc.col.x, cn.y * cc.col.y, cn.z * cc.col.z, cn.w * cc.col.w);
    }
    return cn;
  } else if (EPI == kEpiRopeKV) {
    if (cc.kind == 2) {
      if (valid && kv_dst >= 0)
        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(g.f.v_cache) + kv_dst + cc.off) = pack_bf16x4(x.x, x.y, x.z, x.w);
    } else if (valid && (cc.kind == 0 || kv_dst >= 0)) {
      // x_i' = x_i c - x_j s ;  x_j' = x_j c + x_i s   (j = i + hd/2; aux.a = cos_i, cos_{i+1}, sin_i, sin_{i+1})
      const __nv_bfloat162 lo = __floats2bfloat162_rn(x.x * aux.a.x - x.z * aux.a.z, x.y * aux.a.y - x.w * aux.a.w);
      const __nv_bfloat162 hi = __floats2bfloat162_rn(x.z * aux.a.x + x.x * aux.a.z, x.w * aux.a.y + x.y * aux.a.w);
      __nv_bfloat16* dst = cc.kind == 0 ? reinterpret_cast<__nv_bfloat16*>(g.C) + (long long)row * g.ldc + cc.off
                                        : reinterpret_cast<__nv_bfloat16*>(g.f.k_cache) + kv_dst + cc.off;
      *reinterpret_cast<__nv_bfloat162*>(dst) = lo;
      *reinterpret_cast<__nv_bfloat162*>(dst + (g.f.hd >> 1)) = hi;
    }
  }
  return x;
}

template <int BN, int EPI>
__global__ void __launch_bounds__(kThreads) gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA,
                                                           const __grid_constant__ CUtensorMap tmB, GemmArgs a,
                                                           int* status) {
  using C = Cfg<BN>;
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
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), kEpiWarps); }
    *abort_flag = 0;
    mbar_fence_init();
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
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        const int m0 = (tile % tiles_m) * BM, n0 = (tile / tiles_m) * BN;
        for (int k = 0; k < k_iters; ++k, ++it) {
          const int s = it % STAGES;
          if (it >= STAGES && !mbar_wait_or_abort(empty_bar(s), ((it / STAGES) - 1) & 1, abort_flag)) { ok = false; break; }
          mbar_expect_tx(full_bar(s), C::kStageBytes);
          tma_load_2d(base + s * C::kStageBytes, &tmA, k * BK, m0, full_bar(s));
          tma_load_2d(base + s * C::kStageBytes + kTileBytesA, &tmB, k * BK, n0, full_bar(s));
        }
      }
      if (!ok) {                                 // drain: wait (bounded) for the copies still in flight
        *abort_flag = 1;
        for (int j = max(0, it - STAGES); j < it; ++j) mbar_wait(full_bar(j % STAGES), (j / STAGES) & 1);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int it = 0, t_local = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++t_local) {
        const int b = t_local & 1;
        if (t_local >= 2 && !mbar_wait_or_abort(acc_empty(b), ((t_local >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_acc = tmem_base + (uint32_t)(b * BN);
        for (int k = 0; k < k_iters; ++k, ++it) {
          const int s = it % STAGES;
          if (!mbar_wait_or_abort(full_bar(s), (it / STAGES) & 1, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = base + s * C::kStageBytes, sb = sa + kTileBytesA;
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk)
            tc_mma(tmem_acc, smem_desc(sa + kk * 32), smem_desc(sb + kk * 32), C::kInstrDesc, (k > 0 || kk > 0) ? 1u : 0u);
          tc_commit(empty_bar(s));               // slot free once these MMAs have read it
        }
        if (ok) tc_commit(acc_full(b));          // accumulator complete
      }
      if (!ok) *abort_flag = 1;
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9)
    const int q = warp & 3;                      // TMEM lane quarter this warp may access
    const int half = (warp - 2) >> 2;            // which half of the tile's 32-column groups this warp takes
    float4* stg4 = reinterpret_cast<float4*>(gen_base + STAGES * C::kStageBytes + 256) + (warp - 2) * (32 * 8);
    int t_local = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++t_local) {
      const int tn = tile / tiles_m;
      const int m0 = (tile % tiles_m) * BM, n0 = tn * BN;
      const int b = t_local & 1;
      const int row = m0 + q * 32 + lane;
      float rs = 1.f;                            // RMSNorm scale of the A operand's row (overlaps the main loop)
      if (a.f.ss_in && row < M) {
        float ss = 0.f;
        for (int p = 0; p < a.f.ss_in_parts; ++p) ss += a.f.ss_in[(long long)p * a.f.ss_ld + row];
        rs = rsqrtf(ss * a.f.inv_dim + a.f.eps);
      }
      int pos = 0; long long kvd = -1;
      if (EPI == kEpiRopeKV && row < M) { pos = a.f.tok_pos[row]; kvd = a.f.kv_dst[row]; }
      ok = __all_sync(0xffffffffu, mbar_wait_or_abort(acc_full(b), (t_local >> 1) & 1, abort_flag));   // warp-uniform
      if (!ok) break;
      tc_fence_after();
      const int rows_here = min(32, M - (m0 + q * 32));          // rows of this quarter that exist (may be <= 0)
#pragma unroll 1
      for (int c = half; c < BN / 32; c += 2) {
        const int n_chunk = n0 + c * 32;
        if (n_chunk >= a.N) break;                               // ragged last tile (N is a multiple of 32)
        float v[32];
        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * BN + c * 32), v);
        // transpose through shared memory: from lane = row (how TMEM hands the block out) to 8 lanes per row
#pragma unroll
        for (int j = 0; j < 8; ++j)
          stg4[lane * 8 + (j ^ (lane & 7))] = make_float4(v[4 * j] * rs, v[4 * j + 1] * rs, v[4 * j + 2] * rs, v[4 * j + 3] * rs);
        __syncwarp();
        const int k = lane & 7, rsub = lane >> 3;
        const ChunkCtx cc = chunk_ctx<EPI>(a, n_chunk, k);
        const int n = n_chunk + 4 * k;
#pragma unroll
        for (int it0 = 0; it0 < 8; it0 += 4) {
          if (it0 * 4 >= rows_here) break;                           // warp-uniform
          EpiAux aux[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int r = (it0 + u) * 4 + rsub;
            const int p_r = (EPI == kEpiRopeKV) ? __shfl_sync(0xffffffffu, pos, r) : 0;
            if (r < rows_here) aux[u] = epi_prefetch<EPI>(a, cc, m0 + q * 32 + r, n, p_r);
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int r = (it0 + u) * 4 + rsub;
            const long long kv_r = (EPI == kEpiRopeKV) ? __shfl_sync(0xffffffffu, kvd, r) : -1;
            const float4 x = stg4[r * 8 + (k ^ (r & 7))];
            const float4 back = epi_apply<EPI>(a, cc, r < rows_here, m0 + q * 32 + r, n, k, x, aux[u], kv_r);
            if (EPI == kEpiAddNorm) stg4[r * 8 + (k ^ (r & 7))] = back;
          }
        }
        __syncwarp();
        if (EPI == kEpiAddNorm && lane < rows_here) {
          // one partial sum of squares per 32-column group, added up in column order: the same bits whatever the tile width
          float ssq = 0.f;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float4 t = stg4[lane * 8 + (j ^ (lane & 7))];
            ssq += t.x * t.x; ssq += t.y * t.y; ssq += t.z * t.z; ssq += t.w * t.w;
          }
          a.f.ss_out[(long long)(n_chunk >> 5) * a.f.ss_ld + row] = ssq;
        }
        __syncwarp();
      }
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
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols));
  }
  if (threadIdx.x == 0 && *abort_flag) atomicOr(status, kStInternal);
}

// ---------------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------------
int sm_count() {
  static int n = [] {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0)
      v = 148;
    return v;
  }();
  return n;
}

template <int BN, int EPI>
void launch(const GemmArgs& a, cudaStream_t st) {
  const CUtensorMap* ta = tma_map_bf16(a.A, a.M, a.K, a.lda, BM);
  const CUtensorMap* tb = tma_map_bf16(a.W, a.N, a.K, a.ldw, BN);
  if (!ta || !tb) {                            // cannot happen for shapes gemm_tc_supported accepted; report, do not guess
    static const int flag = kStInternal;
    cudaMemcpyAsync(a.status, &flag, sizeof(int), cudaMemcpyHostToDevice, st);
    return;
  }
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(gemm_tc_kernel<BN, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<BN>::kSmemBytes);
    configured = true;
  }
  const long long tiles = (long long)((a.M + BM - 1) / BM) * ((a.N + BN - 1) / BN);
  const int grid = (int)(tiles < sm_count() ? tiles : sm_count());
  launch_pdl(gemm_tc_kernel<BN, EPI>, dim3(grid), dim3(kThreads), Cfg<BN>::kSmemBytes, st, *ta, *tb, a, a.status);
}

template <int BN>
void launch_bn(const GemmArgs& a, cudaStream_t st) {
  switch (a.epilogue) {
    case kEpiStoreAct: launch<BN, kEpiStoreAct>(a, st); break;
    case kEpiStoreF32: launch<BN, kEpiStoreF32>(a, st); break;
    case kEpiAddF32: launch<BN, kEpiAddF32>(a, st); break;
    case kEpiBiasTanhF32: launch<BN, kEpiBiasTanhF32>(a, st); break;
    case kEpiSwiGLU: launch<BN, kEpiSwiGLU>(a, st); break;
    case kEpiAddNorm: launch<BN, kEpiAddNorm>(a, st); break;
    case kEpiRopeKV: launch<BN, kEpiRopeKV>(a, st); break;
    default: break;
  }
}

}  // namespace

// Output-tile width.  Cost model: waves of tiles over the SMs times the time of one k-step of a tile, which is the
// larger of the tensor-pipe time (2 BN clocks for four M128 N=BN K16 instructions) and the shared-memory feed time
// ((16 KB + BN * 128 B) at 128 B per clock); a 128-wide tile sits exactly on that feed limit, hence its surcharge.
int gemm_tc_tile_n(int M, int N) {
  const long long tiles_m = (M + BM - 1) / BM;
  static const int widths[4] = {256, 128, 64, 32}, step_cost[4] = {512, 288, 192, 160};
  long long best = -1; int best_bn = 32;
  for (int i = 0; i < 4; ++i) {
    const int bn = widths[i];
    if (bn > 32 && N < bn) continue;
    const long long tiles = tiles_m * ((N + bn - 1) / bn);
    const long long cost = ((tiles + sm_count() - 1) / sm_count()) * step_cost[i];
    if (best < 0 || cost < best) { best = cost; best_bn = bn; }
  }
  return best_bn;
}

bool gemm_tc_supported(const GemmArgs& a) {
  if (!a.status || !tma_encode_fn()) return false;
  if (a.K % BK || a.N % 32 || a.M <= 0) return false;
  if ((a.lda * 2) % 16 || (a.ldw * 2) % 16 || ((uintptr_t)a.A & 15) || ((uintptr_t)a.W & 15)) return false;
  if (((uintptr_t)a.C & 15) || (a.ldc & 3)) return false;          // the epilogue stores 8- and 16-byte vectors
  if (a.epilogue == kEpiBiasTanhF32 && ((uintptr_t)a.bias & 15)) return false;
  return a.epilogue >= kEpiStoreAct && a.epilogue <= kEpiRopeKV;
}

void launch_gemm_tc(const GemmArgs& a, cudaStream_t st) {
  LaunchScope ls(kcGemm, st);
  switch (gemm_tc_tile_n(a.M_expected > 0 && a.M_expected < a.M ? a.M_expected : a.M, a.N)) {
    case 256: launch_bn<256>(a, st); break;
    case 128: launch_bn<128>(a, st); break;
    case 64: launch_bn<64>(a, st); break;
    default: launch_bn<32>(a, st); break;
  }
}

}  // namespace nz
