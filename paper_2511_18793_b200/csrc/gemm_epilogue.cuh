// Pieces shared by the tensor-core GEMM kernels: tcgen05 / TMEM helpers, shared-memory operand descriptors, and the
// epilogue that turns a 128 x BN fp32 accumulator in TMEM into the launch's outputs (see GemmFuse for the fused forms).
#pragma once

#include "tma.cuh"

namespace nz {
namespace gemm_detail {

constexpr int BM = 128, BK = 64;
constexpr int kTileBytesA = BM * BK * 2;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr int kTransposeBytes = kEpiWarps * 32 * 32 * 4;   // per epilogue warp: a 32 x 32 fp32 block, chunks swizzled

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

// The four MMAs of one 64-deep k-step (K = 16 each) in one statement: the operands' descriptors advance by 32 bytes
// (2 in the descriptor's 16-byte address units) per MMA; only the first may overwrite the accumulator.  One thread
// issues every MMA of a CTA, so the instructions around each one are the floor of a short k-loop.
__device__ __forceinline__ void tc_mma_kstep(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate_first) {
  asm volatile(
      "{\n\t.reg .pred p, t;\n\t.reg .b64 a1, b1, a2, b2, a3, b3;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "setp.eq.b32 t, %4, %4;\n\t"
      "add.s64 a1, %1, 2;\n\tadd.s64 b1, %2, 2;\n\t"
      "add.s64 a2, %1, 4;\n\tadd.s64 b2, %2, 4;\n\t"
      "add.s64 a3, %1, 6;\n\tadd.s64 b3, %2, 6;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], a1, b1, %3, t;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], a2, b2, %3, t;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], a3, b3, %3, t;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate_first) : "memory");
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

// Per-row inputs of the epilogue that can be fetched before the accumulator is ready.
struct EpiRow { float rs; int pos; long long kvd; };

template <int EPI>
__device__ __forceinline__ EpiRow epilogue_row(const GemmArgs& a, int row, int M) {
  EpiRow r{1.f, 0, -1};
  if (a.f.ss_in && row < M) {                  // RMSNorm scale of the A operand's row
    float ss = 0.f;
    for (int p = 0; p < a.f.ss_in_parts; ++p) ss += a.f.ss_in[(long long)p * a.f.ss_ld + row];
    r.rs = rsqrtf(ss * a.f.inv_dim + a.f.eps);
  }
  if (EPI == kEpiRopeKV && row < M) { r.pos = a.f.tok_pos[row]; r.kvd = a.f.kv_dst[row]; }
  return r;
}

// The epilogue proper on one staged 32 x 32 block (rows row0 .. row0 + 31, columns n_chunk .. n_chunk + 31) that sits in
// the warp's transpose tile in the swizzled "8 lanes per row" image described above.  er = epilogue_row of row
// row0 + lane; rows_here = how many of the 32 rows exist (> 0).  The caller has made the tile visible to the warp.
template <int EPI>
__device__ __forceinline__ void epilogue_block(const GemmArgs& a, float4* stg4, int lane, int row0, int rows_here, int n_chunk,
                                               const EpiRow& er) {
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
      const int p_r = (EPI == kEpiRopeKV) ? __shfl_sync(0xffffffffu, er.pos, r) : 0;
      if (r < rows_here) aux[u] = epi_prefetch<EPI>(a, cc, row0 + r, n, p_r);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int r = (it0 + u) * 4 + rsub;
      const long long kv_r = (EPI == kEpiRopeKV) ? __shfl_sync(0xffffffffu, er.kvd, r) : -1;
      const float4 x = stg4[r * 8 + (k ^ (r & 7))];
      const float4 back = epi_apply<EPI>(a, cc, r < rows_here, row0 + r, n, k, x, aux[u], kv_r);
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
    a.f.ss_out[(long long)(n_chunk >> 5) * a.f.ss_ld + row0 + lane] = ssq;
  }
  __syncwarp();
}

// One epilogue warp's share of a finished accumulator: TMEM lanes [32 q, 32 q + 32) (= rows m0 + 32 q ..) and the
// 32-column groups half, half + 2, ... of the BN columns starting at TMEM column `tmem_acc`.  er = epilogue_row of
// the lane's own row (lane = row while the block comes out of TMEM).
// CHAINS > 1: the tile's K range was accumulated in that many partial accumulators, BN columns apart (one per MMA
// issuer); they are added up here, in order, as the block leaves TMEM.
template <int BN, int EPI, int CHAINS = 1>
__device__ __forceinline__ void drain_accumulator(const GemmArgs& a, uint32_t tmem_acc, int q, int half, int lane,
                                                  float4* stg4, int m0, int n0, int M, const EpiRow& er) {
  const int rows_here = min(32, M - (m0 + q * 32));          // rows of this quarter that exist (may be <= 0)
#pragma unroll 1
  for (int c = half; c < BN / 32; c += 2) {
    const int n_chunk = n0 + c * 32;
    if (n_chunk >= a.N) break;                               // ragged last tile (N is a multiple of 32)
    float v[32];
    tmem_ld32(tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * 32), v);
#pragma unroll
    for (int ch = 1; ch < CHAINS; ++ch) {
      float w[32];
      tmem_ld32(tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)(ch * BN + c * 32), w);
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] += w[j];
    }
    // transpose through shared memory: from lane = row (how TMEM hands the block out) to 8 lanes per row
#pragma unroll
    for (int j = 0; j < 8; ++j)
      stg4[lane * 8 + (j ^ (lane & 7))] =
          make_float4(v[4 * j] * er.rs, v[4 * j + 1] * er.rs, v[4 * j + 2] * er.rs, v[4 * j + 3] * er.rs);
    __syncwarp();
    if (rows_here > 0) epilogue_block<EPI>(a, stg4, lane, m0 + q * 32, rows_here, n_chunk, er);
    __syncwarp();
  }
}

}  // namespace gemm_detail
}  // namespace nz
