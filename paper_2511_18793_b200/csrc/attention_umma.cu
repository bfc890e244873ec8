// KV-cache attention on the Blackwell tensor path (tcgen05 + TMEM), for many query rows per (request, KV head).
//
// One CTA = (request, KV head, tile of 128 query rows): the rows are the request's tokens of this pass times the G query
// heads of the group, so the context K/V is streamed once per 128 rows.  Per 64-position K/V tile (brought in by TMA,
// 128-byte swizzle; K and V in rings of two slots each, because a K tile is free again right after S = Q K^T while
// its V tile is needed until the end of the tile):
//   S = Q K^T      tcgen05.mma M128 N64 K16 x hd/16, Q resident in shared memory, S in 64 TMEM columns
//   softmax        4 warps, one thread per row (a TMEM lane is a row, so row maximum and row sum need no shuffles):
//                  tcgen05.ld the row's 64 scores (after which S is free for the next tile's product, which therefore
//                  runs under this tile's exponentials), base-2 exponentials against a running reference maximum that
//                  is only raised when the true maximum has grown by more than 8 (then the O accumulator in TMEM is
//                  rescaled with tcgen05.ld / st); P goes to shared memory as the bf16 A operand of the second product
//   O += P V       tcgen05.mma M128 N=hd K16 x 4, V taken as it lies in the cache ([position][hd] = N-major operand)
// A CTA is a chain whose softmax takes most of a tile's time, so the kernel keeps every buffer single (65 KB of shared
// memory and 128 TMEM columns at hd = 64, 113 KB and 256 at hd = 128) and lets three (two) CTAs share an SM instead.
// The request's block of draft-token KV rows (every beam's, every level's) follows the context as further tiles of the
// same loop; a row masks them with the bit set of the positions it may see (its own tuple's codes).  At the end each
// thread normalises and stores its row.  Every mbarrier wait is bounded (abort flag, error status, TMEM freed).
#include <math.h>
#include <stdlib.h>

#include "gemm_epilogue.cuh"

namespace nz {

namespace {

using namespace gemm_detail;

constexpr int kPosU = 64;          // KV positions per tile
constexpr int kRowsU = 128;        // query rows per CTA
constexpr int kRingU = 2;          // K tiles in flight, and V tiles in flight (separate rings: K is free again after
                                   // S = Q K^T, long before V, which waits for the end of the tile's softmax)
constexpr int kThreadsU = 192;     // warp 0: TMA producer, warp 1: MMA issuer, warps 2-5: softmax (one thread per row)
constexpr float kRaise = 8.f;      // the reference maximum follows the true one only in steps larger than this (log2 units)

// PT ("P in TMEM"): the softmax threads write P straight back into the TMEM columns its scores came from (bf16 pairs, the
// A operand of the second product read from TMEM) instead of through a shared-memory buffer, and S is double-buffered:
// S_{j+2} = Q K_{j+2}^T is issued right behind P_j V_j, the softmax of tile j + 1 never waits for the P V product of tile
// j, and the 16 KB that P took hold a third K slot (S runs two tiles ahead).  Without PT: one S, one P buffer in shared memory (three CTAs per SM
// at hd = 64, where TMEM is what limits the PT form to two).
template <int HD, bool PT> struct UmmaCfg {
  static constexpr int kKRing = PT ? 3 : kRingU, kVRing = kRingU;
  static constexpr int kQBytes = kRowsU * HD * 2;
  static constexpr int kPBytes = PT ? 0 : kRowsU * kPosU * 2;
  static constexpr int kTileBytes = kPosU * HD * 2;            // one K (or V) tile
  // Two CTAs of the hd = 128 shape fit an SM only if each stays below (228 KB - 2 x 1 KB reserved) / 2 = 113 KB: the tiles
  // alone are 112 KB, so the barriers get 192 bytes and the alignment slack 512 (the dynamic array is declared with the
  // tiles' 1024-byte alignment; the kernel checks the slack it really needs and reports instead of overrunning).
  static constexpr int kBarBytes = 192, kSlack = 512;
  static constexpr int kTilesBytes = kQBytes + kPBytes + (kKRing + kVRing) * kTileBytes;
  static constexpr int kSmemBytes = kTilesBytes + kBarBytes + kSlack;
  // TMEM columns.  Plain: S at 0 (64), O at 64 (HD).  PT: S_0 / P_0 at 0, S_1 / P_1 at 64, O at 128.
  static constexpr int kTmemCols = PT ? 256 : (HD == 64 ? 128 : 256);
  static constexpr uint32_t kColO = PT ? 128 : 64;
  static constexpr int kCtasPerSm = PT ? 2 : (HD == 64 ? 3 : 2);
  static constexpr uint32_t kIdescS = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kPosU >> 3) << 17) | ((uint32_t)(kRowsU >> 4) << 24);
  static constexpr uint32_t kIdescPV =
      (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) /* B is N-major */ | ((uint32_t)(HD >> 3) << 17) | ((uint32_t)(kRowsU >> 4) << 24);
};

// D[tmem] (+)= A[tmem] * B[smem]: the A operand (128 rows = lanes, K along the columns, two bf16 per 32-bit cell) is read
// from tensor memory.
__device__ __forceinline__ void tc_mma_a_tmem(uint32_t tmem_d, uint32_t tmem_a, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(tmem_d), "r"(tmem_a), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_st32_bits(uint32_t taddr, const uint32_t* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
        "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]),
        "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]),
        "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31]) : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// N-major (MN-major) operand tile with the 128-byte swizzle: rows of 64 elements along N, 8-row groups along K 1024 B
// apart (SBO), 64-element groups along N `lbo` bytes apart (LBO).
__device__ __forceinline__ uint64_t smem_desc_nmajor(uint32_t addr, uint32_t lbo) {
  return (uint64_t)((addr >> 4) & 0x3FFF) | ((uint64_t)((lbo >> 4) & 0x3FFF) << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]), "f"(v[8]),
        "f"(v[9]), "f"(v[10]), "f"(v[11]), "f"(v[12]), "f"(v[13]), "f"(v[14]), "f"(v[15]), "f"(v[16]), "f"(v[17]),
        "f"(v[18]), "f"(v[19]), "f"(v[20]), "f"(v[21]), "f"(v[22]), "f"(v[23]), "f"(v[24]), "f"(v[25]), "f"(v[26]),
        "f"(v[27]), "f"(v[28]), "f"(v[29]), "f"(v[30]), "f"(v[31]) : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ float ex2u(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Two fp32 values in one 64-bit register pair: the packed fp32 instructions of sm_100 (one issue slot for two lanes of
// arithmetic) carry the scale-subtract and the row sum of the softmax, whose instruction count is what bounds this kernel.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
  f32x2 r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

template <int HD, bool PT>
__global__ void __launch_bounds__(kThreadsU, UmmaCfg<HD, PT>::kCtasPerSm) attn_umma_kernel(const __grid_constant__ CUtensorMap tmK,
                                                             const __grid_constant__ CUtensorMap tmV,
                                                             const __grid_constant__ CUtensorMap tmKx,
                                                             const __grid_constant__ CUtensorMap tmVx, AttnArgs a, int* status) {
  using C = UmmaCfg<HD, PT>;
  constexpr int SK = C::kKRing, SV = C::kVRing;     // K and V ring lengths
  constexpr int NH = HD / 64;                       // 64-column sub-tiles of a K / V / Q tile
  constexpr int KS = HD / 16;                       // k-steps of Q K^T
  constexpr uint32_t kColO = C::kColO;              // TMEM columns: S (and P) buffer b at 64 b, O behind them

  pdl_wait();                                       // before the first global read and before any exit
  pdl_launch();
  // Grid = (KV head, row tile, request): the row tiles of a (request, KV head) are neighbours in launch order, so they run
  // at the same time and the second one finds the K/V tiles the first one pulled in L2 (with the row tile as the slowest
  // index a request of more than 128 rows streamed its context from HBM once per tile: twice the DRAM bytes).  A causal
  // prefill's last tiles see the most context: those go first.
  const int req_local = blockIdx.z, kvh = blockIdx.x;
  const int tile = a.n_ext_max > 0 ? (int)blockIdx.y : (int)(gridDim.y - 1 - blockIdx.y);
  const int G = a.Hq / a.Hkv;
  const int4 info = a.req_info[req_local];          // {first token, token count, cache row, context length or -1}
  const int tok0 = info.x, n_tok = info.y, request = info.z;
  const int R = n_tok * G;
  const int r0 = tile * kRowsU;
  if (r0 >= R) return;
  const int max_ctx = info.w >= 0 ? info.w : min((r0 + kRowsU - 1) / G, n_tok - 1) + 1;
  const int n_tiles = (max_ctx + kPosU - 1) / kPosU;
  // The draft-token KV rows of the request (every beam's, every level's: ext_positions of them, contiguous for one KV
  // head) follow the context as n_xt more tiles of the same loop; a query row sees only its own ancestors and itself
  // among them, through a per-row bit mask.  Rows nobody sees are finite (the cache is zeroed when the engine is made),
  // so their P = 0 contributes exactly nothing.
  const int n_xt = a.n_ext_max > 0 ? (a.ext_positions + kPosU - 1) / kPosU : 0;
  const int NT = n_tiles + n_xt;
  const int kv_row0 = (int)(((long long)request * a.Hkv + kvh) * (a.ctx_head_stride / HD));

  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  if (base - smem_u32(smem_raw) > (uint32_t)C::kSlack) {   // the array came less aligned than declared: report, touch nothing
    if (threadIdx.x == 0) atomicOr(status, kStInternal);
    return;
  }
  uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t q_base = base, p_base = base + C::kQBytes, k_base = p_base + C::kPBytes, v_base = k_base + SK * C::kTileBytes;
  const uint32_t bar_base = v_base + SV * C::kTileBytes;
  auto k_full = [&](int s) { return bar_base + 8u * s; };
  auto k_empty = [&](int s) { return bar_base + 8u * (SK + s); };
  auto v_full = [&](int s) { return bar_base + 8u * (2 * SK + s); };
  auto v_empty = [&](int s) { return bar_base + 8u * (2 * SK + SV + s); };
  // Plain: one phase per tile on each of s_full(0), s_free, p_full(0), pv_done (tile j completes phase j).  PT: s_full(b)
  // and p_full(b) belong to S / P buffer b = j & 1 (tile j completes phase j >> 1 of them); s_free is not used.
  const uint32_t bar_misc = bar_base + 8u * (2 * SK + 2 * SV);
  auto s_full = [&](int b) { return bar_misc + 8u * b; };
  auto p_full = [&](int b) { return bar_misc + 16u + 8u * b; };
  const uint32_t s_free = bar_misc + 32u;
  // "P_j V_j is complete".  Plain: one barrier, one phase per tile, every softmax warp waits for every phase.  PT: the
  // softmax warps wait for it only before a rescale of O and at the end, and may then be up to two products ahead of or
  // behind the tensor core -- more than a parity can tell apart on one barrier -- so the products alternate between two
  // barriers (tile j completes phase j >> 1 of barrier j & 1), on each of which a waiter is never more than one phase off.
  auto pv_done = [&](int j) { return bar_misc + 40u + (PT ? 8u * (uint32_t)(j & 1) : 0u); };
  auto pv_parity = [&](int j) { return (uint32_t)(PT ? (j >> 1) : j) & 1u; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen_base + (bar_misc - base) + 56);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  static_assert(8 * (2 * C::kKRing + 2 * C::kVRing) + 56 + 8 <= C::kBarBytes, "barrier area");
  // where a bounded wait gave up (first one wins): status[1] = wait site, tile and warp; status[2] = the CTA; status[3] = its sizes
  auto gave_up = [&](int site, int j) {
    if (atomicCAS(status + 1, 0, site * 100000 + j * 100 + (int)(threadIdx.x >> 5) * 10 + (PT ? 1 : 0)) == 0) {
      status[2] = (int)(blockIdx.x + 100 * blockIdx.y + 10000 * blockIdx.z) + 1;
      status[3] = NT * 100000 + R;
    }
  };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < SK; ++s) { mbar_init(k_full(s), 1); mbar_init(k_empty(s), 1); }
    for (int s = 0; s < SV; ++s) { mbar_init(v_full(s), 1); mbar_init(v_empty(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(s_full(b), 1); mbar_init(p_full(b), 4); }
    mbar_init(s_free, 4); mbar_init(pv_done(0), 1); mbar_init(pv_done(1), 1);
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)),
                 "r"(C::kTmemCols));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  // the softmax threads bring their own query row into shared memory (K-major, 128-byte swizzle), zeros for dead rows
  int row = -1, tok = 0, head = 0, ctx = 0;
  bool live = false;
  if (warp >= 2) {
    row = (warp & 3) * 32 + lane;                   // = the TMEM lane this thread may read
    live = r0 + row < R;
    const int rr = live ? r0 + row : r0;
    tok = tok0 + rr / G; head = kvh * G + rr % G;
    ctx = !live ? 0 : (info.w >= 0 ? info.w : rr / G + 1);
    const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(a.q) + (long long)tok * a.q_stride +
                                                      (long long)head * HD);
#pragma unroll
    for (int c = 0; c < HD / 8; ++c) {
      const uint4 v = live ? src[c] : make_uint4(0u, 0u, 0u, 0u);
      const uint32_t dst = (c >> 3) * (kRowsU * 128) + row * 128 + (((c & 7) ^ (row & 7)) << 4);
      *reinterpret_cast<uint4*>(gen_base + dst) = v;
    }
    fence_async_smem();                             // generic-proxy writes, read by the tensor core through the async proxy
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const float sc = a.scale * 1.4426950408889634f;   // scores in base 2

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int t = 0, k_issued = 0, v_issued = 0;
      bool ok = true;
      for (; t < NT; ++t) {
        const int sk = t % SK, sv = t % SV;
        const bool ctx_tile = t < n_tiles;
        const int y = ctx_tile ? kv_row0 + t * kPosU : request * a.ext_positions + (t - n_tiles) * kPosU;
        const int x0 = ctx_tile ? 0 : kvh * HD;      // the draft cache is [positions, kv heads * hd]: this head's columns
        if (t >= SK && !mbar_wait_or_abort(k_empty(sk), (uint32_t)((t / SK) - 1) & 1u, abort_flag)) { gave_up(1, t); ok = false; break; }
        mbar_expect_tx(k_full(sk), C::kTileBytes);
#pragma unroll
        for (int h = 0; h < NH; ++h)
          tma_load_2d(k_base + sk * C::kTileBytes + h * (kPosU * 128), ctx_tile ? &tmK : &tmKx, x0 + h * 64, y, k_full(sk));
        ++k_issued;
        if (t >= SV && !mbar_wait_or_abort(v_empty(sv), (uint32_t)((t / SV) - 1) & 1u, abort_flag)) { gave_up(2, t); ok = false; break; }
        mbar_expect_tx(v_full(sv), C::kTileBytes);
#pragma unroll
        for (int h = 0; h < NH; ++h)
          tma_load_2d(v_base + sv * C::kTileBytes + h * (kPosU * 128), ctx_tile ? &tmV : &tmVx, x0 + h * 64, y, v_full(sv));
        ++v_issued;
      }
      if (!ok) {                                     // drain the copies still in flight before the CTA's memory goes away
        *abort_flag = 1;
        for (int j = max(0, k_issued - SK); j < k_issued; ++j) mbar_wait(k_full(j % SK), (j / SK) & 1);
        for (int j = max(0, v_issued - SV); j < v_issued; ++j) mbar_wait(v_full(j % SV), (j / SV) & 1);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      bool ok = true;
      auto issue_s = [&](int j) {                    // S_j = Q K_j^T into S buffer (PT ? j & 1 : 0)
        const int s = j % SK, b = PT ? (j & 1) : 0;
        if (!mbar_wait_or_abort(k_full(s), (uint32_t)(j / SK) & 1u, abort_flag)) { gave_up(3, j); return false; }
        // plain: the scores of tile j - 1 must be in registers.  PT: buffer b last held S_{j-2} / P_{j-2}, whose P V product
        // was issued before this one, and the tensor core runs a CTA's products in issue order: nothing to wait for.
        if (!PT && j >= 1 && !mbar_wait_or_abort(s_free, (uint32_t)(j - 1) & 1u, abort_flag)) { gave_up(4, j); return false; }
        tc_fence_after();
        const uint32_t kt = k_base + s * C::kTileBytes;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks)
          tc_mma(tmem_base + 64u * b, smem_desc(q_base + (ks >> 2) * (kRowsU * 128) + (ks & 3) * 32),
                 smem_desc(kt + (ks >> 2) * (kPosU * 128) + (ks & 3) * 32), C::kIdescS, ks > 0 ? 1u : 0u);
        tc_commit(k_empty(s));                       // K_j may be overwritten
        tc_commit(s_full(b));
        return true;
      };
      if (NT > 0) ok = issue_s(0);
      if (PT && ok && NT > 1) ok = issue_s(1);
      for (int j = 0; j < NT && ok; ++j) {
        if (!PT && j + 1 < NT && !issue_s(j + 1)) { ok = false; break; }   // runs under the softmax of tile j
        const int b = PT ? (j & 1) : 0;
        if (!mbar_wait_or_abort(p_full(b), (uint32_t)(PT ? (j >> 1) : j) & 1u, abort_flag)) { gave_up(5, j); ok = false; break; }
        if (!mbar_wait_or_abort(v_full(j % SV), (uint32_t)(j / SV) & 1u, abort_flag)) { gave_up(6, j); ok = false; break; }
        tc_fence_after();
        const uint32_t vt = v_base + (j % SV) * C::kTileBytes;
#pragma unroll
        for (int ks = 0; ks < kPosU / 16; ++ks) {
          const uint64_t dv = smem_desc_nmajor(vt + ks * (16 * 128), kPosU * 128);
          const uint32_t acc = (j > 0 || ks > 0) ? 1u : 0u;
          if (PT) tc_mma_a_tmem(tmem_base + kColO, tmem_base + 64u * b + 8u * ks, dv, C::kIdescPV, acc);
          else tc_mma(tmem_base + kColO, smem_desc(p_base + ks * 32), dv, C::kIdescPV, acc);
        }
        tc_commit(v_empty(j % SV));                  // V_j may be overwritten
        tc_commit(pv_done(j));                       // O holds tiles 0..j (and, plain, P may be overwritten)
        if (PT && j + 2 < NT && !issue_s(j + 2)) { ok = false; break; }   // behind P_j V_j, into the buffer it has just read
      }
      if (!ok) *abort_flag = 1;
    }
  } else {
    // ------------------------------------------------------------------ softmax, one thread per row
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    float m_ref = -INFINITY, l_run = 0.f;           // reference maximum (scaled log2 domain) and row sum against it
    bool ok = true;
    const int ctx_min = __reduce_min_sync(0xffffffffu, ctx);
    const bool warp_dead = r0 + (warp & 3) * 32 >= R;   // none of this warp's 32 rows exists: it only keeps the barriers going
    int xpos[kMaxLevels];                           // the row's visible draft positions inside the request's block, or -1
#pragma unroll
    for (int e = 0; e < kMaxLevels; ++e) {
      long long off = -1;
      if (live && e < a.n_ext_max) off = a.tok_ext[(long long)tok * a.n_ext_max + e];
      xpos[e] = off >= 0 ? (int)((off - (long long)request * a.ext_req_stride) / a.ext_pos_stride) : -1;
    }
    for (int j = 0; j < NT; ++j) {
      const int sb = PT ? (j & 1) : 0;               // S / P buffer of this tile
      const uint32_t par = (uint32_t)(PT ? (j >> 1) : j) & 1u;
      const uint32_t col_s = 64u * sb;
      ok = warp_wait(s_full(sb), par, abort_flag, lane);
      if (!ok) { if (lane == 0) gave_up(7, j); break; }
      if (warp_dead) {                               // (its P rows stay whatever they are: O rows nobody reads)
        if (!PT) {
          if (lane == 0) mbar_arrive(s_free);
          if (j >= 1) {
            ok = warp_wait(pv_done(j - 1), pv_parity(j - 1), abort_flag, lane);
            if (!ok) { if (lane == 0) gave_up(8, j); break; }
          }
        }
        if (lane == 0) mbar_arrive(p_full(sb));
        continue;
      }
      tc_fence_after();
      float sv[kPosU];
      tmem_ld32(tmem_base + lane_addr + col_s, sv);
      tmem_ld32(tmem_base + lane_addr + col_s + 32u, sv + 32);
      tc_fence_before();
      __syncwarp();
      if (!PT && lane == 0) mbar_arrive(s_free);     // the scores are in registers: S may take tile j + 1
      if (j >= n_tiles) {                            // a tile of draft positions: the row's own mask
        unsigned long long mk = 0ull;
#pragma unroll
        for (int e = 0; e < kMaxLevels; ++e) {
          const int p = xpos[e] - (j - n_tiles) * kPosU;
          if (xpos[e] >= 0 && p >= 0 && p < kPosU) mk |= 1ull << p;
        }
#pragma unroll
        for (int c = 0; c < kPosU; ++c)
          if (!((mk >> c) & 1ull)) sv[c] = -INFINITY;
      } else if ((j + 1) * kPosU > ctx_min) {
#pragma unroll
        for (int c = 0; c < kPosU; ++c)
          if (j * kPosU + c >= ctx) sv[c] = -INFINITY;
      }
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < kPosU; c += 2) mx = max3(mx, sv[c], sv[c + 1]);
      mx *= sc;
      // raise the reference only when the true maximum has run away from it: p stays below 2^8 otherwise
      const bool raise = mx > m_ref + kRaise || (m_ref == -INFINITY && mx > -INFINITY);
      const float m_new = raise ? mx : m_ref;
      const float m_safe = m_new == -INFINITY ? 0.f : m_new;
      const float corr = raise ? ex2u(m_ref - m_safe) : 1.f;     // ex2(-inf) = 0 the first time
      const f32x2 sc2 = pack2(sc, sc), neg_m2 = pack2(-m_safe, -m_safe);
      f32x2 rs2 = pack2(0.f, 0.f);
      uint32_t pk[kPosU / 2];
#pragma unroll
      for (int c = 0; c < kPosU; c += 2) {
        float x0, x1;
        unpack2(fma2(pack2(sv[c], sv[c + 1]), sc2, neg_m2), x0, x1);
        const float p0 = ex2u(x0), p1 = ex2u(x1);
        rs2 = add2(rs2, pack2(p0, p1));
        __nv_bfloat162 pb = __floats2bfloat162_rn(p0, p1);
        pk[c >> 1] = *reinterpret_cast<uint32_t*>(&pb);
      }
      float rs_lo, rs_hi;
      unpack2(rs2, rs_lo, rs_hi);
      const float rs = rs_lo + rs_hi;
      l_run = l_run * corr + rs;
      m_ref = m_new;
      // Plain: the P V product of tile j - 1 must be done before P is overwritten.  PT: P_j has a buffer of its own (last
      // read by P_{j-2} V_{j-2}, which completed before S_j did); only a rescale of O has to wait for P_{j-1} V_{j-1}.
      const bool rescale = j > 0 && __any_sync(0xffffffffu, raise);
      if (j >= 1 && (!PT || rescale)) {
        ok = warp_wait(pv_done(j - 1), pv_parity(j - 1), abort_flag, lane);
        if (!ok) { if (lane == 0) gave_up(9, j); break; }
      }
      if (rescale) {                                 // rescale O
        tc_fence_after();
#pragma unroll 1
        for (int c = 0; c < HD / 32; ++c) {
          float ov[32];
          tmem_ld32(tmem_base + lane_addr + kColO + (uint32_t)(c * 32), ov);
#pragma unroll
          for (int i = 0; i < 32; ++i) ov[i] *= corr;
          tmem_st32(tmem_base + lane_addr + kColO + (uint32_t)(c * 32), ov);
        }
      }
      if (PT) {                                      // P over the first half of the columns its scores came from
        tmem_st32_bits(tmem_base + lane_addr + col_s, pk);
      } else {
#pragma unroll
        for (int c = 0; c < 8; ++c)
          *reinterpret_cast<uint4*>(gen_base + (p_base - base) + row * 128 + ((c ^ (row & 7)) << 4)) =
              make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
        fence_async_smem();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(p_full(sb));
    }
    if (ok && NT > 0) {
      ok = warp_wait(pv_done(NT - 1), pv_parity(NT - 1), abort_flag, lane);
      if (!ok && lane == 0) gave_up(10, NT);
      tc_fence_after();
    }
    if (!ok) { if (lane == 0) *abort_flag = 1; }
    else {
      // ---- normalise and store (thread = row)
      const float l_tot = l_run;
      const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;
      __nv_bfloat16* op = reinterpret_cast<__nv_bfloat16*>(a.out) + (long long)tok * a.out_stride + (long long)head * HD;
#pragma unroll 1
      for (int c = 0; c < HD / 32; ++c) {
        float ov[32];
        tmem_ld32(tmem_base + lane_addr + kColO + (uint32_t)(c * 32), ov);   // warp-collective: dead rows take part too
        if (live && l_tot > 0.f) {
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            uint32_t w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              __nv_bfloat162 t = __floats2bfloat162_rn(ov[u * 8 + 2 * i] * inv, ov[u * 8 + 2 * i + 1] * inv);
              w[i] = *reinterpret_cast<uint32_t*>(&t);
            }
            reinterpret_cast<uint4*>(op + c * 32)[u] = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols));
  }
  if (threadIdx.x == 0 && *abort_flag) atomicOr(status, kStInternal);
}

template <int HD, bool PT>
void launch_umma(const CUtensorMap* tk, const CUtensorMap* tv, const AttnArgs& a, cudaStream_t st) {
  using C = UmmaCfg<HD, PT>;
  static PerDeviceOnce configured;
  configured.run([] {
    cudaFuncSetAttribute(attn_umma_kernel<HD, PT>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
  });
  const int G = a.Hq / a.Hkv;
  dim3 grid(a.Hkv, (a.max_tokens_per_row * G + kRowsU - 1) / kRowsU, a.n_rows);
  // the layer's draft-token caches as [positions of all requests, kv heads * hd] (a prefill has none: any valid map)
  CUtensorMap tkx = *tk, tvx = *tv;
  if (a.n_ext_max > 0) {
    const long long rows = a.ext_rows_total, cols = (long long)a.Hkv * HD;
    if (!tma_map_bf16(a.k_ext, rows, cols, cols, kPosU, &tkx) || !tma_map_bf16(a.v_ext, rows, cols, cols, kPosU, &tvx)) {
      static const int flag = kStInternal;
      cudaMemcpyAsync(a.status, &flag, sizeof(int), cudaMemcpyHostToDevice, st);
      return;
    }
  }
  launch_pdl(attn_umma_kernel<HD, PT>, grid, dim3(kThreadsU), C::kSmemBytes, st, *tk, *tv, tkx, tvx, a, a.status);
}

}  // namespace

// tk / tv: tensor maps of the layer's context K and V caches with boxes of 64 positions x 64 columns.
void launch_attention_umma(const AttnArgs& a, const CUtensorMap* tk, const CUtensorMap* tv, cudaStream_t st) {
  // P through TMEM with two S buffers pays where the CTA's chain S -> softmax -> P V is the bound: several row tiles per
  // (request, KV head) at hd = 128 (measured: -7 % on the 7B shape's 240-row passes, -6.5 % on the 1.5B shape).  One-tile
  // passes of the 7B shape are bound by HBM and lose 20 % with it (the two-slot K ring then has to run two tiles ahead);
  // at hd = 64 it costs the third CTA per SM for nothing.  NEZHA_ATTN_PT = 0 / 1 forces it off / on.
  static const int pt = getenv("NEZHA_ATTN_PT") ? atoi(getenv("NEZHA_ATTN_PT")) : 2;
  const int G = a.Hq / a.Hkv;
  const long long r_bound = (long long)a.max_tokens_per_row * G;
  const long long r = a.rows_expected > 0 && a.rows_expected < r_bound ? a.rows_expected : r_bound;
  const bool use_pt = pt == 1 || (pt == 2 && a.hd == 128 && r > kRowsU);
  if (a.hd == 64) { if (use_pt) launch_umma<64, true>(tk, tv, a, st); else launch_umma<64, false>(tk, tv, a, st); }
  else { if (use_pt) launch_umma<128, true>(tk, tv, a, st); else launch_umma<128, false>(tk, tv, a, st); }
}

}  // namespace nz
