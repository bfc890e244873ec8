// Tensor-core KV-cache attention (bf16) with TMA-staged K/V tiles.
//
// One CTA = (request, KV head, tile of 16 * RW query rows).  The query rows of a (request, KV head) pair are all of the
// request's tokens in this pass times the G query heads of the group, so the request's context K/V is streamed once
// per (request, KV head, layer) and shared by every beam, draft level and grouped head -- not re-read per token.
// A producer warp brings K/V tiles of 64 positions into a shared-memory ring with TMA (128-byte swizzle); RW x KW
// consumer warps run S = Q K^T and O += P V on mma.sync m16n8k16 (fp32 accumulation) with an online softmax in
// registers.  Two shapes of the same kernel:
//   RW = 4, KW = 1   64 rows per CTA, every warp walks all tiles                       (many query rows per request)
//   RW = 1, KW = 4   16 rows per CTA, the four warps take every fourth tile and their   (few rows: one beam set of a
//                    softmax states are merged through shared memory at the end          small model, plain decode)
// Ring slots are handed back to the producer with per-slot "empty" mbarriers, so warps never wait for each other.
// The draft-token KV rows (a token sees its own tuple's drafted codes, at most L of them) are not gathered per token:
// the request's whole block of draft positions -- every beam's, every level's, contiguous in the cache for one KV head --
// follows the context as one or more further tiles of the same loop, and each query row masks them with the bit set
// of the positions it may see (tree attention over the drafted tuples).  Every barrier wait is bounded (abort flag +
// error status + return).
#include <math.h>
#include <stdlib.h>

#include "tma.cuh"

namespace nz {

namespace {

constexpr int kPos = 64;         // KV positions per tile

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float ex2(float x) {      // 2^x, flushing; ex2(-inf) = 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Address of the 16-byte chunk `chunk` (dims chunk*8 .. +7) of position `pos` inside a K or V stage buffer made of
// HD/64 sub-tiles of [64 positions x 128 bytes], each written by TMA with the 128-byte swizzle.
template <int HD>
__device__ __forceinline__ uint32_t kv_addr(uint32_t tile, int pos, int chunk) {
  const int sub = chunk >> 3, c = chunk & 7;
  return tile + sub * (kPos * 128) + pos * 128 + ((c ^ (pos & 7)) << 4);
}

template <int HD, int RW, int KW>
struct AttnCfg {
  static constexpr int kStages = KW == 1 ? 3 : KW;                // a multiple of KW: slot s always serves warp group s % KW
  static constexpr int kConsumers = RW * KW;
  static constexpr int kThreads = (kConsumers + 1) * 32;          // + the producer warp
  static constexpr int kTileBytes = kPos * HD * 2;                // one K (or V) tile
  static constexpr int kStageBytes = 2 * kTileBytes;
  static constexpr int kMergeFloats = (HD / 8) * 4 + 4;           // o fragments + (m, l) of two rows, per thread
  static constexpr int kMergeBytes = (KW - 1) * RW * kMergeFloats * 32 * 4;
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 + 128 + kMergeBytes;
};

template <int HD, int RW, int KW>
__global__ void __launch_bounds__(AttnCfg<HD, RW, KW>::kThreads) attn_tc_kernel(const __grid_constant__ CUtensorMap tmK,
                                                                               const __grid_constant__ CUtensorMap tmV,
                                                                               const __grid_constant__ CUtensorMap tmKx,
                                                                               const __grid_constant__ CUtensorMap tmVx,
                                                                               AttnArgs a, int* status) {
  using C = AttnCfg<HD, RW, KW>;
  constexpr int S = C::kStages;
  constexpr int NH = HD / 64;                       // 64-column halves per tile
  constexpr int KS = HD / 16;                       // k-steps of Q K^T
  constexpr int NB = HD / 8;                        // n-blocks of the output
  constexpr int kRows = 16 * RW;

  pdl_wait();                                       // before the first global read and before any exit
  pdl_launch();
  // the row tile is the slowest grid index: tiles beyond a request's rows (the grid covers the largest row count a
  // call may have) are scheduled after every tile that has work, instead of holding its place in the first wave
  // (a causal prefill has no such tiles to speak of, and its last tiles see the most context: those go first)
  const int req_local = blockIdx.y, kvh = blockIdx.x;
  const int tile = a.n_ext_max > 0 ? (int)blockIdx.z : (int)(gridDim.z - 1 - blockIdx.z);
  const int G = a.Hq / a.Hkv;
  const int4 info = a.req_info[req_local];          // {first token, token count, cache row, context length or -1}
  const int tok0 = info.x, n_tok = info.y, request = info.z;
  const int R = n_tok * G;                          // query rows of this (request, kv head)
  const int r0 = tile * kRows;
  if (r0 >= R) return;
  // context positions this tile needs: all of them, or (causal prefill) up to its last token's own position
  const int max_ctx = info.w >= 0 ? info.w : min((r0 + kRows - 1) / G, n_tok - 1) + 1;
  const int n_tiles = (max_ctx + kPos - 1) / kPos;
  // The draft-token KV rows of the request (every beam's, every level's: ext_positions of them, contiguous for one KV
  // head) follow the context as n_xt more tiles of the same loop; a query row sees only its own ancestors and itself
  // among them, through a per-row bit mask.  Rows nobody sees are finite (the cache is zeroed when the engine is made),
  // so their P = 0 contributes exactly nothing.
  const int n_xt = a.n_ext_max > 0 ? (a.ext_positions + kPos - 1) / kPos : 0;
  const int NT = n_tiles + n_xt;
  const int kv_row0 = (int)(((long long)request * a.Hkv + kvh) * (a.ctx_head_stride / HD));   // first cache row

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bar_base = base + S * C::kStageBytes;            // full[S], empty[S], then the abort flag
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (S + s); };
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(gen_base + S * C::kStageBytes + 8 * 2 * S);
  float* merge = reinterpret_cast<float*>(gen_base + S * C::kStageBytes + 128);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), RW); }
    *abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();

  float o[NB][4];
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};   // m in the scaled log2 domain
  int tok[2] = {0, 0}, head[2] = {0, 0};
  bool live[2] = {false, false};
  const int qr = lane >> 2, qc = lane & 3;          // fragment row (and +8) / column pair
  const float sc = a.scale * 1.4426950408889634f;   // scores are kept in base 2
  const int rw = warp % RW, g = warp / RW;          // consumer coordinates (the last warp is the producer)

  if (warp == C::kConsumers) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int t = 0;
      bool ok = true;
      for (; t < NT; ++t) {
        const int s = t % S;
        if (t >= S && !mbar_wait_or_abort(empty_bar(s), ((t / S) - 1) & 1, abort_flag)) { ok = false; break; }
        mbar_expect_tx(full_bar(s), C::kStageBytes);
#pragma unroll
        for (int h = 0; h < NH; ++h) {
          const uint32_t kd = base + s * C::kStageBytes + h * (kPos * 128), vd = kd + C::kTileBytes;
          if (t < n_tiles) {
            tma_load_2d(kd, &tmK, h * 64, kv_row0 + t * kPos, full_bar(s));
            tma_load_2d(vd, &tmV, h * 64, kv_row0 + t * kPos, full_bar(s));
          } else {                                   // [positions, kv heads * hd]: this head's columns of 64 draft positions
            const int y = request * a.ext_positions + (t - n_tiles) * kPos;
            tma_load_2d(kd, &tmKx, kvh * HD + h * 64, y, full_bar(s));
            tma_load_2d(vd, &tmVx, kvh * HD + h * 64, y, full_bar(s));
          }
        }
      }
      if (!ok) {                                     // drain the copies still in flight before the CTA's smem goes away
        *abort_flag = 1;
        for (int j = max(0, t - S); j < t; ++j) mbar_wait(full_bar(j % S), (j / S) & 1);
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers
    int ctx[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int row = r0 + rw * 16 + qr + i * 8;
      live[i] = row < R;
      const int rr = live[i] ? row : r0;            // dead rows shadow the tile's first row (never stored)
      tok[i] = tok0 + rr / G;
      head[i] = kvh * G + rr % G;
      ctx[i] = !live[i] ? 0 : (info.w >= 0 ? info.w : rr / G + 1);
    }
    // Q fragments (A operand): a0 = (qr, k0..1), a1 = (qr+8, k0..1), a2 = (qr, k8..9), a3 = (qr+8, k8..9)
    uint32_t qf[KS][4];
    {
      const __nv_bfloat16* q = reinterpret_cast<const __nv_bfloat16*>(a.q);
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const __nv_bfloat16* qp = q + (long long)tok[i] * a.q_stride + (long long)head[i] * HD + qc * 2;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
          qf[ks][i] = *reinterpret_cast<const uint32_t*>(qp + ks * 16);
          qf[ks][i + 2] = *reinterpret_cast<const uint32_t*>(qp + ks * 16 + 8);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < NB; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
    const int ctx_min = __reduce_min_sync(0xffffffffu, min(ctx[0], ctx[1]));   // tiles below it need no masking
    int xpos[2][kMaxLevels];                        // the rows' visible draft positions inside the request's block, or -1
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int e = 0; e < kMaxLevels; ++e) {
        long long off = -1;
        if (live[i] && e < a.n_ext_max) off = a.tok_ext[(long long)tok[i] * a.n_ext_max + e];
        xpos[i][e] = off >= 0 ? (int)((off - (long long)request * a.ext_req_stride) / a.ext_pos_stride) : -1;
      }

    for (int t = g; t < NT; t += KW) {
      const int s = t % S;
      const bool got = mbar_wait_or_abort(full_bar(s), (t / S) & 1, abort_flag);
      if (!__all_sync(0xffffffffu, got)) { if (lane == 0) *abort_flag = 1; break; }
      const uint32_t kt = base + s * C::kStageBytes, vt = kt + C::kTileBytes;

      // ---- S = Q K^T (16 rows x 64 positions per warp)
      float sacc[8][4];
#pragma unroll
      for (int j = 0; j < 8; ++j) { sacc[j][0] = sacc[j][1] = sacc[j][2] = sacc[j][3] = 0.f; }
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
        for (int jp = 0; jp < 4; ++jp) {             // pairs of n-blocks (16 positions)
          const int m = lane >> 3;                   // which 8x8 matrix this lane addresses
          const int pos = jp * 16 + (m >> 1) * 8 + (lane & 7);
          const int chunk = ks * 2 + (m & 1);
          uint32_t b0, b1, b2, b3;
          ldsm_x4(kv_addr<HD>(kt, pos, chunk), b0, b1, b2, b3);
          mma_bf16(sacc[jp * 2], qf[ks], b0, b1);
          mma_bf16(sacc[jp * 2 + 1], qf[ks], b2, b3);
        }
      }
      // ---- mask (only tiles that reach past some row's context), online softmax in base 2
      // rows qr and qr+8; columns j*8 + qc*2 + {0,1}
      if (t >= n_tiles) {                            // a tile of draft positions: each row's own mask
        unsigned long long mk[2] = {0ull, 0ull};
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
          for (int e = 0; e < kMaxLevels; ++e) {
            const int p = xpos[i][e] - (t - n_tiles) * kPos;
            if (xpos[i][e] >= 0 && p >= 0 && p < kPos) mk[i] |= 1ull << p;
          }
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
          for (int e = 0; e < 4; ++e)
            if (!((mk[e >> 1] >> (j * 8 + qc * 2 + (e & 1))) & 1ull)) sacc[j][e] = -INFINITY;
      } else if ((t + 1) * kPos > ctx_min) {
        const int p_base = t * kPos + qc * 2;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
#pragma unroll
          for (int e = 0; e < 4; ++e)
            if (p_base + j * 8 + (e & 1) >= ctx[e >> 1]) sacc[j][e] = -INFINITY;
        }
      }
      float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        mx[0] = fmaxf(mx[0], fmaxf(sacc[j][0], sacc[j][1]));
        mx[1] = fmaxf(mx[1], fmaxf(sacc[j][2], sacc[j][3]));
      }
      float corr[2], neg_m[2];
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        mx[i] = fmaxf(mx[i], __shfl_xor_sync(0xffffffffu, mx[i], 1));
        mx[i] = fmaxf(mx[i], __shfl_xor_sync(0xffffffffu, mx[i], 2));
        const float m_new = fmaxf(m_run[i], mx[i] * sc);
        const float m_safe = m_new == -INFINITY ? 0.f : m_new;     // a row that has seen nothing yet
        corr[i] = ex2(m_run[i] - m_safe);
        m_run[i] = m_new;
        neg_m[i] = -m_safe;
      }
      float rs[2] = {0.f, 0.f};
      uint32_t pf[4][4];                             // P as A fragments for the 4 k-steps of P V
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float p0 = ex2(fmaf(sacc[j][0], sc, neg_m[0])), p1 = ex2(fmaf(sacc[j][1], sc, neg_m[0]));
        const float p2 = ex2(fmaf(sacc[j][2], sc, neg_m[1])), p3 = ex2(fmaf(sacc[j][3], sc, neg_m[1]));
        rs[0] += p0 + p1; rs[1] += p2 + p3;
        pf[j >> 1][(j & 1) * 2] = pack_bf16(p0, p1);
        pf[j >> 1][(j & 1) * 2 + 1] = pack_bf16(p2, p3);
      }
#pragma unroll
      for (int i = 0; i < 2; ++i) l_run[i] = l_run[i] * corr[i] + rs[i];
#pragma unroll
      for (int j = 0; j < NB; ++j) { o[j][0] *= corr[0]; o[j][1] *= corr[0]; o[j][2] *= corr[1]; o[j][3] *= corr[1]; }
      // ---- O += P V
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
        for (int np = 0; np < NB / 2; ++np) {        // pairs of n-blocks (16 dims)
          const int m = lane >> 3;
          const int pos = ks * 16 + (m & 1) * 8 + (lane & 7);
          const int chunk = np * 2 + (m >> 1);
          uint32_t b0, b1, b2, b3;
          ldsm_x4_t(kv_addr<HD>(vt, pos, chunk), b0, b1, b2, b3);
          mma_bf16(o[np * 2], pf[ks], b0, b1);
          mma_bf16(o[np * 2 + 1], pf[ks], b2, b3);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar(s));      // this warp is done with slot s
    }
    if (KW > 1 && g > 0) {                           // hand the partial softmax state to warp group 0
      float* dst = merge + ((size_t)((g - 1) * RW + rw) * C::kMergeFloats) * 32 + lane;
#pragma unroll
      for (int j = 0; j < NB; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) dst[(j * 4 + e) * 32] = o[j][e];
      dst[(NB * 4 + 0) * 32] = m_run[0]; dst[(NB * 4 + 1) * 32] = m_run[1];
      dst[(NB * 4 + 2) * 32] = l_run[0]; dst[(NB * 4 + 3) * 32] = l_run[1];
    }
  }
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicOr(status, kStInternal);
    return;
  }
  if (warp >= RW) return;                            // the rest is warp group 0's

  if (KW > 1) {
#pragma unroll 1
    for (int og = 1; og < KW; ++og) {
      const float* src = merge + ((size_t)((og - 1) * RW + rw) * C::kMergeFloats) * 32 + lane;
      const float m_o[2] = {src[(NB * 4 + 0) * 32], src[(NB * 4 + 1) * 32]};
      const float l_o[2] = {src[(NB * 4 + 2) * 32], src[(NB * 4 + 3) * 32]};
      float c_s[2], c_o[2];
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const float m_new = fmaxf(m_run[i], m_o[i]);
        const float m_safe = m_new == -INFINITY ? 0.f : m_new;
        c_s[i] = ex2(m_run[i] - m_safe); c_o[i] = ex2(m_o[i] - m_safe);
        l_run[i] = l_run[i] * c_s[i] + l_o[i] * c_o[i];
        m_run[i] = m_new;
      }
#pragma unroll
      for (int j = 0; j < NB; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) o[j][e] = o[j][e] * c_s[e >> 1] + src[(j * 4 + e) * 32] * c_o[e >> 1];
    }
  }

  // ---- normalise and store
  __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(a.out);
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    float l = l_run[i];
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    if (!live[i] || !(l > 0.f)) continue;
    const float inv = 1.f / l;
    __nv_bfloat16* op = out + (long long)tok[i] * a.out_stride + (long long)head[i] * HD + qc * 2;
#pragma unroll
    for (int j = 0; j < NB; ++j)
      *reinterpret_cast<__nv_bfloat162*>(op + j * 8) = __floats2bfloat162_rn(o[j][i * 2] * inv, o[j][i * 2 + 1] * inv);
  }
}

template <int HD, int RW, int KW>
void launch(const CUtensorMap* tk, const CUtensorMap* tv, const AttnArgs& a, cudaStream_t st) {
  using C = AttnCfg<HD, RW, KW>;
  static PerDeviceOnce configured;
  configured.run([] {
    cudaFuncSetAttribute(attn_tc_kernel<HD, RW, KW>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
  });
  const int G = a.Hq / a.Hkv;
  dim3 grid(a.Hkv, a.n_rows, (a.max_tokens_per_row * G + 16 * RW - 1) / (16 * RW));
  // the layer's draft-token caches as [positions of all requests, kv heads * hd] (a prefill has none: any valid map)
  CUtensorMap tkx = *tk, tvx = *tv;
  if (a.n_ext_max > 0) {
    const long long rows = a.ext_rows_total, cols = (long long)a.Hkv * HD;
    if (!tma_map_bf16(a.k_ext, rows, cols, cols, kPos, &tkx) || !tma_map_bf16(a.v_ext, rows, cols, cols, kPos, &tvx)) {
      static const int flag = kStInternal;
      cudaMemcpyAsync(a.status, &flag, sizeof(int), cudaMemcpyHostToDevice, st);
      return;
    }
  }
  launch_pdl(attn_tc_kernel<HD, RW, KW>, dim3(grid), dim3(C::kThreads), C::kSmemBytes, st, *tk, *tv, tkx, tvx, a, a.status);
}

}  // namespace

void launch_attention_umma(const AttnArgs& a, const CUtensorMap* tk, const CUtensorMap* tv, cudaStream_t st);

bool attention_tc_supported(const AttnArgs& a) {
  if (!a.status || !a.req_info || a.n_rows <= 0 || a.n_rows > 65535 || a.max_tokens_per_row <= 0) return false;
  if (a.hd != 64 && a.hd != 128) return false;
  if (!tma_encode_fn()) return false;
  if (a.ctx_head_stride % a.hd || a.ctx_row_stride != a.ctx_head_stride * a.Hkv) return false;
  return true;
}

void launch_attention_tc(const AttnArgs& a, cudaStream_t st) {
  // the whole context cache of the layer as one [requests * kv_heads * positions, hd] matrix
  const long long rows = (long long)a.ctx_rows_total;
  CUtensorMap tk_map, tv_map;
  if (!tma_map_bf16(a.k_ctx, rows, a.hd, a.hd, kPos, &tk_map) || !tma_map_bf16(a.v_ctx, rows, a.hd, a.hd, kPos, &tv_map)) {
    launch_attention_simt(a, true, st);
    return;
  }
  const CUtensorMap *tk = &tk_map, *tv = &tv_map;
  LaunchScope ls(kcAttention, st);
  // Query rows per (request, KV head): the bound the grid must cover, and what the caller expects (shapes the tile only).
  const int G = a.Hq / a.Hkv;
  const long long r_bound = (long long)a.max_tokens_per_row * G;
  const long long r = a.rows_expected > 0 && a.rows_expected < r_bound ? a.rows_expected : r_bound;
  if (r <= 32) {                                     // 16-row CTAs whose two consumer warps split the KV tiles
    if (a.hd == 64) launch<64, 1, 2>(tk, tv, a, st); else launch<128, 1, 2>(tk, tv, a, st);
    return;
  }
  static const bool umma = getenv("NEZHA_NO_UMMA_ATTENTION") == nullptr;
  if (umma && r >= 64) { launch_attention_umma(a, tk, tv, st); return; }   // many rows: the tcgen05 kernel, 128 rows per CTA
  // otherwise the fewest CTAs of at most 128 rows, each as short as covers the rows: little padding, K/V streamed
  // as few times as possible
  const int groups = (int)((r + 15) / 16), n_ctas = (groups + 7) / 8;
  const int rw = (groups + n_ctas - 1) / n_ctas;     // 3 .. 8 warps of 16 rows
#define NZ_ATTN_CASE(RW_) \
  case RW_: if (a.hd == 64) launch<64, RW_, 1>(tk, tv, a, st); else launch<128, RW_, 1>(tk, tv, a, st); break;
  switch (rw) {
    NZ_ATTN_CASE(3) NZ_ATTN_CASE(4) NZ_ATTN_CASE(5) NZ_ATTN_CASE(6) NZ_ATTN_CASE(7)
    default: if (a.hd == 64) launch<64, 8, 1>(tk, tv, a, st); else launch<128, 8, 1>(tk, tv, a, st); break;
  }
#undef NZ_ATTN_CASE
}

}  // namespace nz
