// Tensor-core KV-cache attention (bf16) with TMA-staged K/V tiles.
//
// One CTA = (request, KV head, tile of 64 query rows).  The query rows of a (request, KV head) pair are all of the
// request's tokens in this pass times the G query heads of the group, so the request's context K/V is streamed
// from HBM once per (request, KV head, layer) and shared by every beam, draft level and grouped head -- not
// re-read per token.  K/V tiles of 64 positions are brought into shared memory by TMA (128-byte swizzle, a
// 3-deep ring), S = Q K^T and O += P V run on mma.sync m16n8k16 with fp32 accumulation and an online softmax in
// registers.  The per-token extra KV rows (the token's own tuple's drafted codes, at most L-1 of them) are
// folded in afterwards straight from global memory.  The full-barrier wait is bounded (error flag + return).
#include <math.h>

#include "tma.cuh"

namespace nz {

namespace {

constexpr int kRows = 64;        // query rows per CTA (4 warps x 16)
constexpr int kPos = 64;         // KV positions per tile
constexpr int kStages = 3;
constexpr int kThreads = 128;

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

// Address of the 16-byte chunk `chunk` (dims chunk*8 .. +7) of position `pos` inside a K or V stage buffer made of
// HD/64 sub-tiles of [64 positions x 128 bytes], each written by TMA with the 128-byte swizzle.
template <int HD>
__device__ __forceinline__ uint32_t kv_addr(uint32_t tile, int pos, int chunk) {
  const int sub = chunk >> 3, c = chunk & 7;
  return tile + sub * (kPos * 128) + pos * 128 + ((c ^ (pos & 7)) << 4);
}

// The token's own extra KV rows (drafted codes of its tuple), straight from global memory, folded into the running
// softmax state of the thread's two rows.  The loads of all (row, entry) pairs are issued together -- offsets, then
// every K row, then every V row -- so the chain of dependent memory round trips is three long whatever the number
// of entries.  E = compile-time bound of the entries per token (n_ext_max <= E).
template <int HD, int E>
__device__ __forceinline__ void fold_extra_rows(const AttnArgs& a, const int* tok, const int* head, const bool* live, int kvh,
                                                int qc, float sc, float* m_run, float* l_run, float (*o)[4]) {
  constexpr int NB = HD / 8;
    const __nv_bfloat16* q = reinterpret_cast<const __nv_bfloat16*>(a.q);
    const __nv_bfloat16* ke = reinterpret_cast<const __nv_bfloat16*>(a.k_ext);
    const __nv_bfloat16* ve = reinterpret_cast<const __nv_bfloat16*>(a.v_ext);
    long long off[2][E];
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int e = 0; e < E; ++e)
        off[i][e] = (live[i] && e < a.n_ext_max) ? a.tok_ext[(long long)tok[i] * a.n_ext_max + e] : -1;
    // the 4 lanes of a quad own the same rows, so `off` is uniform inside the quad shuffles below
    float sdot[2][E];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const __nv_bfloat16* qp = q + (long long)tok[i] * a.q_stride + (long long)head[i] * HD + qc * 2;
      __nv_bfloat162 qq[NB];
#pragma unroll
      for (int j = 0; j < NB; ++j) qq[j] = *reinterpret_cast<const __nv_bfloat162*>(qp + j * 8);
#pragma unroll
      for (int e = 0; e < E; ++e) {
        float sd = 0.f;
        if (off[i][e] >= 0) {
          const __nv_bfloat16* kp = ke + off[i][e] + (long long)kvh * a.ext_head_stride + qc * 2;
#pragma unroll
          for (int j = 0; j < NB; ++j) {
            const __nv_bfloat162 kk = *reinterpret_cast<const __nv_bfloat162*>(kp + j * 8);
            sd += __bfloat162float(qq[j].x) * __bfloat162float(kk.x) + __bfloat162float(qq[j].y) * __bfloat162float(kk.y);
          }
        }
        sdot[i][e] = sd;
      }
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      float m_new = m_run[i];
#pragma unroll
      for (int e = 0; e < E; ++e) {
        float sd = sdot[i][e];
        sd += __shfl_xor_sync(0xffffffffu, sd, 1);
        sd += __shfl_xor_sync(0xffffffffu, sd, 2);
        sdot[i][e] = off[i][e] >= 0 ? sd * sc : -INFINITY;
        m_new = fmaxf(m_new, sdot[i][e]);
      }
      if (m_new == -INFINITY) continue;              // nothing visible at all (dead row)
      const float c = (m_run[i] == -INFINITY) ? 0.f : exp2f(m_run[i] - m_new);
      l_run[i] *= c;
#pragma unroll
      for (int j = 0; j < NB; ++j) { o[j][i * 2] *= c; o[j][i * 2 + 1] *= c; }
      m_run[i] = m_new;
#pragma unroll
      for (int e = 0; e < E; ++e) {
        if (off[i][e] < 0) continue;
        const float p = exp2f(sdot[i][e] - m_new);
        l_run[i] += (qc == 0 ? p : 0.f);             // row sums are per-lane partials, reduced at the end
        const __nv_bfloat16* vp = ve + off[i][e] + (long long)kvh * a.ext_head_stride + qc * 2;
#pragma unroll
        for (int j = 0; j < NB; ++j) {
          const __nv_bfloat162 vv = *reinterpret_cast<const __nv_bfloat162*>(vp + j * 8);
          o[j][i * 2] += p * __bfloat162float(vv.x);
          o[j][i * 2 + 1] += p * __bfloat162float(vv.y);
        }
      }
    }
}

template <int HD>
__global__ void __launch_bounds__(kThreads, 3) attn_tc_kernel(const __grid_constant__ CUtensorMap tmK,
                                                           const __grid_constant__ CUtensorMap tmV, AttnArgs a,
                                                           int* status) {
  constexpr int NH = HD / 64;                       // 64-column halves per tile
  constexpr int kTileBytes = kPos * HD * 2;         // one K (or V) tile
  constexpr int kStageBytes = 2 * kTileBytes;
  constexpr int KS = HD / 16;                       // k-steps of Q K^T
  constexpr int NB = HD / 8;                        // n-blocks of the output

  const int req_local = blockIdx.z, kvh = blockIdx.y, tile = blockIdx.x;
  const int G = a.Hq / a.Hkv;
  const int4 info = a.req_info[req_local];          // {first token, token count, cache row, context length or -1}
  const int tok0 = info.x, n_tok = info.y, request = info.z;
  const int R = n_tok * G;                          // query rows of this (request, kv head)
  const int r0 = tile * kRows;
  if (r0 >= R) return;
  // context positions this tile needs: all of them, or (causal prefill) up to its last token's own position
  const int max_ctx = info.w >= 0 ? info.w : min((r0 + kRows - 1) / G, n_tok - 1) + 1;
  const int n_tiles = (max_ctx + kPos - 1) / kPos;
  const int kv_row0 = (int)(((long long)request * a.Hkv + kvh) * (a.ctx_head_stride / HD));   // first cache row

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = base + kStages * kStageBytes;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qr = lane >> 2, qc = lane & 3;          // fragment row (and +8) / column pair

  auto issue = [&](int t) {                          // thread 0 only
    const int s = t % kStages;
    const uint32_t bar = bar_base + 8u * s;
    mbar_expect_tx(bar, kStageBytes);
#pragma unroll
    for (int h = 0; h < NH; ++h) {
      tma_load_2d(base + s * kStageBytes + h * (kPos * 128), &tmK, h * 64, kv_row0 + t * kPos, bar);
      tma_load_2d(base + s * kStageBytes + kTileBytes + h * (kPos * 128), &tmV, h * 64, kv_row0 + t * kPos, bar);
    }
  };
  if (threadIdx.x == 0) {                            // the first K/V tiles are on their way before anything else is read
    for (int s = 0; s < kStages; ++s) mbar_init(bar_base + 8u * s, 1);
    mbar_fence_init();
    for (int t = 0; t < min(n_tiles, kStages); ++t) issue(t);
  }

  // the two rows this thread owns
  int row[2], tok[2], head[2], ctx[2];
  bool live[2];
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    row[i] = r0 + warp * 16 + qr + i * 8;
    live[i] = row[i] < R;
    const int rr = live[i] ? row[i] : r0;           // dead rows shadow the tile's first row (never stored)
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
  __syncthreads();                                   // barrier initialisation visible to every waiter

  float o[NB][4];
#pragma unroll
  for (int j = 0; j < NB; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  const float sc = a.scale * 1.4426950408889634f;   // work in base 2
  bool aborted = false;

  for (int t = 0; t < n_tiles; ++t) {
    const int s = t % kStages;
    const int gave_up = mbar_wait(bar_base + 8u * s, (t / kStages) & 1) ? 0 : 1;
    if (__syncthreads_or(gave_up)) { aborted = true; break; }   // uniform exit for the whole CTA
    const uint32_t kt = base + s * kStageBytes, vt = kt + kTileBytes;

    // ---- S = Q K^T (16 rows x 64 positions per warp)
    float sacc[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) { sacc[j][0] = sacc[j][1] = sacc[j][2] = sacc[j][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
      for (int jp = 0; jp < 4; ++jp) {               // pairs of n-blocks (16 positions)
        const int m = lane >> 3;                     // which 8x8 matrix this lane addresses
        const int pos = jp * 16 + (m >> 1) * 8 + (lane & 7);
        const int chunk = ks * 2 + (m & 1);
        uint32_t b0, b1, b2, b3;
        ldsm_x4(kv_addr<HD>(kt, pos, chunk), b0, b1, b2, b3);
        mma_bf16(sacc[jp * 2], qf[ks], b0, b1);
        mma_bf16(sacc[jp * 2 + 1], qf[ks], b2, b3);
      }
    }
    // ---- scale, mask, online softmax (rows qr and qr+8; columns j*8 + qc*2 + {0,1})
    const int p_base = t * kPos + qc * 2;
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int i = e >> 1;
        const int p = p_base + j * 8 + (e & 1);
        const float v = (p < ctx[i]) ? sacc[j][e] * sc : -INFINITY;
        sacc[j][e] = v;
        mx[i] = fmaxf(mx[i], v);
      }
    }
    float corr[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      mx[i] = fmaxf(mx[i], __shfl_xor_sync(0xffffffffu, mx[i], 1));
      mx[i] = fmaxf(mx[i], __shfl_xor_sync(0xffffffffu, mx[i], 2));
      const float m_new = fmaxf(m_run[i], mx[i]);
      corr[i] = (m_run[i] == -INFINITY) ? 0.f : exp2f(m_run[i] - m_new);
      m_run[i] = m_new;
    }
    float rs[2] = {0.f, 0.f};
    uint32_t pf[4][4];                               // P as A fragments for the 4 k-steps of P V
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      float p0 = (m_run[0] == -INFINITY) ? 0.f : exp2f(sacc[j][0] - m_run[0]);
      float p1 = (m_run[0] == -INFINITY) ? 0.f : exp2f(sacc[j][1] - m_run[0]);
      float p2 = (m_run[1] == -INFINITY) ? 0.f : exp2f(sacc[j][2] - m_run[1]);
      float p3 = (m_run[1] == -INFINITY) ? 0.f : exp2f(sacc[j][3] - m_run[1]);
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
      for (int np = 0; np < NB / 2; ++np) {          // pairs of n-blocks (16 dims)
        const int m = lane >> 3;
        const int pos = ks * 16 + (m & 1) * 8 + (lane & 7);
        const int chunk = np * 2 + (m >> 1);
        uint32_t b0, b1, b2, b3;
        ldsm_x4_t(kv_addr<HD>(vt, pos, chunk), b0, b1, b2, b3);
        mma_bf16(o[np * 2], pf[ks], b0, b1);
        mma_bf16(o[np * 2 + 1], pf[ks], b2, b3);
      }
    }
    __syncthreads();                                 // everyone is done with stage s
    if (threadIdx.x == 0 && t + kStages < n_tiles) issue(t + kStages);
  }
  if (aborted) {
    if (threadIdx.x == 0) {
      atomicOr(status, kStInternal);
      // drain copies that may still be in flight (bounded) before the CTA's shared memory goes away
      for (int s = 0; s < kStages; ++s) mbar_wait(bar_base + 8u * s, 0);
    }
    return;
  }

  // ---- the token's own extra KV rows (drafted codes of its tuple)
  if (a.n_ext_max > 4) fold_extra_rows<HD, kMaxLevels>(a, tok, head, live, kvh, qc, sc, m_run, l_run, o);
  else if (a.n_ext_max > 0) fold_extra_rows<HD, 4>(a, tok, head, live, kvh, qc, sc, m_run, l_run, o);

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

template <int HD>
void launch(const CUtensorMap* tk, const CUtensorMap* tv, const AttnArgs& a, cudaStream_t st) {
  constexpr int smem = kStages * 2 * kPos * HD * 2 + 1024 + 64;
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(attn_tc_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    configured = true;
  }
  const int G = a.Hq / a.Hkv;
  dim3 grid((a.max_tokens_per_row * G + kRows - 1) / kRows, a.Hkv, a.n_rows);
  attn_tc_kernel<HD><<<grid, kThreads, smem, st>>>(*tk, *tv, a, a.status);
}

}  // namespace

bool attention_tc_supported(const AttnArgs& a) {
  if (!a.status || !a.req_info || a.n_rows <= 0 || a.max_tokens_per_row <= 0) return false;
  if (a.hd != 64 && a.hd != 128) return false;
  if (!tma_encode_fn()) return false;
  if (a.ctx_head_stride % a.hd || a.ctx_row_stride != a.ctx_head_stride * a.Hkv) return false;
  return true;
}

void launch_attention_tc(const AttnArgs& a, cudaStream_t st) {
  // the whole context cache of the layer as one [requests * kv_heads * positions, hd] matrix
  const long long rows = (long long)a.ctx_rows_total;
  const CUtensorMap* tk = tma_map_bf16(a.k_ctx, rows, a.hd, a.hd, kPos);
  const CUtensorMap* tv = tma_map_bf16(a.v_ctx, rows, a.hd, a.hd, kPos);
  if (!tk || !tv) { launch_attention_simt(a, true, st); return; }
  LaunchScope ls(kcAttention, st);
  if (a.hd == 64) launch<64>(tk, tv, a, st);
  else launch<128>(tk, tv, a, st);
}

}  // namespace nz
