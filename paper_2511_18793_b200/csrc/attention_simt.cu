// CUDA-core attention: each token attends to a prefix of its request's context KV cache plus a few extra
// KV rows (its own tuple's drafted codes).  One warp per (token, query head); the warp is split into 4 groups
// of 8 lanes, each group walks every 4th position with the head dimension spread over its 8 lanes, and the
// 4 partial softmax states are merged at the end.  Exact fp32 arithmetic: this is the attention of the
// fp32 configuration and of head sizes the tensor-core kernel does not take.
#include <math.h>

#include "common.cuh"

namespace nz {

namespace {

template <typename T, int HD>
__global__ void __launch_bounds__(128) attn_simt_kernel(AttnArgs a) {
  constexpr int DPL = HD / 8;
  const int m = a.M_dev ? min(a.M, *a.M_dev) : a.M;
  const long long w = blockIdx.x * (long long)(blockDim.x >> 5) + (threadIdx.x >> 5);
  const int i = (int)(w / a.Hq), h = (int)(w % a.Hq);
  if (i >= m) return;
  const int lane = threadIdx.x & 31, pg = lane >> 3, sub = lane & 7;
  const int kvh = h / (a.Hq / a.Hkv);
  const T* qp = reinterpret_cast<const T*>(a.q) + (long long)i * a.q_stride + (long long)h * HD + sub * DPL;
  float qv[DPL], acc[DPL];
#pragma unroll
  for (int j = 0; j < DPL; ++j) { qv[j] = to_f32(qp[j]) * a.scale; acc[j] = 0.f; }
  float m_run = -INFINITY, l_run = 0.f;

  auto visit = [&](const T* kp, const T* vp) {
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < DPL; ++j) s = fmaf(qv[j], to_f32(kp[j]), s);
    return s;
  };
  auto update = [&](float s, const T* vp) {
    const float m_new = fmaxf(m_run, s);
    const float corr = (m_run == -INFINITY) ? 0.f : expf(m_run - m_new);
    const float pw = expf(s - m_new);
    l_run = l_run * corr + pw;
#pragma unroll
    for (int j = 0; j < DPL; ++j) acc[j] = acc[j] * corr + pw * to_f32(vp[j]);
    m_run = m_new;
  };

  const int ctx_len = a.tok_ctx_len[i];
  const long long base = (long long)a.tok_row[i] * a.ctx_row_stride + (long long)kvh * a.ctx_head_stride + sub * DPL;
  const T* kc = reinterpret_cast<const T*>(a.k_ctx) + base;
  const T* vc = reinterpret_cast<const T*>(a.v_ctx) + base;
  for (int p0 = 0; p0 < ctx_len; p0 += 4) {
    const int p = p0 + pg;
    const bool valid = p < ctx_len;
    float s = valid ? visit(kc + (long long)p * HD, nullptr) : 0.f;
    s += __shfl_xor_sync(0xffffffffu, s, 1);
    s += __shfl_xor_sync(0xffffffffu, s, 2);
    s += __shfl_xor_sync(0xffffffffu, s, 4);
    if (valid) update(s, vc + (long long)p * HD);
  }
  for (int e0 = 0; e0 < a.n_ext_max; e0 += 4) {
    const int e = e0 + pg;
    const long long off = (e < a.n_ext_max) ? a.tok_ext[(long long)i * a.n_ext_max + e] : -1;
    const bool valid = off >= 0;
    const long long eo = off + (long long)kvh * a.ext_head_stride + sub * DPL;
    float s = valid ? visit(reinterpret_cast<const T*>(a.k_ext) + eo, nullptr) : 0.f;
    s += __shfl_xor_sync(0xffffffffu, s, 1);
    s += __shfl_xor_sync(0xffffffffu, s, 2);
    s += __shfl_xor_sync(0xffffffffu, s, 4);
    if (valid) update(s, reinterpret_cast<const T*>(a.v_ext) + eo);
  }
  // merge the 4 position groups
#pragma unroll
  for (int o = 8; o <= 16; o <<= 1) {
    const float m_o = __shfl_xor_sync(0xffffffffu, m_run, o);
    const float l_o = __shfl_xor_sync(0xffffffffu, l_run, o);
    const float m_new = fmaxf(m_run, m_o);
    const float c_s = (m_run == -INFINITY) ? 0.f : expf(m_run - m_new);
    const float c_o = (m_o == -INFINITY) ? 0.f : expf(m_o - m_new);
    l_run = l_run * c_s + l_o * c_o;
#pragma unroll
    for (int j = 0; j < DPL; ++j) {
      const float a_o = __shfl_xor_sync(0xffffffffu, acc[j], o);
      acc[j] = acc[j] * c_s + a_o * c_o;
    }
    m_run = m_new;
  }
  if (pg == 0) {
    T* op = reinterpret_cast<T*>(a.out) + (long long)i * a.out_stride + (long long)h * HD + sub * DPL;
    const float inv = 1.f / l_run;
#pragma unroll
    for (int j = 0; j < DPL; ++j) op[j] = from_f32<T>(acc[j] * inv);
  }
}

template <typename T>
void dispatch(const AttnArgs& a, cudaStream_t st) {
  const long long warps = (long long)a.M * a.Hq;
  const int wpb = 4;
  dim3 grid((unsigned)((warps + wpb - 1) / wpb));
  switch (a.hd) {
    case 16: attn_simt_kernel<T, 16><<<grid, wpb * 32, 0, st>>>(a); break;
    case 32: attn_simt_kernel<T, 32><<<grid, wpb * 32, 0, st>>>(a); break;
    case 64: attn_simt_kernel<T, 64><<<grid, wpb * 32, 0, st>>>(a); break;
    case 128: attn_simt_kernel<T, 128><<<grid, wpb * 32, 0, st>>>(a); break;
    default: break;
  }
}
}  // namespace

void launch_attention_simt(const AttnArgs& a, bool bf16, cudaStream_t st) {
  if (a.M <= 0) return;
  LaunchScope ls(kcAttention, st);
  if (bf16) dispatch<__nv_bfloat16>(a, st);
  else dispatch<float>(a, st);
}

}  // namespace nz
