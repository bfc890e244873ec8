// Glue kernels of the primary model: embedding gather, RMSNorm, rotary embedding + KV-cache append, SwiGLU.
// The residual stream is fp32; activations handed to the GEMMs are in the storage type.
#include "common.cuh"

namespace nz {

// resid[i, :] = embed[tokens[i], :]
template <typename T>
__global__ void embed_kernel(const T* __restrict__ table, const int* __restrict__ tokens, int M, const int* M_dev,
                             int d, float* __restrict__ resid) {
  const int m = M_dev ? min(M, *M_dev) : M;
  const int i = blockIdx.x;
  if (i >= m) return;
  const T* src = table + (long long)tokens[i] * d;
  float* dst = resid + (long long)i * d;
  for (int c = threadIdx.x; c < d; c += blockDim.x) dst[c] = to_f32(src[c]);
}

// out[i, :] = x[row, :] / sqrt(mean(x^2) + eps) * gain,  row = row_index ? row_index[i] : i.  One warp per row.
template <typename T>
__global__ void rmsnorm_kernel(const float* __restrict__ x, long long x_stride, const int* __restrict__ row_index,
                               const T* __restrict__ gain, T* __restrict__ out, float* __restrict__ out_f32, int M,
                               const int* M_dev, int d, float eps) {
  const int m = M_dev ? min(M, *M_dev) : M;
  const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (i >= m) return;
  const long long row = row_index ? row_index[i] : i;
  if (row < 0) return;
  const float* src = x + row * x_stride;
  float ss = 0.f;
  for (int c = lane; c < d; c += 32) { float v = src[c]; ss += v * v; }
  ss = warp_sum(ss);
  const float r = rsqrtf(ss / (float)d + eps);
  for (int c = lane; c < d; c += 32) {
    float v = src[c] * r * to_f32(gain[c]);
    if (out) out[(long long)i * d + c] = from_f32<T>(v);
    if (out_f32) out_f32[(long long)i * d + c] = v;
  }
}

// Rotary embedding on half-split pairs (i, i + hd/2) of q and k, in place in the fused qkv buffer, then
// k and v of the token are appended to the cache.  One block per token, threads over (head, pair).
template <typename T>
__global__ void rope_append_kernel(RopeAppendArgs a) {
  const int m = a.M_dev ? min(a.M, *a.M_dev) : a.M;
  const int i = blockIdx.x;
  if (i >= m) return;
  const int half = a.hd >> 1;
  const int pos = a.tok_pos[i];
  T* row = reinterpret_cast<T*>(a.qkv) + (long long)i * (a.Hq + 2 * a.Hkv) * a.hd;
  const float* ct = a.cos_tab + (long long)pos * half;
  const float* st = a.sin_tab + (long long)pos * half;
  T* kc = reinterpret_cast<T*>(a.k_cache);
  T* vc = reinterpret_cast<T*>(a.v_cache);
  const long long dst = a.kv_dst[i];
  const int n_rot = (a.Hq + a.Hkv) * half;
  for (int t = threadIdx.x; t < n_rot; t += blockDim.x) {
    const int h = t / half, p = t - h * half;
    T* v = row + (long long)h * a.hd;
    const float x0 = to_f32(v[p]), x1 = to_f32(v[p + half]);
    const float c = ct[p], s = st[p];
    const T y0 = from_f32<T>(x0 * c - x1 * s), y1 = from_f32<T>(x1 * c + x0 * s);
    if (h < a.Hq) {
      v[p] = y0; v[p + half] = y1;
    } else if (dst >= 0) {
      T* kd = kc + dst + (long long)(h - a.Hq) * a.kv_head_stride;
      kd[p] = y0; kd[p + half] = y1;
    }
  }
  if (dst >= 0) {
    const T* vsrc = row + (long long)(a.Hq + a.Hkv) * a.hd;
    for (int t = threadIdx.x; t < a.Hkv * a.hd; t += blockDim.x) {
      const int h = t / a.hd, p = t - h * a.hd;
      vc[dst + (long long)h * a.kv_head_stride + p] = vsrc[t];
    }
  }
}

// act[i, f] = silu(gu[i, f]) * gu[i, F + f]
template <typename T>
__global__ void swiglu_kernel(const T* __restrict__ gu, T* __restrict__ act, int M, const int* M_dev, int F) {
  const int m = M_dev ? min(M, *M_dev) : M;
  const long long total = (long long)m * F;
  for (long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x; t < total;
       t += (long long)gridDim.x * blockDim.x) {
    const long long i = t / F; const int f = (int)(t - i * F);
    const float g = to_f32(gu[i * 2 * F + f]), u = to_f32(gu[i * 2 * F + F + f]);
    act[t] = from_f32<T>(g / (1.f + __expf(-g)) * u);
  }
}

// Embedding gather fused with the first layer's RMSNorm input: resid = e (fp32), xg = e * gain (bf16, the first
// GEMM's A operand) and ss[i] = sum(e^2) (the row scale is applied in that GEMM's epilogue).  One block per token.
__global__ void embed_norm_kernel(const __nv_bfloat16* __restrict__ table, const int* __restrict__ tokens, int M,
                                  const int* M_dev, int d, float* __restrict__ resid,
                                  const __nv_bfloat16* __restrict__ gain, __nv_bfloat16* __restrict__ xg,
                                  float* __restrict__ ss) {
  pdl_wait();
  pdl_launch();
  const int m = M_dev ? min(M, *M_dev) : M;
  const int i = blockIdx.x;
  if (i >= m) return;
  const __nv_bfloat16* src = table + (long long)tokens[i] * d;
  float part = 0.f;
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    const float v = __bfloat162float(src[c]);
    resid[(long long)i * d + c] = v;
    xg[(long long)i * d + c] = __float2bfloat16_rn(v * __bfloat162float(gain[c]));
    part += v * v;
  }
  __shared__ float red[4];
  part = warp_sum(part);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = part;
  __syncthreads();
  if (threadIdx.x == 0) ss[i] = red[0] + red[1] + red[2] + red[3];
}

// Weight re-layouts of the fused tensor-core path (run once, at context creation).  The GEMM epilogue hands every
// lane 4 consecutive output columns; the rows are ordered so that those 4 columns are everything the lane needs:
//   rotary:  inside every head of hd rows, the 4 rows 32 g + 4 k .. + 3 are input rows i, i + 1, i + hd/2, i + 1 + hd/2
//            with i = 16 g + 2 k  (two rotary pairs);
//   gate/up: rows 32 t + 4 k .. + 3 are gate rows f, f + 1 and up rows f, f + 1 with f = 16 t + 2 k.
__global__ void permute_rotary_rows_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst,
                                           int hd, int cols) {
  const int r = blockIdx.x;
  const int h = r / hd, w = r % hd, g = w >> 5, j = w & 31, k = j >> 2, c = j & 3;
  const int sr = h * hd + 16 * g + 2 * k + (c & 1) + (c >= 2 ? (hd >> 1) : 0);
  for (int t = threadIdx.x; t < cols; t += blockDim.x) dst[(long long)r * cols + t] = src[(long long)sr * cols + t];
}
__global__ void interleave_gate_up_kernel(const __nv_bfloat16* __restrict__ gate, const __nv_bfloat16* __restrict__ up,
                                          __nv_bfloat16* __restrict__ dst, int cols) {
  const int r = blockIdx.x;
  const int t = r >> 5, j = r & 31, k = j >> 2, c = j & 3;
  const long long f = 16 * t + 2 * k + (c & 1);
  const __nv_bfloat16* src = (c < 2 ? gate : up) + f * cols;
  for (int i = threadIdx.x; i < cols; i += blockDim.x) dst[(long long)r * cols + i] = src[i];
}

void launch_embed_norm(const void* table, const int* tokens, int M, const int* M_dev, int d, float* resid,
                       const void* gain, void* xg, float* ss, cudaStream_t st) {
  if (M <= 0) return;
  LaunchScope ls(kcEmbed, st);
  launch_pdl(embed_norm_kernel, dim3(M), dim3(128), 0, st, (const __nv_bfloat16*)table, tokens, M, M_dev, d, resid,
                                       (const __nv_bfloat16*)gain, (__nv_bfloat16*)xg, ss);
}
void launch_permute_rotary_rows(const void* src, void* dst, int rows, int hd, int cols, cudaStream_t st) {
  LaunchScope ls(kcMisc, st);
  permute_rotary_rows_kernel<<<rows, 128, 0, st>>>((const __nv_bfloat16*)src, (__nv_bfloat16*)dst, hd, cols);
}
void launch_interleave_gate_up(const void* gate, const void* up, void* dst, int F, int cols, cudaStream_t st) {
  LaunchScope ls(kcMisc, st);
  interleave_gate_up_kernel<<<2 * F, 128, 0, st>>>((const __nv_bfloat16*)gate, (const __nv_bfloat16*)up,
                                                   (__nv_bfloat16*)dst, cols);
}

void launch_embed(const void* table, bool bf16, const int* tokens, int M, const int* M_dev, int d, float* resid,
                  cudaStream_t st) {
  if (M <= 0) return;
  LaunchScope ls(kcEmbed, st);
  if (bf16) embed_kernel<__nv_bfloat16><<<M, 128, 0, st>>>((const __nv_bfloat16*)table, tokens, M, M_dev, d, resid);
  else embed_kernel<float><<<M, 128, 0, st>>>((const float*)table, tokens, M, M_dev, d, resid);
}

void launch_rmsnorm(const float* x, long long x_stride, const int* row_index, const void* gain, bool bf16, void* out,
                    float* out_f32, int M, const int* M_dev, int d, float eps, cudaStream_t st) {
  if (M <= 0) return;
  const int wpb = 8;
  LaunchScope ls(kcNorm, st);
  dim3 grid((M + wpb - 1) / wpb);
  if (bf16)
    rmsnorm_kernel<__nv_bfloat16><<<grid, wpb * 32, 0, st>>>(x, x_stride, row_index, (const __nv_bfloat16*)gain,
                                                             (__nv_bfloat16*)out, out_f32, M, M_dev, d, eps);
  else
    rmsnorm_kernel<float><<<grid, wpb * 32, 0, st>>>(x, x_stride, row_index, (const float*)gain, (float*)out, out_f32,
                                                     M, M_dev, d, eps);
}

void launch_rope_append(const RopeAppendArgs& a, bool bf16, cudaStream_t st) {
  if (a.M <= 0) return;
  LaunchScope ls(kcRope, st);
  if (bf16) rope_append_kernel<__nv_bfloat16><<<a.M, 128, 0, st>>>(a);
  else rope_append_kernel<float><<<a.M, 128, 0, st>>>(a);
}

void launch_swiglu(const void* gu, void* act, int M, const int* M_dev, int F, bool bf16, cudaStream_t st) {
  if (M <= 0) return;
  long long total = (long long)M * F;
  LaunchScope ls(kcSwiglu, st);
  int blocks = (int)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
  if (bf16) swiglu_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)gu, (__nv_bfloat16*)act, M, M_dev, F);
  else swiglu_kernel<float><<<blocks, 256, 0, st>>>((const float*)gu, (float*)act, M, M_dev, F);
}

}  // namespace nz
