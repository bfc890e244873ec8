// Plain CUDA-core GEMM, C[M,N] (op)= A[M,K] * W[N,K]^T with fp32 accumulation.
// It is the arithmetic path of the fp32 configuration (exact fp32 FMA, no tensor-core rounding) and serves
// shapes the tensor-core kernel does not take (ragged N or K).
#include "common.cuh"

namespace nz {

namespace {
constexpr int BM = 64, BN = 64, BK = 16, TM = 4, TN = 4;

template <typename T, int EPI>
__global__ void __launch_bounds__(256) gemm_simt_kernel(GemmArgs a) {
  const int M = a.M_dev ? min(a.M, *a.M_dev) : a.M;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  if (m0 >= M) return;
  __shared__ float As[BK][BM + 4];
  __shared__ float Ws[BK][BN + 4];
  const T* A = reinterpret_cast<const T*>(a.A);
  const T* W = reinterpret_cast<const T*>(a.W);
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;          // 16 x 16 threads, each a 4 x 4 micro-tile
  float acc[TM][TN];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

  const int lr = tid >> 2, lc = (tid & 3) * 4;     // loader: row 0..63, k offset 0,4,8,12
  for (int k0 = 0; k0 < a.K; k0 += BK) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int k = k0 + lc + e;
      const int am = m0 + lr, wn = n0 + lr;
      As[lc + e][lr] = (am < M && k < a.K) ? to_f32(A[(long long)am * a.lda + k]) : 0.f;
      Ws[lc + e][lr] = (wn < a.N && k < a.K) ? to_f32(W[(long long)wn * a.ldw + k]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float av[TM], wv[TN];
#pragma unroll
      for (int i = 0; i < TM; ++i) av[i] = As[k][ty * TM + i];
#pragma unroll
      for (int j = 0; j < TN; ++j) wv[j] = Ws[k][tx * TN + j];
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(av[i], wv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const int m = m0 + ty * TM + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      const int n = n0 + tx * TN + j;
      if (n >= a.N) continue;
      const long long o = (long long)m * a.ldc + n;
      if (EPI == kEpiStoreAct) reinterpret_cast<T*>(a.C)[o] = from_f32<T>(acc[i][j]);
      else if (EPI == kEpiStoreF32) reinterpret_cast<float*>(a.C)[o] = acc[i][j];
      else if (EPI == kEpiAddF32) reinterpret_cast<float*>(a.C)[o] += acc[i][j];
      else if (EPI == kEpiBiasTanhF32) reinterpret_cast<float*>(a.C)[o] = tanhf(acc[i][j] + a.bias[n]);
    }
  }
}

template <typename T>
void dispatch(const GemmArgs& a, cudaStream_t st) {
  dim3 grid((a.N + BN - 1) / BN, (a.M + BM - 1) / BM);
  switch (a.epilogue) {
    case kEpiStoreAct: gemm_simt_kernel<T, kEpiStoreAct><<<grid, 256, 0, st>>>(a); break;
    case kEpiStoreF32: gemm_simt_kernel<T, kEpiStoreF32><<<grid, 256, 0, st>>>(a); break;
    case kEpiAddF32: gemm_simt_kernel<T, kEpiAddF32><<<grid, 256, 0, st>>>(a); break;
    case kEpiBiasTanhF32: gemm_simt_kernel<T, kEpiBiasTanhF32><<<grid, 256, 0, st>>>(a); break;
    default: break;
  }
}
}  // namespace

void launch_gemm_simt(const GemmArgs& a, bool bf16, cudaStream_t st) {
  if (a.M <= 0 || a.N <= 0) return;
  LaunchScope ls(kcGemm, st);
  if (bf16) dispatch<__nv_bfloat16>(a, st);
  else dispatch<float>(a, st);
}

}  // namespace nz
