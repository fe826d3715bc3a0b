// K2 (SIMT): out = epilogue(a * w^T + bias) with fp32 FMA arithmetic.
//
// fp32 operands and outputs only: this is the projection kernel of the fp32 configuration (the
// tensor cores have no full-fp32 mode, and TF32 would not meet an fp32-level tolerance).  The
// 16-bit contexts never come here.  Classic shared-memory tiling: 64x64
// output tile, K step 16, 256 threads each owning a 4x4 micro-tile.
#include "common.cuh"
#include "kernels.h"
#include "launch_pdl.h"

namespace marche {

template <typename TA, typename TO, int EPI>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const TA* __restrict__ a, int lda, int M, const TA* __restrict__ w, const float* __restrict__ bias,
                 int N, int K, void* __restrict__ out_) {
  constexpr int BM = 64, BN = 64, BK = 16;
  __shared__ float As[BK][BM + 4];
  __shared__ float Ws[BK][BN + 4];
  const int tid = threadIdx.x;
  pdl_sync();
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const int tx = tid & 15, ty = tid >> 4;       // micro-tile origin: rows ty*4, cols tx*4
  const int lr = tid >> 2, lk = (tid & 3) * 4;  // loader: row lr (0..63), k offset lk (0,4,8,12)

  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < K; k0 += BK) {
    float av[4] = {0.f, 0.f, 0.f, 0.f}, wv[4];
    if (m0 + lr < M) {
#pragma unroll
      for (int i = 0; i < 4; ++i) av[i] = to_float(a[(long)(m0 + lr) * lda + k0 + lk + i]);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) wv[i] = to_float(w[(long)(n0 + lr) * K + k0 + lk + i]);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      As[lk + i][lr] = av[i];
      Ws[lk + i][lr] = wv[i];
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float ar[4], wr[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) ar[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) wr[j] = Ws[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(ar[i], wr[j], acc[i][j]);
    }
    __syncthreads();
  }

  const int col = n0 + tx * 4;
  const float4 bv = *reinterpret_cast<const float4*>(bias + col);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = m0 + ty * 4 + i;
    if (row >= M) continue;
    float v0 = acc[i][0] + bv.x, v1 = acc[i][1] + bv.y, v2 = acc[i][2] + bv.z, v3 = acc[i][3] + bv.w;
    if (EPI == 1) {
      float4* p = reinterpret_cast<float4*>(reinterpret_cast<float*>(out_) + (long)row * N + col);
      float4 o = *p;
      o.x += v0; o.y += v1; o.z += v2; o.w += v3;
      *p = o;
    } else {
      if (EPI == 2) { v0 = gelu_erf(v0); v1 = gelu_erf(v1); v2 = gelu_erf(v2); v3 = gelu_erf(v3); }
      if (EPI == 2) store4(reinterpret_cast<TA*>(out_) + (long)row * N + col, v0, v1, v2, v3);
      else store4(reinterpret_cast<TO*>(out_) + (long)row * N + col, v0, v1, v2, v3);
    }
  }
}

template <typename TA, typename TO>
static cudaError_t launch_t(const TA* a, int lda, int M, const TA* w, const float* bias, int N, int K, int epi,
                            void* out, cudaStream_t st) {
  dim3 grid(N / 64, (M + 63) / 64);
  switch (epi) {
    case 0: return launch_pdl(gemm_simt_kernel<TA, TO, 0>, grid, dim3(256), 0, st, a, lda, M, w, bias, N, K, out);
    case 1: return launch_pdl(gemm_simt_kernel<TA, TO, 1>, grid, dim3(256), 0, st, a, lda, M, w, bias, N, K, out);
    case 2: return launch_pdl(gemm_simt_kernel<TA, TO, 2>, grid, dim3(256), 0, st, a, lda, M, w, bias, N, K, out);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t launch_gemm_simt(const float* a, int lda, int M, const float* w, const float* bias,
                             int N, int K, int epilogue, float* out, cudaStream_t st) {
  if (M == 0) return cudaSuccess;
  if (N % 64 || K % 16) return cudaErrorInvalidValue;
  return launch_t<float, float>(a, lda, M, w, bias, N, K, epilogue, out, st);
}

}  // namespace marche
