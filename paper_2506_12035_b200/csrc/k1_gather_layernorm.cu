// K1: index gather + LayerNorm (Algorithm 1 line 5, input side of the QKV and MLP
// projections).  HBM-bound: each fp32 row is read once with 128-bit loads, kept in
// registers for the two statistics passes, and written once as fp32, fp16 or bf16 (and, at block 0,
// once more as the compact fp32 residual row).
//
// One warp per row: lane l holds float4 number l, l+32, ... of the row (NV per lane),
// so every load/store instruction of a warp covers 512 contiguous bytes.
#include "common.cuh"
#include "kernels.h"
#include "launch_pdl.h"

namespace marche {

constexpr int kLnWarps = 8;

template <typename TOut, int NV>
__global__ void __launch_bounds__(kLnWarps * 32)
gather_layernorm_kernel(const float* __restrict__ src, int src_rows, const int32_t* __restrict__ idx,
                        int n, int total_rows, const float* __restrict__ gamma,
                        const float* __restrict__ beta, float eps, float* __restrict__ x_out,
                        TOut* __restrict__ u_out, const int32_t* __restrict__ out_idx, int out_rows) {
  constexpr int D = NV * 128;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long r = (long)blockIdx.x * kLnWarps + warp;
  if (r >= total_rows) return;
  pdl_sync();
  const int b = (int)(r / n), j = (int)(r - (long)b * n);
  const int srow = idx ? idx[r] : j;
  const float4* __restrict__ in = reinterpret_cast<const float4*>(src + ((long)b * src_rows + srow) * D);

  float4 v[NV];
#pragma unroll
  for (int i = 0; i < NV; ++i) v[i] = __ldg(in + i * 32 + lane);

  float s = 0.f;
#pragma unroll
  for (int i = 0; i < NV; ++i) s += (v[i].x + v[i].y) + (v[i].z + v[i].w);
  const float mean = warp_sum(s) * (1.0f / D);
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const float a = v[i].x - mean, b2 = v[i].y - mean, c = v[i].z - mean, d = v[i].w - mean;
    ss += (a * a + b2 * b2) + (c * c + d * d);
  }
  const float rstd = rsqrtf(warp_sum(ss) * (1.0f / D) + eps);

  if (x_out) {
    float4* xo = reinterpret_cast<float4*>(x_out + r * D);
#pragma unroll
    for (int i = 0; i < NV; ++i) xo[i * 32 + lane] = v[i];
  }
  const float4* g4 = reinterpret_cast<const float4*>(gamma);
  const float4* b4 = reinterpret_cast<const float4*>(beta);
  // out_rows > 0: the normalised row goes to row out_idx[r] (identity when NULL) of a [B][out_rows][D] array
  const long orow = out_rows > 0 ? (long)b * out_rows + (out_idx ? out_idx[r] : j) : r;
  TOut* uo = u_out + orow * D;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const float4 g = __ldg(g4 + i * 32 + lane), be = __ldg(b4 + i * 32 + lane);
    store4(uo + (i * 32 + lane) * 4,
           (v[i].x - mean) * rstd * g.x + be.x, (v[i].y - mean) * rstd * g.y + be.y,
           (v[i].z - mean) * rstd * g.z + be.z, (v[i].w - mean) * rstd * g.w + be.w);
  }
}

template <typename TOut>
static cudaError_t launch_ln_t(const float* src, int src_rows, const int32_t* idx, int B, int n, int D,
                               const float* gamma, const float* beta, float eps, float* x_out, TOut* u_out,
                               cudaStream_t st, const int32_t* out_idx, int out_rows) {
  const long rows = (long)B * n;
  if (rows == 0) return cudaSuccess;
  const unsigned grid = (unsigned)((rows + kLnWarps - 1) / kLnWarps);
  cudaError_t err = cudaSuccess;
#define MARCHE_LN_CASE(NV_)                                                                          \
  case NV_:                                                                                          \
    err = launch_pdl(gather_layernorm_kernel<TOut, NV_>, dim3(grid), dim3(kLnWarps * 32), 0, st, src, src_rows, \
                     idx, n, (int)rows, gamma, beta, eps, x_out, u_out, out_idx, out_rows);          \
    break;
  switch (D / 128) {
    MARCHE_LN_CASE(1) MARCHE_LN_CASE(2) MARCHE_LN_CASE(3) MARCHE_LN_CASE(4) MARCHE_LN_CASE(5)
    MARCHE_LN_CASE(6) MARCHE_LN_CASE(7) MARCHE_LN_CASE(8) MARCHE_LN_CASE(9) MARCHE_LN_CASE(10)
    MARCHE_LN_CASE(11) MARCHE_LN_CASE(12) MARCHE_LN_CASE(13) MARCHE_LN_CASE(14) MARCHE_LN_CASE(15)
    MARCHE_LN_CASE(16)
    default: return cudaErrorInvalidValue;
  }
#undef MARCHE_LN_CASE
  return err;
}

cudaError_t launch_gather_layernorm(int out_kind, const float* src, int src_rows, const int32_t* idx,
                                    int B, int n, int D, const float* gamma, const float* beta, float eps,
                                    float* x_out, void* u_out, cudaStream_t st, const int32_t* out_idx,
                                    int out_rows) {
  if (D % 128 != 0) return cudaErrorInvalidValue;
  if (out_kind == OUT_F16)
    return launch_ln_t<f16>(src, src_rows, idx, B, n, D, gamma, beta, eps, x_out, (f16*)u_out, st, out_idx, out_rows);
  if (out_kind == OUT_BF16)
    return launch_ln_t<bf16>(src, src_rows, idx, B, n, D, gamma, beta, eps, x_out, (bf16*)u_out, st, out_idx, out_rows);
  return launch_ln_t<float>(src, src_rows, idx, B, n, D, gamma, beta, eps, x_out, (float*)u_out, st, out_idx, out_rows);
}

}  // namespace marche
