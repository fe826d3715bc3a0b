// K3 (SIMT): attention of the active queries over all S cached rows of one block
// (Algorithm 1 lines 6-8; by Appendix A this is plain softmax attention, Eq. 5, once
// the active rows' fresh K, V are in the cache), with the relevance reduction of
// Section 4.2 fused in.  fp32 arithmetic and storage; serves the fp32 configuration only.
//
// One CTA per (sample, head); warp w handles queries w, w+NW, ...  A query's whole
// probability row lives in shared memory, so the softmax is the exact two-pass form
// and the column sums use final probabilities.  Each warp accumulates its own column
// sums and the warps are combined in fixed order: scores are bit-reproducible.
#include "common.cuh"
#include "kernels.h"
#include "launch_pdl.h"

namespace marche {

constexpr int kAttWarps = 8;

size_t attention_simt_smem(int S, int dh) {
  return (size_t)kAttWarps * (2 * (size_t)S + dh) * sizeof(float);
}

template <typename T, typename TO>
__global__ void __launch_bounds__(kAttWarps * 32)
attention_simt_kernel(const T* __restrict__ q, int ld_q, int n, int S, int H, int dh,
                      const T* __restrict__ cache_layer, long kv_stride, const uint8_t* __restrict__ is_new,
                      float* __restrict__ score_partial, TO* __restrict__ o) {
  extern __shared__ float smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.x / H, h = blockIdx.x % H;
  pdl_sync();
  const int D = H * dh;
  float* p = smem + (size_t)warp * S;                               // probabilities of the current query
  float* colsum = smem + (size_t)kAttWarps * S + (size_t)warp * S;  // this warp's column sums
  float* qs = smem + (size_t)2 * kAttWarps * S + (size_t)warp * dh;
  const T* Kb = cache_layer + (long)b * S * D + h * dh;
  const T* Vb = Kb + kv_stride;
  const bool scoring = is_new != nullptr;
  const float scale = rsqrtf((float)dh);

  if (scoring)
    for (int t = lane; t < S; t += 32) colsum[t] = 0.f;

  for (int j = warp; j < n; j += kAttWarps) {
    const long r = (long)b * n + j;
    __syncwarp();
    for (int c = lane; c < dh; c += 32) qs[c] = to_float(q[r * ld_q + h * dh + c]) * scale;
    __syncwarp();
    float mx = -INFINITY;
    for (int t = lane; t < S; t += 32) {
      const T* kr = Kb + (long)t * D;
      float acc = 0.f;
      for (int c = 0; c < dh; ++c) acc = fmaf(qs[c], to_float(kr[c]), acc);
      p[t] = acc;
      mx = fmaxf(mx, acc);
    }
    mx = warp_max(mx);
    float sum = 0.f;
    for (int t = lane; t < S; t += 32) {
      const float e = expf(p[t] - mx);
      p[t] = e;
      sum += e;
    }
    const float inv = 1.0f / warp_sum(sum);
    const bool flagged = scoring && is_new[r];
    for (int t = lane; t < S; t += 32) {
      const float pr = p[t] * inv;
      p[t] = pr;
      if (flagged) colsum[t] += pr;
    }
    __syncwarp();
    for (int c = lane; c < dh; c += 32) {
      float acc = 0.f;
      for (int t = 0; t < S; ++t) acc = fmaf(p[t], to_float(Vb[(long)t * D + c]), acc);
      o[r * D + h * dh + c] = from_float<TO>(acc);
    }
  }
  if (scoring) {
    __syncthreads();
    for (int t = threadIdx.x; t < S; t += blockDim.x) {
      float s = 0.f;
      for (int w = 0; w < kAttWarps; ++w) s += smem[(size_t)kAttWarps * S + (size_t)w * S + t];
      score_partial[((long)b * H + h) * S + t] = s;
    }
  }
}

cudaError_t launch_attention_simt(const float* q, int ld_q, int B, int n, int S, int H, int dh,
                                  const float* cache_layer, const uint8_t* is_new, float* score_partial,
                                  float* o, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  const size_t smem = attention_simt_smem(S, dh);
  const long kv_stride = (long)B * S * H * dh;
  static size_t smem_set[kMaxDevices] = {};
  cudaError_t e = ensure_dynamic_smem(attention_simt_kernel<float, float>, smem, smem_set);
  if (e != cudaSuccess) return e;
  return launch_pdl(attention_simt_kernel<float, float>, dim3(B * H), dim3(kAttWarps * 32), smem, st, q, ld_q, n, S, H, dh,
                    cache_layer, kv_stride, is_new, score_partial, o);
}

}  // namespace marche
