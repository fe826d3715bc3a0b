// K4: relevance-score reduction and top-K refresh selection (Section 4.2).
//
// One CTA per sample.  The per-head score partials [H][S] written by the attention
// kernel are summed in fixed head order (bit-reproducible run to run, unlike atomics),
// then every candidate gets its exact rank under (score descending, index ascending)
// by counting, and the K best are emitted in ascending index order through a block
// scan.  S <= 2048, so all keys of a sample live in shared memory; the work per
// sample is S^2 integer compares, which at these sizes is latency- not bandwidth-bound.
#include "common.cuh"
#include "kernels.h"
#include "launch_pdl.h"

namespace marche {

constexpr int kTopkThreads = 512;

// Order-preserving map of a finite float to uint32 (larger float -> larger key), with
// -0 mapped onto +0.
MARCHE_DEVINL uint32_t score_key(float f) {
  uint32_t u = __float_as_uint(f);
  if ((u << 1) == 0u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Counter-based 32-bit mix of (seed, sample, token) for the random-selection ablation: xor the
// three words with odd multipliers, then two xorshift-multiply rounds.
MARCHE_DEVINL uint32_t mix32(uint32_t seed, uint32_t b, uint32_t t) {
  uint32_t x = seed ^ (b * 0x9E3779B1u) ^ (t * 0x85EBCA77u);
  x ^= x >> 16; x *= 0x7FEB352Du;
  x ^= x >> 15; x *= 0x846CA68Bu;
  x ^= x >> 16;
  return x;
}

// policy 0: highest score first (Section 4.2); 1: lowest score first and 2: random order (the
// selection ablations of Section 5.3).  Ties always go to the lower token index.
__global__ void __launch_bounds__(kTopkThreads)
topk_kernel(const float* __restrict__ partial, int H, float* __restrict__ scores,
            const uint8_t* __restrict__ cand, int S, int k, int policy, uint32_t seed,
            int32_t* __restrict__ refresh_idx) {
  extern __shared__ unsigned long long comp[];          // [S] composite keys; 0 = not a candidate
  __shared__ int warp_tot[kTopkThreads / 32];
  const int b = blockIdx.x, tid = threadIdx.x;
  pdl_sync();

  for (int t = tid; t < S; t += kTopkThreads) {
    float s;
    if (partial) {
      s = 0.f;
      for (int h = 0; h < H; ++h) s += partial[((long)b * H + h) * S + t];
      scores[(long)b * S + t] = s;
    } else {
      s = scores[(long)b * S + t];
    }
    // composite key: score key in the high word, reversed index in the low word, so a
    // larger composite means "ranked earlier" and all composites are distinct and > 0.
    const uint32_t key = policy == 0 ? score_key(s) : (policy == 1 ? ~score_key(s) : ~mix32(seed, (uint32_t)b, (uint32_t)t));
    comp[t] = (k > 0 && cand[(long)b * S + t])
                  ? (((unsigned long long)key << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)t))
                  : 0ull;
  }
  if (k <= 0) return;
  __syncthreads();

  // Each thread owns a contiguous chunk of token indices so the scan below emits
  // ascending indices.
  const int per = (S + kTopkThreads - 1) / kTopkThreads;
  const int t0 = tid * per;
  unsigned sel_mask = 0;   // per <= 4 for S <= 2048
  int cnt = 0;
  for (int i = 0; i < per; ++i) {
    const int t = t0 + i;
    if (t < S) {
      const unsigned long long me = comp[t];
      if (me != 0ull) {
        int rank = 0;
        for (int u = 0; u < S; ++u) rank += (comp[u] > me) ? 1 : 0;
        if (rank < k) { sel_mask |= 1u << i; ++cnt; }
      }
    }
  }
  // exclusive block scan of cnt
  const int lane = tid & 31, warp = tid >> 5;
  int inc = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += v;
  }
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  int base = 0;
  for (int w = 0; w < warp; ++w) base += warp_tot[w];
  int pos = base + inc - cnt;
  for (int i = 0; i < per; ++i)
    if (sel_mask & (1u << i)) refresh_idx[(long)b * k + pos++] = t0 + i;
}

cudaError_t launch_topk(const float* partial, int H, float* scores, const uint8_t* cand, int B, int S, int k,
                        int32_t* refresh_idx, cudaStream_t st, int policy, uint32_t seed) {
  if (S > 2048) return cudaErrorInvalidValue;
  return launch_pdl(topk_kernel, dim3(B), dim3(kTopkThreads), (size_t)S * sizeof(unsigned long long), st, partial, H,
                    scores, cand, S, k, policy, seed, refresh_idx);
}

}  // namespace marche
