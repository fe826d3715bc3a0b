// K4: relevance-score reduction and top-K refresh selection (Section 4.2).
//
// One CTA per sample.  The per-head score partials [H][S] written by the attention
// kernel are summed in fixed head order (bit-reproducible run to run, unlike atomics),
// then the K-th best candidate under (score descending, index ascending) is found by a
// radix select and the K best are emitted in ascending index order through a block
// scan.  S <= 2048, so all keys of a sample live in shared memory.
#include "common.cuh"
#include "kernels.h"
#include "launch_pdl.h"

namespace marche {

constexpr int kTopkThreads = 256;

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
//
// Every candidate gets a 44-bit composite (32-bit order key, then 2047 - index, plus one so that
// 0 can mean "not a candidate"); composites are distinct, a larger one ranks earlier.  The k-th
// largest composite is found by a most-significant-digit-first radix select, four passes of 11
// bits over a 2048-bin histogram in shared memory, and every candidate at or above it is emitted.
// O(S) work per sample instead of the S^2 of ranking by counting; the result is the same set.
constexpr int kRadixBits = 11, kRadixBins = 1 << kRadixBits, kRadixPasses = 4;

__global__ void __launch_bounds__(kTopkThreads)
topk_kernel(const float* __restrict__ partial, int H, float* __restrict__ scores,
            const uint8_t* __restrict__ cand, int S, int k, int policy, uint32_t seed,
            int32_t* __restrict__ refresh_idx) {
  extern __shared__ unsigned long long comp[];          // [S] composites; 0 = not a candidate
  __shared__ unsigned int hist[kRadixBins];
  __shared__ int warp_tot[kTopkThreads / 32];
  __shared__ unsigned int sel_digit, sel_above;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
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
    const uint32_t key = policy == 0 ? score_key(s) : (policy == 1 ? ~score_key(s) : ~mix32(seed, (uint32_t)b, (uint32_t)t));
    comp[t] = (k > 0 && cand[(long)b * S + t])
                  ? ((((unsigned long long)key << kRadixBits) | (unsigned long long)(kRadixBins - 1 - t)) + 1ull)
                  : 0ull;
  }
  if (k <= 0) return;

  // ---- radix select of the k-th largest composite
  unsigned long long prefix = 0ull, decided = 0ull;     // bits fixed so far and their mask
  int remaining = k;
#pragma unroll 1
  for (int pass = 0; pass < kRadixPasses; ++pass) {
    const int shift = kRadixBits * (kRadixPasses - 1 - pass);
    for (int i = tid; i < kRadixBins; i += kTopkThreads) hist[i] = 0u;
    __syncthreads();                                     // also orders the writes of comp before the reads
    for (int t = tid; t < S; t += kTopkThreads) {
      const unsigned long long c = comp[t];
      if (c != 0ull && (c & decided) == prefix) atomicAdd(&hist[(unsigned)(c >> shift) & (kRadixBins - 1)], 1u);
    }
    __syncthreads();
    // With fewer than `remaining` candidates left no bin crosses: digit 0 then keeps every candidate.
    // (Reset here: all threads have passed this pass's first barrier, so none still reads the last pass's values.)
    if (tid == 0) { sel_digit = 0u; sel_above = 0u; }
    // thread i owns PER consecutive bins; suffix sums from the top bin downwards
    constexpr int PER = kRadixBins / kTopkThreads;
    unsigned int h[PER], mine = 0u;
#pragma unroll
    for (int j = 0; j < PER; ++j) { h[j] = hist[tid * PER + j]; mine += h[j]; }
    unsigned int inc = mine;                             // inclusive scan over threads in DESCENDING thread order
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned int v = __shfl_down_sync(0xffffffffu, inc, o);
      if (lane + o < 32) inc += v;
    }
    if (lane == 0) warp_tot[warp] = (int)inc;
    __syncthreads();
    unsigned int above = inc - mine;                     // candidates in bins above this thread's bins
    for (int w = warp + 1; w < kTopkThreads / 32; ++w) above += (unsigned)warp_tot[w];
    // the crossing bin: the highest bin d with (count in bins >= d) >= remaining
    if (above < (unsigned)remaining && above + mine >= (unsigned)remaining) {
      unsigned int acc = above;
#pragma unroll
      for (int j = PER - 1; j >= 0; --j) {
        if (acc < (unsigned)remaining && acc + h[j] >= (unsigned)remaining) {
          sel_digit = (unsigned)(tid * PER + j);
          sel_above = acc;
        }
        acc += h[j];
      }
    }
    __syncthreads();
    prefix |= (unsigned long long)sel_digit << shift;
    decided |= (unsigned long long)(kRadixBins - 1) << shift;
    remaining -= (int)sel_above;
  }
  const unsigned long long threshold = prefix;           // the k-th largest composite itself

  // Each thread owns a contiguous chunk of token indices so the scan below emits ascending indices.
  const int per = (S + kTopkThreads - 1) / kTopkThreads;
  const int t0 = tid * per;
  unsigned sel_mask = 0;   // per <= 8 for S <= 2048
  int cnt = 0;
  for (int i = 0; i < per; ++i) {
    const int t = t0 + i;
    if (t < S) {
      const unsigned long long me = comp[t];
      if (me != 0ull && me >= threshold) { sel_mask |= 1u << i; ++cnt; }
    }
  }
  // exclusive block scan of cnt
  int inc2 = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, inc2, o);
    if (lane >= o) inc2 += v;
  }
  __syncthreads();                                       // warp_tot is reused
  if (lane == 31) warp_tot[warp] = inc2;
  __syncthreads();
  int base = 0;
  for (int w = 0; w < warp; ++w) base += warp_tot[w];
  int pos = base + inc2 - cnt;
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
