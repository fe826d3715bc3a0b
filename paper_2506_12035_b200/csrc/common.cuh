// Shared device helpers for the libmarche kernels (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

typedef __nv_bfloat16 bf16;
typedef __half f16;

#define MARCHE_DEVINL __device__ __forceinline__

MARCHE_DEVINL float to_float(float v) { return v; }
MARCHE_DEVINL float to_float(bf16 v) { return __bfloat162float(v); }
MARCHE_DEVINL float to_float(f16 v) { return __half2float(v); }

template <typename T> MARCHE_DEVINL T from_float(float v);
template <> MARCHE_DEVINL float from_float<float>(float v) { return v; }
template <> MARCHE_DEVINL bf16 from_float<bf16>(float v) { return __float2bfloat16_rn(v); }

MARCHE_DEVINL uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&p);
}

// Two floats to packed IEEE fp16, round to nearest even, SATURATING: a magnitude beyond the largest
// finite fp16 value becomes +-65504 instead of infinity (NaN stays NaN).  Every fp16 activation the
// library writes (LayerNorm, attention and GELU outputs in the fp16-operand mode) goes through here.
MARCHE_DEVINL uint32_t pack_f16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// Packed pair in the projections' operand type: bf16 when `bf`, saturating fp16 otherwise.
MARCHE_DEVINL uint32_t pack_a16x2(float lo, float hi, bool bf) { return bf ? pack_bf16x2(lo, hi) : pack_f16x2(lo, hi); }

MARCHE_DEVINL float2 unpack_bf16x2(uint32_t u) {
  __nv_bfloat162 p = *reinterpret_cast<__nv_bfloat162*>(&u);
  return __bfloat1622float2(p);
}

// Programmatic dependent launch: wait for the preceding kernel of the stream (no-op when the
// launch did not opt in), then allow the following kernel to start launching.
MARCHE_DEVINL void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
MARCHE_DEVINL void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
MARCHE_DEVINL void pdl_sync() {
  pdl_wait();
  pdl_launch_dependents();
}

MARCHE_DEVINL float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

MARCHE_DEVINL float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Exact (erf) GELU, the flavour the block uses.
MARCHE_DEVINL float gelu_erf(float x) { return 0.5f * x * (1.0f + erff(x * 0.70710678118654752440f)); }

// GELU for the bf16 tensor-core epilogue: erf by the 5-term rational-exponential formula
// erf(x) = 1 - (a1 t + ... + a5 t^5) exp(-x^2), t = 1/(1 + p x) (absolute error <= 1.5e-7, far
// below the bf16 rounding of the result), about a third of the instructions of erff().
MARCHE_DEVINL float gelu_erf_fast(float x) {
  const float z = fabsf(x) * 0.70710678118654752440f;
  float t;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(fmaf(0.3275911f, z, 1.0f)));
  float poly = fmaf(1.061405429f, t, -1.453152027f);
  poly = fmaf(poly, t, 1.421413741f);
  poly = fmaf(poly, t, -0.284496736f);
  poly = fmaf(poly, t, 0.254829592f);
  float ex;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(ex) : "f"(-z * z * 1.4426950408889634f));
  const float e = poly * t * ex;                      // 1 - erf(z), z >= 0
  const float cdf = x >= 0.f ? 1.0f - 0.5f * e : 0.5f * e;
  return x * cdf;
}

// Stores 4 consecutive outputs of type T starting at a 4-element aligned column.
MARCHE_DEVINL void store4(float* p, float a, float b, float c, float d) {
  *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d);
}
MARCHE_DEVINL void store4(f16* p, float a, float b, float c, float d) {
  uint2 u;
  u.x = pack_f16x2(a, b);
  u.y = pack_f16x2(c, d);
  *reinterpret_cast<uint2*>(p) = u;
}
MARCHE_DEVINL void store4(bf16* p, float a, float b, float c, float d) {
  uint2 u;
  u.x = pack_bf16x2(a, b);
  u.y = pack_bf16x2(c, d);
  *reinterpret_cast<uint2*>(p) = u;
}
