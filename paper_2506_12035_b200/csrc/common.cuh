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

// GELU of two values at once for the tensor-core epilogue, without the special-function unit (which, at a
// quarter of the FP32 rate, was what the fc1 epilogue waited for): GELU(x) = x Phi(x) with
// Phi(x) = sat(0.5 + x R(x^2)), R a degree-8 polynomial fitted to erf(x / sqrt 2) / (2 x) on |x| <= 3 sqrt 2.
// Beyond that range x R(x^2) keeps growing in magnitude (positive leading coefficient, checked numerically: it
// never comes back below 0.49999), so the saturating FMA clamps Phi to 0 or 1 there, infinities included.  The
// polynomial runs for both values in packed fp32-pair instructions.  Error: <= 1.2e-5 in Phi, <= 4.8e-5 absolute
// in the result, a tenth of the 16-bit rounding it is followed by.
MARCHE_DEVINL void gelu_erf_pair(float& a, float& b) {
  float ra, rb;
  asm("{\n"
      ".reg .b64 x, u, acc, k;\n"
      "mov.b64 x, {%2, %3};\n"
      "mul.f32x2 u, x, x;\n"
      "mov.b64 acc, {%4, %4};\n"
      "mov.b64 k, {%5, %5};\n fma.rn.f32x2 acc, acc, u, k;\n"
      "mov.b64 k, {%6, %6};\n fma.rn.f32x2 acc, acc, u, k;\n"
      "mov.b64 k, {%7, %7};\n fma.rn.f32x2 acc, acc, u, k;\n"
      "mov.b64 k, {%8, %8};\n fma.rn.f32x2 acc, acc, u, k;\n"
      "mov.b64 k, {%9, %9};\n fma.rn.f32x2 acc, acc, u, k;\n"
      "mov.b64 k, {%10, %10};\n fma.rn.f32x2 acc, acc, u, k;\n"
      "mov.b64 k, {%11, %11};\n fma.rn.f32x2 acc, acc, u, k;\n"
      "mov.b64 k, {%12, %12};\n fma.rn.f32x2 acc, acc, u, k;\n"
      "mov.b64 {%0, %1}, acc;\n"
      "}\n"
      : "=f"(ra), "=f"(rb)
      : "f"(a), "f"(b), "f"(0.5f * 1.125353213e-10f), "f"(0.5f * -1.074373479e-08f), "f"(0.5f * 4.536591405e-07f),
        "f"(0.5f * -1.129242810e-05f), "f"(0.5f * 1.871812274e-04f), "f"(0.5f * -2.218800364e-03f),
        "f"(0.5f * 1.963623799e-02f), "f"(0.5f * -1.326938421e-01f), "f"(0.5f * 7.978062630e-01f));
  float pa, pb;
  asm("fma.rn.sat.f32 %0, %1, %2, 0f3F000000;" : "=f"(pa) : "f"(a), "f"(ra));
  asm("fma.rn.sat.f32 %0, %1, %2, 0f3F000000;" : "=f"(pb) : "f"(b), "f"(rb));
  a *= pa;
  b *= pb;
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
