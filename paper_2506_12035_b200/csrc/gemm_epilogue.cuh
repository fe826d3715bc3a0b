// Epilogue of the tcgen05 GEMM kernels.  One warp owns 32 accumulator rows (TMEM lanes);
// it converts 128-byte-wide row pieces (32 fp32 or 64 bf16 output columns), writes them into
// its private 4 KB staging box in shared memory using the TMA 128-byte swizzle (conflict-free:
// lane = row), and one lane hands the box to the TMA engine, which writes full 128-byte lines
// to global memory (rows beyond M are clipped by the tensor map).
//   EPI 0: out bf16 = acc + bias
//   EPI 1: out fp32 += acc + bias   -- TMA reduce-add in L2, no read in the SM, one add per element
//   EPI 2: out = GELU_erf(acc + bias) in the operand type, fp16 (saturating) or bf16 (feeds the next
//          projection as its A operand)
//   EPI 4: as EPI 0 for the q columns; the K and V columns go straight into scattered rows of the
//          K/V cache (epilogue_box_scatter), so no separate write-back launch is needed
#pragma once

#include "kernels.h"
#include "sm100_ptx.cuh"

namespace marche {

// Columns covered per call: 32 (EPI 1) or 64 (EPI 0, 2), starting at TMEM column t_col / output
// column `col`.  stage = this warp's 4 KB box (1024-byte aligned shared address).  bias_col may be
// nullptr for EPI 1 (a partial sum of a split K range whose bias another piece adds).
template <int EPI>
MARCHE_DEVINL void epilogue_box(uint32_t t_addr, const float* __restrict__ bias_col, const CUtensorMap* out_map,
                                int col, int row0, uint32_t stage, int lane, bool a_bf16) {
  // the previous box of this warp must have been read out of shared memory
  if (lane == 0) ptx::bulk_wait_read_all();
  __syncwarp();
  const uint32_t row_base = stage + (uint32_t)lane * 128u;
  const float4* b4 = reinterpret_cast<const float4*>(bias_col);
  if (EPI == 1) {
    uint32_t r[32];
    ptx::tmem_ld_32x32(t_addr, r);
    ptx::tmem_ld_wait();
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float4 bv = bias_col ? __ldg(b4 + j) : make_float4(0.f, 0.f, 0.f, 0.f);
      const uint32_t dst = row_base + (uint32_t)((j ^ (lane & 7)) << 4);
      asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(__uint_as_float(r[4 * j + 0]) + bv.x),
                   "f"(__uint_as_float(r[4 * j + 1]) + bv.y), "f"(__uint_as_float(r[4 * j + 2]) + bv.z),
                   "f"(__uint_as_float(r[4 * j + 3]) + bv.w) : "memory");
    }
  } else {
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      uint32_t r[32];
      ptx::tmem_ld_32x32(t_addr + (uint32_t)(hh * 32), r);
      ptx::tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float4 b0 = __ldg(b4 + hh * 8 + 2 * j), b1 = __ldg(b4 + hh * 8 + 2 * j + 1);
        float v0 = __uint_as_float(r[8 * j + 0]) + b0.x, v1 = __uint_as_float(r[8 * j + 1]) + b0.y;
        float v2 = __uint_as_float(r[8 * j + 2]) + b0.z, v3 = __uint_as_float(r[8 * j + 3]) + b0.w;
        float v4 = __uint_as_float(r[8 * j + 4]) + b1.x, v5 = __uint_as_float(r[8 * j + 5]) + b1.y;
        float v6 = __uint_as_float(r[8 * j + 6]) + b1.z, v7 = __uint_as_float(r[8 * j + 7]) + b1.w;
        if (EPI == 2) {
          gelu_erf_pair(v0, v1); gelu_erf_pair(v2, v3); gelu_erf_pair(v4, v5); gelu_erf_pair(v6, v7);
        }
        const uint32_t dst = row_base + (uint32_t)(((hh * 4 + j) ^ (lane & 7)) << 4);
        uint32_t p0, p1, p2, p3;
        if (EPI == 2) { p0 = pack_a16x2(v0, v1, a_bf16); p1 = pack_a16x2(v2, v3, a_bf16); p2 = pack_a16x2(v4, v5, a_bf16); p3 = pack_a16x2(v6, v7, a_bf16); }
        else { p0 = pack_bf16x2(v0, v1); p1 = pack_bf16x2(v2, v3); p2 = pack_bf16x2(v4, v5); p3 = pack_bf16x2(v6, v7); }
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(p0), "r"(p1), "r"(p2), "r"(p3) : "memory");
      }
    }
  }
  ptx::fence_proxy_async();            // generic-proxy writes -> visible to the TMA engine
  __syncwarp();
  if (lane == 0) {
    if (EPI == 1) ptx::tma_reduce_add_2d(out_map, col, row0, stage);
    else ptx::tma_store_2d(out_map, col, row0, stage);
    ptx::bulk_commit();
  }
}

// 64 bf16 columns of 32 accumulator rows, written straight into scattered cache rows.  The values
// are staged through the warp's swizzled 4 KB box exactly as for the TMA store; then every quarter
// warp copies one whole 128-byte row piece per instruction (lane l: chunk l % 8 of row l / 8 + 4 i), so
// each global store instruction of the warp writes four full 128-byte lines.  dst_elem = element
// offset of this lane's row in the cache plus the column of this box, or -1 for a row beyond M.
MARCHE_DEVINL void epilogue_box_scatter(uint32_t t_addr, const float* __restrict__ bias_col, bf16* cache, int dst_elem,
                                        uint32_t stage, int lane) {
  if (lane == 0) ptx::bulk_wait_read_all();            // an earlier TMA store of this warp may still read the box
  __syncwarp();
  const uint32_t row_base = stage + (uint32_t)lane * 128u;
  const float4* b4 = reinterpret_cast<const float4*>(bias_col);
#pragma unroll
  for (int hh = 0; hh < 2; ++hh) {
    uint32_t r[32];
    ptx::tmem_ld_32x32(t_addr + (uint32_t)(hh * 32), r);
    ptx::tmem_ld_wait();
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float4 b0 = __ldg(b4 + hh * 8 + 2 * j), b1 = __ldg(b4 + hh * 8 + 2 * j + 1);
      const uint32_t p0 = pack_bf16x2(__uint_as_float(r[8 * j + 0]) + b0.x, __uint_as_float(r[8 * j + 1]) + b0.y);
      const uint32_t p1 = pack_bf16x2(__uint_as_float(r[8 * j + 2]) + b0.z, __uint_as_float(r[8 * j + 3]) + b0.w);
      const uint32_t p2 = pack_bf16x2(__uint_as_float(r[8 * j + 4]) + b1.x, __uint_as_float(r[8 * j + 5]) + b1.y);
      const uint32_t p3 = pack_bf16x2(__uint_as_float(r[8 * j + 6]) + b1.z, __uint_as_float(r[8 * j + 7]) + b1.w);
      const uint32_t dst = row_base + (uint32_t)(((hh * 4 + j) ^ (lane & 7)) << 4);
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(p0), "r"(p1), "r"(p2), "r"(p3) : "memory");
    }
  }
  __syncwarp();
  const int chunk = lane & 7;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = (lane >> 3) + 4 * i;
    const int dst = __shfl_sync(0xffffffffu, dst_elem, row);
    uint32_t v0, v1, v2, v3;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v0), "=r"(v1), "=r"(v2), "=r"(v3)
                 : "r"(stage + (uint32_t)row * 128u + (uint32_t)((chunk ^ (row & 7)) << 4)) : "memory");
    if (dst >= 0) *reinterpret_cast<uint4*>(cache + dst + chunk * 8) = make_uint4(v0, v1, v2, v3);
  }
  __syncwarp();                                         // the box may be refilled
}

template <int EPI> struct EpiCols { static constexpr int value = (EPI == 1) ? 32 : 64; };

}  // namespace marche
