// Pieces shared by the tensor-core attention kernels: tile geometry, ldmatrix / mma.sync wrappers,
// the shared-memory addressing of TMA-written K/V tiles.
#pragma once

#include "sm100_ptx.cuh"

namespace marche {
namespace att {

constexpr int KT = 64;        // keys per tile
constexpr int NSTAGE = 3;
enum { ST_ATTENTION = 0x21, ST_ATTENTION_TWOSEG = 0x22 };

template <int DH> struct AttCfg {
  static constexpr bool SW = (DH == 64);                 // 128-byte rows: TMA swizzle, conflict-free ldmatrix
  static constexpr int ROWB = DH * 2;
  static constexpr int TILE_BYTES = KT * ROWB;
  static constexpr int STAGE_BYTES = 2 * TILE_BYTES;     // K tile then V tile
  static constexpr int KSTEPS = DH / 16;                 // k16 steps of QK^T
  static constexpr int ONT = DH / 8;                     // n8 tiles of the output
};

MARCHE_DEVINL void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
MARCHE_DEVINL void ldsm_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
MARCHE_DEVINL void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Byte offset of 16-byte chunk c of row r inside a K or V tile.
template <int DH> MARCHE_DEVINL uint32_t tile_off(int r, int c) {
  if (AttCfg<DH>::SW) return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4));
  return (uint32_t)(r * AttCfg<DH>::ROWB + (c << 4));
}

// Ring depth of the mma.sync kernels (plain and persistent): three 16 KB stages at head_dim 64; two 20 KB stages
// at head_dim 80, where a third would cost the fourth resident CTA per SM.
template <int DH> struct ring_stages { static constexpr int N = DH == 64 ? 3 : 2; };

// Byte offset of 16-byte chunk c of key row r inside a K or V tile of those kernels.  head_dim 64: rows of 128
// bytes under TMA's 128-byte swizzle.  head_dim 80: the tile arrives as two boxes, columns 0-63 (same layout)
// and columns 64-79 behind them as rows of 32 bytes under the 32-byte swizzle, so that every ldmatrix phase
// (8 rows x 16 bytes) touches all 32 banks once; packed 160-byte rows would make each phase a 2-way conflict,
// and with two or three warps per CTA reading every tile that is what the kernel was bound by.
template <int DH> MARCHE_DEVINL uint32_t kv_off(int r, int c) {
  if (DH == 64 || c < 8) return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4));
  return (uint32_t)(KT * 128 + r * 32 + (((c - 8) ^ ((r >> 2) & 1)) << 4));
}

MARCHE_DEVINL float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

}  // namespace att
}  // namespace marche
