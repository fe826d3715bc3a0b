// K3, two-segment flavour: Algorithm 1 lines 6-8 and 11 in the paper's own order.
//
// The active queries attend to two separate key/value segments that are merged by one online
// softmax (Eq. 6-10) without being concatenated first:
//   segment A  the fresh K_A, V_A of the active rows, read in place from the QKV projection's
//              output (row j of the compact [B][n][ld] buffer is token active_idx[b][j]);
//   segment C  the cached K_C, V_C: the token-major cache, with the (stale) rows of the active
//              tokens masked out.
// After the last tile the CTA writes its head's fresh K, V rows into the cache (line 11), so the
// step needs no separate write-back kernel and the attention does not depend on one.
// Same machinery as attention_mma_kernel: producer warp + TMA ring + mbarriers, mma.sync tiles,
// fp32 online softmax, optional exact two-pass scoring with fixed-order column sums.  Tiles of
// segment C whose 64 tokens are all active are skipped (a full step reads segment A only).
#include <cuda.h>

#include "attention_common.cuh"
#include "kernels.h"
#include "launch_pdl.h"
#include "tma_host.h"

namespace marche {

namespace {

using namespace att;


template <int DH, int NWARPS, bool SCORING>
__global__ void __launch_bounds__((NWARPS + 1) * 32)
attention_twoseg_kernel(const __grid_constant__ CUtensorMap tmap_c, const __grid_constant__ CUtensorMap tmap_a,
                        const bf16* __restrict__ qkv, int ld, int k_off, int v_off, int n, int S, int H, int B,
                        const int32_t* __restrict__ active_idx, bf16* __restrict__ cache_layer,
                        const uint8_t* __restrict__ is_new, float* __restrict__ score_partial,
                        uint16_t* __restrict__ o, bool o_bf16, int* __restrict__ status) {
  using Cfg = AttCfg<DH>;
  constexpr int QT = NWARPS * 16;
  constexpr int NTHREADS = (NWARPS + 1) * 32;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const uint32_t bar_base = base + NSTAGE * Cfg::STAGE_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (NSTAGE + s); };
  uint8_t* aux = gen + NSTAGE * Cfg::STAGE_BYTES;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(aux + 16 * NSTAGE);            // 2 ints
  volatile int* n_ctiles = reinterpret_cast<volatile int*>(aux + 16 * NSTAGE + 8);          // 1 int
  unsigned long long* cmask = reinterpret_cast<unsigned long long*>(aux + 64);              // [32] active bits per cache tile
  uint8_t* ctile = aux + 64 + 32 * 8;                                                       // [32] cache tiles to visit
  int32_t* tok = reinterpret_cast<int32_t*>(aux + 64 + 32 * 8 + 32);                        // [n] token of fresh row j
  float* colsum = reinterpret_cast<float*>(aux + 64 + 32 * 8 + 32 + ((n * 4 + 15) & ~15)); // [NWARPS][S], scoring only

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, tg = lane & 3;
  const int b = blockIdx.x / H, h = blockIdx.x - b * H;
  const int D = H * DH;
  const int n_kv = (S + KT - 1) / KT, n_qt = (n + QT - 1) / QT, n_at = (n + KT - 1) / KT;
  constexpr int PASSES = SCORING ? 2 : 1;
  const float scale_log2 = rsqrtf((float)DH) * 1.4426950408889634f;

  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGE; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), NWARPS);
    }
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
  }
  for (int t = threadIdx.x; t < 32; t += NTHREADS) cmask[t] = 0ull;
  if (SCORING)
    for (int t = threadIdx.x; t < NWARPS * S; t += NTHREADS) colsum[t] = 0.f;
  __syncthreads();
  pdl_sync();

  // token of each fresh row; bit t of cmask marks token t as active (excluded from segment C)
  for (int j = threadIdx.x; j < n; j += NTHREADS) {
    const int t = active_idx ? active_idx[(size_t)b * n + j] : j;
    tok[j] = t;
    atomicOr(&cmask[t >> 6], 1ull << (t & 63));
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int c = 0;
    for (int kt = 0; kt < n_kv; ++kt) {
      const int valid = (S - kt * KT) < KT ? (S - kt * KT) : KT;
      const unsigned long long all = valid == 64 ? ~0ull : ((1ull << valid) - 1ull);
      if ((cmask[kt] & all) != all) ctile[c++] = (uint8_t)kt;      // some token of the tile is cached
    }
    *n_ctiles = c;
  }
  __syncthreads();
  const int n_ct = *n_ctiles;
  const int n_t = n_at + n_ct;                     // tiles per pass: fresh tiles, then cache tiles
  const int n_loads = n_qt * n_t * PASSES;

  bool ok = true;
  if (warp == NWARPS) {
    // ---------------------------------------------------------------- producer warp (one lane)
    if (lane == 0) {
      ptx::prefetch_tensormap(&tmap_c);
      ptx::prefetch_tensormap(&tmap_a);
      int i = 0;
      for (; i < n_loads; ++i) {
        const int rem = i % (n_t * PASSES);
        const int pass = rem / n_t, u = rem - pass * n_t;
        const bool with_v = !SCORING || pass == 1;
        const int s = i % NSTAGE;
        if (!ptx::mbar_wait(empty_bar(s), ((uint32_t)(i / NSTAGE) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        const uint32_t dst = base + s * Cfg::STAGE_BYTES;
        ptx::mbar_expect_tx(full_bar(s), with_v ? Cfg::STAGE_BYTES : Cfg::TILE_BYTES);
        if (u < n_at) {
          ptx::tma_load_3d(dst, &tmap_a, k_off + h * DH, u * KT, b, full_bar(s));
          if (with_v) ptx::tma_load_3d(dst + Cfg::TILE_BYTES, &tmap_a, v_off + h * DH, u * KT, b, full_bar(s));
        } else {
          const int kt = ctile[u - n_at];
          ptx::tma_load_3d(dst, &tmap_c, h * DH, kt * KT, b, full_bar(s));
          if (with_v) ptx::tma_load_3d(dst + Cfg::TILE_BYTES, &tmap_c, h * DH, kt * KT, B + b, full_bar(s));
        }
      }
      if (!ok) {
        *(volatile int*)status = ST_ATTENTION_TWOSEG;
        for (int j = 1; j <= NSTAGE && j <= i; ++j) {
          const int i2 = i - j;
          ptx::mbar_wait(full_bar(i2 % NSTAGE), (uint32_t)(i2 / NSTAGE) & 1u, abort_flag + 1, 20000000LL);
        }
      }
    }
  } else {
    // ---------------------------------------------------------------- consumer warps
    uint32_t qf[Cfg::KSTEPS][4];
    float oacc[Cfg::ONT][4];
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    bool flag[2] = {false, false};
    bool warp_active = false, warp_flagged = false;

    for (int i = 0; i < n_loads; ++i) {
      const int qt = i / (n_t * PASSES);
      const int rem = i - qt * (n_t * PASSES);
      const int pass = rem / n_t, u = rem - pass * n_t;
      const bool final_pass = !SCORING || pass == 1;
      const bool fresh = u < n_at;
      const int kt = fresh ? u : (int)ctile[u - n_at];
      const int s = i % NSTAGE;

      if (rem == 0) {
        const int r0 = qt * QT + warp * 16 + g, r1 = r0 + 8;
        warp_active = (qt * QT + warp * 16) < n;
        const bf16* q0 = qkv + ((size_t)b * n + r0) * ld + h * DH;
        const bf16* q1 = qkv + ((size_t)b * n + r1) * ld + h * DH;
#pragma unroll
        for (int kk = 0; kk < Cfg::KSTEPS; ++kk) {
          qf[kk][0] = r0 < n ? *reinterpret_cast<const uint32_t*>(q0 + kk * 16 + 2 * tg) : 0u;
          qf[kk][1] = r1 < n ? *reinterpret_cast<const uint32_t*>(q1 + kk * 16 + 2 * tg) : 0u;
          qf[kk][2] = r0 < n ? *reinterpret_cast<const uint32_t*>(q0 + kk * 16 + 8 + 2 * tg) : 0u;
          qf[kk][3] = r1 < n ? *reinterpret_cast<const uint32_t*>(q1 + kk * 16 + 8 + 2 * tg) : 0u;
        }
        m_run[0] = m_run[1] = -INFINITY;
        l_run[0] = l_run[1] = 0.f;
        if (SCORING) {
          flag[0] = r0 < n && is_new[(size_t)b * n + r0];
          flag[1] = r1 < n && is_new[(size_t)b * n + r1];
          warp_flagged = __any_sync(0xffffffffu, flag[0] || flag[1]);
        }
      }
      if (final_pass && u == 0) {
#pragma unroll
        for (int j = 0; j < Cfg::ONT; ++j) oacc[j][0] = oacc[j][1] = oacc[j][2] = oacc[j][3] = 0.f;
      }

      if (!ptx::mbar_wait(full_bar(s), (uint32_t)(i / NSTAGE) & 1u, abort_flag)) { ok = false; break; }

      if (warp_active) {
        const uint32_t k_tile = base + s * Cfg::STAGE_BYTES, v_tile = k_tile + Cfg::TILE_BYTES;
        float sacc[8][4];
#pragma unroll
        for (int j = 0; j < 8; ++j) sacc[j][0] = sacc[j][1] = sacc[j][2] = sacc[j][3] = 0.f;
#pragma unroll
        for (int kk = 0; kk < Cfg::KSTEPS; ++kk) {
#pragma unroll
          for (int jp = 0; jp < 4; ++jp) {
            const int mi = lane >> 3;
            const int key = 8 * (2 * jp + (mi >> 1)) + (lane & 7);
            uint32_t b0, b1, b2, b3;
            ldsm_x4(k_tile + tile_off<DH>(key, 2 * kk + (mi & 1)), b0, b1, b2, b3);
            mma_bf16(sacc[2 * jp], qf[kk], b0, b1);
            mma_bf16(sacc[2 * jp + 1], qf[kk], b2, b3);
          }
        }
        // ---- keys that do not belong to this segment: rows beyond n (fresh), active or beyond S (cache)
        unsigned long long invalid;
        if (fresh) {
          const int valid = n - kt * KT;
          invalid = valid >= 64 ? 0ull : ~((1ull << valid) - 1ull);
        } else {
          const int valid = S - kt * KT;
          invalid = cmask[kt] | (valid >= 64 ? 0ull : ~((1ull << valid) - 1ull));
        }
        if (invalid) {
#pragma unroll
          for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e)
              if ((invalid >> (8 * j + 2 * tg + (e & 1))) & 1ull) sacc[j][e] = -INFINITY;
        }
        if (!SCORING || pass == 0) {
          float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            mx[0] = fmaxf(mx[0], fmaxf(sacc[j][0], sacc[j][1]));
            mx[1] = fmaxf(mx[1], fmaxf(sacc[j][2], sacc[j][3]));
          }
          float corr[2], neg_ms[2];
#pragma unroll
          for (int r = 0; r < 2; ++r) {
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
            const float m_new = fmaxf(m_run[r], mx[r]);
            // a tile may be entirely masked for a row only together with all earlier ones if the
            // first fresh tile were empty, which cannot happen (n >= 1): m_new is finite here
            corr[r] = ex2_approx((m_run[r] - m_new) * scale_log2);
            m_run[r] = m_new;
            neg_ms[r] = -m_new * scale_log2;
          }
          float rs[2] = {0.f, 0.f};
#pragma unroll
          for (int j = 0; j < 8; ++j) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float p = ex2_approx(fmaf(sacc[j][e], scale_log2, neg_ms[e >> 1]));
              sacc[j][e] = p;
              rs[e >> 1] += p;
            }
          }
#pragma unroll
          for (int r = 0; r < 2; ++r) {
            rs[r] += __shfl_xor_sync(0xffffffffu, rs[r], 1);
            rs[r] += __shfl_xor_sync(0xffffffffu, rs[r], 2);
            l_run[r] = l_run[r] * corr[r] + rs[r];
          }
          if (!SCORING) {
#pragma unroll
            for (int j = 0; j < Cfg::ONT; ++j) {
              oacc[j][0] *= corr[0]; oacc[j][1] *= corr[0];
              oacc[j][2] *= corr[1]; oacc[j][3] *= corr[1];
            }
          }
        } else {
          const float inv0 = 1.0f / l_run[0], inv1 = 1.0f / l_run[1];
          const float nm0 = -m_run[0] * scale_log2, nm1 = -m_run[1] * scale_log2;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            sacc[j][0] = ex2_approx(fmaf(sacc[j][0], scale_log2, nm0)) * inv0;
            sacc[j][1] = ex2_approx(fmaf(sacc[j][1], scale_log2, nm0)) * inv0;
            sacc[j][2] = ex2_approx(fmaf(sacc[j][2], scale_log2, nm1)) * inv1;
            sacc[j][3] = ex2_approx(fmaf(sacc[j][3], scale_log2, nm1)) * inv1;
          }
          if (warp_flagged) {
            float* cs = colsum + (size_t)warp * S;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              float c0 = (flag[0] ? sacc[j][0] : 0.f) + (flag[1] ? sacc[j][2] : 0.f);
              float c1 = (flag[0] ? sacc[j][1] : 0.f) + (flag[1] ? sacc[j][3] : 0.f);
#pragma unroll
              for (int sh = 4; sh < 32; sh <<= 1) {
                c0 += __shfl_xor_sync(0xffffffffu, c0, sh);
                c1 += __shfl_xor_sync(0xffffffffu, c1, sh);
              }
              if (g == 0) {
                const int col = 8 * j + 2 * tg;
                if (!((invalid >> col) & 1ull)) cs[fresh ? tok[kt * KT + col] : kt * KT + col] += c0;
                if (!((invalid >> (col + 1)) & 1ull)) cs[fresh ? tok[kt * KT + col + 1] : kt * KT + col + 1] += c1;
              }
            }
          }
        }
        if (final_pass) {
#pragma unroll
          for (int k2 = 0; k2 < KT / 16; ++k2) {
            uint32_t pf[4];
            pf[0] = pack_bf16x2(sacc[2 * k2][0], sacc[2 * k2][1]);
            pf[1] = pack_bf16x2(sacc[2 * k2][2], sacc[2 * k2][3]);
            pf[2] = pack_bf16x2(sacc[2 * k2 + 1][0], sacc[2 * k2 + 1][1]);
            pf[3] = pack_bf16x2(sacc[2 * k2 + 1][2], sacc[2 * k2 + 1][3]);
#pragma unroll
            for (int jd = 0; jd < Cfg::ONT; jd += 2) {
              const int mi = lane >> 3;
              const int key = 16 * k2 + 8 * (mi & 1) + (lane & 7);
              uint32_t b0, b1, b2, b3;
              ldsm_x4_trans(v_tile + tile_off<DH>(key, jd + (mi >> 1)), b0, b1, b2, b3);
              mma_bf16(oacc[jd], pf, b0, b1);
              mma_bf16(oacc[jd + 1], pf, b2, b3);
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(empty_bar(s));

      if (warp_active && final_pass && u == n_t - 1) {
        const float f0 = SCORING ? 1.0f : 1.0f / l_run[0], f1 = SCORING ? 1.0f : 1.0f / l_run[1];
        const int r0 = qt * QT + warp * 16 + g, r1 = r0 + 8;
        uint16_t* o0 = o + ((size_t)b * n + r0) * D + h * DH + 2 * tg;
        uint16_t* o1 = o + ((size_t)b * n + r1) * D + h * DH + 2 * tg;
#pragma unroll
        for (int j = 0; j < Cfg::ONT; ++j) {
          if (r0 < n) *reinterpret_cast<uint32_t*>(o0 + 8 * j) = pack_a16x2(oacc[j][0] * f0, oacc[j][1] * f0, o_bf16);
          if (r1 < n) *reinterpret_cast<uint32_t*>(o1 + 8 * j) = pack_a16x2(oacc[j][2] * f1, oacc[j][3] * f1, o_bf16);
        }
      }
    }
    if (!ok && lane == 0) *(volatile int*)status = ST_ATTENTION_TWOSEG;
  }

  // ---------------------------------------------------------------- epilogue (all warps)
  __syncthreads();                                   // every TMA read of the cache has landed and been consumed
  if (*abort_flag) return;
  // Algorithm 1 line 11: this head's fresh K, V rows go into the cache (16-byte chunks)
  constexpr int CH = DH / 8;
  const size_t kv_stride = (size_t)B * S * D;
  for (int e = threadIdx.x; e < 2 * n * CH; e += NTHREADS) {
    const int which = e / (n * CH), r = e - which * n * CH;
    const int j = r / CH, c = r - j * CH;
    const uint4 v = *reinterpret_cast<const uint4*>(qkv + ((size_t)b * n + j) * ld + (which ? v_off : k_off) + h * DH + c * 8);
    *reinterpret_cast<uint4*>(cache_layer + which * kv_stride + ((size_t)b * S + tok[j]) * D + h * DH + c * 8) = v;
  }
  if (SCORING) {
    float* dst = score_partial + ((size_t)b * H + h) * S;
    for (int t = threadIdx.x; t < S; t += NTHREADS) {
      float sum = 0.f;
#pragma unroll
      for (int w = 0; w < NWARPS; ++w) sum += colsum[(size_t)w * S + t];
      dst[t] = sum;
    }
  }
}

template <int DH, int NWARPS, bool SCORING>
cudaError_t launch_ts(const CUtensorMap& tc, const CUtensorMap& ta, const bf16* qkv, int ld, int k_off, int v_off,
                      int B, int n, int S, int H, const int32_t* idx, bf16* cache, const uint8_t* is_new,
                      float* partial, uint16_t* o, bool o_bf16, int* status, cudaStream_t st) {
  const size_t smem = NSTAGE * AttCfg<DH>::STAGE_BYTES + 1024 + 64 + 32 * 8 + 32 + (((size_t)n * 4 + 15) & ~(size_t)15) +
                      (SCORING ? (size_t)NWARPS * S * sizeof(float) : 0);
  static size_t smem_set[kMaxDevices] = {};
  cudaError_t e = ensure_dynamic_smem(attention_twoseg_kernel<DH, NWARPS, SCORING>, smem, smem_set);
  if (e != cudaSuccess) return e;
  return launch_pdl(attention_twoseg_kernel<DH, NWARPS, SCORING>, dim3(B * H), dim3((NWARPS + 1) * 32), smem, st, tc, ta,
                    qkv, ld, k_off, v_off, n, S, H, B, idx, cache, is_new, partial, o, o_bf16, status);
}

template <int DH>
cudaError_t launch_ts_dh(const CUtensorMap& tc, const CUtensorMap& ta, const bf16* qkv, int ld, int k_off, int v_off,
                         int B, int n, int S, int H, const int32_t* idx, bf16* cache, const uint8_t* is_new,
                         float* partial, uint16_t* o, bool o_bf16, int* status, cudaStream_t st) {
  const bool sc = is_new != nullptr;
  const int nw = n <= 16 ? 1 : (n <= 32 ? 2 : (n <= 48 ? 3 : (n <= 64 ? 4 : 7)));
#define MARCHE_TS_CASE(NW_)                                                                                          \
  if (nw == NW_)                                                                                                     \
    return sc ? launch_ts<DH, NW_, true>(tc, ta, qkv, ld, k_off, v_off, B, n, S, H, idx, cache, is_new, partial, o,   \
                                         o_bf16, status, st)                                                         \
              : launch_ts<DH, NW_, false>(tc, ta, qkv, ld, k_off, v_off, B, n, S, H, idx, cache, is_new, partial, o,  \
                                          o_bf16, status, st);
  MARCHE_TS_CASE(1) MARCHE_TS_CASE(2) MARCHE_TS_CASE(3) MARCHE_TS_CASE(4) MARCHE_TS_CASE(7)
#undef MARCHE_TS_CASE
  return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_attention_twoseg(const void* qkv, int ld, int k_off, int v_off, int B, int n, int S, int H, int dh,
                                    const int32_t* active_idx, void* cache_layer, const uint8_t* is_new,
                                    float* score_partial, void* o, bool o_bf16, int* status, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  if ((dh != 64 && dh != 80) || ld % 8 || k_off % 8 || v_off % 8 || ((uintptr_t)qkv & 15) ||
      ((uintptr_t)cache_layer & 15) || S > 2048 || n > S)
    return cudaErrorInvalidValue;
  const int D = H * dh;
  CUtensorMap tc, ta;
  {
    const uint64_t dims[3] = {(uint64_t)D, (uint64_t)S, (uint64_t)2 * B};
    const uint64_t strides[2] = {(uint64_t)D * 2, (uint64_t)S * D * 2};
    const uint32_t box[3] = {(uint32_t)dh, KT, 1};
    if (!tma_make_map_bf16(&tc, cache_layer, 3, dims, strides, box, dh == 64)) return cudaErrorInvalidValue;
  }
  {
    const uint64_t dims[3] = {(uint64_t)ld, (uint64_t)n, (uint64_t)B};
    const uint64_t strides[2] = {(uint64_t)ld * 2, (uint64_t)n * ld * 2};
    const uint32_t box[3] = {(uint32_t)dh, KT, 1};
    if (!tma_make_map_bf16(&ta, qkv, 3, dims, strides, box, dh == 64)) return cudaErrorInvalidValue;
  }
  if (dh == 64)
    return launch_ts_dh<64>(tc, ta, (const bf16*)qkv, ld, k_off, v_off, B, n, S, H, active_idx, (bf16*)cache_layer, is_new,
                            score_partial, (uint16_t*)o, o_bf16, status, st);
  return launch_ts_dh<80>(tc, ta, (const bf16*)qkv, ld, k_off, v_off, B, n, S, H, active_idx, (bf16*)cache_layer, is_new,
                          score_partial, (uint16_t*)o, o_bf16, status, st);
}

}  // namespace marche
