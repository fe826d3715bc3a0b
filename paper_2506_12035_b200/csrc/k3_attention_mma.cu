// K3: attention of the active queries over ALL S cached rows of one block, unmasked
// (Algorithm 1 lines 6-8; equal to plain softmax attention, Eq. 5, by Appendix A once the
// active rows' fresh K, V sit in the cache), with the relevance reduction of Section 4.2
// fused in: per key, the sum over the generating tokens' queries of the softmax weight.
//
// At the small active sets of a cache-aware step the kernel is bound by streaming the
// K/V cache from HBM (about nA flop per byte), so the design goal is to keep TMA loads
// in flight: one CTA per (sample, head) walks 64-key tiles of K and V, which TMA stages
// through a 3-deep shared-memory ring (128-byte swizzle for head_dim 64) straight from
// the token-major cache [2][B][S][D]; a dedicated producer warp issues the loads and the
// consumer warps hand ring slots back through mbarriers (no CTA-wide barrier per tile);
// several CTAs are resident per SM.  QK^T and PV
// run on the tensor cores (mma.sync m16n8k16, bf16 in, fp32 accumulate; each warp owns
// 16 query rows), softmax statistics stay in fp32 registers.  The output rows are written
// in the projections' operand type (fp16 or bf16): they are the A operand of the output projection.
//
// Two flavours:
//   plain    one pass, online softmax (running max / sum, rescaled accumulators);
//   scoring  (only at the scoring block) two passes: first the exact row max and sum
//            over K alone, then K and V again with final probabilities, so that the
//            per-key column sums use exact softmax weights.  Each warp adds the weights
//            of its flagged rows into its own shared-memory column array; the arrays
//            are combined in fixed order, so scores are bit-reproducible (no atomics).
// Every mbarrier wait is bounded and reports through the status word.
#include <cuda.h>

#include "kernels.h"
#include "launch_pdl.h"
#include "attention_common.cuh"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace marche {

namespace {

using namespace att;

// NWARPS consumer warps (16 query rows each) plus one producer warp.
template <int DH, int NWARPS, bool SCORING>
__global__ void __launch_bounds__((NWARPS + 1) * 32, NWARPS == 3 ? 4 : ((NWARPS == 2 && DH == 80) ? 5 : 1))
attention_mma_kernel(const __grid_constant__ CUtensorMap tmap_kv, const __grid_constant__ CUtensorMap tmap_tail,
                     const bf16* __restrict__ q, int ld_q, int n,
                     int S, int H, int B, const uint8_t* __restrict__ is_new, float* __restrict__ score_partial,
                     uint16_t* __restrict__ o, bool o_bf16, int* __restrict__ status) {
  using Cfg = AttCfg<DH>;
  constexpr int QT = NWARPS * 16;
  constexpr int NSTAGE = ring_stages<DH>::N;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const uint32_t bar_base = base + NSTAGE * Cfg::STAGE_BYTES;          // full[NSTAGE] then empty[NSTAGE]
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (NSTAGE + s); };
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + NSTAGE * Cfg::STAGE_BYTES + 16 * NSTAGE);
  float* colsum = reinterpret_cast<float*>(gen + NSTAGE * Cfg::STAGE_BYTES + 64);   // [NWARPS][S], scoring only

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, tg = lane & 3;
  const int b = blockIdx.x / H, h = blockIdx.x - b * H;
  const int D = H * DH;
  const int n_kv = (S + KT - 1) / KT, n_qt = (n + QT - 1) / QT;
  constexpr int PASSES = SCORING ? 2 : 1;
  const int n_loads = n_qt * n_kv * PASSES;
  const float scale_log2 = rsqrtf((float)DH) * 1.4426950408889634f;

  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGE; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), NWARPS);                // one arrival per consumer warp
    }
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
  }
  if (SCORING)
    for (int t = threadIdx.x; t < NWARPS * S; t += (NWARPS + 1) * 32) colsum[t] = 0.f;
  __syncthreads();
  pdl_sync();                                          // set-up above overlaps the previous kernel's tail

  bool ok = true;
  if (warp == NWARPS) {
    // ---------------------------------------------------------------- producer warp (one lane)
    // Fixed load sequence: per q-tile, [K tiles of the statistics pass,] then K+V tiles.
    if (lane == 0) {
      ptx::prefetch_tensormap(&tmap_kv);
      const uint64_t stream_once = ptx::l2_policy_evict_first();
      int i = 0;
      for (; i < n_loads; ++i) {
        const int rem = i % (n_kv * PASSES);
        const int pass = rem / n_kv, kt = rem - pass * n_kv;
        const bool with_v = !SCORING || pass == 1;
        const int s = i % NSTAGE;
        if (!ptx::mbar_wait(empty_bar(s), ((uint32_t)(i / NSTAGE) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        const uint32_t dst = base + s * Cfg::STAGE_BYTES;
        ptx::mbar_expect_tx(full_bar(s), with_v ? Cfg::STAGE_BYTES : Cfg::TILE_BYTES);
        ptx::tma_load_3d_hint(dst, &tmap_kv, h * DH, kt * KT, b, full_bar(s), stream_once);
        if (with_v) ptx::tma_load_3d_hint(dst + Cfg::TILE_BYTES, &tmap_kv, h * DH, kt * KT, B + b, full_bar(s), stream_once);
        if (DH > 64) {                                     // columns 64 .. DH-1 as a second box behind the first
          ptx::tma_load_3d_hint(dst + KT * 128, &tmap_tail, h * DH + 64, kt * KT, b, full_bar(s), stream_once);
          if (with_v)
            ptx::tma_load_3d_hint(dst + Cfg::TILE_BYTES + KT * 128, &tmap_tail, h * DH + 64, kt * KT, B + b, full_bar(s),
                                  stream_once);
        }
      }
      if (!ok) {
        *(volatile int*)status = ST_ATTENTION;
        // let copies already issued land before the CTA's shared memory is released
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
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};   // running max of the RAW logits, sum
    bool flag[2] = {false, false};
    bool warp_active = false, warp_flagged = false;

    for (int i = 0; i < n_loads; ++i) {
      const int qt = i / (n_kv * PASSES);
      const int rem = i - qt * (n_kv * PASSES);
      const int pass = rem / n_kv, kt = rem - pass * n_kv;
      const bool final_pass = !SCORING || pass == 1;
      const int s = i % NSTAGE;

      if (rem == 0) {
        // new q-tile: fetch this warp's 16 query rows as A fragments, reset the statistics
        const int r0 = qt * QT + warp * 16 + g, r1 = r0 + 8;
        warp_active = (qt * QT + warp * 16) < n;
        const bf16* q0 = q + ((size_t)b * n + r0) * ld_q + h * DH;
        const bf16* q1 = q + ((size_t)b * n + r1) * ld_q + h * DH;
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
      if (final_pass && kt == 0) {
#pragma unroll
        for (int j = 0; j < Cfg::ONT; ++j) oacc[j][0] = oacc[j][1] = oacc[j][2] = oacc[j][3] = 0.f;
      }

      if (!ptx::mbar_wait(full_bar(s), (uint32_t)(i / NSTAGE) & 1u, abort_flag)) { ok = false; break; }

      if (warp_active) {
        const uint32_t k_tile = base + s * Cfg::STAGE_BYTES, v_tile = k_tile + Cfg::TILE_BYTES;
        // ---- raw logits of 16 rows x 64 keys
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
            ldsm_x4(k_tile + kv_off<DH>(key, 2 * kk + (mi & 1)), b0, b1, b2, b3);
            mma_bf16(sacc[2 * jp], qf[kk], b0, b1);
            mma_bf16(sacc[2 * jp + 1], qf[kk], b2, b3);
          }
        }
        // ---- mask keys beyond S, row maxima of the raw logits
        const int t_base = kt * KT;
        if (t_base + KT > S) {
#pragma unroll
          for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e)
              if (t_base + 8 * j + 2 * tg + (e & 1) >= S) sacc[j][e] = -INFINITY;
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
            corr[r] = ex2_approx((m_run[r] - m_new) * scale_log2);
            m_run[r] = m_new;
            neg_ms[r] = -m_new * scale_log2;
          }
          // p = 2^(s*c - m*c): one FMA and one ex2 per element
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
          // second pass of the scoring flavour: exact probabilities with the final max and sum
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
              const int t = t_base + 8 * j + 2 * tg;
              if (g == 0) {
                if (t < S) cs[t] += c0;
                if (t + 1 < S) cs[t + 1] += c1;
              }
            }
          }
        }
        // ---- O += P V
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
              ldsm_x4_trans(v_tile + kv_off<DH>(key, jd + (mi >> 1)), b0, b1, b2, b3);
              mma_bf16(oacc[jd], pf, b0, b1);
              mma_bf16(oacc[jd + 1], pf, b2, b3);
            }
          }
        }
      }
      // this warp is done with the stage: release it to the producer
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(empty_bar(s));

      // ---- end of the q-tile's last pass: write the 16 output rows
      if (warp_active && final_pass && kt == n_kv - 1) {
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
    if (!ok && lane == 0) *(volatile int*)status = ST_ATTENTION;
  }

  if (SCORING) {
    __syncthreads();
    if (!*abort_flag) {
      float* dst = score_partial + ((size_t)b * H + h) * S;
      for (int t = threadIdx.x; t < S; t += (NWARPS + 1) * 32) {
        float sum = 0.f;
#pragma unroll
        for (int w = 0; w < NWARPS; ++w) sum += colsum[(size_t)w * S + t];
        dst[t] = sum;
      }
    }
  }
}

template <int DH, int NWARPS, bool SCORING>
cudaError_t launch_att(const CUtensorMap& tm, const CUtensorMap& tail, const bf16* q, int ld_q, int B, int n, int S, int H,
                       const uint8_t* is_new, float* partial, uint16_t* o, bool o_bf16, int* status, cudaStream_t st) {
  constexpr int NSTAGE = ring_stages<DH>::N;
  const size_t smem = NSTAGE * AttCfg<DH>::STAGE_BYTES + 1024 + 64 + (SCORING ? (size_t)NWARPS * S * sizeof(float) : 0);
  static size_t smem_set[kMaxDevices] = {};
  cudaError_t e = ensure_dynamic_smem(attention_mma_kernel<DH, NWARPS, SCORING>, smem, smem_set);
  if (e != cudaSuccess) return e;
  // (Launching one sample's heads as a cluster, to co-schedule the CTAs that read neighbouring
  // 128-byte pieces of the same cache rows, was measured and does not help: 41.0 -> 41-43 us.)
  return launch_pdl(attention_mma_kernel<DH, NWARPS, SCORING>, dim3(B * H), dim3((NWARPS + 1) * 32), smem, st, tm, tail, q, ld_q,
                    n, S, H, B, is_new, partial, o, o_bf16, status);
}

template <int DH>
cudaError_t launch_dh(const CUtensorMap& tm, const CUtensorMap& tail, const bf16* q, int ld_q, int B, int n, int S, int H,
                      const uint8_t* is_new, float* partial, uint16_t* o, bool o_bf16, int* status, cudaStream_t st) {
  const bool sc = is_new != nullptr;
  // 7 consumer warps + the producer warp = 256 threads: two CTAs per SM still fit the register file
  const int nw = n <= 16 ? 1 : (n <= 32 ? 2 : (n <= 48 ? 3 : (n <= 64 ? 4 : 7)));
#define MARCHE_ATT_CASE(NW_)                                                                              \
  if (nw == NW_)                                                                                          \
    return sc ? launch_att<DH, NW_, true>(tm, tail, q, ld_q, B, n, S, H, is_new, partial, o, o_bf16, status, st) \
              : launch_att<DH, NW_, false>(tm, tail, q, ld_q, B, n, S, H, is_new, partial, o, o_bf16, status, st);
  MARCHE_ATT_CASE(1) MARCHE_ATT_CASE(2) MARCHE_ATT_CASE(3) MARCHE_ATT_CASE(4) MARCHE_ATT_CASE(7)
#undef MARCHE_ATT_CASE
  return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_attention_mma(const void* q, int ld_q, int B, int n, int S, int H, int dh,
                                 const void* cache_layer, const uint8_t* is_new, float* score_partial, void* o,
                                 bool o_bf16, int* status, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  if ((dh != 64 && dh != 80) || ld_q % 2 || ((uintptr_t)q & 3) || ((uintptr_t)cache_layer & 15))
    return cudaErrorInvalidValue;
  const int D = H * dh;
  CUtensorMap tm;
  const uint64_t dims[3] = {(uint64_t)D, (uint64_t)S, (uint64_t)2 * B};
  const uint64_t strides[2] = {(uint64_t)D * 2, (uint64_t)S * D * 2};
  const uint32_t box[3] = {64, KT, 1};                   // columns 0-63 of a head: 128-byte rows, swizzled
  if (!tma_make_map_bf16(&tm, cache_layer, 3, dims, strides, box, true)) return cudaErrorInvalidValue;
  if (dh == 64)
    return launch_dh<64>(tm, tm, (const bf16*)q, ld_q, B, n, S, H, is_new, score_partial, (uint16_t*)o, o_bf16, status, st);
  CUtensorMap tail;                                      // columns 64-79: 32-byte rows, 32-byte swizzle
  const uint32_t box_tail[3] = {16, KT, 1};
  if (!tma_make_map_bf16(&tail, cache_layer, 3, dims, strides, box_tail, false, false, true)) return cudaErrorInvalidValue;
  return launch_dh<80>(tm, tail, (const bf16*)q, ld_q, B, n, S, H, is_new, score_partial, (uint16_t*)o, o_bf16, status, st);
}

}  // namespace marche
