// K3 for very small active sets (up to 32 query rows per sample, no relevance scores): the plain flavour of
// the mma.sync attention kernel (Algorithm 1 lines 6-8 == Eq. 5 by Appendix A, online softmax of Eq. 6-10)
// as a PERSISTENT kernel.
//
// With one or two consumer warps a CTA's arithmetic is short and the launch is bound by how well the K/V stream
// from HBM is kept going; with one CTA per (sample, head) item the stream of an SM thins out every time a CTA
// retires and its successor starts (five 64-key tiles per item at S = 320).  Here as many CTAs as are resident at
// once take equal shares of the items; the producer warp runs ahead across items, so the first tiles of the next
// item, and its query rows (by TMA, into shared memory; fragments by ldmatrix), are in flight while the consumer
// warps finish the current one: 9 % faster than one CTA per item at 4-32 rows (S 320), 3 % slower with three
// consumer warps, which is why the three-warp and larger variants stay with one CTA per item.
// The tile arithmetic is that of attention_mma_kernel; every mbarrier wait is bounded and reports through the
// status word.
#include <cuda.h>

#include "kernels.h"
#include "launch_pdl.h"
#include "attention_common.cuh"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace marche {

namespace {

using namespace att;

// Shared-memory bytes set aside for a unit's query rows (whole kilobytes: the barriers follow).
template <int DH, int NWARPS> struct QRegion { static constexpr int BYTES = (NWARPS * 16 * AttCfg<DH>::ROWB + 1023) & ~1023; };

// NWARPS consumer warps (16 query rows each) plus one producer warp.
template <int DH, int NWARPS>
__global__ void __launch_bounds__((NWARPS + 1) * 32, (NWARPS == 2 && DH == 80) ? 5 : 1)
attention_mma_persist_kernel(const __grid_constant__ CUtensorMap tmap_kv, const __grid_constant__ CUtensorMap tmap_tail,
                             const __grid_constant__ CUtensorMap tmap_q, int n, int S, int H, int B,
                             uint16_t* __restrict__ o, bool o_bf16, int* __restrict__ status) {
  using Cfg = AttCfg<DH>;
  constexpr int QT = NWARPS * 16;
  constexpr int NSTAGE = ring_stages<DH>::N;
  constexpr int Q_BYTES = QT * Cfg::ROWB, Q_REGION = QRegion<DH, NWARPS>::BYTES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  const uint32_t q_tile = base + NSTAGE * Cfg::STAGE_BYTES;            // the unit's query rows, written by TMA
  const uint32_t bar_base = q_tile + Q_REGION;                         // full[NSTAGE], empty[NSTAGE], q_full, q_empty
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (NSTAGE + s); };
  const uint32_t q_full = bar_base + 8u * (2 * NSTAGE), q_empty = q_full + 8u;
  volatile int* abort_flag =
      reinterpret_cast<volatile int*>(gen + NSTAGE * Cfg::STAGE_BYTES + Q_REGION + 8 * (2 * NSTAGE + 2));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, tg = lane & 3;
  const int D = H * DH;
  const int n_kv = (S + KT - 1) / KT, n_qt = (n + QT - 1) / QT;
  // the CTA's items: blockIdx.x, blockIdx.x + gridDim.x, ...; a unit = one query tile of one item
  const int n_items = B * H;
  const int items_cta = (n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
  const int n_units = items_cta * n_qt;
  const float scale_log2 = rsqrtf((float)DH) * 1.4426950408889634f;

  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGE; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), NWARPS);                // one arrival per consumer warp
    }
    ptx::mbar_init(q_full, 1);
    ptx::mbar_init(q_empty, NWARPS);
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
  }
  __syncthreads();
  pdl_sync();                                          // set-up above overlaps the previous kernel's tail

  bool ok = true;
  if (warp == NWARPS) {
    // ---------------------------------------------------------------- producer warp (one lane)
    // Fixed load sequence: per unit the query tile, then its K+V tiles.  The ring runs ahead across units and items.
    if (lane == 0) {
      ptx::prefetch_tensormap(&tmap_kv);
      ptx::prefetch_tensormap(&tmap_q);
      const uint64_t stream_once = ptx::l2_policy_evict_first();
      int i = 0, q_loads = 0;                              // ring loads / query-tile loads so far
      for (int u = 0; u < n_units && ok; ++u) {
        const int item = (int)blockIdx.x + (u / n_qt) * (int)gridDim.x, qt = u % n_qt;
        const int b = item / H, h = item - b * H;
        if (!ptx::mbar_wait(q_empty, ((uint32_t)u & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        ptx::mbar_expect_tx(q_full, Q_BYTES);
        ptx::tma_load_3d(q_tile, &tmap_q, h * DH, qt * QT, b, q_full);
        ++q_loads;
        for (int kt = 0; kt < n_kv; ++kt, ++i) {
          const int s = i % NSTAGE;
          if (!ptx::mbar_wait(empty_bar(s), ((uint32_t)(i / NSTAGE) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t dst = base + s * Cfg::STAGE_BYTES;
          ptx::mbar_expect_tx(full_bar(s), Cfg::STAGE_BYTES);
          ptx::tma_load_3d_hint(dst, &tmap_kv, h * DH, kt * KT, b, full_bar(s), stream_once);
          ptx::tma_load_3d_hint(dst + Cfg::TILE_BYTES, &tmap_kv, h * DH, kt * KT, B + b, full_bar(s), stream_once);
          if (DH > 64) {                                   // columns 64 .. DH-1 as a second box behind the first
            ptx::tma_load_3d_hint(dst + KT * 128, &tmap_tail, h * DH + 64, kt * KT, b, full_bar(s), stream_once);
            ptx::tma_load_3d_hint(dst + Cfg::TILE_BYTES + KT * 128, &tmap_tail, h * DH + 64, kt * KT, B + b, full_bar(s),
                                  stream_once);
          }
        }
      }
      if (!ok) {
        *(volatile int*)status = ST_ATTENTION;
        // let copies already issued land before the CTA's shared memory is released
        for (int j = 1; j <= NSTAGE && j <= i; ++j) {
          const int i2 = i - j;
          ptx::mbar_wait(full_bar(i2 % NSTAGE), (uint32_t)(i2 / NSTAGE) & 1u, abort_flag + 1, 20000000LL);
        }
        if (q_loads > 0) ptx::mbar_wait(q_full, (uint32_t)(q_loads - 1) & 1u, abort_flag + 1, 20000000LL);
      }
    }
  } else {
    // ---------------------------------------------------------------- consumer warps
    uint32_t qf[Cfg::KSTEPS][4];
    float oacc[Cfg::ONT][4];
    int s = 0;                                             // ring slot of the next tile, and its phase
    uint32_t ring_phase = 0;
    for (int u = 0; u < n_units && ok; ++u) {
      const int item = (int)blockIdx.x + (u / n_qt) * (int)gridDim.x, qt = u % n_qt;
      const int b = item / H, h = item - b * H;
      // this warp's 16 query rows as A fragments (rows beyond n arrive as zeros)
      const bool warp_active = (qt * QT + warp * 16) < n;
      if (!ptx::mbar_wait(q_full, (uint32_t)u & 1u, abort_flag)) { ok = false; break; }
#pragma unroll
      for (int kk = 0; kk < Cfg::KSTEPS; ++kk)
        ldsm_x4(q_tile + tile_off<DH>(warp * 16 + (lane & 15), 2 * kk + (lane >> 4)), qf[kk][0], qf[kk][1], qf[kk][2],
                qf[kk][3]);
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(q_empty);            // the producer may fetch the next unit's rows
      float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};   // running max of the RAW logits, sum
#pragma unroll
      for (int j = 0; j < Cfg::ONT; ++j) oacc[j][0] = oacc[j][1] = oacc[j][2] = oacc[j][3] = 0.f;

      for (int kt = 0; kt < n_kv; ++kt) {
        if (!ptx::mbar_wait(full_bar(s), ring_phase, abort_flag)) { ok = false; break; }
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
#pragma unroll
          for (int j = 0; j < Cfg::ONT; ++j) {
            oacc[j][0] *= corr[0]; oacc[j][1] *= corr[0];
            oacc[j][2] *= corr[1]; oacc[j][3] *= corr[1];
          }
          // ---- O += P V
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
        // this warp is done with the stage: release it to the producer
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(empty_bar(s));
        if (++s == NSTAGE) { s = 0; ring_phase ^= 1u; }
      }
      if (!ok) break;
      // ---- end of the unit: write the 16 output rows
      if (warp_active) {
        const float f0 = 1.0f / l_run[0], f1 = 1.0f / l_run[1];
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
}

template <int DH, int NWARPS>
cudaError_t launch_persist(const CUtensorMap& tm, const CUtensorMap& tail, const void* q, int ld_q, int B, int n, int S,
                           int H, uint16_t* o, bool o_bf16, int* status, cudaStream_t st) {
  constexpr int NSTAGE = ring_stages<DH>::N;
  const size_t smem = NSTAGE * AttCfg<DH>::STAGE_BYTES + QRegion<DH, NWARPS>::BYTES + 1024 + 128;
  static size_t smem_set[kMaxDevices] = {};
  cudaError_t e = ensure_dynamic_smem(attention_mma_persist_kernel<DH, NWARPS>, smem, smem_set);
  if (e != cudaSuccess) return e;
  CUtensorMap tq;
  {
    const uint64_t dims[3] = {(uint64_t)ld_q, (uint64_t)n, (uint64_t)B};
    const uint64_t strides[2] = {(uint64_t)ld_q * 2, (uint64_t)n * ld_q * 2};
    const uint32_t box[3] = {(uint32_t)DH, (uint32_t)(NWARPS * 16), 1};
    if (!tma_make_map_bf16(&tq, q, 3, dims, strides, box, DH == 64)) return cudaErrorInvalidValue;
  }
  // as many CTAs as are resident at once, each with an equal share of the items (ceil(items / resident) per CTA)
  static int per_sm[kMaxDevices] = {};
  int dev = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (!per_sm[dev]) {
    int occ = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, attention_mma_persist_kernel<DH, NWARPS>, (NWARPS + 1) * 32,
                                                      smem);
    if (e != cudaSuccess) return e;
    per_sm[dev] = occ > 0 ? occ : 1;
  }
  const int resident = per_sm[dev] * device_sm_count();
  int grid = B * H;
  if (grid > resident) {
    const int per_cta = (grid + resident - 1) / resident;
    grid = (grid + per_cta - 1) / per_cta;
  }
  return launch_pdl(attention_mma_persist_kernel<DH, NWARPS>, dim3(grid), dim3((NWARPS + 1) * 32), smem, st, tm, tail, tq,
                    n, S, H, B, o, o_bf16, status);
}

}  // namespace

cudaError_t launch_attention_mma_persist(const void* q, int ld_q, int B, int n, int S, int H, int dh,
                                         const void* cache_layer, void* o, bool o_bf16, int* status, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  if ((dh != 64 && dh != 80) || n > 32 || ld_q % 8 || ((uintptr_t)q & 15) || ((uintptr_t)cache_layer & 15))
    return cudaErrorInvalidValue;
  const int D = H * dh;
  CUtensorMap tm, tail;
  const uint64_t dims[3] = {(uint64_t)D, (uint64_t)S, (uint64_t)2 * B};
  const uint64_t strides[2] = {(uint64_t)D * 2, (uint64_t)S * D * 2};
  const uint32_t box[3] = {64, KT, 1};                   // columns 0-63 of a head: 128-byte rows, swizzled
  if (!tma_make_map_bf16(&tm, cache_layer, 3, dims, strides, box, true)) return cudaErrorInvalidValue;
  tail = tm;
  if (dh == 80) {                                        // columns 64-79: 32-byte rows, 32-byte swizzle
    const uint32_t box_tail[3] = {16, KT, 1};
    if (!tma_make_map_bf16(&tail, cache_layer, 3, dims, strides, box_tail, false, false, true)) return cudaErrorInvalidValue;
  }
  uint16_t* op = (uint16_t*)o;
  if (dh == 64)
    return n <= 16 ? launch_persist<64, 1>(tm, tail, q, ld_q, B, n, S, H, op, o_bf16, status, st)
                   : launch_persist<64, 2>(tm, tail, q, ld_q, B, n, S, H, op, o_bf16, status, st);
  return n <= 16 ? launch_persist<80, 1>(tm, tail, q, ld_q, B, n, S, H, op, o_bf16, status, st)
                 : launch_persist<80, 2>(tm, tail, q, ld_q, B, n, S, H, op, o_bf16, status, st);
}

}  // namespace marche
