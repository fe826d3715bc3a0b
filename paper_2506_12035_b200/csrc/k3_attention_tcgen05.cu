// K3 on the 5th-generation tensor cores (head_dim 64): attention of the active queries over all
// S cached rows of one block (Algorithm 1 lines 6-8 == Eq. 5 by Appendix A) with the relevance
// column sums of Section 4.2.
//
// One CTA per (sample, head), 128 query rows per q-tile (rows beyond n are zero-filled by TMA and
// never stored).  Roles:
//   warp 0     TMA producer: Q tile once per q-tile; 64-key K (and, in pass 2, V) tiles through a
//              3-deep ring, straight from the token-major cache
//   warp 1     issues tcgen05.mma: S = Q K^T (M128 x N64 x K64, fp32 in TMEM, double-buffered) and
//              O += P V (M128 x N64 x K64; P from shared memory, V as an MN-major operand)
//   warps 2-5  softmax: one thread per query row reads its S row from TMEM (tcgen05.ld); no
//              cross-lane reductions are needed for the row statistics
// Softmax is exact two-pass: pass 1 streams K only and takes the row maxima, pass 2 streams K and V,
// forms p = 2^((s - m)/sqrt(d) log2 e) with the final maximum, accumulates the row sums in registers
// and O in TMEM, so O is never rescaled; the epilogue divides by the row sum.  The second reading
// of K comes from L2.  With scoring on, each softmax warp reduces the weights of its flagged rows
// per key with a 62-shuffle butterfly and adds them to its own shared-memory column array; the four
// arrays are combined in fixed order (bit-reproducible).
// All mbarrier waits are bounded and report through the status word.
#include <cuda.h>

#include "kernels.h"
#include "launch_pdl.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace marche {

namespace {

constexpr int DH = 64;
constexpr int QT = 128;                    // query rows per tile
constexpr int KT = 64;                     // keys per tile
constexpr int NSTAGE = 3;
constexpr int TILE_BYTES = KT * DH * 2;    // 8 KB (K or V tile)
constexpr int STAGE_BYTES = 2 * TILE_BYTES;
constexpr int Q_BYTES = QT * DH * 2;       // 16 KB
constexpr int P_BYTES = QT * KT * 2;       // 16 KB
constexpr int kThreads = 192;
constexpr int TMEM_COLS = 256;             // S0 0..63, S1 64..127, O 128..191
enum { ST_ATT_TC = 0x41 };

// smem layout (from a 1024-byte aligned base)
constexpr int OFF_Q = 0;
constexpr int OFF_KV = OFF_Q + Q_BYTES;
constexpr int OFF_P = OFF_KV + NSTAGE * STAGE_BYTES;
constexpr int OFF_BAR = OFF_P + 2 * P_BYTES;
// barriers (8 bytes each)
enum { B_KV_FULL = 0, B_KV_EMPTY = NSTAGE, B_S_FULL = 2 * NSTAGE, B_S_EMPTY = 2 * NSTAGE + 2, B_P_FULL = 2 * NSTAGE + 4,
       B_P_EMPTY = 2 * NSTAGE + 6, B_Q_FULL = 2 * NSTAGE + 8, B_Q_EMPTY = 2 * NSTAGE + 9, B_O_FULL = 2 * NSTAGE + 10,
       B_O_EMPTY = 2 * NSTAGE + 11, N_BARS = 2 * NSTAGE + 12 };
constexpr int OFF_MISC = OFF_BAR + 8 * N_BARS;       // tmem slot (4), abort flags (8)
constexpr int OFF_COLSUM = (OFF_MISC + 16 + 15) & ~15;
constexpr int SMEM_FIXED = OFF_COLSUM + 1024;        // + alignment slack

// bf16 A and B, fp32 D; both K-major, or B MN-major (b_major bit 16)
MARCHE_DEVINL constexpr uint32_t idesc_bf16(int M, int N, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major ? (1u << 16) : 0u) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}
// MN-major operand tile written by TMA as [k rows][64 elements = 128 bytes] with the 128-byte
// swizzle: 8 k-rows form a 1024-byte atom (stride byte offset), one atom wide in MN.
MARCHE_DEVINL uint64_t smem_desc_mn_sw128(uint32_t addr) {
  const uint32_t lo = ((addr & 0x3FFFFu) >> 4) | ((1024u >> 4) << 16);
  const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
  return ((uint64_t)hi << 32) | lo;
}
MARCHE_DEVINL float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <bool SCORING>
__global__ void __launch_bounds__(kThreads)
attention_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_kv, const __grid_constant__ CUtensorMap tmap_q,
                         int n, int S, int H, int B, const uint8_t* __restrict__ is_new,
                         float* __restrict__ score_partial, uint16_t* __restrict__ o, bool o_bf16,
                         int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  auto bar = [&](int i) { return base + OFF_BAR + 8u * i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + OFF_MISC);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + OFF_MISC + 8);
  float* colsum = reinterpret_cast<float*>(gen + OFF_COLSUM);           // [4][S], scoring only

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.x / H, h = blockIdx.x - b * H;
  const int D = H * DH;
  const int n_kv = (S + KT - 1) / KT, n_qt = (n + QT - 1) / QT;
  const float c_log2 = rsqrtf((float)DH) * 1.4426950408889634f;

  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGE; ++s) { ptx::mbar_init(bar(B_KV_FULL + s), 1); ptx::mbar_init(bar(B_KV_EMPTY + s), 1); }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(bar(B_S_FULL + a), 1);  ptx::mbar_init(bar(B_S_EMPTY + a), 4);
      ptx::mbar_init(bar(B_P_FULL + a), 4);  ptx::mbar_init(bar(B_P_EMPTY + a), 1);
    }
    ptx::mbar_init(bar(B_Q_FULL), 1);  ptx::mbar_init(bar(B_Q_EMPTY), 1);
    ptx::mbar_init(bar(B_O_FULL), 1);  ptx::mbar_init(bar(B_O_EMPTY), 4);
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
  }
  if (warp == 2) {
    ptx::tmem_alloc(ptx::smem_u32((const void*)tmem_slot), TMEM_COLS);
    ptx::tmem_relinquish();
  }
  if (SCORING)
    for (int t = threadIdx.x; t < 4 * S; t += kThreads) colsum[t] = 0.f;
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_sync();

  bool ok = true;
  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      ptx::prefetch_tensormap(&tmap_kv);
      ptx::prefetch_tensormap(&tmap_q);
      int it = 0;                                          // K/V loads issued so far
      for (int qt = 0; qt < n_qt && ok; ++qt) {
        if (!ptx::mbar_wait(bar(B_Q_EMPTY), ((uint32_t)qt & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        ptx::mbar_expect_tx(bar(B_Q_FULL), Q_BYTES);
        ptx::tma_load_3d(base + OFF_Q, &tmap_q, h * DH, qt * QT, b, bar(B_Q_FULL));
        for (int pass = 0; pass < 2 && ok; ++pass) {
          for (int kt = 0; kt < n_kv; ++kt, ++it) {
            const int s = it % NSTAGE;
            if (!ptx::mbar_wait(bar(B_KV_EMPTY + s), ((uint32_t)(it / NSTAGE) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
            const uint32_t dst = base + OFF_KV + s * STAGE_BYTES;
            ptx::mbar_expect_tx(bar(B_KV_FULL + s), pass ? STAGE_BYTES : TILE_BYTES);
            ptx::tma_load_3d(dst, &tmap_kv, h * DH, kt * KT, b, bar(B_KV_FULL + s));
            if (pass) ptx::tma_load_3d(dst + TILE_BYTES, &tmap_kv, h * DH, kt * KT, B + b, bar(B_KV_FULL + s));
          }
        }
      }
      if (!ok) *(volatile int*)status = ST_ATT_TC;
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_bf16(QT, KT, false);
      constexpr uint32_t idesc_o = idesc_bf16(QT, DH, true);
      const uint32_t q_addr = base + OFF_Q;
      int it = 0;        // K/V tiles consumed (ring index)
      int sc = 0;        // S accumulators produced
      int pc = 0;        // P tiles consumed
      auto s_mma = [&](int s, int a) {
#pragma unroll
        for (int k = 0; k < DH / 16; ++k)
          ptx::umma_f16(tmem_base + (uint32_t)(a * KT), ptx::smem_desc_k_sw128(q_addr + k * 32),
                        ptx::smem_desc_k_sw128(base + OFF_KV + s * STAGE_BYTES + k * 32), idesc_s, k ? 1u : 0u);
      };
      auto pv_mma = [&](int s, int a, bool first) {
#pragma unroll
        for (int k = 0; k < KT / 16; ++k)
          ptx::umma_f16(tmem_base + 128u, ptx::smem_desc_k_sw128(base + OFF_P + a * P_BYTES + k * 32),
                        smem_desc_mn_sw128(base + OFF_KV + s * STAGE_BYTES + TILE_BYTES + k * 2048), idesc_o,
                        (first && k == 0) ? 0u : 1u);
      };
      for (int qt = 0; qt < n_qt && ok; ++qt) {
        if (!ptx::mbar_wait(bar(B_Q_FULL), (uint32_t)qt & 1u, abort_flag)) { ok = false; break; }
        // pass 1: logits only
        for (int kt = 0; kt < n_kv; ++kt, ++it, ++sc) {
          const int s = it % NSTAGE, a = sc & 1;
          if (!ptx::mbar_wait(bar(B_KV_FULL + s), (uint32_t)(it / NSTAGE) & 1u, abort_flag) ||
              !ptx::mbar_wait(bar(B_S_EMPTY + a), ((uint32_t)(sc >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after();
          s_mma(s, a);
          ptx::umma_commit(bar(B_S_FULL + a));
          ptx::umma_commit(bar(B_KV_EMPTY + s));
        }
        if (!ok) break;
        // pass 2: logits of tile kt, then O += P V of tile kt-1 (so the softmax of kt overlaps it)
        if (!ptx::mbar_wait(bar(B_O_EMPTY), ((uint32_t)qt & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        int prev_s = 0;
        for (int kt = 0; kt <= n_kv; ++kt) {
          if (kt < n_kv) {
            const int s = it % NSTAGE, a = sc & 1;
            if (!ptx::mbar_wait(bar(B_KV_FULL + s), (uint32_t)(it / NSTAGE) & 1u, abort_flag) ||
                !ptx::mbar_wait(bar(B_S_EMPTY + a), ((uint32_t)(sc >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
            ptx::tc_fence_after();
            s_mma(s, a);
            ptx::umma_commit(bar(B_S_FULL + a));
            ++sc;
          }
          if (kt > 0) {
            const int a = pc & 1;
            if (!ptx::mbar_wait(bar(B_P_FULL + a), (uint32_t)(pc >> 1) & 1u, abort_flag)) { ok = false; break; }
            ptx::tc_fence_after();
            pv_mma(prev_s, a, kt == 1);
            ptx::umma_commit(bar(B_P_EMPTY + a));
            ptx::umma_commit(bar(B_KV_EMPTY + prev_s));
            ++pc;
          }
          if (kt < n_kv) { prev_s = it % NSTAGE; ++it; }
        }
        if (!ok) break;
        ptx::umma_commit(bar(B_O_FULL));                   // all MMAs of this q-tile done: O complete,
        ptx::umma_commit(bar(B_Q_EMPTY));                  // and Q may be overwritten
      }
      if (!ok) *(volatile int*)status = ST_ATT_TC;
    }
  } else {
    // ---------------------------------------------------------------- softmax warps (one thread per row)
    const int quarter = warp & 3;
    const int row_in_tile = quarter * 32 + lane;
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    int sc = 0, pc = 0;
    for (int qt = 0; qt < n_qt && ok; ++qt) {
      const int row = qt * QT + row_in_tile;
      const bool valid = row < n;
      const bool flagged = SCORING && valid && is_new[(size_t)b * n + row];
      const bool warp_flagged = SCORING && __any_sync(0xffffffffu, flagged);
      const bool warp_valid = (qt * QT + quarter * 32) < n;
      // ---- pass 1: row maxima of the raw logits (and, when scoring, the row sums, online)
      float m = -INFINITY, l = 0.f;
      for (int kt = 0; kt < n_kv; ++kt, ++sc) {
        const int a = sc & 1;
        if (!ptx::mbar_wait(bar(B_S_FULL + a), (uint32_t)(sc >> 1) & 1u, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after();
        uint32_t r[64];
        {
          uint32_t (&r0)[32] = *reinterpret_cast<uint32_t (*)[32]>(&r[0]);
          uint32_t (&r1)[32] = *reinterpret_cast<uint32_t (*)[32]>(&r[32]);
          ptx::tmem_ld_32x32(t_lane + (uint32_t)(a * KT), r0);
          ptx::tmem_ld_32x32(t_lane + (uint32_t)(a * KT + 32), r1);
        }
        ptx::tmem_ld_wait();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bar(B_S_EMPTY + a));
        const int lim = S - kt * KT;                      // keys of this tile that exist
        float tmax = -INFINITY;
#pragma unroll
        for (int c = 0; c < 64; ++c)
          if (c < lim) tmax = fmaxf(tmax, __uint_as_float(r[c]));
        if (SCORING && warp_valid) {
          const float m_new = fmaxf(m, tmax);
          const float neg = -m_new * c_log2;
          float sum = 0.f;
#pragma unroll
          for (int c = 0; c < 64; ++c)
            if (c < lim) sum += ex2_approx(fmaf(__uint_as_float(r[c]), c_log2, neg));
          l = l * ex2_approx((m - m_new) * c_log2) + sum;
          m = m_new;
        } else {
          m = fmaxf(m, tmax);
        }
      }
      if (!ok) break;
      // ---- pass 2: weights with the final maximum (normalised right away when scoring), P tiles
      const float neg_mc = -m * c_log2;
      const float p_scale = SCORING ? 1.0f / l : 1.0f;
      if (!SCORING) l = 0.f;
      for (int kt = 0; kt < n_kv; ++kt, ++sc, ++pc) {
        const int a = sc & 1, pa = pc & 1;
        if (!ptx::mbar_wait(bar(B_S_FULL + a), (uint32_t)(sc >> 1) & 1u, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after();
        uint32_t r[64];
        {
          uint32_t (&r0)[32] = *reinterpret_cast<uint32_t (*)[32]>(&r[0]);
          uint32_t (&r1)[32] = *reinterpret_cast<uint32_t (*)[32]>(&r[32]);
          ptx::tmem_ld_32x32(t_lane + (uint32_t)(a * KT), r0);
          ptx::tmem_ld_32x32(t_lane + (uint32_t)(a * KT + 32), r1);
        }
        ptx::tmem_ld_wait();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bar(B_S_EMPTY + a));
        const int lim = S - kt * KT;
        if (warp_valid) {
#pragma unroll
          for (int c = 0; c < 64; ++c) {
            float p = c < lim ? ex2_approx(fmaf(__uint_as_float(r[c]), c_log2, neg_mc)) : 0.f;
            if (SCORING) p *= p_scale; else l += p;
            r[c] = __float_as_uint(p);
          }
        } else {
#pragma unroll
          for (int c = 0; c < 64; ++c) r[c] = 0u;
        }
        // P tile (bf16, K-major, 128-byte swizzle): this thread's row
        if (!ptx::mbar_wait(bar(B_P_EMPTY + pa), ((uint32_t)(pc >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        const uint32_t prow = base + OFF_P + pa * P_BYTES + (uint32_t)row_in_tile * 128u;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint32_t dst = prow + (uint32_t)((j ^ (row_in_tile & 7)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst),
                       "r"(pack_bf16x2(__uint_as_float(r[8 * j + 0]), __uint_as_float(r[8 * j + 1]))),
                       "r"(pack_bf16x2(__uint_as_float(r[8 * j + 2]), __uint_as_float(r[8 * j + 3]))),
                       "r"(pack_bf16x2(__uint_as_float(r[8 * j + 4]), __uint_as_float(r[8 * j + 5]))),
                       "r"(pack_bf16x2(__uint_as_float(r[8 * j + 6]), __uint_as_float(r[8 * j + 7]))) : "memory");
        }
        ptx::fence_proxy_async();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bar(B_P_FULL + pa));
        // ---- relevance: per key, the sum of the (final) weights of this warp's flagged rows.
        // Butterfly over the 32 lanes: after 5 rounds (62 shuffles) lane i holds keys 2i and 2i+1.
        if (SCORING && warp_flagged) {
          float v[64];
#pragma unroll
          for (int c = 0; c < 64; ++c) v[c] = flagged ? __uint_as_float(r[c]) : 0.f;
#pragma unroll
          for (int off = 16, cnt = 32; off >= 1; off >>= 1, cnt >>= 1) {
            const bool up = (lane & off) != 0;
#pragma unroll
            for (int i = 0; i < cnt; ++i) {
              const float send = up ? v[i] : v[i + cnt];
              const float keep = up ? v[i + cnt] : v[i];
              v[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
            }
          }
          float* cs = colsum + (size_t)quarter * S + kt * KT;
          if (2 * lane < lim) cs[2 * lane] += v[0];
          if (2 * lane + 1 < lim) cs[2 * lane + 1] += v[1];
        }
      }
      if (!ok) break;
      // ---- epilogue of the q-tile: O / l -> fp16 rows
      if (!ptx::mbar_wait(bar(B_O_FULL), (uint32_t)qt & 1u, abort_flag)) { ok = false; break; }
      ptx::tc_fence_after();
      {
        uint32_t r0[32], r1[32];
        ptx::tmem_ld_32x32(t_lane + 128u, r0);
        ptx::tmem_ld_32x32(t_lane + 160u, r1);
        ptx::tmem_ld_wait();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bar(B_O_EMPTY));
        if (valid) {
          const float inv = SCORING ? 1.0f : 1.0f / l;
          uint4* dst = reinterpret_cast<uint4*>(o + ((size_t)b * n + row) * D + h * DH);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint4 v;
            v.x = pack_a16x2(__uint_as_float(r0[8 * j + 0]) * inv, __uint_as_float(r0[8 * j + 1]) * inv, o_bf16);
            v.y = pack_a16x2(__uint_as_float(r0[8 * j + 2]) * inv, __uint_as_float(r0[8 * j + 3]) * inv, o_bf16);
            v.z = pack_a16x2(__uint_as_float(r0[8 * j + 4]) * inv, __uint_as_float(r0[8 * j + 5]) * inv, o_bf16);
            v.w = pack_a16x2(__uint_as_float(r0[8 * j + 6]) * inv, __uint_as_float(r0[8 * j + 7]) * inv, o_bf16);
            dst[j] = v;
          }
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint4 v;
            v.x = pack_a16x2(__uint_as_float(r1[8 * j + 0]) * inv, __uint_as_float(r1[8 * j + 1]) * inv, o_bf16);
            v.y = pack_a16x2(__uint_as_float(r1[8 * j + 2]) * inv, __uint_as_float(r1[8 * j + 3]) * inv, o_bf16);
            v.z = pack_a16x2(__uint_as_float(r1[8 * j + 4]) * inv, __uint_as_float(r1[8 * j + 5]) * inv, o_bf16);
            v.w = pack_a16x2(__uint_as_float(r1[8 * j + 6]) * inv, __uint_as_float(r1[8 * j + 7]) * inv, o_bf16);
            dst[4 + j] = v;
          }
        }
      }
    }
    if (!ok && lane == 0) *(volatile int*)status = ST_ATT_TC;
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
  if (SCORING && !*abort_flag) {
    float* dst = score_partial + ((size_t)b * H + h) * S;
    for (int t = threadIdx.x; t < S; t += kThreads)
      dst[t] = ((colsum[t] + colsum[(size_t)S + t]) + colsum[(size_t)2 * S + t]) + colsum[(size_t)3 * S + t];
  }
}

template <bool SCORING>
cudaError_t launch_tc(const CUtensorMap& tkv, const CUtensorMap& tq, int B, int n, int S, int H, const uint8_t* is_new,
                      float* partial, uint16_t* o, bool o_bf16, int* status, cudaStream_t st) {
  const size_t smem = SMEM_FIXED + (SCORING ? (size_t)4 * S * sizeof(float) : 0);
  static size_t smem_set[kMaxDevices] = {};
  cudaError_t e = ensure_dynamic_smem(attention_tcgen05_kernel<SCORING>, smem, smem_set);
  if (e != cudaSuccess) return e;
  return launch_pdl(attention_tcgen05_kernel<SCORING>, dim3(B * H), dim3(kThreads), smem, st, tkv, tq, n, S, H, B, is_new,
                    partial, o, o_bf16, status);
}

}  // namespace

cudaError_t launch_attention_tcgen05(const void* q, int ld_q, int B, int n, int S, int H, int dh,
                                     const void* cache_layer, const uint8_t* is_new, float* score_partial, void* o,
                                     bool o_bf16, int* status, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  if (dh != DH || ld_q % 8 || ((uintptr_t)q & 15) || ((uintptr_t)cache_layer & 15) || S > 2048)
    return cudaErrorInvalidValue;
  const int D = H * dh;
  CUtensorMap tkv, tq;
  {
    const uint64_t dims[3] = {(uint64_t)D, (uint64_t)S, (uint64_t)2 * B};
    const uint64_t strides[2] = {(uint64_t)D * 2, (uint64_t)S * D * 2};
    const uint32_t box[3] = {(uint32_t)DH, KT, 1};
    if (!tma_make_map_bf16(&tkv, cache_layer, 3, dims, strides, box, true)) return cudaErrorInvalidValue;
  }
  {
    const uint64_t dims[3] = {(uint64_t)ld_q, (uint64_t)n, (uint64_t)B};
    const uint64_t strides[2] = {(uint64_t)ld_q * 2, (uint64_t)n * ld_q * 2};
    const uint32_t box[3] = {(uint32_t)DH, QT, 1};
    if (!tma_make_map_bf16(&tq, q, 3, dims, strides, box, true)) return cudaErrorInvalidValue;
  }
  return is_new ? launch_tc<true>(tkv, tq, B, n, S, H, is_new, score_partial, (uint16_t*)o, o_bf16, status, st)
                : launch_tc<false>(tkv, tq, B, n, S, H, is_new, score_partial, (uint16_t*)o, o_bf16, status, st);
}

}  // namespace marche
