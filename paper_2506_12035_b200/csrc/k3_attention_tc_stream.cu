// K3 on the 5th-generation tensor cores, single pass (head_dim 64, no relevance scores): attention of
// the active queries over all S cached rows of one block (Algorithm 1 lines 6-8 == Eq. 5 by
// Appendix A), with the running-maximum / running-sum merge of Eq. 6-10 applied tile by tile.
//
// Persistent CTAs (one per SM).  The work of a CTA is a list of units, one unit = one 128-row query
// tile of one (sample, head) item against all S keys; THREE independent streams inside the CTA take
// the units in turn.  A unit is a latency chain (Q K^T -> read logits -> exponentials -> write weights
// -> P V ...), and the exponentials - 16 per clock and SM - are the scarce resource once the active set
// is large; three chains in flight per SM partition keep those units and the tensor core busy while
// each chain waits on its own hand-overs.  Each stream owns a query buffer, a 3-deep TMA ring of 64-key
// K/V tiles that runs ahead across units (the HBM queue never drains between items) and accumulators in
// tensor memory: S_j 64 columns (fp32 logits), P_j 32 columns (weights as packed bf16), O_j 64 columns.
// Roles (20 warps; the eight control warps hand most of their registers to the twelve softmax warps):
//   warps 0-11    softmax: warps 4j .. 4j+3 serve stream j, one thread per query row.  A thread pulls its
//                 S row into registers (tcgen05.ld), hands the S buffer straight back so that the next
//                 tile's Q K^T runs during the exponentials, and writes the weights to tensor memory
//                 (tcgen05.st), from where the tensor core reads them as the A operand of P V
//   warps 12-14   TMA producer of stream 0 / 1 / 2: Q tile per unit, K/V ring
//   warps 15-17   issue tcgen05.mma for stream 0 / 1 / 2: S_j = Q_j K^T (M128 x N64 x K64) as soon as the S
//                 buffer is free, O_j += P_j V (M128 x N64 x K64, V as an MN-major operand from shared
//                 memory) as soon as the weights are there; warp 17 also allocates / frees tensor memory
// Online softmax with a lazy reference maximum: the exponent reference of a row only moves when a
// tile's maximum exceeds it by more than 2^8 in the exponent, and only then is the row's O accumulator
// rescaled in tensor memory (by the row's own thread, after the previous P V has completed); weights
// therefore never exceed 256 and the final division by the row sum makes the result exact up to
// rounding.  All waits are bounded and report through the status word.
#include <cuda.h>

#include "kernels.h"
#include "launch_pdl.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace marche {

namespace {

constexpr int DH = 64;
constexpr int QT = 128;                    // query rows per unit (= TMEM lanes)
constexpr int KT = 64;                     // keys per tile
constexpr int NS = 3;                      // streams per CTA
constexpr int NST = 3;                     // K/V ring stages per stream
constexpr int K_BYTES = KT * DH * 2;       // 8 KB
constexpr int STAGE_BYTES = 2 * K_BYTES;   // K tile then V tile
constexpr int Q_BYTES = QT * DH * 2;       // 16 KB
constexpr int kThreads = 640;               // 12 softmax warps, then 8 control warps: 3 producers, 3 MMA issuers, 2 idle
constexpr int W_PROD = NS * 4, W_MMA = NS * 5;   // (whole groups of four warps, as the register reallocation requires)
constexpr int TMEM_COLS = 512;
constexpr uint32_t COL_S = 0;                       // S_j: KT columns each
constexpr uint32_t COL_P = NS * KT;                 // P_j: KT / 2 columns each (KT bf16)
constexpr uint32_t COL_O = COL_P + NS * (KT / 2);   // O_j: 64 columns each
static_assert(COL_O + NS * DH <= TMEM_COLS, "tensor memory budget");
enum { ST_ATT_STREAM = 0x51 };

// shared memory (from a 1024-byte aligned base)
constexpr int OFF_Q = 0;                                   // [stream]
constexpr int OFF_KV = OFF_Q + NS * Q_BYTES;               // [stream][stage]
constexpr int OFF_BAR = OFF_KV + NS * NST * STAGE_BYTES;
// barriers of one stream (8 bytes each); stream j's block starts at j * NB
enum { B_KV_FULL = 0, B_KV_EMPTY = NST, B_Q_FULL = 2 * NST, B_Q_EMPTY, B_S_FULL, B_S_EMPTY, B_P_FULL, B_P_EMPTY, B_O_FULL,
       B_O_FREE, NB };
constexpr int OFF_MISC = OFF_BAR + 8 * NS * NB;            // tmem slot (4), abort flags (8)
constexpr int SMEM_BYTES = OFF_MISC + 32 + 1024;

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
// D[tmem] (+)= A[tmem] * B[smem desc]: the A operand (128 lanes x K 16-bit values, two per column) is
// read from tensor memory.
MARCHE_DEVINL void umma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n"
      "}\n"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 32 lanes x N consecutive 32-bit columns: thread i of the warp accesses lane (base + i).
MARCHE_DEVINL void tmem_ld_32x64(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x64.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
      : "r"(taddr)
      : "memory");
}
MARCHE_DEVINL void tmem_ld_32x16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
MARCHE_DEVINL void tmem_st_32x16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
MARCHE_DEVINL void tmem_st_32x32(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
MARCHE_DEVINL void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
MARCHE_DEVINL float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// Packed fp32 pairs (one instruction for two values): (a0, a1) * m + (b, b), and pairwise accumulate.
MARCHE_DEVINL void ffma2_bcast(float a0, float a1, float m, float b, float& r0, float& r1) {
  asm("{\n"
      ".reg .b64 ra, rm, rb, rr;\n"
      "mov.b64 ra, {%2, %3};\n"
      "mov.b64 rm, {%4, %4};\n"
      "mov.b64 rb, {%5, %5};\n"
      "fma.rn.f32x2 rr, ra, rm, rb;\n"
      "mov.b64 {%0, %1}, rr;\n"
      "}\n"
      : "=f"(r0), "=f"(r1) : "f"(a0), "f"(a1), "f"(m), "f"(b));
}
MARCHE_DEVINL void fadd2(float& acc0, float& acc1, float p0, float p1) {
  asm("{\n"
      ".reg .b64 ra, rp;\n"
      "mov.b64 ra, {%0, %1};\n"
      "mov.b64 rp, {%2, %3};\n"
      "add.f32x2 ra, ra, rp;\n"
      "mov.b64 {%0, %1}, ra;\n"
      "}\n"
      : "+f"(acc0), "+f"(acc1) : "f"(p0), "f"(p1));
}
MARCHE_DEVINL float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// The CTA's units in order: unit k = query tile (k % n_qt) of the CTA's (k / n_qt)-th item; stream j
// takes k = j, j + NS, ...
struct Unit { int b, h, qt; };
MARCHE_DEVINL Unit unit_of(int j, int u, int n_qt, int H) {
  const int k = NS * u + j;
  const int item = (int)blockIdx.x + (k / n_qt) * (int)gridDim.x;
  Unit r;
  r.b = item / H;
  r.h = item - r.b * H;
  r.qt = k % n_qt;
  return r;
}

__global__ void __launch_bounds__(kThreads, 1)
attention_tc_stream_kernel(const __grid_constant__ CUtensorMap tmap_kv, const __grid_constant__ CUtensorMap tmap_q,
                           int n, int S, int H, int B, uint16_t* __restrict__ o, int o_bf16, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - raw);
  auto bar = [&](int j, int i) { return base + OFF_BAR + 8u * (uint32_t)(j * NB + i); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + OFF_MISC);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + OFF_MISC + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int D = H * DH;
  const int n_kv = (S + KT - 1) / KT, n_qt = (n + QT - 1) / QT;
  const int n_items = B * H;
  const int items_cta = (n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
  const int units_cta = items_cta * n_qt;
  int n_units[NS];
#pragma unroll
  for (int j = 0; j < NS; ++j) n_units[j] = (units_cta + NS - 1 - j) / NS;
  const float c_log2 = rsqrtf((float)DH) * 1.4426950408889634f;

  if (threadIdx.x == 0) {
    for (int j = 0; j < NS; ++j) {
      for (int s = 0; s < NST; ++s) { ptx::mbar_init(bar(j, B_KV_FULL + s), 1); ptx::mbar_init(bar(j, B_KV_EMPTY + s), 1); }
      ptx::mbar_init(bar(j, B_Q_FULL), 1);   ptx::mbar_init(bar(j, B_Q_EMPTY), 1);
      ptx::mbar_init(bar(j, B_S_FULL), 1);   ptx::mbar_init(bar(j, B_S_EMPTY), 4);
      ptx::mbar_init(bar(j, B_P_FULL), 4);   ptx::mbar_init(bar(j, B_P_EMPTY), 1);
      ptx::mbar_init(bar(j, B_O_FULL), 1);   ptx::mbar_init(bar(j, B_O_FREE), 4);
    }
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
  }
  if (warp == W_MMA + NS - 1) {
    ptx::tmem_alloc(ptx::smem_u32((const void*)tmem_slot), TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_sync();
  // Register reallocation (per group of four warps): 256 control threads x 40 + 384 softmax threads x 128 <= 640 x 96.
  if (warp >= W_PROD) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
   if (warp < W_MMA) {
    // ---------------------------------------------------------------- TMA producer of stream j
    if (lane == 0) {
      const int j = warp - W_PROD;
      ptx::prefetch_tensormap(&tmap_kv);
      ptx::prefetch_tensormap(&tmap_q);
      const uint64_t stream_once = ptx::l2_policy_evict_first();
      int tl = 0;                                          // K/V tiles issued so far
      bool ok = true;
      for (int u = 0; u < n_units[j] && ok; ++u) {
        const Unit un = unit_of(j, u, n_qt, H);
        if (!ptx::mbar_wait(bar(j, B_Q_EMPTY), ((uint32_t)u & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        ptx::mbar_expect_tx(bar(j, B_Q_FULL), Q_BYTES);
        ptx::tma_load_3d(base + OFF_Q + j * Q_BYTES, &tmap_q, un.h * DH, un.qt * QT, un.b, bar(j, B_Q_FULL));
        for (int kt = 0; kt < n_kv; ++kt, ++tl) {
          const int s = tl % NST;
          if (!ptx::mbar_wait(bar(j, B_KV_EMPTY + s), ((uint32_t)(tl / NST) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t dst = base + OFF_KV + (j * NST + s) * STAGE_BYTES;
          ptx::mbar_expect_tx(bar(j, B_KV_FULL + s), STAGE_BYTES);
          ptx::tma_load_3d_hint(dst, &tmap_kv, un.h * DH, kt * KT, un.b, bar(j, B_KV_FULL + s), stream_once);
          ptx::tma_load_3d_hint(dst + K_BYTES, &tmap_kv, un.h * DH, kt * KT, B + un.b, bar(j, B_KV_FULL + s), stream_once);
        }
      }
      if (!ok) {
        *(volatile int*)status = ST_ATT_STREAM;
        // let copies already issued land before the CTA's shared memory is released
        for (int back = 1; back <= NST && back <= tl; ++back) {
          const int i2 = tl - back;
          ptx::mbar_wait(bar(j, B_KV_FULL + i2 % NST), (uint32_t)(i2 / NST) & 1u, abort_flag + 1, 20000000LL);
        }
      }
    }
   } else if (warp < W_MMA + NS) {
    // ---------------------------------------------------------------- MMA issuer of stream j
    // Within a stream the events arrive in a fixed order (S buffer handed back, then the weights of the same
    // tile), so a plain sequence of waits is optimal: S(0); for each tile t: [S buffer free] S(t+1), [weights] P V(t).
    if (lane == 0) {
      const int j = warp - W_MMA;
      constexpr uint32_t idesc_s = idesc_bf16(QT, KT, false);
      constexpr uint32_t idesc_o = idesc_bf16(QT, DH, true);
      const int total = n_units[j] * n_kv;
      const uint32_t q_addr = base + OFF_Q + j * Q_BYTES;
      bool ok = true;
      auto issue_s = [&](int t) -> bool {                  // t: tile counter of the stream
        const int i = t % n_kv, u = t / n_kv;
        if (t > 0 && !ptx::mbar_wait(bar(j, B_S_EMPTY), (uint32_t)(t - 1) & 1u, abort_flag)) return false;
        if (i == 0 && !ptx::mbar_wait(bar(j, B_Q_FULL), (uint32_t)u & 1u, abort_flag)) return false;
        if (!ptx::mbar_wait(bar(j, B_KV_FULL + t % NST), (uint32_t)(t / NST) & 1u, abort_flag)) return false;
        const uint32_t k_addr = base + OFF_KV + (j * NST + t % NST) * STAGE_BYTES;
        ptx::tc_fence_after();
#pragma unroll
        for (int k = 0; k < DH / 16; ++k)
          ptx::umma_f16(tmem_base + COL_S + (uint32_t)(j * KT), ptx::smem_desc_k_sw128(q_addr + k * 32),
                        ptx::smem_desc_k_sw128(k_addr + k * 32), idesc_s, k ? 1u : 0u);
        ptx::umma_commit(bar(j, B_S_FULL));
        if (i == n_kv - 1) ptx::umma_commit(bar(j, B_Q_EMPTY));   // the unit's last Q K^T: Q_j may be overwritten
        return true;
      };
      if (total > 0) ok = issue_s(0);
      for (int t = 0; t < total && ok; ++t) {
        const int i = t % n_kv, u = t / n_kv;
        if (t + 1 < total && !issue_s(t + 1)) { ok = false; break; }
        // O_j += P_j V: needs the weights, and for a unit's first tile the previous output read out
        if (!ptx::mbar_wait(bar(j, B_P_FULL), (uint32_t)t & 1u, abort_flag)) { ok = false; break; }
        if (i == 0 && u > 0 && !ptx::mbar_wait(bar(j, B_O_FREE), (uint32_t)(u - 1) & 1u, abort_flag)) { ok = false; break; }
        const uint32_t v_addr = base + OFF_KV + (j * NST + t % NST) * STAGE_BYTES + K_BYTES;
        ptx::tc_fence_after();
#pragma unroll
        for (int k = 0; k < KT / 16; ++k)
          umma_f16_ts(tmem_base + COL_O + (uint32_t)(j * DH), tmem_base + COL_P + (uint32_t)(j * (KT / 2) + k * 8),
                      smem_desc_mn_sw128(v_addr + k * 2048), idesc_o, (i == 0 && k == 0) ? 0u : 1u);
        ptx::umma_commit(bar(j, B_KV_EMPTY + t % NST));    // K was read by the S of this tile, V just now
        ptx::umma_commit(bar(j, B_P_EMPTY));
        if (i == n_kv - 1) ptx::umma_commit(bar(j, B_O_FULL));
      }
      if (!ok) *(volatile int*)status = ST_ATT_STREAM;
    }
   }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 128;");
    // ---------------------------------------------------------------- softmax streams (one thread per row)
    const int j = warp >> 2;                               // stream (warps 4j .. 4j+3)
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;                     // row inside the query tile = TMEM lane
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const uint32_t t_s = t_lane + COL_S + (uint32_t)(j * KT);
    const uint32_t t_p = t_lane + COL_P + (uint32_t)(j * (KT / 2));
    const uint32_t t_o = t_lane + COL_O + (uint32_t)(j * DH);
    bool ok = true;
    int t = 0;                                             // tiles of this stream so far
    for (int u = 0; u < n_units[j] && ok; ++u) {
      const Unit un = unit_of(j, u, n_qt, H);
      const int row = un.qt * QT + r;
      const bool warp_valid = (un.qt * QT + quarter * 32) < n;
      float m_ref = -INFINITY, l = 0.f;                    // exponent reference (raw logit units), running sum
      uint32_t v[KT];
      for (int i = 0; i < n_kv; ++i, ++t) {
        if (!ptx::mbar_wait(bar(j, B_S_FULL), (uint32_t)t & 1u, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after();
        const int lim = S - i * KT;                        // keys of this tile that exist
        if (warp_valid) {
          tmem_ld_32x64(t_s, v);
          ptx::tmem_ld_wait();
        }
        // the row is in registers: the next tile's logits may overwrite S_j while we work on this one
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bar(j, B_S_EMPTY));
        bool move = false;
        float tmax = -INFINITY;
        if (warp_valid) {
          float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
          if (lim >= KT) {
#pragma unroll
            for (int c = 0; c < KT; c += 2)
              mx[(c >> 1) & 3] = max3(mx[(c >> 1) & 3], __uint_as_float(v[c]), __uint_as_float(v[c + 1]));
          } else {
#pragma unroll
            for (int c = 0; c < KT; ++c)
              if (c < lim) mx[c & 3] = fmaxf(mx[c & 3], __uint_as_float(v[c]));
          }
          tmax = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
          // lazy reference maximum: move it only when this tile exceeds it by more than 2^8
          move = (tmax - m_ref) * c_log2 > 8.0f;           // also true for a unit's first tile (m_ref = -inf)
        }
        // the previous P_j V has read the weights we are about to overwrite, and has finished adding to O_j
        if (t > 0 && !ptx::mbar_wait(bar(j, B_P_EMPTY), (uint32_t)(t - 1) & 1u, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after();
        if (warp_valid) {
          if (i > 0 && __any_sync(0xffffffffu, move)) {
            // rescale this row's accumulator in tensor memory to the new reference
            const float f = move ? ex2_approx((m_ref - tmax) * c_log2) : 1.0f;
#pragma unroll 1
            for (int qc = 0; qc < 4; ++qc) {
              uint32_t ov[16];
              tmem_ld_32x16(t_o + (uint32_t)(qc * 16), ov);
              ptx::tmem_ld_wait();
#pragma unroll
              for (int c = 0; c < 16; ++c) ov[c] = __float_as_uint(__uint_as_float(ov[c]) * f);
              tmem_st_32x16(t_o + (uint32_t)(qc * 16), ov);
            }
            l *= f;
          }
          if (move) m_ref = tmax;
          const float neg = -m_ref * c_log2;
          // weights: p = 2^((s - m_ref) / sqrt(d) * log2 e), packed bf16 pairs, in place (pair c -> v[c])
          float ls[4] = {0.f, 0.f, 0.f, 0.f};
          bool half_stored = false;
          if (lim >= KT) {                                 // (two copies of the loop: no per-element selects on the
#pragma unroll                                             //  common, full tile)
            for (int c = 0; c < KT / 2; ++c) {
              float x0, x1;
              ffma2_bcast(__uint_as_float(v[2 * c]), __uint_as_float(v[2 * c + 1]), c_log2, neg, x0, x1);
              const float p0 = ex2_approx(x0), p1 = ex2_approx(x1);
              fadd2(ls[2 * (c & 1)], ls[2 * (c & 1) + 1], p0, p1);
              v[c] = pack_bf16x2(p0, p1);
              if (c == KT / 4 - 1) tmem_st_32x16(t_p, v);  // first half on its way while the second is computed
            }
            half_stored = true;
          } else {
#pragma unroll
            for (int c = 0; c < KT / 2; ++c) {
              float p0 = ex2_approx(fmaf(__uint_as_float(v[2 * c]), c_log2, neg));
              float p1 = ex2_approx(fmaf(__uint_as_float(v[2 * c + 1]), c_log2, neg));
              if (2 * c >= lim) p0 = 0.f;
              if (2 * c + 1 >= lim) p1 = 0.f;
              ls[c & 3] += p0 + p1;
              v[c] = pack_bf16x2(p0, p1);
            }
          }
          l += (ls[0] + ls[1]) + (ls[2] + ls[3]);
          if (half_stored) tmem_st_32x16(t_p + 16u, v + 16);
          else tmem_st_32x32(t_p, v);
          tmem_st_wait();
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bar(j, B_P_FULL));
      }
      if (!ok) break;
      // ---- end of the unit: O / l -> output rows
      if (!ptx::mbar_wait(bar(j, B_O_FULL), (uint32_t)u & 1u, abort_flag)) { ok = false; break; }
      ptx::tc_fence_after();
      const float inv = 1.0f / l;
      uint4* dst = reinterpret_cast<uint4*>(o + ((size_t)un.b * n + row) * D + un.h * DH);
#pragma unroll 1
      for (int qc = 0; qc < 4; ++qc) {                       // 16 output columns at a time
        uint32_t ov[16];
        if (warp_valid) {
          tmem_ld_32x16(t_o + (uint32_t)(qc * 16), ov);
          ptx::tmem_ld_wait();
        }
        if (qc == 3) {
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(bar(j, B_O_FREE));
        }
        if (warp_valid && row < n) {
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            uint4 w;
            w.x = pack_a16x2(__uint_as_float(ov[8 * q + 0]) * inv, __uint_as_float(ov[8 * q + 1]) * inv, o_bf16 != 0);
            w.y = pack_a16x2(__uint_as_float(ov[8 * q + 2]) * inv, __uint_as_float(ov[8 * q + 3]) * inv, o_bf16 != 0);
            w.z = pack_a16x2(__uint_as_float(ov[8 * q + 4]) * inv, __uint_as_float(ov[8 * q + 5]) * inv, o_bf16 != 0);
            w.w = pack_a16x2(__uint_as_float(ov[8 * q + 6]) * inv, __uint_as_float(ov[8 * q + 7]) * inv, o_bf16 != 0);
            dst[2 * qc + q] = w;
          }
        }
      }
    }
    if (!ok && lane == 0) *(volatile int*)status = ST_ATT_STREAM;
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == W_MMA + NS - 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

}  // namespace

cudaError_t launch_attention_tc_stream(const void* q, int ld_q, int B, int n, int S, int H, int dh,
                                       const void* cache_layer, void* o, bool o_bf16, int* status, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  if (dh != DH || ld_q % 8 || ((uintptr_t)q & 15) || ((uintptr_t)cache_layer & 15) || ((uintptr_t)o & 15) || S > 2048)
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
  static size_t smem_set[kMaxDevices] = {};
  cudaError_t e = ensure_dynamic_smem(attention_tc_stream_kernel, (size_t)SMEM_BYTES, smem_set);
  if (e != cudaSuccess) return e;
  const int sms = device_sm_count();
  const int grid = B * H < sms ? B * H : sms;
  return launch_pdl(attention_tc_stream_kernel, dim3(grid), dim3(kThreads), (size_t)SMEM_BYTES, st, tkv, tq, n, S, H, B,
                    (uint16_t*)o, o_bf16 ? 1 : 0, status);
}

}  // namespace marche
