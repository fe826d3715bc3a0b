// K2: out = epilogue(a * w^T + bias) on the 5th-generation tensor cores.
//
// The QKV, output and MLP projections of the active rows (Algorithm 1 lines 5 and 9)
// are dense 16-bit contractions (both operands fp16, or both bf16, -> fp32), so they run as a persistent, warp-specialised tcgen05
// kernel: one CTA per SM walks over 128 x BN output tiles;
//   warp 0   (one lane)  TMA producer: 128x64 A tile and BNx64 W tile per K step into a
//                        shared-memory ring (128-byte swizzle), completion on mbarriers
//   warp 1   (one lane)  issues tcgen05.mma (M 128, N BN, K 16; fp16 in, fp32 accumulate
//                        in TMEM), frees ring slots and publishes accumulators with
//                        tcgen05.commit
//   warps 2-5            epilogue: tcgen05.ld of the accumulator (thread = output row),
//                        bias / GELU, swizzled staging box in shared memory, TMA bulk store
//                        (TMA reduce-add for the fp32 residual)
// The accumulator is double-buffered in TMEM (2 x BN columns) so the epilogue of tile i
// overlaps the MMAs of tile i+1.  Rows beyond M are zero-filled by TMA on load and
// masked on store, so M needs no padding.  Every mbarrier wait is bounded; on a
// give-up the kernel records a status code and drains instead of hanging.
#include <cuda.h>

#include "gemm_epilogue.cuh"
#include "kernels.h"
#include "launch_pdl.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace marche {

namespace {

constexpr int BM = 128;
constexpr int BK = 64;                    // one 128-byte swizzle row of bf16
constexpr int kGemmThreads = 192;
constexpr int A_BYTES = BM * BK * 2;      // 16 KB

template <int BN> struct GemmCfg {
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int STAGES = (BN == 256) ? 4 : 6;
  static constexpr int RING_BYTES = STAGES * (A_BYTES + B_BYTES);
  static constexpr int STAGING_BYTES = 4 * 4096;            // one 32-row x 128-byte box per epilogue warp
  static constexpr int SMEM_BYTES = RING_BYTES + STAGING_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
  static constexpr int TMEM_COLS = 2 * BN;
};

enum { ST_PRODUCER = 0x11, ST_MMA = 0x12, ST_EPILOGUE = 0x13 };

template <int BN, int EPI>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
                    const __grid_constant__ CUtensorMap tmap_out, int M, int N, int K,
                    const float* __restrict__ bias, int* __restrict__ status, int a_bf16) {
  using Cfg = GemmCfg<BN>;
  constexpr int STAGES = Cfg::STAGES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;             // swizzled tiles need 1024-byte alignment
  const uint32_t a_base = base;
  const uint32_t w_base = base + STAGES * A_BYTES;
  const uint32_t staging = base + Cfg::RING_BYTES;
  const uint32_t bar_base = staging + Cfg::STAGING_BYTES;   // 8-byte barriers
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
  uint8_t* gen_base = smem_raw + (base - raw);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen_base + Cfg::RING_BYTES + Cfg::STAGING_BYTES + 8 * (2 * STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen_base + Cfg::RING_BYTES + Cfg::STAGING_BYTES + 8 * (2 * STAGES + 4) + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_m = (M + BM - 1) / BM, n_n = N / BN, n_tiles = n_m * n_n, n_kb = K / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(tfull_bar(a), 1);
      ptx::mbar_init(tempty_bar(a), 4);                     // one arrival per epilogue warp
    }
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
  }
  if (warp == 2) {
    ptx::tmem_alloc(ptx::smem_u32((const void*)tmem_slot), Cfg::TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_sync();                                               // set-up above overlaps the previous kernel's tail

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      ptx::prefetch_tensormap(&tmap_a);
      ptx::prefetch_tensormap(&tmap_w);
      ptx::prefetch_tensormap(&tmap_out);
      int it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        const int m_blk = tile / n_n, n_blk = tile - m_blk * n_n;
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
          if (!ptx::mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { ok = false; break; }
          ptx::mbar_expect_tx(full_bar(s), A_BYTES + Cfg::B_BYTES);
          ptx::tma_load_2d(a_base + s * A_BYTES, &tmap_a, kb * BK, m_blk * BM, full_bar(s));
          ptx::tma_load_2d(w_base + s * Cfg::B_BYTES, &tmap_w, kb * BK, n_blk * BN, full_bar(s));
        }
      }
      if (!ok) {
        *(volatile int*)status = ST_PRODUCER;
        // let copies already issued land before the CTA's shared memory is released
        for (int j = 1; j <= STAGES && j <= it; ++j) {
          const int i2 = it - j;
          ptx::mbar_wait(full_bar(i2 % STAGES), (uint32_t)(i2 / STAGES) & 1u, abort_flag + 1, 20000000LL);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc = ptx::idesc_16_f32(BM, BN, a_bf16 != 0);
      int it = 0, tile_i = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++tile_i) {
        const int acc = tile_i & 1;
        const uint32_t acc_ph = (uint32_t)(tile_i >> 1) & 1u;
        if (!ptx::mbar_wait(tempty_bar(acc), acc_ph ^ 1u, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
          if (!ptx::mbar_wait(full_bar(s), ph, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after();
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            const uint64_t da = ptx::smem_desc_k_sw128(a_base + s * A_BYTES + k * 32);
            const uint64_t dw = ptx::smem_desc_k_sw128(w_base + s * Cfg::B_BYTES + k * 32);
            ptx::umma_f16(d_tmem, da, dw, idesc, (kb | k) ? 1u : 0u);
          }
          ptx::umma_commit(empty_bar(s));                   // slot free once these MMAs have read it
        }
        if (ok) ptx::umma_commit(tfull_bar(acc));           // accumulator complete
      }
      if (!ok) *(volatile int*)status = ST_MMA;
    }
  } else {
    // ---------------------------------------------------------------- epilogue (warps 2..5)
    const int quarter = warp & 3;                           // TMEM lanes 32*quarter .. +31
    int tile_i = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++tile_i) {
      const int m_blk = tile / n_n, n_blk = tile - m_blk * n_n;
      const int acc = tile_i & 1;
      const uint32_t acc_ph = (uint32_t)(tile_i >> 1) & 1u;
      if (!ptx::mbar_wait(tfull_bar(acc), acc_ph, abort_flag)) { ok = false; break; }
      ptx::tc_fence_after();
      const int row0 = m_blk * BM + quarter * 32;
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
      const uint32_t my_stage = staging + (uint32_t)(warp - 2) * 4096u;
      if (row0 < M) {
        constexpr int EC = EpiCols<EPI>::value;
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += EC)
          epilogue_box<EPI>(t_row + (uint32_t)c0, bias + n_blk * BN + c0, &tmap_out, n_blk * BN + c0, row0, my_stage,
                            lane, a_bf16 != 0);
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(tempty_bar(acc));
    }
    if (!ok && lane == 0) *(volatile int*)status = ST_EPILOGUE;
    if (lane == 0) ptx::bulk_wait_all();                    // this warp's stores have landed
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
  }
}

// ---------------------------------------------------------------- host side
// Row-major bf16 matrix [rows][cols] with row stride ld elements; box = 64 columns x box_rows rows.
bool make_map_2d(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows,
                 bool ieee_half) {
  const uint64_t dims[2] = {cols, rows};
  const uint64_t strides[1] = {ld * 2};
  const uint32_t box[2] = {BK, box_rows};
  return tma_make_map_bf16(map, ptr, 2, dims, strides, box, true, ieee_half);
}

int sm_count() { return device_sm_count(); }

template <int BN, int EPI>
cudaError_t launch_one(const CUtensorMap& ta, const CUtensorMap& tw, const CUtensorMap& to, int M, int N, int K,
                       const float* bias, int* status, int a_bf16, cudaStream_t st) {
  static size_t smem_set[kMaxDevices] = {};
  cudaError_t e = ensure_dynamic_smem(gemm_tcgen05_kernel<BN, EPI>, (size_t)GemmCfg<BN>::SMEM_BYTES, smem_set);
  if (e != cudaSuccess) return e;
  const int n_tiles = ((M + BM - 1) / BM) * (N / BN);
  const int grid = n_tiles < sm_count() ? n_tiles : sm_count();
  return launch_pdl(gemm_tcgen05_kernel<BN, EPI>, dim3(grid), dim3(kGemmThreads), (size_t)GemmCfg<BN>::SMEM_BYTES, st, ta,
                    tw, to, M, N, K, bias, status, a_bf16);
}

}  // namespace

int gemm_tcgen05_pick_bn(int M, int N) {
  const int n_m = (M + BM - 1) / BM, sms = sm_count();
  if (N % 256) return 128;
  const long t256 = (long)n_m * (N / 256), t128 = (long)n_m * (N / 128);
  const double c256 = (double)((t256 + sms - 1) / sms) * 256.0;
  const double c128 = (double)((t128 + sms - 1) / sms) * 128.0 * 1.08;   // smaller tiles re-read A more often
  return c256 <= c128 ? 256 : 128;
}

cudaError_t launch_gemm_tcgen05(const void* a, int lda, int M, const void* w, const float* bias, int N, int K,
                                int epilogue, void* out, bool a_bf16, int* status, cudaStream_t st) {
  if (M == 0) return cudaSuccess;
  if (N % 128 || K % BK || lda % 8 || ((uintptr_t)a & 15) || ((uintptr_t)w & 15)) return cudaErrorInvalidValue;
  const int bn = gemm_tcgen05_pick_bn(M, N);
  CUtensorMap ta, tw, to;
  if (!make_map_2d(&ta, a, (uint64_t)M, (uint64_t)K, (uint64_t)lda, BM, !a_bf16)) return cudaErrorInvalidValue;
  if (!make_map_2d(&tw, w, (uint64_t)N, (uint64_t)K, (uint64_t)K, (uint32_t)bn, !a_bf16)) return cudaErrorInvalidValue;
  if (((uintptr_t)out & 15) || !tma_make_store_map(&to, out, (uint64_t)M, (uint64_t)N, epilogue == 1 ? 4 : 2))
    return cudaErrorInvalidValue;
#define MARCHE_GEMM_CASE(BN_, EPI_) \
  if (bn == BN_ && epilogue == EPI_) return launch_one<BN_, EPI_>(ta, tw, to, M, N, K, bias, status, a_bf16 ? 1 : 0, st);
  MARCHE_GEMM_CASE(256, 0) MARCHE_GEMM_CASE(256, 1) MARCHE_GEMM_CASE(256, 2)
  MARCHE_GEMM_CASE(128, 0) MARCHE_GEMM_CASE(128, 1) MARCHE_GEMM_CASE(128, 2)
#undef MARCHE_GEMM_CASE
  return cudaErrorInvalidValue;
}

}  // namespace marche
