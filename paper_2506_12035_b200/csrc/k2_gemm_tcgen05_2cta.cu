// K2, 2-CTA flavour: the same projections as k2_gemm_tcgen05.cu with tcgen05.mma
// cta_group::2.  Two CTAs on neighbouring SMs (a cluster of 2) share one 256 x BN output
// tile: each CTA loads its own 128 rows of A and HALF of the W tile per K step, the pair's
// tensor cores read both halves, and each CTA keeps its 128 x BN accumulator in its own
// TMEM.  Per CTA a ring stage is 32 KB instead of 48 KB for the same MMA work, so the ring
// hides more TMA latency per byte of shared memory and L2 -> shared-memory traffic per flop
// drops by a third.  No TMA multicast is used: every CTA fetches its own tiles.
//
// Protocol (rank 0 of the pair is the leader, rank 1 the peer):
//   full[s]    leader's barrier; the leader's producer arms it with the bytes of BOTH CTAs'
//              tiles and both producers' TMA loads complete on it
//   empty[s]   one per CTA; the leader's MMA thread frees a slot in both CTAs with one
//              multicast tcgen05.commit
//   tfull[a]   one per CTA; multicast commit when an accumulator is complete
//   tempty[a]  leader's barrier; the 8 epilogue warps of each CTA arrive (remotely for the peer)
// Epilogue: TMEM -> registers -> swizzled staging box in shared memory -> TMA bulk store (TMA
// reduce-add for the fp32 residual), see gemm_epilogue.cuh.
// All waits are bounded; both CTAs meet at a final cluster barrier so that neither exits
// while its shared memory or TMEM can still be touched by the other.
#include <cuda.h>

#include "gemm_epilogue.cuh"
#include "kernels.h"
#include "launch_pdl.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace marche {

namespace {

constexpr int BM = 128;                   // rows per CTA (256 per pair)
constexpr int BK = 64;
constexpr int kThreads = 320;             // producer warp, MMA warp, 8 epilogue warps
constexpr int A_BYTES = BM * BK * 2;

template <int BN> struct PairCfg {
  static constexpr int BH_BYTES = (BN / 2) * BK * 2;            // this CTA's half of the W tile
  static constexpr int STAGE_BYTES = A_BYTES + BH_BYTES;
  static constexpr int STAGES = (BN == 256) ? 5 : 6;
  static constexpr int RING_BYTES = STAGES * STAGE_BYTES;
  static constexpr int STAGING_BYTES = 8 * 4096;                 // one 32-row x 128-byte box per epilogue warp
  static constexpr int SMEM_BYTES = RING_BYTES + STAGING_BYTES + 1024 + 256;
  static constexpr int TMEM_COLS = 2 * BN;
};

enum { ST2_PRODUCER = 0x31, ST2_MMA = 0x32, ST2_EPILOGUE = 0x33 };

template <int BN, int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_tcgen05_2cta_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
                         const __grid_constant__ CUtensorMap tmap_out, int M, int N, int K,
                         const float* __restrict__ bias, int* __restrict__ status, int* __restrict__ turn,
                         const KvScatter kv, int tail_split, int a_bf16) {
  using Cfg = PairCfg<BN>;
  constexpr int STAGES = Cfg::STAGES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const uint32_t staging = base + Cfg::RING_BYTES;
  const uint32_t bar_base = staging + Cfg::STAGING_BYTES;
  auto a_tile = [&](int s) { return base + (uint32_t)s * Cfg::STAGE_BYTES; };
  auto w_tile = [&](int s) { return base + (uint32_t)s * Cfg::STAGE_BYTES + A_BYTES; };
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
  uint8_t* gen_base = smem_raw + (base - raw);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen_base + Cfg::RING_BYTES + Cfg::STAGING_BYTES + 8 * (2 * STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen_base + Cfg::RING_BYTES + Cfg::STAGING_BYTES + 8 * (2 * STAGES + 4) + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();           // 0 = leader
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int n_m2 = (M + 2 * BM - 1) / (2 * BM), n_n = N / BN, n_tiles = n_m2 * n_n, n_kb = K / BK;

  // Work list of this CTA pair, as pieces (tile, K-block range).
  //  * turn == nullptr: whole tiles, pair p takes tiles p, p + n_pairs, ...
  //  * turn != nullptr (residual epilogue only): stream-K.  The tiles' K-blocks, laid end to end, are cut
  //    into n_pairs equal ranges, so no pair idles in a partial last wave.  A range is at least one
  //    tile long, hence a tile is shared by at most two pairs: the one that owns its first K-blocks
  //    (it adds the bias) and the one that owns the rest.  Each pair walks its range from the LAST tile
  //    to the first, so the piece that starts at K-block 0 is computed early and the completing piece
  //    late; the two TMA reduce-adds into the fp32 output are ordered by a per-(tile, rank, warp) turn
  //    flag in global memory (0 -> 1 by the first piece, back to 0 by the second), which keeps the
  //    result bit-reproducible.
  //  * tail_split > 1 (whole-tile mode only): the tiles left over after the last full round
  //    (n_tiles mod n_pairs of them) are cut along N into tail_split column slices each, and the slices
  //    are dealt round-robin, so the last round costs about 1/tail_split of a tile instead of a whole one.
  //    A slice loads the same W box (only its first rows are used) and issues MMAs with N = BN / tail_split.
  int n_pieces, sk_u0 = 0, sk_u1 = 0, sk_t_last = 0, full_rounds = 0;
  if (turn) {
    const long U = (long)n_tiles * n_kb;
    const long W = (U + n_pairs - 1) / n_pairs;
    sk_u0 = (int)((long)pair * W < U ? (long)pair * W : U);
    sk_u1 = (int)((long)sk_u0 + W < U ? (long)sk_u0 + W : U);
    sk_t_last = sk_u1 > sk_u0 ? (sk_u1 - 1) / n_kb : 0;
    n_pieces = sk_u1 > sk_u0 ? sk_t_last - sk_u0 / n_kb + 1 : 0;
  } else if (tail_split > 1) {
    full_rounds = n_tiles / n_pairs;
    const int slices = (n_tiles - full_rounds * n_pairs) * tail_split;
    n_pieces = full_rounds + (slices > pair ? (slices - pair + n_pairs - 1) / n_pairs : 0);
  } else {
    n_pieces = pair < n_tiles ? (n_tiles - pair + n_pairs - 1) / n_pairs : 0;
  }
  // piece i of this pair: output tile, K-block range, and the column slice [n_off, n_off + n_w) of the tile
  auto get_piece = [&](int i, int& tile, int& kb0, int& kb1, int& n_off, int& n_w) {
    n_off = 0;
    n_w = BN;
    if (turn) {
      tile = sk_t_last - i;
      const int lo = tile * n_kb, hi = lo + n_kb;
      kb0 = (sk_u0 > lo ? sk_u0 : lo) - lo;
      kb1 = (sk_u1 < hi ? sk_u1 : hi) - lo;
    } else {
      kb0 = 0;
      kb1 = n_kb;
      if (tail_split > 1 && i >= full_rounds) {
        const int j = pair + (i - full_rounds) * n_pairs;
        tile = full_rounds * n_pairs + j / tail_split;
        n_w = BN / tail_split;
        n_off = (j % tail_split) * n_w;
      } else {
        tile = pair + i * n_pairs;
      }
    }
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(tfull_bar(a), 1);
      ptx::mbar_init(tempty_bar(a), 16);                  // 8 epilogue warps x 2 CTAs
    }
    abort_flag[0] = 0;
    abort_flag[1] = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async();
  }
  if (warp == 2) {
    ptx::tmem_alloc_pair(ptx::smem_u32((const void*)tmem_slot), Cfg::TMEM_COLS);
    ptx::tmem_relinquish_pair();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();                                // both CTAs' barriers exist before any remote signal
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Programmatic dependent launch: everything above overlapped the previous kernel's tail.  The
  // producer additionally fetches the first weight tiles (weights are never written by a kernel)
  // before it waits for the previous kernel; every other thread waits right here.
  if (!(warp == 0 && lane == 0)) pdl_sync();

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer (both CTAs)
    if (lane == 0) {
      ptx::prefetch_tensormap(&tmap_a);
      ptx::prefetch_tensormap(&tmap_w);
      ptx::prefetch_tensormap(&tmap_out);
      int prefetched = 0;                                  // ring slots whose barrier is armed and W half loaded
      if (n_pieces > 0) {
        int tile, kb0, kb1, n_off, n_w;
        get_piece(0, tile, kb0, kb1, n_off, n_w);
        const int wrow0 = (tile % n_n) * BN + n_off + (int)rank * (n_w / 2);
        for (; prefetched < STAGES && kb0 + prefetched < kb1; ++prefetched) {
          const uint32_t leader_full = ptx::mapa(full_bar(prefetched), 0);
          if (rank == 0) ptx::mbar_expect_tx(full_bar(prefetched), 2 * Cfg::STAGE_BYTES);
          ptx::tma_load_2d_pair(w_tile(prefetched), &tmap_w, (kb0 + prefetched) * BK, wrow0, leader_full);
        }
      }
      pdl_sync();
      int it = 0;
      bool ok = true;
      for (int i = 0; i < n_pieces && ok; ++i) {
        int tile, kb0, kb1, n_off, n_w;
        get_piece(i, tile, kb0, kb1, n_off, n_w);
        const int m2 = tile / n_n, n_blk = tile - m2 * n_n;
        const int row0 = m2 * 2 * BM + (int)rank * BM;                // this CTA's 128 rows of A
        const int wrow0 = n_blk * BN + n_off + (int)rank * (n_w / 2);  // this CTA's half of the W rows of the slice
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t leader_full = ptx::mapa(full_bar(s), 0);
          if (it < prefetched) {                           // slot armed and W already in flight
            ptx::tma_load_2d_pair(a_tile(s), &tmap_a, kb * BK, row0, leader_full);
            continue;
          }
          const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
          if (!ptx::mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { ok = false; break; }
          if (rank == 0) ptx::mbar_expect_tx(full_bar(s), 2 * Cfg::STAGE_BYTES);
          ptx::tma_load_2d_pair(a_tile(s), &tmap_a, kb * BK, row0, leader_full);
          ptx::tma_load_2d_pair(w_tile(s), &tmap_w, kb * BK, wrow0, leader_full);
        }
      }
      if (!ok) *(volatile int*)status = ST2_PRODUCER;
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer (leader only)
    if (lane == 0 && rank == 0) {
      int it = 0;
      bool ok = true;
      for (int i = 0; i < n_pieces && ok; ++i) {
        int tile, kb0, kb1, n_off, n_w;
        get_piece(i, tile, kb0, kb1, n_off, n_w);
        const uint32_t idesc = ptx::idesc_16_f32(2 * BM, n_w, a_bf16 != 0);
        const int acc = i & 1;
        const uint32_t acc_ph = (uint32_t)(i >> 1) & 1u;
        if (!ptx::mbar_wait(tempty_bar(acc), acc_ph ^ 1u, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
          if (!ptx::mbar_wait(full_bar(s), ph, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after();
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            const uint64_t da = ptx::smem_desc_k_sw128(a_tile(s) + k * 32);
            const uint64_t dw = ptx::smem_desc_k_sw128(w_tile(s) + k * 32);
            ptx::umma_f16_pair(d_tmem, da, dw, idesc, (kb > kb0 || k) ? 1u : 0u);
          }
          ptx::umma_commit_pair(empty_bar(s), 3);           // frees the slot in both CTAs
        }
        if (ok) ptx::umma_commit_pair(tfull_bar(acc), 3);   // accumulator complete in both CTAs
      }
      if (!ok) *(volatile int*)status = ST2_MMA;
    }
  } else {
    // ---------------------------------------------------------------- epilogue (warps 2..9, both CTAs)
    const int quarter = warp & 3;                           // TMEM lanes 32*quarter .. +31
    const int half = (warp - 2) >> 2;                       // which half of the BN columns
    bool ok = true;
    for (int i = 0; i < n_pieces && ok; ++i) {
      int tile, kb0, kb1, n_off, n_w;
      get_piece(i, tile, kb0, kb1, n_off, n_w);
      const int m2 = tile / n_n, n_blk = tile - m2 * n_n;
      const int acc = i & 1;
      const uint32_t acc_ph = (uint32_t)(i >> 1) & 1u;
      if (!ptx::mbar_wait(tfull_bar(acc), acc_ph, abort_flag)) { ok = false; break; }
      ptx::tc_fence_after();
      const int row0 = m2 * 2 * BM + (int)rank * BM + quarter * 32;
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
      const uint32_t my_stage = staging + (uint32_t)(warp - 2) * 4096u;
      int* my_turn = turn ? turn + ((size_t)tile * 2 + rank) * 8 + (warp - 2) : nullptr;
      if (row0 < M) {
        if (my_turn && kb0 > 0) {
          // second piece of a shared tile: its reduce-add must follow the first piece's
          if (lane == 0) {
            const long long t0 = clock64();
            int v;
            do {
              asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(my_turn) : "memory");
              if (v != 1 && (*abort_flag || clock64() - t0 > 2000000000LL)) { *abort_flag = 1; break; }
            } while (v != 1);
            asm volatile("fence.proxy.async.global;" ::: "memory");   // the TMA reduce-adds below follow the acquire
          }
          __syncwarp();
          if (*abort_flag) { ok = false; break; }
        }
        constexpr int EC = EpiCols<EPI>::value;
        const int col_tile = n_blk * BN + n_off;                            // first output column of this piece
        const float* bias_tile = kb0 == 0 ? bias + col_tile : nullptr;     // the piece with K-block 0 adds the bias
        // the two warps of a TMEM lane quarter share the piece's n_w columns (a 64-column slice of a
        // 64-column-box epilogue is handled by the first of them alone)
        const int hw = n_w / 2 > EC ? n_w / 2 : EC;
        const int c_begin = half * hw, c_end = (half + 1) * hw < n_w ? (half + 1) * hw : n_w;
        if (EPI == 4 && col_tile >= kv.D) {
          // a K or V tile of the fused QKV projection: straight into the cache rows of the active tokens
          const int which = col_tile / kv.D - 1;                            // 0 = K, 1 = V
          const int col0 = col_tile - (which + 1) * kv.D;
          const int grow = row0 + lane;
          int dst_row = -1;
          if (grow < M) {
            const int b = grow / kv.n;
            const int t = kv.idx ? kv.idx[grow] : grow - b * kv.n;
            dst_row = ((which * kv.B + b) * kv.S + t) * kv.D + col0;
          }
#pragma unroll 1
          for (int c0 = c_begin; c0 < c_end; c0 += 64)
            epilogue_box_scatter(t_row + (uint32_t)c0, bias_tile + c0, (bf16*)kv.cache, dst_row < 0 ? -1 : dst_row + c0,
                                 my_stage, lane);
        } else {
#pragma unroll 1
          for (int c0 = c_begin; c0 < c_end; c0 += EC)
            epilogue_box<(EPI == 4) ? 0 : EPI>(t_row + (uint32_t)c0, bias_tile ? bias_tile + c0 : nullptr, &tmap_out,
                                               col_tile + c0, row0, my_stage, lane, a_bf16 != 0);
        }
        if (my_turn && lane == 0) {
          if (kb0 == 0 && kb1 < n_kb) {
            ptx::bulk_wait_all();                           // this warp's reduce-adds have been performed
            __threadfence();
            asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(my_turn), "r"(1) : "memory");
          } else if (kb0 > 0) {
            *(volatile int*)my_turn = 0;                    // leave the flag clean for the next launch
          }
        }
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive_cluster(ptx::mapa(tempty_bar(acc), 0));
    }
    if (!ok && lane == 0) *(volatile int*)status = ST2_EPILOGUE;
    if (lane == 0) ptx::bulk_wait_read_all();               // the TMA engine has read this warp's staging box;
                                                            // the writes complete with the grid
  }

  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();                                  // peer done with our smem / TMEM and vice versa
  if (warp == 2) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc_pair(tmem_base, Cfg::TMEM_COLS);
  }
}

bool make_map_2d(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows,
                 bool ieee_half) {
  const uint64_t dims[2] = {cols, rows};
  const uint64_t strides[1] = {ld * 2};
  const uint32_t box[2] = {BK, box_rows};
  return tma_make_map_bf16(map, ptr, 2, dims, strides, box, true, ieee_half);
}

// Number of CTA pairs of this kernel that can be resident at once on the current device (queried
// once per device and instantiation).  The grid never exceeds it, so that every pair of a launch is
// running while stream-K pieces wait for each other's turn flags.
template <int BN, int EPI>
cudaError_t max_resident_pairs(int* out) {
  static int cached[kMaxDevices] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (!cached[dev]) {
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (sms / 2 > 0 ? sms / 2 : 1));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = (size_t)PairCfg<BN>::SMEM_BYTES;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    e = cudaOccupancyMaxActiveClusters(&clusters, gemm_tcgen05_2cta_kernel<BN, EPI>, &cfg);
    if (e != cudaSuccess) return e;
    if (clusters > sms / 2) clusters = sms / 2;
    cached[dev] = clusters > 0 ? clusters : 1;
  }
  *out = cached[dev];
  return cudaSuccess;
}

template <int BN, int EPI>
cudaError_t launch_pair(const CUtensorMap& ta, const CUtensorMap& tw, const CUtensorMap& to, int M, int N, int K,
                        const float* bias, int* status, int* turn, const KvScatter& kv, int a_bf16, const GemmTuning& tune,
                        cudaStream_t st) {
  static size_t smem_set[kMaxDevices] = {};
  cudaError_t e = ensure_dynamic_smem(gemm_tcgen05_2cta_kernel<BN, EPI>, (size_t)PairCfg<BN>::SMEM_BYTES, smem_set);
  if (e != cudaSuccess) return e;
  const int n_tiles = ((M + 2 * BM - 1) / (2 * BM)) * (N / BN);
  int max_pairs = 1;
  e = max_resident_pairs<BN, EPI>(&max_pairs);
  if (e != cudaSuccess) return e;
  const int pairs = n_tiles < max_pairs ? n_tiles : max_pairs;
  // stream-K only for the reduce-add epilogue and only where whole tiles would waste a large part of
  // the last wave: a few waves at most (measured: +2 % on the cache-aware step, but -4 % on the
  // 9-wave full step, where the ordering costs more than the 4 % of idle SMs it removes)
  // ... and only for long tiles (K >= 2048, i.e. fc2): the completing piece has to wait until the first
  // piece's reduce-adds are complete, about 3 us after its last MMA, which a 16-K-block tile (7 us of MMA
  // work, the out-projection) cannot hide: measured 18 us with and without stream-K there.
  int* use_turn = (EPI == 1 && turn && tune.stream_k && K >= 2048 && n_tiles > max_pairs && n_tiles % max_pairs != 0 &&
                   n_tiles < 4 * max_pairs) ? turn : nullptr;
  // Whole-tile mode: cut the tiles of the last, partial round into 2 or 4 column slices when that
  // shortens the round (cost model in tile units, below).
  const int split_on = tune.tail_split;              // 0 off, 1 cost model, 2 / 4 forced (measurement only)
  int tail_split = 1;
  const int left = n_tiles % pairs;
  if (!use_turn && (split_on == 2 || split_on == 4) && BN == 256 && left > 0) {
    tail_split = split_on;
  } else if (!use_turn && split_on && BN == 256 && left > 0) {
    double best = 1.0;
    for (int sp = 2; sp <= 4; sp *= 2) {
      // measured at K = 1024: a half-width slice costs about 0.75 of a tile, a quarter-width one about 0.65
      // (every slice loads the whole A tile again and pays its own ramp and epilogue)
      const double cost = (double)((left * sp + pairs - 1) / pairs) * (1.0 / sp + (sp == 2 ? 0.25 : 0.40));
      if (cost < best - 0.05) { best = cost; tail_split = sp; }
    }
  }
  return launch_pdl(gemm_tcgen05_2cta_kernel<BN, EPI>, dim3(2 * pairs), dim3(kThreads), (size_t)PairCfg<BN>::SMEM_BYTES,
                    st, ta, tw, to, M, N, K, bias, status, use_turn, kv, tail_split, a_bf16);
}

}  // namespace

// Tile width: 256 whenever N allows it.  Measured on B200 at M = 4.3-5.8 k rows, the 128-wide
// pair tile costs about 0.7x a 256-wide one (1.5x the operand bytes per flop), so it never wins
// back what it gains in wave balance.  tile_n = 128 overrides (measurement only).
int gemm_tcgen05_2cta_pick_bn(int M, int N, int tile_n) {
  (void)M;
  if (N % 256) return 128;
  return tile_n == 128 ? 128 : 256;
}

size_t gemm_tcgen05_2cta_turn_bytes(int M, int N) {
  const size_t n_m2 = ((size_t)M + 2 * BM - 1) / (2 * BM);
  return n_m2 * (size_t)(N / 128) * 16 * sizeof(int);
}

cudaError_t launch_gemm_tcgen05_2cta(const void* a, int lda, int M, const void* w, const float* bias, int N, int K,
                                     int epilogue, void* out, bool a_bf16, int* status, cudaStream_t st,
                                     const GemmTuning& tune, int* turn, const KvScatter* kv_scatter) {
  if (M == 0) return cudaSuccess;
  KvScatter kv = {nullptr, nullptr, 1, 1, 1, 1 << 30};
  if (epilogue == 4) {
    // q, K and V column ranges must each be whole tiles, and cache offsets must fit 32 bits
    if (!kv_scatter || !kv_scatter->cache || N != 3 * kv_scatter->D || kv_scatter->D % 256 ||
        (long)2 * kv_scatter->B * kv_scatter->S * kv_scatter->D >= (1L << 31) || ((uintptr_t)kv_scatter->cache & 15))
      return cudaErrorInvalidValue;
    kv = *kv_scatter;
  }
  if (N % 128 || K % BK || lda % 8 || ((uintptr_t)a & 15) || ((uintptr_t)w & 15)) return cudaErrorInvalidValue;
  const int bn = gemm_tcgen05_2cta_pick_bn(M, N, tune.tile_n);
  CUtensorMap ta, tw, to;
  if (!make_map_2d(&ta, a, (uint64_t)M, (uint64_t)K, (uint64_t)lda, BM, !a_bf16)) return cudaErrorInvalidValue;
  if (!make_map_2d(&tw, w, (uint64_t)N, (uint64_t)K, (uint64_t)K, (uint32_t)(bn / 2), !a_bf16)) return cudaErrorInvalidValue;
  if (((uintptr_t)out & 15) || !tma_make_store_map(&to, out, (uint64_t)M, (uint64_t)N, epilogue == 1 ? 4 : 2))
    return cudaErrorInvalidValue;
#define MARCHE_GEMM2_CASE(BN_, EPI_) \
  if (bn == BN_ && epilogue == EPI_)   \
    return launch_pair<BN_, EPI_>(ta, tw, to, M, N, K, bias, status, turn, kv, a_bf16 ? 1 : 0, tune, st);
  MARCHE_GEMM2_CASE(256, 0) MARCHE_GEMM2_CASE(256, 1) MARCHE_GEMM2_CASE(256, 2) MARCHE_GEMM2_CASE(256, 4)
  MARCHE_GEMM2_CASE(128, 0) MARCHE_GEMM2_CASE(128, 1) MARCHE_GEMM2_CASE(128, 2)
#undef MARCHE_GEMM2_CASE
  return cudaErrorInvalidValue;
}

}  // namespace marche
