// Host-side launch wrappers, one per kernel; raw device pointers and a stream.
// Every wrapper only enqueues work and returns the launch's cudaError_t.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace marche {

// Element type of an activation output: fp32, saturating IEEE fp16, or bf16.
enum { OUT_F32 = 0, OUT_F16 = 1, OUT_BF16 = 2 };

// K1: gather + LayerNorm (output type out_kind).  rows = B*n; src row of (b, j) is src[b][idx ? idx[b][j] : j].
cudaError_t launch_gather_layernorm(int out_kind, const float* src, int src_rows, const int32_t* idx,
                                    int B, int n, int D, const float* gamma, const float* beta, float eps,
                                    float* x_out, void* u_out, cudaStream_t st, const int32_t* out_idx = nullptr,
                                    int out_rows = 0);

// K5: K/V write-back into one block's cache slice [2][B][S][D]; idx NULL = identity.
cudaError_t launch_scatter_kv(bool bf16_t, const void* k, const void* v, int ld_kv, const int32_t* idx,
                              int B, int n, int S, int D, void* cache_layer, cudaStream_t st);

// fp32 row scatter dst[b][idx ? idx[b][j] : j] = rows[b][j].
cudaError_t launch_scatter_rows(const float* rows, const int32_t* idx, int B, int n, int S, int D,
                                float* dst, cudaStream_t st);

// fp32 row gather out[b][j] = src[b][idx[b][j]].
cudaError_t launch_gather_rows(const float* src, const int32_t* idx, int B, int n, int S, int D, float* out,
                               cudaStream_t st);

// out[r] = table[idx[r]] for total_rows rows of D floats (table shared by all samples).
cudaError_t launch_gather_table_rows(const float* table, const int32_t* idx, long total_rows, int D, float* out,
                                     cudaStream_t st);

// out[b][s] = mask_token + pos[s], float [B][S][D] (Eq. 2, masked positions of the decoder's input).
cudaError_t launch_fill_mask_rows(const float* mask_token, const float* pos, int B, int S, int D, float* out,
                                  cudaStream_t st);

// a0 prologue: is_new[b][j] (may be NULL with n_active = 0) and the candidate mask cand[b][t].
cudaError_t launch_step_flags(const int32_t* active_idx, int n_active, const int32_t* new_idx, int n_new,
                              const int32_t* excl_idx, int n_excl, int B, int S, uint8_t* is_new,
                              uint8_t* cand, cudaStream_t st);

cudaError_t launch_build_active(const int32_t* a, int na, const int32_t* b, int nb, const int32_t* c, int nc,
                                int B, int32_t* out, cudaStream_t st);

// Index validation; *status (device or mapped host int) is set non-zero on a violation.
cudaError_t launch_validate(const int32_t* active_idx, int n_active, const int32_t* new_idx, int n_new,
                            const int32_t* excl_idx, int n_excl, int B, int S, int* status, cudaStream_t st);

// K4: optional fixed-order head reduction of score partials [B][H][S] into scores [B][S],
// then top-k among cand (k may be 0: reduction only).
// policy 0 = highest scores, 1 = lowest scores, 2 = random (counter-based hash of seed, sample, token).
cudaError_t launch_topk(const float* partial, int H, float* scores, const uint8_t* cand, int B, int S, int k,
                        int32_t* refresh_idx, cudaStream_t st, int policy = 0, uint32_t seed = 0);

// K2 of the fp32 configuration (SIMT, fp32 operands and outputs).
cudaError_t launch_gemm_simt(const float* a, int lda, int M, const float* w, const float* bias,
                             int N, int K, int epilogue, float* out, cudaStream_t st);

// K2 (16-bit operands, tcgen05/TMEM fed by TMA).  N % 128 == 0, K % 64 == 0, lda % 8 == 0, 16-byte aligned
// operands.  a_bf16: both operands (and the GELU epilogue's output) are bf16, otherwise IEEE fp16.
// `status` is a device-visible int that bounded waits set when they give up.
cudaError_t launch_gemm_tcgen05(const void* a, int lda, int M, const void* w, const float* bias, int N, int K,
                                int epilogue, void* out, bool a_bf16, int* status, cudaStream_t st);
int gemm_tcgen05_pick_bn(int M, int N);
// Where the K and V columns of a fused QKV projection go (Algorithm 1 line 11 done by the projection's
// epilogue, epilogue code 4): row r of the GEMM is active token j = r % n of sample b = r / n, its cache row is
// idx[r] (identity when idx is NULL).  cache is one block's [2][B][S][D] slice (bf16).  Needs N == 3 D,
// D a multiple of 256 and 2 B S D < 2^31.
struct KvScatter {
  const int32_t* idx;
  void* cache;
  int n, S, B, D;
};

// Same contract, tcgen05.mma cta_group::2: CTA pairs share 256 x BN tiles (cluster of 2, no multicast).
// `turn`: optional zero-filled device scratch of gemm_tcgen05_2cta_turn_bytes(M, N) bytes; with it the
// residual epilogue may use stream-K (ordered reduce-adds; the flags are left zero again).
struct GemmTuning {
  bool stream_k = true;   // residual epilogue: stream-K with ordered reduce-adds where it pays
  int tail_split = 1;     // partial last round of tiles cut into column slices: 0 off, 1 cost model, 2 / 4 forced
  int tile_n = 0;         // 0: 256-wide tiles whenever N allows; 128 forces the narrow tile
};
cudaError_t launch_gemm_tcgen05_2cta(const void* a, int lda, int M, const void* w, const float* bias, int N, int K,
                                     int epilogue, void* out, bool a_bf16, int* status, cudaStream_t st,
                                     const GemmTuning& tune, int* turn = nullptr,
                                     const KvScatter* kv_scatter = nullptr);
size_t gemm_tcgen05_2cta_turn_bytes(int M, int N);
int gemm_tcgen05_2cta_pick_bn(int M, int N, int tile_n);

// K3 of the fp32 configuration (SIMT): attention of n queries per sample over all S cache rows.
cudaError_t launch_attention_simt(const float* q, int ld_q, int B, int n, int S, int H, int dh,
                                  const float* cache_layer, const uint8_t* is_new, float* score_partial,
                                  float* o, cudaStream_t st);
size_t attention_simt_smem(int S, int dh);

// K3 (bf16 q / cache, TMA-staged K/V tiles, tensor-core QK^T and PV, fused score column sums).
// head_dim 64 or 80; ld_q even; cache_layer 16-byte aligned.  o is written in the projections'
// operand type: bf16 when o_bf16, saturating fp16 otherwise.
cudaError_t launch_attention_mma(const void* q, int ld_q, int B, int n, int S, int H, int dh,
                                 const void* cache_layer, const uint8_t* is_new, float* score_partial, void* o,
                                 bool o_bf16, int* status, cudaStream_t st);

// The same kernel's plain flavour for n <= 32 as a persistent launch (equal item shares per resident CTA, loads
// running ahead across items, query rows by TMA).  ld_q % 8 == 0; q and cache_layer 16-byte aligned.
cudaError_t launch_attention_mma_persist(const void* q, int ld_q, int B, int n, int S, int H, int dh,
                                         const void* cache_layer, void* o, bool o_bf16, int* status, cudaStream_t st);

// K3 on tcgen05 (head_dim 64 only): S = Q K^T and O = P V as tcgen05.mma with TMEM accumulators.
// ld_q % 8 == 0; q and cache_layer 16-byte aligned.
cudaError_t launch_attention_tcgen05(const void* q, int ld_q, int B, int n, int S, int H, int dh,
                                     const void* cache_layer, const uint8_t* is_new, float* score_partial, void* o,
                                     bool o_bf16, int* status, cudaStream_t st);

// K3 on tcgen05, single pass with online softmax, persistent over (sample, head) items, P kept in tensor
// memory (head_dim 64, no relevance scores).  Same alignment rules as launch_attention_tcgen05, o 16-byte aligned.
cudaError_t launch_attention_tc_stream(const void* q, int ld_q, int B, int n, int S, int H, int dh,
                                       const void* cache_layer, void* o, bool o_bf16, int* status, cudaStream_t st);

// K3, two-segment flavour (Eq. 6-10 without concatenation, then the cache write-back of Algorithm 1
// line 11 by the same kernel): fresh K/V are columns k_off / v_off of the compact qkv buffer
// [B*n][ld]; active_idx NULL = identity.  Same type and alignment rules as launch_attention_mma.
cudaError_t launch_attention_twoseg(const void* qkv, int ld, int k_off, int v_off, int B, int n, int S, int H, int dh,
                                    const int32_t* active_idx, void* cache_layer, const uint8_t* is_new,
                                    float* score_partial, void* o, bool o_bf16, int* status, cudaStream_t st);

// Diagnostic: one thread waits, with the library's bounded mbarrier wait, on a barrier nothing ever
// arrives on; after limit_cycles it gives up, writes a code to *status and the kernel returns.
cudaError_t launch_bounded_wait_probe(long long limit_cycles, int* status, cudaStream_t st);

}  // namespace marche
