// C ABI of libmarche (see include/marche.h) and the per-step kernel sequence.
//
// The step is a fixed chain of launches on the caller's stream, per block:
//   K1 LayerNorm (with the row gather at block 0) -> K2 QKV projection -> K5 K/V
//   write-back -> K3 attention over the whole cache (+ score partials at the scoring
//   block) -> K2 output projection (+residual) -> K1 LayerNorm -> K2 fc1 (+GELU) ->
//   K2 fc2 (+residual);
// then once per step the fp32 row scatter into hidden_out and K4 (score reduction +
// top-K).  Nothing here allocates device memory or synchronises, except where the
// header says a call is synchronous.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <utility>
#include <vector>

#include "../../include/marche.h"
#include "kernels.h"
#include "launch_pdl.h"

using namespace marche;

struct marche_ctx {
  marche_config cfg;
  std::vector<marche_block_weights> blocks;
  marche_mar_weights mar{};                           // glue of the two-stage model (marche_set_mar_weights)
  bool has_mar = false;
  int device = 0;
  bool bf16 = false;                                  // 16-bit context: q/k/v and the cache are bf16
  bool a_bf16 = false;                                // ... and the projections' operands are bf16 too (else fp16)
  int a_kind = OUT_F32;                               // element type of LayerNorm / attention / GELU outputs
  size_t eb = 4;
  float eps = 1e-6f;
  int score_layer = 0;
  std::vector<int> extra_score_layers;                // blocks that also accumulate scores (analysis only)
  marche_tuning tune;                                 // kernel-selection switches (marche_set_tuning)
  unsigned skip_mask = 0;                             // measurement hook: kernel classes that are not launched
  unsigned repeat_mask = 0;                           // measurement hook: kernel classes that are launched twice
  std::vector<std::pair<const void*, bool>> caches;  // (cache pointer, filled)
  int* status_host = nullptr;                         // pinned, mapped
  int* status_dev = nullptr;
  std::string last_error;
  // launch accounting and optional per-kernel-class timing
  unsigned long long launches = 0;
  bool profiling = false;
  std::vector<cudaEvent_t> events;     // pool, reused between profile runs
  std::vector<int> event_class;        // class of the launch that follows event i
};

namespace {

inline size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

struct WsLayout {
  size_t scores, partial, cand, is_new, turn, turn_bytes, x, x2, x3, u, qkv, o, g, total;
};

WsLayout ws_layout(const marche_ctx* c, int nA) {
  const size_t B = c->cfg.batch, S = c->cfg.seq_len, D = c->cfg.width, F = c->cfg.mlp_dim, H = c->cfg.n_heads;
  const size_t M = B * (size_t)nA, eb = c->eb;
  WsLayout w;
  size_t off = 0;
  w.scores = off;  off += align256(B * S * sizeof(float));
  w.partial = off; off += align256((1 + c->extra_score_layers.size()) * B * H * S * sizeof(float));
  w.cand = off;    off += align256(B * S);
  w.is_new = off;  off += align256(M);
  w.turn_bytes = gemm_tcgen05_2cta_turn_bytes((int)M, (int)D);   // stream-K turn flags of the residual GEMMs
  w.turn = off;    off += align256(w.turn_bytes);
  w.x = off;       off += align256(M * D * sizeof(float));
  w.x2 = off;      off += align256(M * D * sizeof(float));   // second residual buffer (in-step selection)
  w.x3 = off;      off += align256(M * D * sizeof(float));   // decoder input of the two-stage step
  w.u = off;       off += align256(M * D * eb);
  w.qkv = off;     off += align256(M * 3 * D * eb);
  w.o = off;       off += align256(M * D * eb);
  w.g = off;       off += align256(M * F * eb);
  w.total = off;
  return w;
}

int cuda_fail(marche_ctx* c, cudaError_t e, const char* what) {
  if (c) c->last_error = std::string(what) + ": " + cudaGetErrorString(e);
  return MARCHE_ECUDA;
}

#define MARCHE_TRY(call, what)                              \
  do {                                                      \
    cudaError_t e__ = (call);                               \
    if (e__ != cudaSuccess) return cuda_fail(ctx, e__, what); \
  } while (0)

// Counts a launch and, while profiling, records an event in front of it.  The time from
// this event to the next one (kernel plus the gap before its successor) is charged to `cls`.
void mark(marche_ctx* ctx, int cls, cudaStream_t st) {
  ++ctx->launches;
  if (!ctx->profiling) return;
  const size_t i = ctx->event_class.size();
  if (i >= ctx->events.size()) {
    cudaEvent_t e;
    if (cudaEventCreate(&e) != cudaSuccess) return;
    ctx->events.push_back(e);
  }
  cudaEventRecord(ctx->events[i], st);
  ctx->event_class.push_back(cls);
}

marche_tuning default_tuning() {
  marche_tuning t;
  t.stream_k = 1;
  t.fuse_qkv_scatter = 1;
  t.attention_kernel = MARCHE_ATTENTION_AUTO;
  t.attention_tc_min_rows = 48;
  t.two_segment_attention = 0;
  t.gemm_kernel = MARCHE_GEMM_AUTO;
  t.tail_split = 1;
  t.tile_n = 0;
  t.pdl = 1;
  return t;
}

// Every call that touches the device starts here: the context belongs to the device that was
// current at marche_create, and its pointers mean nothing on another one.
int enter(marche_ctx* ctx) {
  if (!ctx) return MARCHE_EINVAL;
  int dev = -1;
  const cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaGetDevice");
  if (dev != ctx->device) {
    char msg[128];
    snprintf(msg, sizeof msg, "the context was created on device %d but device %d is current", ctx->device, dev);
    ctx->last_error = msg;
    return MARCHE_EINVAL;
  }
  return MARCHE_OK;
}
#define MARCHE_ENTER(ctx)        \
  do {                           \
    const int rc__ = enter(ctx); \
    if (rc__) return rc__;       \
  } while (0)

int misaligned(marche_ctx* ctx, const char* what) {
  ctx->last_error = std::string(what) + ": a 16-bit context needs 16-byte aligned operands and row strides "
                    "that are multiples of 8 elements (there is no slow path to fall back to)";
  return MARCHE_EINVAL;
}

GemmTuning gemm_tuning(const marche_ctx* ctx) {
  GemmTuning g;
  g.stream_k = ctx->tune.stream_k != 0;
  g.tail_split = ctx->tune.tail_split;
  g.tile_n = ctx->tune.tile_n;
  return g;
}

inline bool skipped(const marche_ctx* ctx, int cls) { return (ctx->skip_mask >> cls) & 1u; }
inline int launches_of(const marche_ctx* ctx, int cls) { return ((ctx->repeat_mask >> cls) & 1u) ? 2 : 1; }

int refresh_count(float ratio, int S, int n_cand) {
  const int want = (int)std::floor((double)ratio * (double)S + 0.5);
  return want < n_cand ? (want < 0 ? 0 : want) : n_cand;
}

// Slot of block l in the per-head score partials: 0 = the scoring block that drives the selection,
// 1.. = the extra analysis blocks, -1 = this block accumulates no scores.
int score_slot(const marche_ctx* ctx, int l) {
  if (l == ctx->score_layer) return 0;
  for (size_t i = 0; i < ctx->extra_score_layers.size(); ++i)
    if (ctx->extra_score_layers[i] == l) return (int)i + 1;
  return -1;
}

// True when the QKV projection of M rows can write K and V into the cache itself (CTA-pair GEMM,
// whole 256-column tiles per q / K / V range, 32-bit cache offsets): no scatter_kv launch then.
bool qkv_scatter_fused(const marche_ctx* ctx, int M, int S) {
  const marche_config& c = ctx->cfg;
  return ctx->tune.fuse_qkv_scatter && ctx->bf16 && !ctx->tune.two_segment_attention && ctx->tune.tile_n != 128 &&
         (ctx->tune.gemm_kernel == MARCHE_GEMM_PAIR || (ctx->tune.gemm_kernel == MARCHE_GEMM_AUTO && M > 128)) &&
         c.width % 256 == 0 &&
         (long)2 * c.batch * S * c.width < (1L << 31);
}

int do_linear(marche_ctx* ctx, int cls, const void* a, int lda, int M, const void* w, const float* bias, int N, int K,
              int epi, void* out, cudaStream_t st, int* turn = nullptr, const KvScatter* kv = nullptr) {
  if (skipped(ctx, cls)) return MARCHE_OK;
  if (!ctx->bf16) {
    if (M > 0) mark(ctx, cls, st);
    MARCHE_TRY(launch_gemm_simt((const float*)a, lda, M, (const float*)w, bias, N, K, epi, (float*)out, st), "gemm");
    return MARCHE_OK;
  }
  // 16-bit contexts run on the tensor cores or not at all
  if (N % 128 || K % 64) return MARCHE_ESHAPE;
  if (lda % 8 || (((uintptr_t)a | (uintptr_t)w | (uintptr_t)out) & 15)) return misaligned(ctx, "projection");
  const bool pair = ctx->tune.gemm_kernel == MARCHE_GEMM_PAIR || (ctx->tune.gemm_kernel == MARCHE_GEMM_AUTO && M > 128);
  for (int r = 0; r < launches_of(ctx, cls); ++r) {
    if (M > 0) mark(ctx, cls, st);
    if (pair)
      MARCHE_TRY(launch_gemm_tcgen05_2cta(a, lda, M, w, bias, N, K, epi, out, ctx->a_bf16, ctx->status_dev, st,
                                          gemm_tuning(ctx), turn, kv), "gemm_tcgen05_2cta");
    else
      MARCHE_TRY(launch_gemm_tcgen05(a, lda, M, w, bias, N, K, epi, out, ctx->a_bf16, ctx->status_dev, st), "gemm_tcgen05");
  }
  return MARCHE_OK;
}

int do_attention(marche_ctx* ctx, const void* q, int ld_q, int n, const void* cache_layer, const uint8_t* is_new,
                 float* partial, void* o, cudaStream_t st, int S_kv = 0) {
  const marche_config& c = ctx->cfg;
  const int S = S_kv > 0 ? S_kv : c.seq_len;            // tokens per sample in cache_layer [2][B][S][D]
  if (skipped(ctx, MARCHE_KC_ATTENTION)) return MARCHE_OK;
  if (!ctx->bf16) {
    if (n > 0) mark(ctx, MARCHE_KC_ATTENTION, st);
    MARCHE_TRY(launch_attention_simt((const float*)q, ld_q, c.batch, n, S, c.n_heads, c.head_dim, (const float*)cache_layer,
                                     is_new, partial, (float*)o, st), "attention");
    return MARCHE_OK;
  }
  if (ld_q % 2 || ((uintptr_t)q & 3) || ((uintptr_t)cache_layer & 15) || ((uintptr_t)o & 15)) return misaligned(ctx, "attention");
  for (int rep_i = 0; rep_i < launches_of(ctx, MARCHE_KC_ATTENTION); ++rep_i) {
  if (n > 0) mark(ctx, MARCHE_KC_ATTENTION, st);
  // Three tensor-core kernels.  At small active sets the step is bound by streaming the cache and the
  // mma.sync kernel (several small CTAs per SM, one pass) is fastest: 40 us vs 50 us at n = 41..48 (S 320).
  // From 49 rows, where the mma.sync kernel needs a fourth consumer warp and drops to two CTAs per SM, the
  // single-pass tcgen05 kernel wins (S 320: 50 vs 56 us at n = 49..64, 54 vs 110 us at n = 77, 141 vs 303 us at
  // n = 320; S 1088: 77 vs 82 us at n = 49..64, 81 vs 252 us at n = 116, 129 vs 256 us at n = 159).  The
  // relevance scores need final weights, hence the two-pass tcgen05 kernel there (74 vs 143 us at n = 77).
  // marche_tuning.attention_kernel forces one of them; head_dim 80 has only the mma.sync kernel.
  const int tc_min = is_new ? 64 : ctx->tune.attention_tc_min_rows;
  const int ak = ctx->tune.attention_kernel;
  const bool tc5 = c.head_dim == 64 && ld_q % 8 == 0 && ((uintptr_t)q & 15) == 0 &&
                   (ak == MARCHE_ATTENTION_TCGEN05 || ak == MARCHE_ATTENTION_TCGEN05_TWO_PASS ||
                    (ak == MARCHE_ATTENTION_AUTO && n > tc_min));
  // plain flavour: single-pass streaming kernel; the relevance scores need final weights, i.e. two passes
  if (tc5 && !is_new && ak != MARCHE_ATTENTION_TCGEN05_TWO_PASS)
    MARCHE_TRY(launch_attention_tc_stream(q, ld_q, c.batch, n, S, c.n_heads, c.head_dim, cache_layer, o, ctx->a_bf16,
                                          ctx->status_dev, st), "attention_tc_stream");
  else if (tc5)
    MARCHE_TRY(launch_attention_tcgen05(q, ld_q, c.batch, n, S, c.n_heads, c.head_dim, cache_layer, is_new,
                                        partial, o, ctx->a_bf16, ctx->status_dev, st), "attention_tcgen05");
  else if (!is_new && n <= 32 && ld_q % 8 == 0 && ((uintptr_t)q & 15) == 0)
    // very small active sets, no scores: the persistent launch of the same arithmetic (31 vs 34 us at n = 8,
    // 32 vs 36 us at n = 24..32, S 320); above 32 rows one CTA per item is as fast or faster
    MARCHE_TRY(launch_attention_mma_persist(q, ld_q, c.batch, n, S, c.n_heads, c.head_dim, cache_layer, o, ctx->a_bf16,
                                            ctx->status_dev, st), "attention_mma_persist");
  else
    MARCHE_TRY(launch_attention_mma(q, ld_q, c.batch, n, S, c.n_heads, c.head_dim, cache_layer, is_new,
                                    partial, o, ctx->a_bf16, ctx->status_dev, st), "attention_mma");
  }
  return MARCHE_OK;
}

struct StackBufs {
  float* scores; float* partial; uint8_t* cand; uint8_t* is_new;
  float* x; float* x2; float* x3; char* u; char* qkv; char* o; char* g;
  int* turn;
};

StackBufs carve(void* workspace, const WsLayout& w) {
  char* ws = (char*)workspace;
  StackBufs b;
  b.scores = (float*)(ws + w.scores);
  b.partial = (float*)(ws + w.partial);
  b.cand = (uint8_t*)(ws + w.cand);
  b.is_new = (uint8_t*)(ws + w.is_new);
  b.turn = (int*)(ws + w.turn);
  b.x = (float*)(ws + w.x);
  b.x2 = (float*)(ws + w.x2);
  b.x3 = (float*)(ws + w.x3);
  b.u = ws + w.u;
  b.qkv = ws + w.qkv;
  b.o = ws + w.o;
  b.g = ws + w.g;
  return b;
}

// Blocks [l_begin, l_end) for M = B*nA rows whose token positions are idx (nullptr = identity,
// nA == S).  When gather_src is non-null the first block's LayerNorm gathers its rows from
// gather_src[b][idx][:] (float [B][src_rows][D]) and writes the compact residual rows to x;
// otherwise x already holds them.  is_new (flags of the scoring queries) is used at the scoring block.
// S_kv > 0: these blocks keep only S_kv tokens per sample, laid out [2][B][S_kv][D] at the start of each
// block's cache slice (the encoder over the known tokens, whose K/V do not outlive the step).
int run_blocks(marche_ctx* ctx, int l_begin, int l_end, const float* gather_src, int src_rows, const int32_t* idx,
               int nA, float* x, const StackBufs& bf, void* kv_cache, const uint8_t* is_new, cudaStream_t st,
               int S_kv = 0) {
  const marche_config& c = ctx->cfg;
  const int B = c.batch, S = S_kv > 0 ? S_kv : c.seq_len, D = c.width, F = c.mlp_dim;
  const int M = B * nA;
  const size_t eb = ctx->eb;
  const size_t layer_bytes = (size_t)2 * B * c.seq_len * D * eb;
  const int32_t* kv_idx = S_kv > 0 ? nullptr : idx;   // compact layout: row j of the sample is token j
  for (int l = l_begin; l < l_end; ++l) {
    const marche_block_weights& bw = ctx->blocks[l];
    char* cache_l = (char*)kv_cache + (size_t)l * layer_bytes;
    const int slot = is_new ? score_slot(ctx, l) : -1;
    const uint8_t* flags_l = slot >= 0 ? is_new : nullptr;
    float* partial_l = bf.partial + (size_t)(slot > 0 ? slot : 0) * B * c.n_heads * c.seq_len;
    const bool skip_ln = skipped(ctx, MARCHE_KC_GATHER_LN);
    if (!skip_ln) mark(ctx, MARCHE_KC_GATHER_LN, st);
    for (int r = 0; r < (skip_ln ? 0 : launches_of(ctx, MARCHE_KC_GATHER_LN)); ++r) {
      if (r) mark(ctx, MARCHE_KC_GATHER_LN, st);
      if (l == l_begin && gather_src)
        MARCHE_TRY(launch_gather_layernorm(ctx->a_kind, gather_src, src_rows, idx, B, nA, D, bw.ln1_g, bw.ln1_b, ctx->eps,
                                           x, bf.u, st), "gather_layernorm");
      else
        MARCHE_TRY(launch_gather_layernorm(ctx->a_kind, x, nA, nullptr, B, nA, D, bw.ln1_g, bw.ln1_b, ctx->eps,
                                           nullptr, bf.u, st), "layernorm1");
    }
    const bool fused_kv = qkv_scatter_fused(ctx, M, S);
    const KvScatter kvs = {kv_idx, cache_l, nA, S, B, D};
    int rc = do_linear(ctx, MARCHE_KC_GEMM_QKV, bf.u, D, M, bw.w_qkv, bw.b_qkv, 3 * D, D, fused_kv ? 4 : MARCHE_EPI_BIAS,
                       bf.qkv, st, nullptr, fused_kv ? &kvs : nullptr);
    if (rc) return rc;
    if (fused_kv) {
      // the projection's epilogue has written K and V into the cache (Algorithm 1 line 11)
      rc = do_attention(ctx, bf.qkv, 3 * D, nA, cache_l, flags_l, partial_l, bf.o, st, S);
      if (rc) return rc;
    } else if (ctx->tune.two_segment_attention && ctx->bf16) {
      // two-segment attention: fresh K/V read in place, cache write-back by the same kernel
      mark(ctx, MARCHE_KC_ATTENTION, st);
      MARCHE_TRY(launch_attention_twoseg(bf.qkv, 3 * D, D, 2 * D, B, nA, S, c.n_heads, c.head_dim, kv_idx, cache_l,
                                         flags_l, partial_l, bf.o, ctx->a_bf16, ctx->status_dev, st),
                 "attention_twoseg");
    } else {
      mark(ctx, MARCHE_KC_SCATTER_KV, st);
      MARCHE_TRY(launch_scatter_kv(ctx->bf16, bf.qkv + (size_t)D * eb, bf.qkv + (size_t)2 * D * eb, 3 * D, kv_idx, B, nA,
                                   S, D, cache_l, st), "scatter_kv");
      rc = do_attention(ctx, bf.qkv, 3 * D, nA, cache_l, flags_l, partial_l, bf.o, st,
                        S);
      if (rc) return rc;
    }
    rc = do_linear(ctx, MARCHE_KC_GEMM_O, bf.o, D, M, bw.w_o, bw.b_o, D, D, MARCHE_EPI_BIAS_RESIDUAL, x, st, bf.turn);
    if (rc) return rc;
    for (int r = 0; r < (skip_ln ? 0 : launches_of(ctx, MARCHE_KC_GATHER_LN)); ++r) {
      mark(ctx, MARCHE_KC_GATHER_LN, st);
      MARCHE_TRY(launch_gather_layernorm(ctx->a_kind, x, nA, nullptr, B, nA, D, bw.ln2_g, bw.ln2_b, ctx->eps, nullptr,
                                         bf.u, st), "layernorm2");
    }
    rc = do_linear(ctx, MARCHE_KC_GEMM_FC1, bf.u, D, M, bw.w_fc1, bw.b_fc1, F, D, MARCHE_EPI_BIAS_GELU, bf.g, st);
    if (rc) return rc;
    rc = do_linear(ctx, MARCHE_KC_GEMM_FC2, bf.g, F, M, bw.w_fc2, bw.b_fc2, D, F, MARCHE_EPI_BIAS_RESIDUAL, x, st, bf.turn);
    if (rc) return rc;
  }
  return MARCHE_OK;
}

// The whole stack for M = B*nA rows.  active_idx == nullptr means every token (nA == S).
int run_stack(marche_ctx* ctx, const float* hidden, void* kv_cache, const int32_t* active_idx, int nA,
              const int32_t* new_idx, int n_new, const int32_t* excl_idx, int n_excl, float ratio,
              float* hidden_out, int32_t* refresh_idx, int* n_refresh, void* workspace, size_t ws_bytes,
              cudaStream_t st) {
  const marche_config& c = ctx->cfg;
  const int B = c.batch, S = c.seq_len, D = c.width, H = c.n_heads, L = c.n_blocks;
  if (!hidden || !kv_cache || !hidden_out || !workspace || hidden == hidden_out) return MARCHE_EINVAL;
  if (((uintptr_t)hidden | (uintptr_t)hidden_out | (uintptr_t)kv_cache) & 15) return MARCHE_EINVAL;
  if (nA < 1 || nA > S || n_new < 0 || n_new > nA || n_excl < 0 || n_new + n_excl > S) return MARCHE_EINVAL;
  if ((n_new > 0 && !new_idx) || (n_excl > 0 && !excl_idx)) return MARCHE_EINVAL;
  if (((uintptr_t)workspace & 255) != 0) return MARCHE_EINVAL;
  const WsLayout w = ws_layout(ctx, nA);
  if (ws_bytes < w.total) return MARCHE_EWORKSPACE;
  const int k = refresh_idx ? refresh_count(ratio, S, S - n_new - n_excl) : 0;
  if (n_refresh) *n_refresh = k;
  const StackBufs bf = carve(workspace, w);

  // the workspace is scratch between calls: make sure the stream-K turn flags start at zero
  if (ctx->bf16 && ctx->tune.stream_k) MARCHE_TRY(cudaMemsetAsync(bf.turn, 0, w.turn_bytes, st), "memset");
  mark(ctx, MARCHE_KC_FLAGS, st);
  MARCHE_TRY(launch_step_flags(active_idx, nA, new_idx, n_new, excl_idx, n_excl, B, S, bf.is_new, bf.cand, st), "flags");
  const int rc = run_blocks(ctx, 0, L, hidden, S, active_idx, nA, bf.x, bf, kv_cache, bf.is_new, st);
  if (rc) return rc;
  mark(ctx, MARCHE_KC_SCATTER_ROWS, st);
  MARCHE_TRY(launch_scatter_rows(bf.x, active_idx, B, nA, S, D, hidden_out, st), "scatter_rows");
  mark(ctx, MARCHE_KC_TOPK, st);
  MARCHE_TRY(launch_topk(bf.partial, H, bf.scores, bf.cand, B, S, k, refresh_idx, st), "topk");
  return MARCHE_OK;
}

// One step under the paper's own schedule: blocks 0..score_layer on every token, top-K there,
// blocks after it on A = new | prev | refresh.
int run_in_step(marche_ctx* ctx, const float* hidden, void* kv_cache, const int32_t* new_idx, int n_new,
                const int32_t* prev_idx, int n_prev, int k, const int32_t* forced_refresh, float* hidden_out,
                int32_t* refresh_idx, int32_t* active_idx, void* workspace, size_t ws_bytes, cudaStream_t st) {
  const marche_config& c = ctx->cfg;
  const int B = c.batch, S = c.seq_len, D = c.width, H = c.n_heads, L = c.n_blocks, sl = ctx->score_layer;
  if (!hidden || !kv_cache || !hidden_out || !workspace || !refresh_idx || !active_idx || hidden == hidden_out)
    return MARCHE_EINVAL;
  if (((uintptr_t)hidden | (uintptr_t)hidden_out | (uintptr_t)kv_cache) & 15) return MARCHE_EINVAL;
  if (n_new < 0 || n_prev < 0 || k < 0 || n_new + n_prev + k > S || n_new + n_prev + k < 1) return MARCHE_EINVAL;
  if ((n_new > 0 && !new_idx) || (n_prev > 0 && !prev_idx)) return MARCHE_EINVAL;
  if (sl >= L - 1) return MARCHE_EINVAL;                     // needs at least one cache-aware block
  if (((uintptr_t)workspace & 255) != 0) return MARCHE_EINVAL;
  const WsLayout w = ws_layout(ctx, S);
  if (ws_bytes < w.total) return MARCHE_EWORKSPACE;
  const StackBufs bf = carve(workspace, w);
  const int nA = n_new + n_prev + k;
  if (ctx->bf16 && ctx->tune.stream_k) MARCHE_TRY(cudaMemsetAsync(bf.turn, 0, w.turn_bytes, st), "memset");

  // phase 1: every token; generating rows flagged for the scores; candidates = all \ (new u prev)
  mark(ctx, MARCHE_KC_FLAGS, st);
  MARCHE_TRY(launch_step_flags(nullptr, S, new_idx, n_new, prev_idx, n_prev, B, S, bf.is_new, bf.cand, st), "flags");
  int rc = run_blocks(ctx, 0, sl + 1, hidden, S, nullptr, S, bf.x, bf, kv_cache, bf.is_new, st);
  if (rc) return rc;
  mark(ctx, MARCHE_KC_TOPK, st);
  MARCHE_TRY(launch_topk(bf.partial, H, bf.scores, bf.cand, B, S, k, refresh_idx, st), "topk");
  mark(ctx, MARCHE_KC_OTHER, st);
  MARCHE_TRY(launch_build_active(new_idx, n_new, prev_idx, n_prev, forced_refresh ? forced_refresh : refresh_idx, k, B,
                                 active_idx, st), "build_active");
  // phase 2: rows of A, gathered from the full residual rows of phase 1
  rc = run_blocks(ctx, sl + 1, L, bf.x, S, active_idx, nA, bf.x2, bf, kv_cache, nullptr, st);
  if (rc) return rc;
  mark(ctx, MARCHE_KC_SCATTER_ROWS, st);
  MARCHE_TRY(launch_scatter_rows(bf.x2, active_idx, B, nA, S, D, hidden_out, st), "scatter_rows");
  return MARCHE_OK;
}

// One step of the two-stage model: encoder blocks [0, E) on the known tokens only (Eq. 1), the
// decoder's input assembled from the projected encoder rows and the mask embedding (Eq. 2), then
// the decoder blocks [E, L) either on every token or under the in-step selection schedule.
int run_mar(marche_ctx* ctx, bool full_decoder, const float* tokens, const int32_t* known_idx, int n_known,
            void* kv_cache, const int32_t* new_idx, int n_new, const int32_t* prev_idx, int n_prev, int k,
            const int32_t* forced_refresh, float* z_out, int32_t* refresh_idx, int32_t* active_idx, void* workspace,
            size_t ws_bytes, cudaStream_t st) {
  const marche_config& c = ctx->cfg;
  const int B = c.batch, S = c.seq_len, D = c.width, H = c.n_heads, L = c.n_blocks, E = c.n_enc_blocks;
  const int sl = ctx->score_layer;
  if (!ctx->has_mar) return MARCHE_EINVAL;
  if (!tokens || !known_idx || !kv_cache || !z_out || !workspace || tokens == z_out) return MARCHE_EINVAL;
  if (((uintptr_t)tokens | (uintptr_t)z_out | (uintptr_t)kv_cache) & 15) return MARCHE_EINVAL;
  if (E < 1 || E >= L || sl < E) return MARCHE_EINVAL;
  if (n_known < 1 || n_known > S || n_new < 0 || n_prev < 0 || k < 0 || n_new + n_prev + k > S) return MARCHE_EINVAL;
  if ((n_new > 0 && !new_idx) || (n_prev > 0 && !prev_idx) || (k > 0 && !refresh_idx)) return MARCHE_EINVAL;
  const int nA = n_new + n_prev + k;
  if (!full_decoder && (sl >= L - 1 || nA < 1 || !active_idx)) return MARCHE_EINVAL;
  if (((uintptr_t)workspace & 255) != 0) return MARCHE_EINVAL;
  const WsLayout w = ws_layout(ctx, S);
  if (ws_bytes < w.total) return MARCHE_EWORKSPACE;
  const StackBufs bf = carve(workspace, w);
  const marche_mar_weights& mw = ctx->mar;
  if (ctx->bf16 && ctx->tune.stream_k) MARCHE_TRY(cudaMemsetAsync(bf.turn, 0, w.turn_bytes, st), "memset");

  mark(ctx, MARCHE_KC_FLAGS, st);
  MARCHE_TRY(launch_step_flags(nullptr, S, new_idx, n_new, prev_idx, n_prev, B, S, bf.is_new, bf.cand, st), "flags");
  // ---- Eq. 1: encoder on the compacted known tokens; its K/V live only inside this step
  int rc = run_blocks(ctx, 0, E, tokens, S, known_idx, n_known, bf.x, bf, kv_cache, nullptr, st, n_known);
  if (rc) return rc;
  // ---- Eq. 2: x3[b][s] = mask + pos[s];  x3[b][known] = W_de * LN(h_enc) + b_de + pos[known]
  mark(ctx, MARCHE_KC_GATHER_LN, st);
  MARCHE_TRY(launch_gather_layernorm(ctx->a_kind, bf.x, n_known, nullptr, B, n_known, D, mw.enc_norm_g, mw.enc_norm_b,
                                     ctx->eps, nullptr, bf.u, st), "encoder_norm");
  mark(ctx, MARCHE_KC_OTHER, st);
  MARCHE_TRY(launch_gather_table_rows(mw.dec_pos, known_idx, (long)B * n_known, D, bf.x2, st), "gather_table_rows");
  rc = do_linear(ctx, MARCHE_KC_OTHER, bf.u, D, B * n_known, mw.w_dec_embed, mw.b_dec_embed, D, D,
                 MARCHE_EPI_BIAS_RESIDUAL, bf.x2, st, bf.turn);
  if (rc) return rc;
  mark(ctx, MARCHE_KC_OTHER, st);
  MARCHE_TRY(launch_fill_mask_rows(mw.mask_token, mw.dec_pos, B, S, D, bf.x3, st), "fill_mask_rows");
  mark(ctx, MARCHE_KC_SCATTER_ROWS, st);
  MARCHE_TRY(launch_scatter_rows(bf.x2, known_idx, B, n_known, S, D, bf.x3, st), "scatter_rows");

  // ---- decoder
  if (full_decoder) {
    rc = run_blocks(ctx, E, L, bf.x3, S, nullptr, S, bf.x, bf, kv_cache, bf.is_new, st);
    if (rc) return rc;
    mark(ctx, MARCHE_KC_TOPK, st);
    MARCHE_TRY(launch_topk(bf.partial, H, bf.scores, bf.cand, B, S, k, refresh_idx, st), "topk");
    mark(ctx, MARCHE_KC_GATHER_LN, st);
    MARCHE_TRY(launch_gather_layernorm(OUT_F32, bf.x, S, nullptr, B, S, D, mw.dec_norm_g, mw.dec_norm_b, ctx->eps,
                                       nullptr, z_out, st), "decoder_norm");
    return MARCHE_OK;
  }
  rc = run_blocks(ctx, E, sl + 1, bf.x3, S, nullptr, S, bf.x, bf, kv_cache, bf.is_new, st);
  if (rc) return rc;
  mark(ctx, MARCHE_KC_TOPK, st);
  MARCHE_TRY(launch_topk(bf.partial, H, bf.scores, bf.cand, B, S, k, refresh_idx, st), "topk");
  mark(ctx, MARCHE_KC_OTHER, st);
  MARCHE_TRY(launch_build_active(new_idx, n_new, prev_idx, n_prev, forced_refresh ? forced_refresh : refresh_idx, k, B,
                                 active_idx, st), "build_active");
  rc = run_blocks(ctx, sl + 1, L, bf.x, S, active_idx, nA, bf.x2, bf, kv_cache, nullptr, st);
  if (rc) return rc;
  mark(ctx, MARCHE_KC_GATHER_LN, st);
  MARCHE_TRY(launch_gather_layernorm(OUT_F32, bf.x2, nA, nullptr, B, nA, D, mw.dec_norm_g, mw.dec_norm_b, ctx->eps,
                                     nullptr, z_out, st, active_idx, S), "decoder_norm");
  return MARCHE_OK;
}

std::pair<const void*, bool>* find_cache(marche_ctx* ctx, const void* p) {
  for (auto& e : ctx->caches)
    if (e.first == p) return &e;
  return nullptr;
}

}  // namespace

extern "C" {

int marche_create(const marche_config* cfg, const marche_block_weights* blocks, marche_ctx** out) {
  if (!cfg || !blocks || !out) return MARCHE_EINVAL;
  *out = nullptr;
  const marche_config& c = *cfg;
  if (c.n_blocks < 1 || c.batch < 1 || c.seq_len < 1 || c.n_heads < 1 || c.head_dim < 1) return MARCHE_EINVAL;
  if (c.dtype != MARCHE_F32 && c.dtype != MARCHE_BF16 && c.dtype != MARCHE_BF16_F16OP) return MARCHE_EINVAL;
  if (c.width != c.n_heads * c.head_dim) return MARCHE_EINVAL;
  if (c.width % 128 || c.width > 2048 || c.mlp_dim % 128 || c.mlp_dim < 128 || c.seq_len > 2048)
    return MARCHE_ESHAPE;
  if (c.head_dim % 16 || c.head_dim > 128) return MARCHE_ESHAPE;
  if (c.dtype != MARCHE_F32 && c.head_dim != 64 && c.head_dim != 80) return MARCHE_ESHAPE;
  if (c.score_layer >= c.n_blocks) return MARCHE_EINVAL;
  marche_ctx* ctx = new (std::nothrow) marche_ctx();
  if (!ctx) return MARCHE_EINVAL;
  ctx->cfg = c;
  ctx->blocks.assign(blocks, blocks + c.n_blocks);
  for (const marche_block_weights& b : ctx->blocks) {
    // vector loads / TMA: every parameter array starts on a 16-byte boundary
    const void* ptrs[12] = {b.ln1_g, b.ln1_b, b.w_qkv, b.b_qkv, b.w_o, b.b_o, b.ln2_g, b.ln2_b, b.w_fc1, b.b_fc1, b.w_fc2, b.b_fc2};
    for (const void* q : ptrs)
      if (!q || ((uintptr_t)q & 15)) { delete ctx; return MARCHE_EINVAL; }
  }
  ctx->bf16 = c.dtype != MARCHE_F32;
  ctx->a_bf16 = c.dtype == MARCHE_BF16;
  ctx->a_kind = !ctx->bf16 ? OUT_F32 : (ctx->a_bf16 ? OUT_BF16 : OUT_F16);
  ctx->eb = ctx->bf16 ? 2 : 4;
  ctx->tune = default_tuning();
  ctx->eps = c.ln_eps > 0.f ? c.ln_eps : 1e-6f;
  int sl = c.score_layer >= 0 ? c.score_layer : c.n_enc_blocks + 1;
  if (sl >= c.n_blocks) sl = c.n_blocks - 1;
  ctx->score_layer = sl;
  cudaError_t e = cudaGetDevice(&ctx->device);
  if (e == cudaSuccess) e = cudaHostAlloc((void**)&ctx->status_host, 64, cudaHostAllocMapped);
  if (e == cudaSuccess) {
    memset(ctx->status_host, 0, 64);
    e = cudaHostGetDevicePointer((void**)&ctx->status_dev, ctx->status_host, 0);
  }
  if (e != cudaSuccess) {
    if (ctx->status_host) cudaFreeHost(ctx->status_host);
    delete ctx;
    return MARCHE_ECUDA;
  }
  *out = ctx;
  return MARCHE_OK;
}

void marche_destroy(marche_ctx* ctx) {
  if (!ctx) return;
  if (ctx->status_host) cudaFreeHost(ctx->status_host);
  for (cudaEvent_t e : ctx->events) cudaEventDestroy(e);
  delete ctx;
}

size_t marche_cache_bytes(const marche_ctx* ctx) {
  if (!ctx) return 0;
  const marche_config& c = ctx->cfg;
  return (size_t)c.n_blocks * 2 * c.batch * c.seq_len * c.width * ctx->eb;
}

size_t marche_workspace_bytes(const marche_ctx* ctx, int max_active) {
  if (!ctx || max_active < 1 || max_active > ctx->cfg.seq_len) return 0;
  return ws_layout(ctx, max_active).total;
}

int marche_init_cache(marche_ctx* ctx, void* kv_cache, size_t bytes, marche_stream stream) {
  if (!ctx || !kv_cache) return MARCHE_EINVAL;
  MARCHE_ENTER(ctx);
  if (bytes < marche_cache_bytes(ctx)) return MARCHE_EWORKSPACE;
  MARCHE_TRY(cudaMemsetAsync(kv_cache, 0, marche_cache_bytes(ctx), (cudaStream_t)stream), "memset");
  if (auto* e = find_cache(ctx, kv_cache)) e->second = false;
  else ctx->caches.emplace_back(kv_cache, false);
  return MARCHE_OK;
}

int marche_step(marche_ctx* ctx, const float* hidden, void* kv_cache, const int32_t* active_idx, int n_active,
                const int32_t* new_idx, int n_new, const int32_t* exclude_idx, int n_excl, float refresh_ratio,
                float* hidden_out, int32_t* refresh_idx, int* n_refresh, void* workspace, size_t workspace_bytes,
                marche_stream stream) {
  if (!ctx || !active_idx) return MARCHE_EINVAL;
  MARCHE_ENTER(ctx);
  auto* e = find_cache(ctx, kv_cache);
  if (!e || !e->second) return MARCHE_ECACHE;
  return run_stack(ctx, hidden, kv_cache, active_idx, n_active, new_idx, n_new, exclude_idx, n_excl, refresh_ratio,
                   hidden_out, refresh_idx, n_refresh, workspace, workspace_bytes, (cudaStream_t)stream);
}

int marche_full_step(marche_ctx* ctx, const float* hidden, void* kv_cache, const int32_t* new_idx, int n_new,
                     const int32_t* exclude_idx, int n_excl, float refresh_ratio, float* hidden_out,
                     int32_t* refresh_idx, int* n_refresh, void* workspace, size_t workspace_bytes,
                     marche_stream stream) {
  MARCHE_ENTER(ctx);
  const int rc = run_stack(ctx, hidden, kv_cache, nullptr, ctx->cfg.seq_len, new_idx, n_new, exclude_idx, n_excl,
                           refresh_ratio, hidden_out, refresh_idx, n_refresh, workspace, workspace_bytes,
                           (cudaStream_t)stream);
  if (rc == MARCHE_OK) {
    if (auto* e = find_cache(ctx, kv_cache)) e->second = true;
    else ctx->caches.emplace_back(kv_cache, true);
  }
  return rc;
}

int marche_step_in_step_selection(marche_ctx* ctx, const float* hidden, void* kv_cache, const int32_t* new_idx,
                                  int n_new, const int32_t* prev_idx, int n_prev, int n_refresh,
                                  const int32_t* forced_refresh, float* hidden_out, int32_t* refresh_idx,
                                  int32_t* active_idx, void* workspace, size_t workspace_bytes, marche_stream stream) {
  MARCHE_ENTER(ctx);
  auto* e = find_cache(ctx, kv_cache);
  if (!e || !e->second) return MARCHE_ECACHE;
  return run_in_step(ctx, hidden, kv_cache, new_idx, n_new, prev_idx, n_prev, n_refresh, forced_refresh, hidden_out,
                     refresh_idx, active_idx, workspace, workspace_bytes, (cudaStream_t)stream);
}

int marche_set_mar_weights(marche_ctx* ctx, const marche_mar_weights* w) {
  if (!ctx || !w) return MARCHE_EINVAL;
  if (!w->enc_norm_g || !w->enc_norm_b || !w->w_dec_embed || !w->b_dec_embed || !w->mask_token || !w->dec_pos ||
      !w->dec_norm_g || !w->dec_norm_b)
    return MARCHE_EINVAL;
  if (((uintptr_t)w->enc_norm_g | (uintptr_t)w->enc_norm_b | (uintptr_t)w->w_dec_embed | (uintptr_t)w->b_dec_embed |
       (uintptr_t)w->mask_token | (uintptr_t)w->dec_pos | (uintptr_t)w->dec_norm_g | (uintptr_t)w->dec_norm_b) & 15)
    return MARCHE_EINVAL;
  if (ctx->cfg.n_enc_blocks < 1 || ctx->cfg.n_enc_blocks >= ctx->cfg.n_blocks) return MARCHE_EINVAL;
  ctx->mar = *w;
  ctx->has_mar = true;
  return MARCHE_OK;
}

int marche_mar_step(marche_ctx* ctx, int full_decoder, const float* tokens, const int32_t* known_idx, int n_known,
                    void* kv_cache, const int32_t* new_idx, int n_new, const int32_t* prev_idx, int n_prev,
                    int n_refresh, const int32_t* forced_refresh, float* z_out, int32_t* refresh_idx,
                    int32_t* active_idx, void* workspace, size_t workspace_bytes, marche_stream stream) {
  MARCHE_ENTER(ctx);
  auto* e = find_cache(ctx, kv_cache);
  if (!full_decoder && (!e || !e->second)) return MARCHE_ECACHE;
  const int rc = run_mar(ctx, full_decoder != 0, tokens, known_idx, n_known, kv_cache, new_idx, n_new, prev_idx, n_prev,
                         n_refresh, forced_refresh, z_out, refresh_idx, active_idx, workspace, workspace_bytes,
                         (cudaStream_t)stream);
  if (rc == MARCHE_OK && full_decoder) {
    if (e) e->second = true;
    else ctx->caches.emplace_back(kv_cache, true);
  }
  return rc;
}

int marche_select_refresh(marche_ctx* ctx, const float* scores, const int32_t* new_idx, int n_new,
                          const int32_t* exclude_idx, int n_excl, int k, int32_t* refresh_idx, void* mask_scratch,
                          marche_stream stream) {
  return marche_select_refresh_policy(ctx, scores, new_idx, n_new, exclude_idx, n_excl, k, MARCHE_SELECT_HIGH, 0u,
                                      refresh_idx, mask_scratch, stream);
}

int marche_select_refresh_policy(marche_ctx* ctx, const float* scores, const int32_t* new_idx, int n_new,
                                 const int32_t* exclude_idx, int n_excl, int k, int policy, uint32_t seed,
                                 int32_t* refresh_idx, void* mask_scratch, marche_stream stream) {
  if (!ctx || !scores || !mask_scratch || n_new < 0 || n_excl < 0 || k < 0) return MARCHE_EINVAL;
  MARCHE_ENTER(ctx);
  if (policy < MARCHE_SELECT_HIGH || policy > MARCHE_SELECT_RANDOM) return MARCHE_EINVAL;
  if ((n_new > 0 && !new_idx) || (n_excl > 0 && !exclude_idx)) return MARCHE_EINVAL;
  const int B = ctx->cfg.batch, S = ctx->cfg.seq_len;
  if (k > S - n_new - n_excl) return MARCHE_EINVAL;
  if (k == 0) return MARCHE_OK;
  if (!refresh_idx) return MARCHE_EINVAL;
  cudaStream_t st = (cudaStream_t)stream;
  mark(ctx, MARCHE_KC_FLAGS, st);
  MARCHE_TRY(launch_step_flags(nullptr, 0, new_idx, n_new, exclude_idx, n_excl, B, S, nullptr, (uint8_t*)mask_scratch,
                               st), "flags");
  mark(ctx, MARCHE_KC_TOPK, st);
  MARCHE_TRY(launch_topk(nullptr, 0, const_cast<float*>(scores), (const uint8_t*)mask_scratch, B, S, k, refresh_idx,
                         st, policy, seed), "topk");
  return MARCHE_OK;
}

int marche_set_score_layers(marche_ctx* ctx, const int32_t* layers, int n) {
  if (!ctx || n < 0 || n > 64 || (n > 0 && !layers)) return MARCHE_EINVAL;
  std::vector<int> v;
  for (int i = 0; i < n; ++i) {
    if (layers[i] < 0 || layers[i] >= ctx->cfg.n_blocks) return MARCHE_EINVAL;
    bool dup = layers[i] == ctx->score_layer;
    for (int x : v) dup = dup || x == layers[i];
    if (!dup) v.push_back(layers[i]);
  }
  ctx->extra_score_layers = v;
  return MARCHE_OK;
}

int marche_get_layer_scores(marche_ctx* ctx, void* workspace, int layer, float* scores_out, marche_stream stream) {
  if (!ctx || !workspace || !scores_out) return MARCHE_EINVAL;
  MARCHE_ENTER(ctx);
  const int slot = score_slot(ctx, layer);
  if (slot < 0) return MARCHE_EINVAL;
  const marche_config& c = ctx->cfg;
  const WsLayout w = ws_layout(ctx, 1);
  const float* partial = (const float*)((const char*)workspace + w.partial) + (size_t)slot * c.batch * c.n_heads * c.seq_len;
  mark(ctx, MARCHE_KC_TOPK, (cudaStream_t)stream);
  // k = 0: the kernel only adds the per-head partials in head order and writes the sums
  MARCHE_TRY(launch_topk(partial, c.n_heads, scores_out, nullptr, c.batch, c.seq_len, 0, nullptr, (cudaStream_t)stream),
             "score_sum");
  return MARCHE_OK;
}

int marche_get_scores(marche_ctx* ctx, const void* workspace, float* scores_out, marche_stream stream) {
  if (!ctx || !workspace || !scores_out) return MARCHE_EINVAL;
  MARCHE_ENTER(ctx);
  const size_t bytes = (size_t)ctx->cfg.batch * ctx->cfg.seq_len * sizeof(float);
  MARCHE_TRY(cudaMemcpyAsync(scores_out, (const char*)workspace + ws_layout(ctx, 1).scores, bytes,
                             cudaMemcpyDeviceToDevice, (cudaStream_t)stream), "memcpy");
  return MARCHE_OK;
}

int marche_build_active(marche_ctx* ctx, const int32_t* new_idx, int n_new, const int32_t* prev_idx, int n_prev,
                        const int32_t* refresh_idx, int n_refresh, int32_t* active_idx, marche_stream stream) {
  if (!ctx || !active_idx || n_new < 0 || n_prev < 0 || n_refresh < 0) return MARCHE_EINVAL;
  MARCHE_ENTER(ctx);
  if ((n_new && !new_idx) || (n_prev && !prev_idx) || (n_refresh && !refresh_idx)) return MARCHE_EINVAL;
  if (n_new + n_prev + n_refresh > ctx->cfg.seq_len) return MARCHE_EINVAL;
  mark(ctx, MARCHE_KC_OTHER, (cudaStream_t)stream);
  MARCHE_TRY(launch_build_active(new_idx, n_new, prev_idx, n_prev, refresh_idx, n_refresh, ctx->cfg.batch, active_idx,
                                 (cudaStream_t)stream), "build_active");
  return MARCHE_OK;
}

int marche_scatter_rows(marche_ctx* ctx, const float* rows, const int32_t* idx, int n, float* dst,
                        marche_stream stream) {
  if (!ctx || !rows || !dst || n < 0 || n > ctx->cfg.seq_len || (n && !idx)) return MARCHE_EINVAL;
  MARCHE_ENTER(ctx);
  if (n == 0) return MARCHE_OK;
  mark(ctx, MARCHE_KC_SCATTER_ROWS, (cudaStream_t)stream);
  MARCHE_TRY(launch_scatter_rows(rows, idx, ctx->cfg.batch, n, ctx->cfg.seq_len, ctx->cfg.width, dst,
                                 (cudaStream_t)stream), "scatter_rows");
  return MARCHE_OK;
}

int marche_validate_indices(marche_ctx* ctx, const int32_t* active_idx, int n_active, const int32_t* new_idx,
                            int n_new, const int32_t* exclude_idx, int n_excl, marche_stream stream) {
  if (!ctx || n_active < 0 || n_new < 0 || n_excl < 0) return MARCHE_EINVAL;
  MARCHE_ENTER(ctx);
  if ((n_active && !active_idx) || (n_new && !new_idx) || (n_excl && !exclude_idx)) return MARCHE_EINVAL;
  const int S = ctx->cfg.seq_len;
  if (n_active > S || n_new > S || n_excl > S) return MARCHE_EINDEX;
  cudaStream_t st = (cudaStream_t)stream;
  volatile int* flag = ctx->status_host + 8;   // second word group: index validation
  *flag = 0;
  MARCHE_TRY(launch_validate(n_active ? active_idx : nullptr, n_active, new_idx, n_new, exclude_idx, n_excl,
                             ctx->cfg.batch, S, ctx->status_dev + 8, st), "validate");
  MARCHE_TRY(cudaStreamSynchronize(st), "sync");
  if (*(volatile int*)ctx->status_host) return MARCHE_ETIMEOUT;   // an earlier kernel of the stream gave up a wait
  return *flag ? MARCHE_EINDEX : MARCHE_OK;
}

int marche_gather_layernorm(marche_ctx* ctx, const float* src, int src_rows, const int32_t* idx, int n,
                            const float* gamma, const float* beta, float* x_out, void* u_out,
                            marche_stream stream) {
  if (!ctx || !src || !gamma || !beta || !u_out || n < 0 || src_rows < 1) return MARCHE_EINVAL;
  MARCHE_ENTER(ctx);
  if (!idx && n > src_rows) return MARCHE_EINVAL;
  mark(ctx, MARCHE_KC_GATHER_LN, (cudaStream_t)stream);
  MARCHE_TRY(launch_gather_layernorm(ctx->a_kind, src, src_rows, idx, ctx->cfg.batch, n, ctx->cfg.width, gamma, beta,
                                     ctx->eps, x_out, u_out, (cudaStream_t)stream), "gather_layernorm");
  return MARCHE_OK;
}

int marche_linear(marche_ctx* ctx, const void* a, int lda, int M, const void* w, const float* bias, int N, int K,
                  int epilogue, void* out, marche_stream stream) {
  if (!ctx || !a || !w || !bias || !out || M < 0 || N < 1 || K < 1 || lda < K) return MARCHE_EINVAL;
  if (epilogue < 0 || epilogue > 2) return MARCHE_EINVAL;
  MARCHE_ENTER(ctx);
  if (ctx->bf16 ? (N % 128 || K % 64 || lda % 8) : (N % 64 || K % 16 || lda % 4)) return MARCHE_ESHAPE;
  return do_linear(ctx, MARCHE_KC_OTHER, a, lda, M, w, bias, N, K, epilogue, out, (cudaStream_t)stream);
}

int marche_scatter_kv(marche_ctx* ctx, const void* k, const void* v, int ld_kv, const int32_t* idx, int n,
                      void* cache_layer, marche_stream stream) {
  if (!ctx || !k || !v || !cache_layer || n < 0 || n > ctx->cfg.seq_len || ld_kv < ctx->cfg.width)
    return MARCHE_EINVAL;
  if (!idx && n != ctx->cfg.seq_len) return MARCHE_EINVAL;
  MARCHE_ENTER(ctx);
  mark(ctx, MARCHE_KC_SCATTER_KV, (cudaStream_t)stream);
  MARCHE_TRY(launch_scatter_kv(ctx->bf16, k, v, ld_kv, idx, ctx->cfg.batch, n, ctx->cfg.seq_len, ctx->cfg.width,
                               cache_layer, (cudaStream_t)stream), "scatter_kv");
  return MARCHE_OK;
}

int marche_attention_two_segment(marche_ctx* ctx, const void* qkv, int ld, int n, const int32_t* active_idx,
                                 void* cache_layer, const uint8_t* is_new, float* score_partial, void* o,
                                 marche_stream stream) {
  if (!ctx || !qkv || !cache_layer || !o || n < 0 || n > ctx->cfg.seq_len || ld < 3 * ctx->cfg.width)
    return MARCHE_EINVAL;
  if (!active_idx && n != ctx->cfg.seq_len) return MARCHE_EINVAL;
  if (is_new && !score_partial) return MARCHE_EINVAL;
  if (!ctx->bf16) return MARCHE_ESHAPE;
  MARCHE_ENTER(ctx);
  if (n == 0) return MARCHE_OK;
  const marche_config& c = ctx->cfg;
  mark(ctx, MARCHE_KC_ATTENTION, (cudaStream_t)stream);
  MARCHE_TRY(launch_attention_twoseg(qkv, ld, c.width, 2 * c.width, c.batch, n, c.seq_len, c.n_heads, c.head_dim,
                                     active_idx, cache_layer, is_new, score_partial, o, ctx->a_bf16, ctx->status_dev,
                                     (cudaStream_t)stream), "attention_twoseg");
  return MARCHE_OK;
}

int marche_attention(marche_ctx* ctx, const void* q, int ld_q, int n, const void* cache_layer,
                     const uint8_t* is_new, float* score_partial, void* o, marche_stream stream) {
  if (!ctx || !q || !cache_layer || !o || n < 0 || n > ctx->cfg.seq_len || ld_q < ctx->cfg.width)
    return MARCHE_EINVAL;
  if (is_new && !score_partial) return MARCHE_EINVAL;
  MARCHE_ENTER(ctx);
  return do_attention(ctx, q, ld_q, n, cache_layer, is_new, score_partial, o, (cudaStream_t)stream);
}

int marche_gather_rows(marche_ctx* ctx, const float* src, const int32_t* idx, int n, float* rows_out,
                       marche_stream stream) {
  if (!ctx || !src || !rows_out || n < 0 || n > ctx->cfg.seq_len || (n && !idx)) return MARCHE_EINVAL;
  MARCHE_ENTER(ctx);
  if (n == 0) return MARCHE_OK;
  mark(ctx, MARCHE_KC_OTHER, (cudaStream_t)stream);
  MARCHE_TRY(launch_gather_rows(src, idx, ctx->cfg.batch, n, ctx->cfg.seq_len, ctx->cfg.width, rows_out,
                                (cudaStream_t)stream), "gather_rows");
  return MARCHE_OK;
}

size_t marche_staging_bytes(const marche_ctx* ctx, int max_new) {
  if (!ctx || max_new < 0 || max_new > ctx->cfg.seq_len) return 0;
  const size_t B = ctx->cfg.batch, S = ctx->cfg.seq_len, D = ctx->cfg.width, n = max_new;
  return 2 * align256(B * n * D * sizeof(float)) + 3 * align256(B * n * sizeof(int32_t)) +
         align256(B * S * sizeof(int32_t));
}

int marche_step_host(marche_ctx* ctx, int full, float* hidden, void* kv_cache, const float* h_prev_rows,
                     const int32_t* h_prev_idx, int n_prev, const int32_t* h_new_idx, int n_new,
                     const int32_t* h_excl_idx, int n_excl, const int32_t* refresh_in, int n_refresh_in,
                     float refresh_ratio, float* hidden_out, int32_t* refresh_out, float* h_out_rows,
                     int32_t* h_refresh_out, int* n_refresh, int max_new, void* staging, size_t staging_bytes,
                     void* workspace, size_t workspace_bytes, marche_stream stream) {
  if (!ctx || !hidden || !staging || !refresh_out || n_prev < 0 || n_new < 0 || n_excl < 0 || n_refresh_in < 0)
    return MARCHE_EINVAL;
  if (n_prev > max_new || n_new > max_new || n_excl > max_new) return MARCHE_EINVAL;
  if ((n_prev && (!h_prev_rows || !h_prev_idx)) || (n_new && !h_new_idx) || (n_excl && !h_excl_idx) ||
      (n_refresh_in && !refresh_in))
    return MARCHE_EINVAL;
  if (((uintptr_t)staging & 255) != 0) return MARCHE_EINVAL;
  MARCHE_ENTER(ctx);
  if (staging_bytes < marche_staging_bytes(ctx, max_new)) return MARCHE_EWORKSPACE;
  const size_t B = ctx->cfg.batch, D = ctx->cfg.width, mn = max_new;
  cudaStream_t st = (cudaStream_t)stream;
  char* p = (char*)staging;
  float* d_prev_rows = (float*)p;  p += align256(B * mn * D * sizeof(float));
  float* d_out_rows = (float*)p;   p += align256(B * mn * D * sizeof(float));
  int32_t* d_prev_idx = (int32_t*)p; p += align256(B * mn * sizeof(int32_t));
  int32_t* d_new_idx = (int32_t*)p;  p += align256(B * mn * sizeof(int32_t));
  int32_t* d_excl_idx = (int32_t*)p; p += align256(B * mn * sizeof(int32_t));
  int32_t* d_active = (int32_t*)p;
  if (n_prev) {
    MARCHE_TRY(cudaMemcpyAsync(d_prev_rows, h_prev_rows, B * n_prev * D * sizeof(float), cudaMemcpyHostToDevice, st), "h2d");
    MARCHE_TRY(cudaMemcpyAsync(d_prev_idx, h_prev_idx, B * n_prev * sizeof(int32_t), cudaMemcpyHostToDevice, st), "h2d");
  }
  if (n_new)
    MARCHE_TRY(cudaMemcpyAsync(d_new_idx, h_new_idx, B * n_new * sizeof(int32_t), cudaMemcpyHostToDevice, st), "h2d");
  if (n_excl)
    MARCHE_TRY(cudaMemcpyAsync(d_excl_idx, h_excl_idx, B * n_excl * sizeof(int32_t), cudaMemcpyHostToDevice, st), "h2d");
  int rc = marche_scatter_rows(ctx, d_prev_rows, d_prev_idx, n_prev, hidden, stream);
  if (rc) return rc;
  int k = 0;
  if (full) {
    rc = marche_full_step(ctx, hidden, kv_cache, d_new_idx, n_new, n_excl ? d_excl_idx : nullptr, n_excl,
                          refresh_ratio, hidden_out, refresh_out, &k, workspace, workspace_bytes, stream);
  } else {
    const int nA = n_new + n_prev + n_refresh_in;
    rc = marche_build_active(ctx, d_new_idx, n_new, d_prev_idx, n_prev, refresh_in, n_refresh_in, d_active, stream);
    if (rc) return rc;
    rc = marche_step(ctx, hidden, kv_cache, d_active, nA, d_new_idx, n_new, n_excl ? d_excl_idx : nullptr, n_excl,
                     refresh_ratio, hidden_out, refresh_out, &k, workspace, workspace_bytes, stream);
  }
  if (rc) return rc;
  if (n_refresh) *n_refresh = k;
  if (h_out_rows && n_new) {
    rc = marche_gather_rows(ctx, hidden_out, d_new_idx, n_new, d_out_rows, stream);
    if (rc) return rc;
    MARCHE_TRY(cudaMemcpyAsync(h_out_rows, d_out_rows, B * n_new * D * sizeof(float), cudaMemcpyDeviceToHost, st), "d2h");
  }
  if (h_refresh_out && k)
    MARCHE_TRY(cudaMemcpyAsync(h_refresh_out, refresh_out, B * k * sizeof(int32_t), cudaMemcpyDeviceToHost, st), "d2h");
  return MARCHE_OK;
}

unsigned long long marche_launch_count(const marche_ctx* ctx) { return ctx ? ctx->launches : 0ull; }

int marche_profile_begin(marche_ctx* ctx) {
  if (!ctx) return MARCHE_EINVAL;
  ctx->event_class.clear();
  ctx->profiling = true;
  return MARCHE_OK;
}

int marche_profile_end(marche_ctx* ctx, marche_stream stream, float* ms_per_class, int* launches_per_class) {
  if (!ctx || !ms_per_class || !launches_per_class) return MARCHE_EINVAL;
  MARCHE_ENTER(ctx);
  cudaStream_t st = (cudaStream_t)stream;
  const size_t n = ctx->event_class.size();
  mark(ctx, MARCHE_KC_OTHER, st);              // closing event
  --ctx->launches;
  ctx->profiling = false;
  for (int c = 0; c < MARCHE_N_KERNEL_CLASSES; ++c) { ms_per_class[c] = 0.f; launches_per_class[c] = 0; }
  if (ctx->event_class.size() != n + 1) { ctx->event_class.clear(); return MARCHE_ECUDA; }
  MARCHE_TRY(cudaStreamSynchronize(st), "sync");
  for (size_t i = 0; i < n; ++i) {
    float ms = 0.f;
    MARCHE_TRY(cudaEventElapsedTime(&ms, ctx->events[i], ctx->events[i + 1]), "elapsed");
    ms_per_class[ctx->event_class[i]] += ms;
    ++launches_per_class[ctx->event_class[i]];
  }
  ctx->event_class.clear();
  return *(volatile int*)ctx->status_host ? MARCHE_ETIMEOUT : MARCHE_OK;
}

const char* marche_kernel_class_name(int cls) {
  static const char* names[MARCHE_N_KERNEL_CLASSES] = {
      "step_flags", "gather_layernorm", "gemm_qkv", "scatter_kv", "attention", "gemm_out_proj",
      "gemm_fc1_gelu", "gemm_fc2", "scatter_rows", "topk", "other"};
  return (cls >= 0 && cls < MARCHE_N_KERNEL_CLASSES) ? names[cls] : "?";
}

// ---------------------------------------------------------------- allocation-free selection
// Candidate-mask scratch of marche_select_refresh_static.  It lives in the library image, so every
// GPU that loads the library holds these bytes until the process exits.  In host code the name
// below is only a stand-in for the device object; its device address is obtained once per device
// with cudaGetSymbolAddress and handed to the kernels.
static __device__ __align__(256) uint8_t g_static_mask_scratch[MARCHE_STATIC_SCRATCH_BYTES];

namespace {
uint8_t* g_static_mask_ptr[kMaxDevices] = {};

// Device address of the scratch array on device `dev`, which must be the current device (looked up on
// first use: cudaGetSymbolAddress answers for the current device).
cudaError_t static_mask_address(int dev, uint8_t** out) {
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (!g_static_mask_ptr[dev]) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_static_mask_scratch);
    if (e != cudaSuccess) return e;
    g_static_mask_ptr[dev] = static_cast<uint8_t*>(p);
  }
  *out = g_static_mask_ptr[dev];
  return cudaSuccess;
}
}  // namespace

int marche_select_refresh_static(marche_ctx* ctx, const float* scores, const int32_t* new_idx, int n_new,
                                 const int32_t* exclude_idx, int n_excl, int k, int32_t* refresh_idx,
                                 marche_stream stream) {
  if (!ctx || !scores || n_new < 0 || n_excl < 0 || k < 0) return MARCHE_EINVAL;
  MARCHE_ENTER(ctx);                                   // the context's device is the current one from here on
  if ((n_new > 0 && !new_idx) || (n_excl > 0 && !exclude_idx)) return MARCHE_EINVAL;
  const int B = ctx->cfg.batch, S = ctx->cfg.seq_len;
  if (k > S - n_new - n_excl) return MARCHE_EINVAL;
  if (k == 0) return MARCHE_OK;
  if (!refresh_idx) return MARCHE_EINVAL;
  if ((size_t)B * (size_t)S > (size_t)MARCHE_STATIC_SCRATCH_BYTES) {
    char msg[160];
    snprintf(msg, sizeof msg, "marche_select_refresh_static: batch*seq_len = %zu exceeds the built-in scratch of %d bytes",
             (size_t)B * (size_t)S, (int)MARCHE_STATIC_SCRATCH_BYTES);
    ctx->last_error = msg;
    return MARCHE_EWORKSPACE;
  }
  uint8_t* mask = nullptr;
  MARCHE_TRY(static_mask_address(ctx->device, &mask), "cudaGetSymbolAddress");
  cudaStream_t st = (cudaStream_t)stream;
  // The mask kernel writes all B*S bytes it uses, so nothing left over from an earlier call
  // (of this or any other context) can leak into this one.
  mark(ctx, MARCHE_KC_FLAGS, st);
  MARCHE_TRY(launch_step_flags(nullptr, 0, new_idx, n_new, exclude_idx, n_excl, B, S, nullptr, mask, st), "flags");
  mark(ctx, MARCHE_KC_TOPK, st);
  MARCHE_TRY(launch_topk(nullptr, 0, const_cast<float*>(scores), mask, B, S, k, refresh_idx, st), "topk");
  return MARCHE_OK;
}

// ---------------------------------------------------------------- tuning, status, diagnostics
int marche_get_tuning(const marche_ctx* ctx, marche_tuning* out) {
  if (!ctx || !out) return MARCHE_EINVAL;
  *out = ctx->tune;
  return MARCHE_OK;
}

int marche_set_tuning(marche_ctx* ctx, const marche_tuning* t) {
  if (!ctx || !t) return MARCHE_EINVAL;
  if (t->attention_kernel < MARCHE_ATTENTION_AUTO || t->attention_kernel > MARCHE_ATTENTION_TCGEN05_TWO_PASS) return MARCHE_EINVAL;
  if (t->gemm_kernel < MARCHE_GEMM_AUTO || t->gemm_kernel > MARCHE_GEMM_PAIR) return MARCHE_EINVAL;
  if (t->tail_split != 0 && t->tail_split != 1 && t->tail_split != 2 && t->tail_split != 4) return MARCHE_EINVAL;
  if (t->tile_n != 0 && t->tile_n != 128) return MARCHE_EINVAL;
  if (t->attention_tc_min_rows < 0) return MARCHE_EINVAL;
  ctx->tune = *t;
  pdl_switch() = t->pdl != 0;
  return MARCHE_OK;
}

namespace {
constexpr unsigned kHookClasses = (1u << MARCHE_KC_GATHER_LN) | (1u << MARCHE_KC_GEMM_QKV) | (1u << MARCHE_KC_ATTENTION) |
                                  (1u << MARCHE_KC_GEMM_O) | (1u << MARCHE_KC_GEMM_FC1) | (1u << MARCHE_KC_GEMM_FC2);
}

int marche_debug_skip_classes(marche_ctx* ctx, unsigned class_mask) {
  if (!ctx || (class_mask & ~kHookClasses)) return MARCHE_EINVAL;
  ctx->skip_mask = class_mask;
  return MARCHE_OK;
}

int marche_debug_repeat_classes(marche_ctx* ctx, unsigned class_mask) {
  if (!ctx || (class_mask & ~kHookClasses)) return MARCHE_EINVAL;
  ctx->repeat_mask = class_mask;
  return MARCHE_OK;
}

int marche_check_status(marche_ctx* ctx, marche_stream stream) {
  MARCHE_ENTER(ctx);
  MARCHE_TRY(cudaStreamSynchronize((cudaStream_t)stream), "sync");
  return *(volatile int*)ctx->status_host ? MARCHE_ETIMEOUT : MARCHE_OK;
}

int marche_debug_bounded_wait(marche_ctx* ctx, long long limit_cycles, marche_stream stream) {
  MARCHE_ENTER(ctx);
  if (limit_cycles < 1 || limit_cycles > 2000000000LL) return MARCHE_EINVAL;
  mark(ctx, MARCHE_KC_OTHER, (cudaStream_t)stream);
  MARCHE_TRY(launch_bounded_wait_probe(limit_cycles, ctx->status_dev, (cudaStream_t)stream), "bounded_wait_probe");
  return MARCHE_OK;
}

const char* marche_strerror(int code) {
  switch (code) {
    case MARCHE_OK: return "ok";
    case MARCHE_EINVAL: return "invalid argument";
    case MARCHE_ESHAPE: return "unsupported shape";
    case MARCHE_EWORKSPACE: return "workspace or cache buffer too small";
    case MARCHE_ECACHE: return "cache-aware step on a cache that no full step has filled";
    case MARCHE_EINDEX: return "invalid index set";
    case MARCHE_ECUDA: return "CUDA error";
    case MARCHE_ETIMEOUT: return "bounded device wait timed out";
    default: return "unknown error";
  }
}

const char* marche_last_error(const marche_ctx* ctx) { return ctx ? ctx->last_error.c_str() : ""; }

int marche_device_status(const marche_ctx* ctx) { return ctx ? *(volatile int*)ctx->status_host : 0; }

void marche_clear_device_status(marche_ctx* ctx) {
  if (ctx) *(volatile int*)ctx->status_host = 0;
}

}  // extern "C"
