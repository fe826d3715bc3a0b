/*
 * marche.h - C ABI of libmarche: the per-decoding-step hot path of MARche
 * (cache-aware attention with selective KV refresh for masked autoregressive
 * image generation) on one NVIDIA B200 (sm_100a).
 *
 * Conventions that hold for every call unless a call says otherwise
 * -----------------------------------------------------------------
 * Pointers   "device" pointers address global memory of the GPU that was current
 *            when marche_create() ran, and that GPU must be the current device in
 *            every later call on the context (MARCHE_EINVAL otherwise, nothing
 *            enqueued); "host" pointers address ordinary host memory.  Device
 *            arrays start on 16-byte boundaries (cudaMalloc gives 256).
 *            The library never allocates or frees device memory: the
 *            caller owns hidden states, the K/V cache, index arrays, weights
 *            and the workspace, and keeps them alive until the stream has
 *            finished the call.  The library owns only the small host-side
 *            marche_ctx.
 * Streams    `stream` is a cudaStream_t passed as an opaque pointer (NULL = the
 *            default stream).  All device work is enqueued on it and the call
 *            returns without waiting for it (asynchronous), except where noted.
 * Notation   B batch rows, S tokens per sample, D width = H heads x dh,
 *            F MLP width, L blocks, nA active tokens per sample, nG generating
 *            ("new") tokens per sample, M = B*nA rows.
 * Types      marche_config.dtype selects two element types.  `T` (q/k/v and the
 *            K/V cache, i.e. everything attention reads) and `A` (both operands of
 *            the four projections: the weight matrices, and the activation
 *            matrices that feed them - LayerNorm, attention and GELU outputs):
 *              MARCHE_F32         T = A = float   (plain fp32 kernels, no tensor cores)
 *              MARCHE_BF16        T = A = bf16    (fp32 accumulation everywhere)
 *              MARCHE_BF16_F16OP  T = bf16, A = IEEE fp16: the weight matrices are
 *                                 handed over in fp16
 *            Why the third exists: with 16-bit operands the rounding of exactly the
 *            A activations dominates the end-to-end error (all-bf16 gives max-abs
 *            about 5e-2 against an fp64 reference at 32 blocks; fp16 there gives
 *            under 1e-2), fp16 runs at the same tensor-core rate and size, and the
 *            tensor core wants both operands of one MMA in the same format.
 *            Range rule of MARCHE_BF16_F16OP: every A activation is converted with
 *            saturation, so a magnitude above 65504 is stored as +-65504, never as
 *            infinity (NaN stays NaN); weight matrices must already be finite fp16.
 *            Contexts with 16-bit types have no fp32 fall-back path: a misaligned
 *            operand is MARCHE_EINVAL, not a slower kernel.
 * Index sets int32, device, row-major [B][n] with the same n for every sample;
 *            entries are token positions in [0, S), unique within a sample.
 * Layouts    hidden / hidden_out  float [B][S][D]
 *            K/V cache            T [L][2][B][S][D]; [l][0] holds K, [l][1] V;
 *                                 head h occupies columns h*dh .. (h+1)*dh-1
 *            weight matrices      A [out][in] row-major; LayerNorm parameters
 *                                 and all biases are float
 * Errors     0 (MARCHE_OK) on success, a negative MARCHE_E* code otherwise; no
 *            C++ exception crosses the boundary and no device code traps.  When
 *            a code other than MARCHE_OK is returned because of argument
 *            checking, nothing was enqueued.  CUDA launch errors are reported
 *            as MARCHE_ECUDA (text via marche_last_error()).  Index contents
 *            are not validated on the device (out-of-range or duplicate
 *            entries are undefined behaviour) unless the call says so.
 * Threads    a marche_ctx may be used from one host thread at a time.
 */
#ifndef MARCHE_H_
#define MARCHE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct marche_ctx marche_ctx;
typedef void* marche_stream; /* cudaStream_t */

enum { MARCHE_F32 = 0, MARCHE_BF16 = 1, MARCHE_BF16_F16OP = 2 };

enum {
  MARCHE_OK = 0,
  MARCHE_EINVAL = -1,     /* NULL pointer, negative size, inconsistent arguments          */
  MARCHE_ESHAPE = -2,     /* dimensions this build has no kernel for                      */
  MARCHE_EWORKSPACE = -3, /* workspace (or cache buffer) smaller than required            */
  MARCHE_ECACHE = -4,     /* cache-aware step on a cache no full step has filled          */
  MARCHE_EINDEX = -5,     /* marche_validate_indices found a bad index set                */
  MARCHE_ECUDA = -6,      /* a CUDA runtime / driver call failed                          */
  MARCHE_ETIMEOUT = -7    /* a bounded device-side wait gave up (see marche_device_status)*/
};

/* Epilogues of marche_linear. */
enum {
  MARCHE_EPI_BIAS = 0,          /* out T[M][N]      = acc + bias                          */
  MARCHE_EPI_BIAS_RESIDUAL = 1, /* out float[M][N] += acc + bias   (read-modify-write)    */
  MARCHE_EPI_BIAS_GELU = 2      /* out A[M][N]      = GELU_erf(acc + bias)                */
};

/* Kernel classes of marche_profile_end / marche_kernel_class_name. */
enum {
  MARCHE_KC_FLAGS = 0, MARCHE_KC_GATHER_LN = 1, MARCHE_KC_GEMM_QKV = 2, MARCHE_KC_SCATTER_KV = 3,
  MARCHE_KC_ATTENTION = 4, MARCHE_KC_GEMM_O = 5, MARCHE_KC_GEMM_FC1 = 6, MARCHE_KC_GEMM_FC2 = 7,
  MARCHE_KC_SCATTER_ROWS = 8, MARCHE_KC_TOPK = 9, MARCHE_KC_OTHER = 10,
  MARCHE_N_KERNEL_CLASSES = 11
};

typedef struct {
  int32_t n_blocks;     /* L                                                              */
  int32_t n_enc_blocks; /* E; only used for the default score layer                       */
  int32_t width;        /* D, multiple of 128, <= 2048                                    */
  int32_t n_heads;      /* H                                                              */
  int32_t head_dim;     /* dh = D / H; 64 or 80 for bf16, any multiple of 16 <= 128 f32   */
  int32_t mlp_dim;      /* F, multiple of 128                                             */
  int32_t seq_len;      /* S = image tokens + buffer tokens, <= 2048                      */
  int32_t n_buffer;     /* informational (buffer tokens are ordinary tokens here)         */
  int32_t batch;        /* B, already doubled for classifier-free guidance                */
  int32_t dtype;        /* MARCHE_F32, MARCHE_BF16 or MARCHE_BF16_F16OP (see Types above) */
  int32_t score_layer;  /* 0-based block whose attention yields the relevance scores;
                           -1 selects the second decoder block, E+1 (Section 4.2)         */
  float ln_eps;         /* LayerNorm epsilon; <= 0 selects 1e-6                           */
} marche_config;

/* One entry per block; all device pointers.  The block is the standard pre-LN
 * transformer block that Algorithm 1 abbreviates:  x += Wo*Attn(LN1(x)) + bo;
 * x += W2*GELU(W1*LN2(x) + b1) + b2.  w_qkv is [3D][D] with rows ordered q, k, v. */
typedef struct {
  const float* ln1_g; const float* ln1_b;
  const void* w_qkv;  const float* b_qkv;
  const void* w_o;    const float* b_o;
  const float* ln2_g; const float* ln2_b;
  const void* w_fc1;  const float* b_fc1;
  const void* w_fc2;  const float* b_fc2;
} marche_block_weights;

/* ---------------------------------------------------------------- life cycle */

/* Creates the host-side context for one model shape on the current device.
 * `blocks` is a host array of cfg->n_blocks structs (copied).  Synchronous; no
 * device memory is allocated.  MARCHE_ESHAPE for unsupported dimensions, MARCHE_EINVAL for a
 * NULL or misaligned parameter array.  Weight matrices and biases must be complete in memory
 * before any call that uses them is enqueued (the projection kernels start fetching weight tiles
 * before they wait for the preceding kernel of the stream). */
int marche_create(const marche_config* cfg, const marche_block_weights* blocks, marche_ctx** out);
void marche_destroy(marche_ctx* ctx);

/* Bytes of the K/V cache, L*2*B*S*D*sizeof(T), and of the scratch workspace a
 * step with up to `max_active` active tokens per sample needs (S for a full
 * step).  The workspace must be 256-byte aligned. */
size_t marche_cache_bytes(const marche_ctx* ctx);
size_t marche_workspace_bytes(const marche_ctx* ctx, int max_active);

/* Zero-fills `kv_cache` (device) and records it as "not filled": a cache-aware
 * step on it fails with MARCHE_ECACHE until a full step has run on it (the
 * initial full refresh of Section 4.3). */
int marche_init_cache(marche_ctx* ctx, void* kv_cache, size_t bytes, marche_stream stream);

/* ---------------------------------------------------------------- the step */

/* One cache-aware decoding step: Algorithm 1 lines 4-11 for every block, with
 * the relevance scores of Section 4.2 taken at block `score_layer` and the
 * top-K refresh selection applied to them (the selection feeds the NEXT step).
 *
 *   hidden       in   device float [B][S][D]  stack input (token embeddings)
 *   kv_cache     i/o  device T [L][2][B][S][D]; rows active_idx of every block
 *                     are overwritten with fresh K, V, all other rows keep their
 *                     bytes
 *   active_idx   in   device int32 [B][n_active]   A = G u N u R
 *   new_idx      in   device int32 [B][n_new]      G, a subset of active_idx; the
 *                     queries of these tokens produce the relevance scores
 *   exclude_idx  in   device int32 [B][n_excl] or NULL: tokens that must not be
 *                     selected besides new_idx (the caller passes the tokens
 *                     the next step generates); disjoint from new_idx
 *   refresh_ratio     K = min(S - n_new - n_excl, floor(ratio*S + 1/2))
 *   hidden_out   out  device float [B][S][D]; rows active_idx receive the stack
 *                     output, other rows keep their bytes.  May not alias hidden.
 *   refresh_idx  out  device int32 [B][K], ascending token index per sample; K
 *                     highest scores, ties broken towards the lower index.  Must
 *                     hold B*floor(ratio*S+1/2) entries.  May be NULL: no selection.
 *   n_refresh    out  host int, receives K (may be NULL)
 *   workspace         device scratch of marche_workspace_bytes(ctx, n_active)
 * Errors: MARCHE_ECACHE if kv_cache was never filled by marche_full_step;
 * MARCHE_EINVAL for n_active < 1 or > S, n_new > n_active, NULL buffers;
 * MARCHE_EWORKSPACE. */
int marche_step(marche_ctx* ctx, const float* hidden, void* kv_cache,
                const int32_t* active_idx, int n_active,
                const int32_t* new_idx, int n_new,
                const int32_t* exclude_idx, int n_excl,
                float refresh_ratio, float* hidden_out,
                int32_t* refresh_idx, int* n_refresh,
                void* workspace, size_t workspace_bytes, marche_stream stream);

/* The same stack with every token active (active_idx = 0..S-1): the initial
 * full refresh that fills the cache (Section 4.3) and the full-recompute MAR
 * baseline (Section 3, Motivation).  Marks kv_cache as filled.  Workspace of
 * marche_workspace_bytes(ctx, S). */
int marche_full_step(marche_ctx* ctx, const float* hidden, void* kv_cache,
                     const int32_t* new_idx, int n_new,
                     const int32_t* exclude_idx, int n_excl,
                     float refresh_ratio, float* hidden_out,
                     int32_t* refresh_idx, int* n_refresh,
                     void* workspace, size_t workspace_bytes, marche_stream stream);

/* One decoding step under the paper's own schedule (Section 4.2 and Figure 3, Section 4.3):
 * blocks 0 .. score_layer run full attention on every token (their cache layers are fully
 * refreshed), the relevance scores are taken at block score_layer from the queries of new_idx,
 * the n_refresh highest-scoring tokens outside new_idx u prev_idx become the refreshing tokens,
 * and the blocks after score_layer run cache-aware on A = new | prev | refresh (Algorithm 1).
 * With a fixed active budget the caller passes n_refresh = budget - n_new - n_prev.
 *   prev_idx        device int32 [B][n_prev]: tokens generated in the previous step (N), or NULL
 *   forced_refresh  device int32 [B][n_refresh] or NULL: when given it is used as R instead of the
 *                   selection (which is still written to refresh_idx) - for teacher-forced tests
 *   refresh_idx     out, device int32 [B][n_refresh];  active_idx out, device int32 [B][nA],
 *                   nA = n_new + n_prev + n_refresh
 *   hidden_out      rows active_idx receive the stack output; other rows keep their bytes
 *   workspace       marche_workspace_bytes(ctx, S)
 * Needs score_layer < L-1 (MARCHE_EINVAL otherwise) and a filled cache (MARCHE_ECACHE). */
int marche_step_in_step_selection(marche_ctx* ctx, const float* hidden, void* kv_cache,
                                  const int32_t* new_idx, int n_new, const int32_t* prev_idx, int n_prev,
                                  int n_refresh, const int32_t* forced_refresh, float* hidden_out,
                                  int32_t* refresh_idx, int32_t* active_idx,
                                  void* workspace, size_t workspace_bytes, marche_stream stream);

/* ---------------------------------------------------------------- two-stage model (Section 3) */

/* Glue of MAR's encoder/decoder shape around the L blocks; all device pointers, borrowed like the
 * block weights.  Reading: the encoder output passes a final LayerNorm and a linear map into the
 * decoder width (equal to D here), the decoder adds its own learned positional embedding to every
 * position and ends in a final LayerNorm. */
typedef struct {
  const float* enc_norm_g;  const float* enc_norm_b;   /* [D]   final encoder norm                 */
  const void* w_dec_embed;  const float* b_dec_embed;  /* A [D][D] ([out][in]), float [D]          */
  const float* mask_token;                             /* [D]   embedding of a masked position     */
  const float* dec_pos;                                /* [S][D] decoder positional embedding      */
  const float* dec_norm_g;  const float* dec_norm_b;   /* [D]   final decoder norm                 */
} marche_mar_weights;

/* Registers the glue weights; needs 1 <= n_enc_blocks < n_blocks (MARCHE_EINVAL otherwise, also
 * for a NULL member).  Nothing is enqueued. */
int marche_set_mar_weights(marche_ctx* ctx, const marche_mar_weights* w);

/* One decoding step of the two-stage model.
 *   Eq. 1   blocks 0 .. E-1 (E = n_enc_blocks) run on the known tokens only: rows known_idx of
 *           `tokens` are gathered, attend to one another and to nothing else.  These blocks are
 *           recomputed in every step and cache nothing across steps (the paper keeps cached
 *           projections only in decoder layers); their slices of kv_cache serve as per-step
 *           scratch in a compact [2][B][n_known][D] layout.
 *   Eq. 2   the decoder's input is, at a known position, w_dec_embed * LN_enc(encoder row) +
 *           b_dec_embed, at every other position mask_token; dec_pos is added everywhere.
 *   decoder blocks E .. L-1.  full_decoder != 0: on every token (the first step and the periodic
 *           full refresh of Section 4.3); all S rows of z_out are written; marks kv_cache filled.
 *           full_decoder == 0: the schedule of Section 4.2 - blocks E .. score_layer on every
 *           token, the n_refresh best-scoring tokens outside new_idx u prev_idx selected there,
 *           the later blocks cache-aware on A = new | prev | refresh (Algorithm 1); rows A of
 *           z_out are written, other rows keep their bytes.
 *   z_out   device float [B][S][D]: decoder output after the final decoder norm (the vectors the
 *           sampler of Eq. 3 is conditioned on).
 *   tokens  device float [B][S][D]: embedded input tokens; rows outside known_idx are never read.
 *   known_idx  device int32 [B][n_known], ascending within a sample; 1 <= n_known <= S.
 *   new_idx / prev_idx / forced_refresh / refresh_idx / active_idx: as for
 *           marche_step_in_step_selection; refresh_idx may be NULL when n_refresh == 0 and
 *           active_idx may be NULL when full_decoder != 0.  The relevance scores of block
 *           score_layer are computed in both modes (marche_get_scores).
 *   workspace  marche_workspace_bytes(ctx, S).
 * Needs marche_set_mar_weights, E <= score_layer, and for full_decoder == 0 score_layer < L-1
 * (MARCHE_EINVAL) and a filled cache (MARCHE_ECACHE).  A cache driven by this call holds encoder
 * scratch in its first E slices: run marche_full_step before using it with the uniform-stack calls. */
int marche_mar_step(marche_ctx* ctx, int full_decoder, const float* tokens,
                    const int32_t* known_idx, int n_known, void* kv_cache,
                    const int32_t* new_idx, int n_new, const int32_t* prev_idx, int n_prev,
                    int n_refresh, const int32_t* forced_refresh, float* z_out,
                    int32_t* refresh_idx, int32_t* active_idx,
                    void* workspace, size_t workspace_bytes, marche_stream stream);

/* Top-K refresh selection alone (Section 4.2, "select the top-K tokens with the
 * highest relevance scores"): scores device float [B][S] (finite); candidates
 * are all tokens outside new_idx and exclude_idx; writes refresh_idx device
 * int32 [B][k] ascending; order (score descending, index ascending); -0 == +0.
 * `mask_scratch` is device scratch of B*S bytes.  MARCHE_EINVAL if
 * k > S - n_new - n_excl or k < 0; k == 0 enqueues nothing. */
int marche_select_refresh(marche_ctx* ctx, const float* scores,
                          const int32_t* new_idx, int n_new,
                          const int32_t* exclude_idx, int n_excl,
                          int k, int32_t* refresh_idx, void* mask_scratch, marche_stream stream);

/* Selection ablations of Section 5.3 (Table 3): the same call with a policy.  MARCHE_SELECT_HIGH is
 * the method (highest relevance first); MARCHE_SELECT_LOW picks the lowest scores; and
 * MARCHE_SELECT_RANDOM ignores the scores and orders the candidates by a 32-bit counter-based hash
 * of (seed, sample index, token index): x = seed ^ b*0x9E3779B1 ^ t*0x85EBCA77; x ^= x>>16;
 * x *= 0x7FEB352D; x ^= x>>15; x *= 0x846CA68B; x ^= x>>16 (mod 2^32), smaller first.  Ties go to
 * the lower token index in every policy.  (The active-set ablations of Table 2 need no kernel: pass
 * n_prev = 0 or n_new = 0 to marche_build_active.) */
enum { MARCHE_SELECT_HIGH = 0, MARCHE_SELECT_LOW = 1, MARCHE_SELECT_RANDOM = 2 };
int marche_select_refresh_policy(marche_ctx* ctx, const float* scores,
                                 const int32_t* new_idx, int n_new,
                                 const int32_t* exclude_idx, int n_excl,
                                 int k, int policy, uint32_t seed, int32_t* refresh_idx,
                                 void* mask_scratch, marche_stream stream);

/* The same selection as marche_select_refresh for callers that have no scratch buffer to give
 * and cannot obtain one: code running where device allocation is not allowed (inside a region
 * whose memory was sized up front, a latency-critical serving loop that must never touch the
 * allocator, a plug-in that is handed only its input and output tensors).  The paper has no
 * counterpart; this is a packaging variant of the same kernels.
 *   - The candidate mask lives in a fixed array inside the library, MARCHE_STATIC_SCRATCH_BYTES
 *     (256 KiB) per GPU, which every GPU that loads the library holds until the process exits.
 *     batch*seq_len must not exceed that size; otherwise MARCHE_EWORKSPACE is returned, nothing
 *     is enqueued and marche_last_error() names both numbers.
 *   - No device memory is allocated or freed by this call, now or later.  Its first call on a
 *     device looks up the array's device address (a synchronous, one-time driver query), so make
 *     that first call before starting any stream capture on that device.
 *   - All calls on a device, from every context, share the one array and it keeps the bytes of
 *     the last call.  Each call rewrites every byte it reads, so stale contents are harmless, but
 *     two calls whose kernels overlap on the GPU (different streams, no dependency) race on it:
 *     keep them on one stream or order them with events.
 * Arguments, result and errors otherwise exactly as marche_select_refresh without mask_scratch. */
#define MARCHE_STATIC_SCRATCH_BYTES (256 * 1024)
int marche_select_refresh_static(marche_ctx* ctx, const float* scores,
                                 const int32_t* new_idx, int n_new,
                                 const int32_t* exclude_idx, int n_excl,
                                 int k, int32_t* refresh_idx, marche_stream stream);

/* Copies the relevance scores float [B][S] that the last step left in
 * `workspace` to `scores_out` (device).  Section 4.2: attention probability
 * from the generating tokens to each token, summed over heads and queries. */
int marche_get_scores(marche_ctx* ctx, const void* workspace, float* scores_out, marche_stream stream);

/* Relevance scores at more than one block (the top-K overlap statistics across decoder layers of
 * Section 5.3 / Appendix G need them).  marche_set_score_layers registers up to 64 blocks that
 * accumulate scores in addition to score_layer (which alone drives the selection); it changes the
 * workspace size, so call it before marche_workspace_bytes.  n = 0 clears the list.  The extra
 * blocks are honoured by marche_step and marche_full_step, and by the every-token phase of
 * marche_step_in_step_selection / marche_mar_step (full decoder only); each costs the two-pass
 * scoring variant of the attention kernel.  marche_get_layer_scores sums the per-head partials of
 * one registered block (or of score_layer) left in `workspace` by the last step, in head order,
 * into scores_out, device float [B][S].  MARCHE_EINVAL for a block that is not registered. */
int marche_set_score_layers(marche_ctx* ctx, const int32_t* layers /* host */, int n);
int marche_get_layer_scores(marche_ctx* ctx, void* workspace, int layer, float* scores_out, marche_stream stream);

/* Algorithm 1 line 4, A = G u N u R, built on the device so that a generation
 * loop needs no host round trip: active_idx[b] = new_idx[b] | prev_idx[b] |
 * refresh_idx[b] (concatenation; the caller guarantees disjointness).  Any of
 * the three may have n = 0 (pointer then ignored).  active_idx device int32
 * [B][n_new + n_prev + n_refresh]. */
int marche_build_active(marche_ctx* ctx, const int32_t* new_idx, int n_new,
                        const int32_t* prev_idx, int n_prev,
                        const int32_t* refresh_idx, int n_refresh,
                        int32_t* active_idx, marche_stream stream);

/* Row scatter dst[b][idx[b][j]][:] = rows[b][j][:] for float [B][n][D] rows into
 * float [B][S][D]; the step uses it for hidden_out (only active rows are
 * written, cf. Algorithm 1 line 9) and a generation driver uses it to insert the
 * tokens sampled after a step (Eq. 3-4) into the stack input. */
int marche_scatter_rows(marche_ctx* ctx, const float* rows, const int32_t* idx, int n,
                        float* dst, marche_stream stream);

/* Inverse of marche_scatter_rows: rows_out[b][j][:] = src[b][idx[b][j]][:], float
 * [B][S][D] -> float [B][n][D]: the stack outputs z_i of the tokens being generated,
 * which are all that the sampler consumes (Eq. 3). */
int marche_gather_rows(marche_ctx* ctx, const float* src, const int32_t* idx, int n, float* rows_out,
                       marche_stream stream);

/* One decoding step driven from HOST buffers (a sampler that lives on the host): copies
 * this step's inputs to the device, runs the step, copies its results back, all on
 * `stream` (asynchronous when the host buffers are pinned; synchronise before reading).
 *   full            non-zero: marche_full_step (first step); zero: cache-aware step with
 *                   A = new | prev | refresh_in (Algorithm 1 line 4)
 *   hidden          i/o device float [B][S][D], the stack input kept on the device; rows
 *                   prev_idx are first overwritten with h_prev_rows (the tokens sampled
 *                   after the previous step, Eq. 3-4)
 *   h_prev_rows     host float [B][n_prev][D];  h_prev_idx host int32 [B][n_prev]
 *   h_new_idx       host int32 [B][n_new] (G);  h_excl_idx host int32 [B][n_excl] or NULL
 *   refresh_in      device int32 [B][n_refresh_in]: the previous call's refresh_out
 *   refresh_out     device int32, room for B*floor(ratio*S+1/2) entries (the next call's
 *                   refresh_in; use two buffers alternately)
 *   h_out_rows      host float [B][n_new][D] or NULL: hidden_out rows of new_idx
 *   h_refresh_out   host int32 [B][K] or NULL;  n_refresh host int, receives K
 *   staging         device scratch of marche_staging_bytes(ctx, max_new), 256-byte aligned,
 *                   where max_new bounds n_prev, n_new and n_excl
 * Other arguments and errors as for marche_step / marche_full_step. */
size_t marche_staging_bytes(const marche_ctx* ctx, int max_new);
int marche_step_host(marche_ctx* ctx, int full, float* hidden, void* kv_cache, const float* h_prev_rows,
                     const int32_t* h_prev_idx, int n_prev, const int32_t* h_new_idx, int n_new,
                     const int32_t* h_excl_idx, int n_excl, const int32_t* refresh_in, int n_refresh_in,
                     float refresh_ratio, float* hidden_out, int32_t* refresh_out, float* h_out_rows,
                     int32_t* h_refresh_out, int* n_refresh, int max_new, void* staging, size_t staging_bytes,
                     void* workspace, size_t workspace_bytes, marche_stream stream);

/* Checks index sets on the device (range, uniqueness within a sample, new_idx a
 * subset of active_idx, exclude_idx disjoint from new_idx) and waits for the
 * result: MARCHE_OK or MARCHE_EINDEX.  Synchronous.  active_idx may be NULL
 * (n_active = 0) to skip its checks. */
int marche_validate_indices(marche_ctx* ctx, const int32_t* active_idx, int n_active,
                            const int32_t* new_idx, int n_new,
                            const int32_t* exclude_idx, int n_excl, marche_stream stream);

/* ---------------------------------------------------------------- single kernels
 * The step is a fixed sequence of the calls below; they are exported so that
 * each kernel can be checked and measured on its own. */

/* Gather + LayerNorm (Algorithm 1 line 5, input side): for r = b*n + j,
 *   x = src[b][idx ? idx[b][j] : j][:]   (src float [B][src_rows][D])
 *   x_out[r][:] = x                      (float [B*n][D], skipped when NULL)
 *   u_out[r][:] = (x-mean)/sqrt(var+eps)*gamma + beta   (A [B*n][D])
 * Statistics in fp32 from the row held in registers (two passes). */
int marche_gather_layernorm(marche_ctx* ctx, const float* src, int src_rows, const int32_t* idx, int n,
                            const float* gamma, const float* beta, float* x_out, void* u_out,
                            marche_stream stream);

/* out = epilogue(a * w^T + bias): a A [M][K] with row stride lda elements,
 * w A [N][K], bias float [N], out [M][N] dense (type per epilogue).  The QKV,
 * output and MLP projections on active rows only (Algorithm 1 lines 5 and 9).
 * 16-bit contexts: K % 64 == 0, N % 128 == 0, lda % 8 == 0 (MARCHE_ESHAPE), 16-byte aligned a, w,
 * out (MARCHE_EINVAL).  fp32 accumulation.  w and bias must be complete in memory before the call
 * is enqueued: synchronise after writing them, or keep at least one other kernel of the same
 * stream between the write and this call. */
int marche_linear(marche_ctx* ctx, const void* a, int lda, int M, const void* w, const float* bias,
                  int N, int K, int epilogue, void* out, marche_stream stream);

/* Cache write-back (Algorithm 1 line 11): for r = b*n + j,
 *   cache_layer[0][b][idx[b][j]][:] = k[r][:], cache_layer[1][b][..] = v[r][:]
 * k, v T [B*n][D] with row stride ld_kv elements; cache_layer = T [2][B][S][D]
 * (one block's slice of the cache); idx NULL means the identity (n == S). */
int marche_scatter_kv(marche_ctx* ctx, const void* k, const void* v, int ld_kv,
                      const int32_t* idx, int n, void* cache_layer, marche_stream stream);

/* Attention of the active queries over ALL S cached rows of one block, unmasked
 * (Algorithm 1 lines 6-8, equal to Eq. 5 by Appendix A once the fresh K, V of
 * the active rows are in the cache), with the fused relevance reduction of
 * Section 4.2:
 *   q T [B*n][D] with row stride ld_q; o A [B*n][D] dense;
 *   is_new  device uint8 [B][n] flags of the scoring queries, or NULL: no scores;
 *   score_partial device float [B][H][S]: per head, sum over flagged queries of
 *   the softmax weights (overwritten, not accumulated); ignored when is_new NULL. */
int marche_attention(marche_ctx* ctx, const void* q, int ld_q, int n, const void* cache_layer,
                     const uint8_t* is_new, float* score_partial, void* o, marche_stream stream);

/* The paper's own attention kernel shape (Section 4.1, Appendix A.2 and B): the active queries
 * attend to the fresh segment (K_A, V_A) and to the cached segment (K_C, V_C) separately, the two
 * are merged with one shared maximum and normaliser (Eq. 6-10), nothing is concatenated, and the
 * cache rows of the active tokens are written afterwards (Algorithm 1 line 11) by the same kernel.
 *   qkv   T [B*n][ld]: columns 0..D-1 hold q, D..2D-1 the fresh k, 2D..3D-1 the fresh v (the QKV
 *         projection's output, read in place); ld >= 3D, ld % 8 == 0
 *   active_idx  device int32 [B][n] (token of each row; NULL = identity, n == S)
 *   cache_layer i/o T [2][B][S][D]: rows outside active_idx are read, rows active_idx are written
 *   is_new / score_partial / o  as for marche_attention
 * Results equal marche_scatter_kv followed by marche_attention.  MARCHE_BF16 contexts only
 * (MARCHE_ESHAPE otherwise).  marche_tuning.two_segment_attention makes the step use this kernel. */
int marche_attention_two_segment(marche_ctx* ctx, const void* qkv, int ld, int n, const int32_t* active_idx,
                                 void* cache_layer, const uint8_t* is_new, float* score_partial, void* o,
                                 marche_stream stream);

/* ---------------------------------------------------------------- tuning
 * Kernel-selection switches of one context.  The defaults (marche_get_tuning after marche_create)
 * are the measured winners on B200; the alternatives exist for measurements and for the tests that
 * pin them to the same results.  None of them changes what is computed, only which kernel does it;
 * `pdl` is process-wide (it is a property of how kernels are launched). */
enum { MARCHE_ATTENTION_AUTO = 0, MARCHE_ATTENTION_MMA = 1, MARCHE_ATTENTION_TCGEN05 = 2,
       MARCHE_ATTENTION_TCGEN05_TWO_PASS = 3 /* the two-pass tcgen05 kernel also where no scores are taken */ };
enum { MARCHE_GEMM_AUTO = 0, MARCHE_GEMM_SINGLE = 1, MARCHE_GEMM_PAIR = 2 };
typedef struct {
  int32_t stream_k;              /* 1: fc2-sized residual projections use stream-K with ordered reduce-adds   */
  int32_t fuse_qkv_scatter;      /* 1: the QKV projection's epilogue writes K, V into the cache (no K5 launch)*/
  int32_t attention_kernel;      /* MARCHE_ATTENTION_*: AUTO picks by active rows and head_dim                 */
  int32_t attention_tc_min_rows; /* AUTO: tcgen05 attention above this many active rows (head_dim 64; 48)      */
  int32_t two_segment_attention; /* 1: the step uses marche_attention_two_segment instead of K5 + K3           */
  int32_t gemm_kernel;           /* MARCHE_GEMM_*: AUTO = CTA-pair kernel above 128 rows                       */
  int32_t tail_split;            /* 0 off, 1 cost model, 2 / 4 forced: column slices in a partial last round   */
  int32_t tile_n;                /* 0 = 256-wide tiles whenever N allows, 128 = narrow tiles                   */
  int32_t pdl;                   /* 1: programmatic dependent launch along the kernel chain (process-wide)     */
} marche_tuning;
int marche_get_tuning(const marche_ctx* ctx, marche_tuning* out);
/* MARCHE_EINVAL for a value outside the ranges above; nothing is enqueued. */
int marche_set_tuning(marche_ctx* ctx, const marche_tuning* tuning);

/* ---------------------------------------------------------------- diagnostics */
const char* marche_strerror(int code);
/* Text of the last CUDA error this context saw ("" if none). */
const char* marche_last_error(const marche_ctx* ctx);
/* Status word that bounded waits inside the kernels set when they give up
 * (0 = none; otherwise a kernel-specific code, and the step's results are
 * invalid).  It lives in pinned host memory owned by the context; synchronise
 * the stream before reading it. */
int marche_device_status(const marche_ctx* ctx);
/* Waits for `stream` and reports whether any kernel of this context gave up a bounded wait since the
 * status word was last cleared: MARCHE_ETIMEOUT (the results of the calls enqueued since then are
 * invalid; marche_device_status() names the kernel) or MARCHE_OK.  Synchronous.  The other
 * synchronous calls, marche_validate_indices and marche_profile_end, report the same condition. */
int marche_check_status(marche_ctx* ctx, marche_stream stream);
/* Test hook for that path: enqueues a one-warp kernel whose single waiting thread uses the library's
 * bounded wait on a barrier that nothing arrives on.  After `limit_cycles` SM clock cycles (1 ..
 * 2e9; a million is about half a millisecond) the wait gives up, the status word is set and the
 * kernel returns; nothing traps and the context stays usable.  Asynchronous. */
int marche_debug_bounded_wait(marche_ctx* ctx, long long limit_cycles, marche_stream stream);
/* Number of kernels this context has launched so far. */
unsigned long long marche_launch_count(const marche_ctx* ctx);
/* Per-kernel-class device time of the calls made between marche_profile_begin and
 * marche_profile_end: while profiling, a CUDA event is recorded on the stream in front
 * of every launch, and the time up to the next event (the kernel plus the gap before its
 * successor) is charged to the launch's class.  marche_profile_end synchronises the
 * stream and fills two host arrays of MARCHE_N_KERNEL_CLASSES entries. */
int marche_profile_begin(marche_ctx* ctx);
int marche_profile_end(marche_ctx* ctx, marche_stream stream, float* ms_per_class, int* launches_per_class);
const char* marche_kernel_class_name(int kernel_class);
/* Measurement hook for the cost of a kernel class INSIDE the real launch chain (launch overlap on, no
 * events between kernels): while bit c of `class_mask` is set, the step calls do not launch the kernels
 * of class c, so (time of a step) - (time of the same step with the class left out) is what that
 * class costs in the chain.  The results of such a step are garbage (stale buffers are read) but every
 * index stays in range.  Only MARCHE_KC_GATHER_LN, _GEMM_QKV, _ATTENTION, _GEMM_O, _GEMM_FC1 and
 * _GEMM_FC2 may be left out (MARCHE_EINVAL otherwise); 0 restores the normal step. */
int marche_debug_skip_classes(marche_ctx* ctx, unsigned class_mask);
/* The complementary hook: while bit c is set, every launch of class c is issued twice in a row (same
 * arguments).  (time with the class doubled) - (time of the normal step) is the class's cost in the real
 * chain under the clocks and power the real chain runs at, which leaving a class out does not preserve
 * on a power-capped GPU.  Doubling is harmless for the values except that the two residual projections
 * add their result twice; use it for timing only.  Same classes, same errors. */
int marche_debug_repeat_classes(marche_ctx* ctx, unsigned class_mask);
void marche_clear_device_status(marche_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* MARCHE_H_ */
