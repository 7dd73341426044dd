/*
 * edgefm.h -- C ABI of the batch-1 decode step of a Qwen2.5-style decoder on one NVIDIA B200.
 *
 * The library implements the decode phase of Eq. 4 of the paper,
 *     y_t <- DecodeStep(y_{t-1}, KV; theta_d),   KV <- UpdateKV(KV, y_t),
 * for one request slot (Sec. 3.7, 3.9: a slot owns a pre-allocated KV cache) with greedy sampling
 * (Sec. 4.2: temperature 0, top_k = 1), replayed as one fixed CUDA graph per token whose dynamic
 * parameters (token, position, cache length) live in device memory (Sec. 3.10).
 *
 * Conventions
 *   - "device" pointers are CUDA device pointers on the device that was current at edgefm_create;
 *     "host" pointers are ordinary host memory.  All bf16 data is raw 16-bit patterns.
 *   - Weights are BORROWED: the caller allocates them, keeps them alive and unmodified until
 *     edgefm_destroy.  The context OWNS its KV cache, work buffers, device state and CUDA graph.
 *   - edgefm_prefill_kv and edgefm_decode_step only enqueue work on `stream` (a cudaStream_t passed
 *     as void*; NULL = the legacy default stream) and return without synchronising.  All calls on
 *     one context must be issued on one stream or be externally ordered; a context is not
 *     thread-safe; distinct contexts are independent.
 *   - Every call returns an edgefm_status; nothing throws or aborts.  Arguments are validated on the
 *     host before anything is launched; a call that returns an error has launched nothing and
 *     changed no state (except edgefm_last_error's message).
 *   - There is no CPU fallback: without a CUDA device every call that needs one returns
 *     EDGEFM_ERR_CUDA.
 */
#ifndef EDGEFM_H_
#define EDGEFM_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct edgefm_ctx edgefm_ctx; /* opaque: one request slot */

typedef enum {
    EDGEFM_OK = 0,
    EDGEFM_ERR_INVALID_ARG = 1,   /* null pointer, token out of range, negative size ...            */
    EDGEFM_ERR_BAD_SHAPE = 2,     /* model shape the kernels do not support (see edgefm_create)      */
    EDGEFM_ERR_CONTEXT_FULL = 3,  /* the KV cache has no free slot / prefill longer than max_context */
    EDGEFM_ERR_OUT_OF_MEMORY = 4, /* device or host allocation failed                                */
    EDGEFM_ERR_CUDA = 5,          /* a CUDA runtime call failed; see edgefm_last_error               */
    EDGEFM_ERR_TIMEOUT = 6        /* a bounded device-side wait expired or a device self-check failed
                                     (reported by edgefm_sync_status)                                 */
} edgefm_status;

/* Model shape (the public Qwen2.5 decoder block). */
typedef struct {
    int32_t n_layers;
    int32_t hidden;      /* H, multiple of 8                                        */
    int32_t n_q_heads;   /* multiple of n_kv_heads, group size n_q/n_kv in 1..8     */
    int32_t n_kv_heads;
    int32_t head_dim;    /* d: 64 or 128                                            */
    int32_t ffn;         /* F, multiple of 8                                        */
    int32_t vocab;       /* V                                                       */
    float rms_eps;       /* RMSNorm epsilon (inside the square root)                */
    float rope_theta;    /* RoPE base; rotate-half pairs (i, i+d/2)                 */
    int32_t qkv_bias;    /* 1: bqkv is used; 0: it is ignored                       */
} edgefm_shape;

/* Per-layer DEVICE pointers, bf16, row-major [out][in]. */
typedef struct {
    const void *input_norm; /* [H]                                                        */
    const void *wqkv;       /* [(n_q + 2 n_kv) d][H]; rows: q heads, then k heads, then v */
    const void *bqkv;       /* [(n_q + 2 n_kv) d], or NULL when qkv_bias == 0              */
    const void *wo;         /* [H][n_q d]                                                 */
    const void *post_norm;  /* [H]                                                        */
    const void *w_gate_up;  /* [2F][H]; rows 0..F-1 gate, F..2F-1 up                      */
    const void *w_down;     /* [H][F]                                                     */
} edgefm_layer_weights;

typedef struct {
    const void *embed;                  /* device bf16 [V][H]                                  */
    const void *final_norm;             /* device bf16 [H]                                     */
    const void *lm_head;                /* device bf16 [V][H]; may equal embed (tied)          */
    const edgefm_layer_weights *layers; /* HOST array [n_layers] of structs of device pointers */
} edgefm_weights;

/*
 * edgefm_create -- build a context for one request slot (Sec. 3.7 step 1, Sec. 3.9 pre-allocation).
 * Allocates the KV cache K,V : bf16 [n_layers][n_kv_heads][max_context][head_dim] (cache length 0),
 * the work buffers and the device state, and records the step as a CUDA graph.
 * All matrix base pointers must be 16-byte aligned.  `shape` and `weights` (and the `layers` array)
 * are read during the call only; the device buffers they point to are borrowed until destroy.
 * Errors: INVALID_ARG (null pointers, max_context < 1), BAD_SHAPE, OUT_OF_MEMORY, CUDA.
 * On error *out is set to NULL.
 */
edgefm_status edgefm_create(const edgefm_shape *shape, const edgefm_weights *weights, int32_t max_context,
                            edgefm_ctx **out);

/*
 * edgefm_create_with_options -- edgefm_create with a choice of cache format (Sec. 3.9, "KV Cache Compression":
 * KV~ = C(KV) with on-demand reconstruction; the paper leaves C open).
 *   options->kv_format = EDGEFM_KV_BF16 : the plain cache of edgefm_create (options == NULL means the same);
 *                        EDGEFM_KV_INT8 : every cached row (one position of one kv head, head_dim values) of K and of V is
 *     kept as head_dim signed 8-bit codes and one fp32 scale: scale = amax / 127, code_j = clamp(rint(x_j * (127 / amax)),
 *     -127, 127), both in fp32 (round to nearest even; an all-zero row has scale 0).  Attention multiplies with
 *     code * scale wherever the plain cache is read, the row appended by the step itself included; that row is
 *     compressed from the fp32 k (after RoPE) and v.  Rows given to edgefm_prefill_kv / edgefm_append_kv (bf16) are
 *     compressed as they are copied in.  The cache takes head_dim + 4 bytes per row instead of 2 head_dim.
 *     edgefm_export_kv is refused on such a context (use edgefm_export_kv_int8), and so is edgefm_decode_step_static.
 *   options->block_tokens = 0 or 1 : plain decode steps only;
 *                           2 or 4 : the context can also verify a block of up to that many tokens per call
 *     (edgefm_verify_block).  It then runs a build of the step kernel that carries the tokens side by side (work buffers
 *     per token, somewhat smaller weight tiles); edgefm_decode_step works as before on such a context.  The 2-token
 *     build multiplies with the same 24-bit activations as the plain step; the 4-token build stages every activation as
 *     two bf16 pieces (16 mantissa bits) so that four tokens fit one tensor-core operand.  Needs the plain bf16 cache and
 *     max_context <= 8192.
 *   options->reserved must be zero.
 * Errors: as edgefm_create; INVALID_ARG for an unknown format, an unsupported block size or non-zero reserved fields;
 * BAD_SHAPE when block_tokens > 1 is combined with the compressed cache or a context beyond 8192 positions.
 */
enum { EDGEFM_KV_BF16 = 0, EDGEFM_KV_INT8 = 1 };
typedef struct {
    int32_t kv_format;
    int32_t block_tokens;
    int32_t reserved[6];
} edgefm_options;
edgefm_status edgefm_create_with_options(const edgefm_shape *shape, const edgefm_weights *weights, int32_t max_context,
                                         const edgefm_options *options, edgefm_ctx **out);

/*
 * edgefm_prefill_kv -- load an already computed KV cache (Eq. 3: KV <- Prefill(x_1:T); here the
 * result of the prefill is given, vision-token positions included; Sec. 3.9 Eq. 5 prefix reuse).
 * k, v: DEVICE bf16; element (layer l, kv head g, position t, j) is read at
 *       l*stride_layer + g*stride_head + t*stride_pos + j  (strides in elements; the last
 *       dimension is contiguous).  Keys must already carry their rotary embedding.
 * Copies positions 0 .. n_positions-1 into cache slots 0 .. n_positions-1 and sets the cache
 * length to n_positions (n_positions = 0 empties the cache; k, v may then be NULL).
 * The copy is asynchronous on `stream`; k and v must stay valid until it has run.
 * Errors: INVALID_ARG, CONTEXT_FULL (n_positions > max_context; nothing is written), CUDA.
 */
edgefm_status edgefm_prefill_kv(edgefm_ctx *ctx, const void *k, const void *v, int32_t n_positions,
                                int64_t stride_layer, int64_t stride_head, int64_t stride_pos, void *stream);

/*
 * edgefm_decode_step -- one decode step (Eq. 4): consume one token, append its K/V at cache slot
 * cur_len, attend over slots 0 .. cur_len, produce the logits and the greedy next token.
 *   token_id  >= 0 : the input token.  -1 : the token the previous step on this context produced
 *                    (kept on the device, no host round trip).
 *   position  >= 0 : rotary position of the input token (it may differ from the cache slot, e.g.
 *                    after vision tokens).  -1 : previous step's position + 1 (cache length for the
 *                    first step after prefill).
 *   logits_out      : DEVICE fp32 [vocab] or NULL.
 *   next_token_out  : DEVICE int32 [1] or NULL (lowest index among the maxima of the logits).
 * Outputs are valid once `stream` has executed the step.  The cache length grows by one.
 * Errors: INVALID_ARG (token_id >= vocab or < -1, position < -1, token_id == -1 before any step),
 * CONTEXT_FULL (cache length == max_context; nothing is launched), CUDA.
 */
edgefm_status edgefm_decode_step(edgefm_ctx *ctx, int32_t token_id, int32_t position, void *stream,
                                 float *logits_out, int32_t *next_token_out);

/*
 * edgefm_verify_block -- verification of a proposed block (Sec. 3.11 of the paper, "Verification" and "Commit"; the draft
 * model that proposes the block is not part of this library).  tokens[0] is the token to decode (or -1: the token the
 * previous call left on the device), tokens[1 .. m-1] the proposed continuation.  All m tokens pass through the model in
 * ONE step at rotary positions position, position + 1, ... (position = -1: continue from the previous call) and cache slots
 * cur_len, cur_len + 1, ...: the weights are streamed once, token t attends to the cache and to tokens 0 .. t of the block.
 * With g_t the greedy token after token t, proposal t + 1 is accepted if tokens[t + 1] == g_t, and acceptance stops at the
 * first mismatch.  n_accepted = 1 + accepted proposals (>= 1: tokens[0] itself always enters the cache); the cache length
 * grows by n_accepted (the rows of rejected tokens stay behind it and are overwritten later); the next token is
 * g_{n_accepted - 1}.  The result is what n_accepted plain decode steps would have produced.
 *   tokens          : HOST int32 [m], read during the call.  m = 1 .. block_tokens of the context (m = 1 is a decode step)
 *                     through the step kernel.  Longer blocks, up to 8 tokens (on any context, also block_tokens = 0), take the
 *                     DENSE path: the prefill kernels of edgefm_prefill for the m tokens, one pass over the output matrix for
 *                     all m rows, the same acceptance rule on the device.  That path needs tokens[0] and position given (no
 *                     -1) and an exact host-side cache length: after a verified block, edgefm_sync_length comes first.
 *   logits_out      : DEVICE fp32 [m][vocab] (row t: the logits after token t; rows >= n_accepted belong to rejected
 *                     tokens) or NULL.  With a vocabulary subset of n ids (edgefm_set_vocab_subset) the rows are n long,
 *                     [m][n], and the greedy tokens -- hence the acceptance -- are taken over the subset.
 *   n_accepted_out, next_token_out : DEVICE int32 [1] or NULL.
 * The host-side cache length (edgefm_get_length) cannot know n_accepted: after this call it is the upper bound
 * cur_len + m until edgefm_sync_length has been called.
 * Errors: INVALID_ARG (context created without block_tokens, m out of range, token out of range, tokens[0] == -1 before
 * any step), CONTEXT_FULL (fewer than m free slots; nothing is launched), CUDA.
 */
edgefm_status edgefm_verify_block(edgefm_ctx *ctx, const int32_t *tokens, int32_t m, int32_t position, void *stream,
                                  float *logits_out, int32_t *n_accepted_out, int32_t *next_token_out);

/*
 * edgefm_prefill_tokens -- compute the cache rows of n given tokens from the weights (Eq. 3 of the paper, KV <- Prefill(x);
 * Sec. 3.9: KV_u of a request's own suffix behind a prefix).  The tokens pass through the decode-step kernel, as many per
 * call as the context's build carries (1, or block_tokens), at rotary positions position, position + 1, ... and
 * cache slots cur_len, cur_len + 1, ...; every token enters the cache.  Afterwards the device holds the greedy token that
 * follows tokens[n-1], so decoding continues with edgefm_decode_step(ctx, -1, -1, ...).
 * This is prefill at the weight traffic of n / block_tokens decode steps, in the step's own arithmetic (24- or 16-bit
 * activations); meant for short suffixes and for the compressed cache.  Long prompts: edgefm_prefill.
 *   tokens : HOST int32 [n], read during the call.
 * Errors: INVALID_ARG, CONTEXT_FULL (fewer than n free slots; nothing is launched), CUDA.
 */
edgefm_status edgefm_prefill_tokens(edgefm_ctx *ctx, const int32_t *tokens, int32_t n, int32_t position, void *stream);

/*
 * edgefm_prefill -- the prefill phase (Eq. 3 of the paper, KV <- Prefill(x_1:T; theta_p); with a prefix already in the cache,
 * Eq. 5: KV = Concat(KV_p, KV_u)) as dense contractions.  The prompt's tokens pass through the layers TOGETHER (at most 4096
 * per pass): every projection is one [tokens x K] x [K x N] product on the tensor cores (tcgen05, fp32 accumulation in
 * tensor memory; every activation enters as two bf16 pieces, hi + lo = 16 mantissa bits, the weights are bf16 exactly; fp32
 * residual stream), attention is causal over the cache rows 0 .. cur_len + t; the K and V rows go to cache slots cur_len ..
 * The output layer then runs for the last token alone (final norm, one matrix-vector pass, greedy token), and the device
 * state is what a decode step of that token leaves behind: decoding continues with edgefm_decode_step(ctx, -1, -1, ...).
 * (Prompts of fewer than 8 tokens: all but the last token dense, the last one an ordinary decode step.)
 * The cache rows agree with those of n decode steps up to the last bf16 step of a value.
 *   tokens     : HOST int32 [n], n >= 1, read during the call.
 *   position   : rotary position of tokens[0] (>= 0); token i has position + i.
 *   logits_out : DEVICE fp32 [vocab] (or the subset's length) or NULL;  next_token_out : DEVICE int32 [1] or NULL.
 * The work buffers (about (40 H + 8 n_q d + 4 F) bytes per token of a pass) are allocated at the first call and kept.
 * After edgefm_verify_block call edgefm_sync_length first: the rows are placed behind the host's cache length (the call is
 * refused with INVALID_ARG while that length is only an upper bound).
 * On a context with the compressed cache (EDGEFM_KV_INT8) the new K and V rows are compressed from their fp32 values (k after
 * RoPE, v) as the decode step compresses its own row, and attention reads codes x scales for every row, the new ones
 * included (the codes are expanded to bf16 exactly on their way into the tensor cores, the scales multiply the scores and
 * the probabilities).
 * Errors: INVALID_ARG, CONTEXT_FULL (fewer than n free slots; nothing is launched),
 * OUT_OF_MEMORY, CUDA.  A bounded wait of a contraction that runs out is reported by edgefm_sync_status (TIMEOUT).
 */
edgefm_status edgefm_prefill(edgefm_ctx *ctx, const int32_t *tokens, int32_t n, int32_t position, void *stream,
                             float *logits_out, int32_t *next_token_out);

/* Wait for `stream`, then read the cache length from the device (exact again after edgefm_verify_block calls). */
edgefm_status edgefm_sync_length(edgefm_ctx *ctx, void *stream, int32_t *cur_len_host);

/* edgefm_destroy -- synchronise the device, then free everything the context owns (Sec. 3.7 step 4). NULL is a no-op. */
edgefm_status edgefm_destroy(edgefm_ctx *ctx);

/* ---- small helpers (tests, benchmarks) ---------------------------------------------------------- */

/* Host-side cache length (number of filled slots) after all calls enqueued so far; no sync. */
edgefm_status edgefm_get_length(const edgefm_ctx *ctx, int32_t *cur_len_host);

/* Copy the whole cache, internal layout bf16 [n_layers][n_kv_heads][max_context][head_dim], to the
 * DEVICE buffers k_out / v_out (asynchronous on `stream`). */
edgefm_status edgefm_export_kv(edgefm_ctx *ctx, void *k_out, void *v_out, void *stream);

/* The same for a context with the EDGEFM_KV_INT8 cache: codes int8 [n_layers][n_kv_heads][max_context][head_dim] and
 * scales fp32 [n_layers][n_kv_heads][max_context] of K and of V, to DEVICE buffers (asynchronous on `stream`).
 * Errors: INVALID_ARG (null pointers, or the context has the plain cache), CUDA. */
edgefm_status edgefm_export_kv_int8(edgefm_ctx *ctx, void *k_codes_out, void *v_codes_out, float *k_scales_out,
                                    float *v_scales_out, void *stream);

/* Number of kernel launches one decode step performs (nodes of the step graph). */
edgefm_status edgefm_get_launches_per_step(const edgefm_ctx *ctx, int32_t *n_launches_host);

/* Synchronise `stream`, then report whether a bounded device-side wait of the persistent step kernel
 * expired or one of its self-checks failed (EDGEFM_ERR_TIMEOUT; the context is then unusable and must be destroyed)
 * or all is well.  ctx == NULL: the status left by the last edgefm_decode_step_static on the current device. */
edgefm_status edgefm_sync_status(edgefm_ctx *ctx, void *stream);

/*
 * edgefm_append_kv -- fixed-prefix cache reuse (Sec. 3.9, Eq. 5: KV = Concat(KV_p, KV_u)).
 * Copies n_positions of caller-provided KV (same element layout and strides as edgefm_prefill_kv, keys already
 * rotated) into cache slots [start, start + n_positions) and sets the cache length to start + n_positions.
 *   start == current length: plain append behind what the cache holds;
 *   start <  current length: slots from `start` on are dropped first -- the first `start` slots (a prefix computed
 *                            once at start-up) are kept as they are and serve the next request without being copied again;
 *   n_positions == 0       : only the truncation (k, v may be NULL).
 * start > current length is INVALID_ARG (the cache has no holes); start + n_positions > max_context is CONTEXT_FULL;
 * in both cases nothing is written.  Asynchronous on `stream` like edgefm_prefill_kv; the next step's default
 * position (position = -1) becomes start + n_positions.
 */
edgefm_status edgefm_append_kv(edgefm_ctx *ctx, const void *k, const void *v, int32_t start, int32_t n_positions,
                               int64_t stride_layer, int64_t stride_head, int64_t stride_pos, void *stream);

/*
 * edgefm_set_vocab_subset -- vocabulary pruning of the output layer (named among the base-layer optimisations in
 * the caption of Fig. 2; the paper gives no algorithm, so the reading is: greedy decoding restricted to a
 * caller-chosen set of token ids).
 *   token_ids  HOST int32 [n], strictly ascending, each in [0, vocab); read before the call returns.
 *   n          subset size; n == 0 (token_ids may be NULL) restores the full vocabulary.
 * After the call every decode step of this context computes only the n logits  W_lm[token_ids[r]] . x_f  and
 *   next token = token_ids[argmax_r logit_r]   (equal maxima: the lowest token id wins, as without pruning);
 *   logits_out, when given, receives fp32 [n] in subset order (entries past n are left untouched).
 * The rows are gathered once into a contiguous bf16 [n][hidden] matrix owned by the context (n * hidden * 2 bytes of
 * device memory, freed by the next call or by edgefm_destroy), so the pruned step streams n rows instead of vocab.
 * Input token ids stay full-vocabulary ids.  The call synchronises `stream` (steps already enqueued there finish with
 * the previous subset) and returns after its own copies are done; use the stream the decode steps run on.
 * Errors: INVALID_ARG (unsorted, duplicate or out-of-range ids, n outside [0, vocab], debug kernel path),
 * BAD_SHAPE (the subset does not fit the tile plan), OUT_OF_MEMORY, CUDA.  On error the previous subset stays.
 */
edgefm_status edgefm_set_vocab_subset(edgefm_ctx *ctx, const int32_t *token_ids, int32_t n, void *stream);

/* Diagnostics.  When the environment variable EDGEFM_PROFILE=1 was set at edgefm_create (the only environment
 * variable the library reads), every CTA of the persistent step kernel records device timestamps (ns) at fixed points
 * of the last step: start, then per layer {QKV: staged, done, released; attention: done, released; O, gate/up, down:
 * staged, done, released}, then lm_head staged, done.  Synchronises the device and copies the [n_ctas][stride] table to
 * out_host (capacity in elements).  n_ctas = 0 when profiling is off; out_host may be NULL to query the sizes. */
edgefm_status edgefm_debug_profile(edgefm_ctx *ctx, uint64_t *out_host, int64_t capacity, int32_t *n_ctas, int32_t *stride);

/* Launch geometry of the context's step kernel: out8 = {CTAs, consumer warps per CTA, ring slots per warp, bytes per slot,
 * dynamic shared memory, tiles of the busiest CTA, shared-memory bytes reserved for the tile lists, 1 = long-context
 * build of the kernel}.  Host only. */
edgefm_status edgefm_debug_plan(const edgefm_ctx *ctx, int32_t *out8);

/* Every device-side wait of the step kernel (tile arrival, grid barrier) gives up after a bound (1 s by default), records
 * EDGEFM_ERR_TIMEOUT in the device state and lets the kernel return; edgefm_sync_status reports it.  This call changes
 * the bound (limit_ns >= 1000) of the steps enqueued afterwards and, for testing that path without any fault, can make the
 * grid barrier expect one arrival more than there are CTAs (extra_barrier_arrivals = 1; 0 in production), so that the
 * first barrier of the next step runs into the bound.  Synchronises the device and re-records the step graph. */
edgefm_status edgefm_debug_set_wait_limit(edgefm_ctx *ctx, uint32_t limit_ns, int32_t extra_barrier_arrivals);

/* The same for the contractions of edgefm_prefill: every wait on a shared-memory barrier gives up after `polls` polls
 * (2^24 by default; >= 1024), raises an error word that edgefm_sync_status reports as EDGEFM_ERR_TIMEOUT, waits (bounded) for
 * its own copies and multiplies in flight, frees its tensor memory and returns.  extra_arrivals = 1 (0 in production) makes
 * the stage barriers expect an arrival nobody makes, so that the first wait of every contraction enqueued afterwards runs
 * into the bound without any fault.  Host only. */
edgefm_status edgefm_debug_set_prefill_wait(edgefm_ctx *ctx, uint32_t polls, int32_t extra_arrivals);

/* How edgefm_prefill tiles a contraction of [M tokens x K] x [K x N] on num_sms SMs: out2 = {1 = 256-column output tiles
 * (0 = 128), K units per output tile}.  epilogue: 0 = QKV, 1 = added to the residual stream (O and down projection; only
 * these split K), 2 = gate/up (always wide, never split).  Host only: for checking the planner without a GPU. */
edgefm_status edgefm_debug_prefill_plan(int32_t epilogue, int32_t M, int32_t N, int32_t K, int32_t num_sms, int32_t *out2);

/* Host-only check of the planner: the tile schedule of one weight-streaming operator (kind: 0 QKV pairs, 1 residual rows,
 * 2 gate/up pairs, 3 output-layer rows; units rows or pairs; K columns; head_half = head_dim / 2 for kind 0) for n_ctas CTAs
 * of n_warps consumer warps whose ring slots hold slot_rows rows.  tiles_out receives one 64-bit descriptor per tile, CTA by
 * CTA and warp by warp (tiles_per_warp [n_ctas * n_warps] counts them); combines_out four 32-bit words per entry
 * (combines_per_cta [n_ctas]); variant_rows [4] the box heights of the operator's tensor maps; *n_tiles / *n_combines the
 * totals (call once with NULL outputs to size the buffers).  Needs no GPU.  BAD_SHAPE when the operator does not fit. */
edgefm_status edgefm_debug_plan_operator(int32_t kind, int32_t units, int32_t K, int32_t head_half, int32_t op_index, int32_t n_ctas,
                                         int32_t n_warps, int32_t slot_rows, uint64_t *tiles_out, int64_t tiles_cap,
                                         int32_t *tiles_per_warp, uint32_t *combines_out, int64_t combines_cap,
                                         int32_t *combines_per_cta, int32_t *variant_rows, int64_t *n_tiles, int64_t *n_combines);

/*
 * edgefm_decode_step_static -- one decode step that allocates nothing (the paper has no counterpart; this
 * entry point exists for callers that cannot allocate device memory).
 *
 * Who needs it: code that runs inside another framework's allocation-free region (a phase in which that framework has
 * frozen its memory plan), processes whose device memory is handed out entirely by a pool they do not own, and
 * latency-critical threads that cannot take the implicit device synchronisation of cudaMalloc / cudaFree.
 * edgefm_create allocates a KV cache and work buffers; this call does neither.  It is the same persistent step
 * kernel as edgefm_decode_step, with all its work buffers (residual stream, queries, attention partials, MLP
 * activations, operator table, tile schedule, tensor maps, counters, device state) carved out of a fixed 4 MiB array
 * that is part of the loaded library image on every GPU, and with the KV cache owned by the caller:
 *   shape, weights   as for edgefm_create (read during the call; device buffers borrowed until the step has run);
 *                    at most 96 layers, and the work buffers of the shape must fit the 4 MiB, else
 *                    EDGEFM_ERR_BAD_SHAPE with a message that states the limit.
 *   k_cache, v_cache DEVICE bf16 [n_layers][n_kv_heads][max_context][head_dim] (the layout edgefm_export_kv
 *                    writes), 16-byte aligned; slots 0 .. cur_len-1 are read, slot cur_len is written.
 *   cur_len          filled slots before the step (the caller keeps the count; 0 <= cur_len < max_context).
 *   token_id, position  both explicit (>= 0); nothing is remembered between calls.
 *   logits_out       DEVICE fp32 [vocab] or NULL;  next_token_out  DEVICE int32 [1] or NULL.
 * The work is enqueued on `stream` (stream-ordered copies of the schedule and one memset of the counters, then the
 * kernel) and the call returns without synchronising.  It calls no cudaMalloc, cudaFree or other allocating
 * routine.  The first call on a device also looks up the device address of the scratch array (once per device,
 * with that device current).  The copies read host memory of the call itself, so `stream` must NOT be in capture
 * mode: a capturing stream is refused with EDGEFM_ERR_INVALID_ARG before anything is enqueued.
 * All calls on a device share the one scratch array, which keeps the previous call's contents: the call
 * clears what must start at zero itself, but two calls that overlap on the GPU (different streams, different
 * threads; a context created by edgefm_create is NOT affected -- it has its own buffers) race on it and
 * give wrong results; order them on one stream or with events.  A bounded wait that expired inside such a step is
 * reported by edgefm_sync_status(NULL, stream).
 * Errors: INVALID_ARG, BAD_SHAPE, CONTEXT_FULL (cur_len == max_context), CUDA; message via edgefm_last_error(NULL).
 */
edgefm_status edgefm_decode_step_static(const edgefm_shape *shape, const edgefm_weights *weights, void *k_cache, void *v_cache,
                                        int32_t max_context, int32_t cur_len, int32_t token_id, int32_t position, void *stream,
                                        float *logits_out, int32_t *next_token_out);

/* Message of the last error on this context ("" if none); ctx == NULL: last error of edgefm_create
 * on the calling thread. The string is owned by the library. */
const char *edgefm_last_error(const edgefm_ctx *ctx);

/* Library version string. */
const char *edgefm_version(void);

#ifdef __cplusplus
}
#endif
#endif /* EDGEFM_H_ */
