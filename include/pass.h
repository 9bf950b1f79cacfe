/*
 * pass.h - C boundary of the B200 (sm_100a) PaSS decoder-step library.
 *
 * PaSS = Parallel Speculative Sampling (Monea, Joulin, Grave; arXiv 2311.13581).
 * One model call scores the tokens drafted by the previous call and, through k
 * look-ahead embeddings appended to the input, drafts the next k tokens
 * (Algorithm 1; section "Look-ahead embeddings"); the speculative-sampling rule
 * of Algorithm 1 / Algorithm 2 then accepts a prefix of the drafts, resamples or
 * adds one token, and the KV cache is cut back to what was kept (section
 * "Baselines": the cache is updated after every call according to the number of
 * drafted and accepted tokens).
 *
 * Naming: the paper writes q for the target law and p for the draft law, other
 * texts the opposite; this library says P_tgt (target) and Q_dft (draft).
 *
 * General rules
 *   - Plain C ABI.  Pointers are HOST pointers unless the name ends in _device /
 *     the comment says "device".  No call allocates device memory: the KV cache
 *     and the workspace are the caller's, borrowed until pass_destroy.
 *   - Every call returns PASS_OK (0) or a negative PASS_ERR_*.  Nothing throws,
 *     aborts or traps.  On error the state of every sequence is unchanged
 *     (except after PASS_ERR_CUDA, where the CUDA context decides).
 *   - All work is enqueued on the stream given to pass_create.  Calls are not
 *     thread-safe per context.
 *   - There is no CPU fallback: without a CUDA device every compute call fails.
 */
#ifndef PASS_B200_H
#define PASS_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PASS_OK                 0
#define PASS_ERR_INVALID_ARG   -1   /* NULL pointer, bad shape, k out of range, bad token id ... */
#define PASS_ERR_CAPACITY      -2   /* KV capacity, workspace size or row limit exceeded */
#define PASS_ERR_STATE         -3   /* e.g. pass_step before pass_prefill / pass_load_weights */
#define PASS_ERR_CUDA          -4   /* a CUDA runtime or driver call failed */
#define PASS_ERR_NONFINITE     -5   /* a non-finite logit reached the verify kernel */
#define PASS_ERR_TIMEOUT       -6   /* a bounded device-side wait ran out */

#define PASS_MAX_LOOKAHEAD     8    /* upper limit of k_max */
#define PASS_MAX_ROWS        128    /* rows of one forward call: batch * (1 + 2k) <= 128 */

#define PASS_DTYPE_FP32        0
#define PASS_DTYPE_BF16        1

typedef struct pass_ctx pass_ctx;   /* opaque */

/* Shape of a LLaMA-style decoder (pre-norm, RMSNorm, rotary positions on adjacent
 * pairs, SwiGLU, no biases, n_kv_heads == n_heads, untied output head): the
 * paper's experiments use a re-implementation of the 7B LLaMA model. */
typedef struct {
    int n_layers, d_model, n_heads, d_head, d_ffn, vocab;
    int k_max;        /* rows of the look-ahead embedding table, 1..PASS_MAX_LOOKAHEAD */
    int max_batch;    /* independent sequences held by the context */
    int kv_capacity;  /* positions per sequence */
    int dtype;        /* PASS_DTYPE_*: type of weights AND of the KV cache */
    float rms_eps, rope_theta;
} pass_config;

/* Device pointers to the weights, canonical [out_features, in_features] row-major,
 * all of type cfg.dtype.  Per-layer entries are HOST arrays of n_layers device pointers.
 * la_emb is the [k_max, d_model] look-ahead table (section "Look-ahead embeddings":
 * extra rows of the INPUT embedding only; the output head keeps the original vocabulary). */
typedef struct {
    const void *tok_emb;      /* [vocab, d_model] */
    const void *la_emb;       /* [k_max, d_model] */
    const void *lm_head;      /* [vocab, d_model] */
    const void *final_norm;   /* [d_model] */
    const void *const *wq, *const *wk, *const *wv, *const *wo;   /* [d_model, d_model] */
    const void *const *wg, *const *wu;                            /* [d_ffn, d_model] */
    const void *const *wd;                                        /* [d_model, d_ffn] */
    const void *const *norm_attn, *const *norm_ffn;               /* [d_model] */
} pass_weights;

/* Bytes the caller must provide.  kv: EACH of kv_k and kv_v.  Returns 0 on a bad config. */
size_t pass_kv_bytes(const pass_config *cfg);
size_t pass_workspace_bytes(const pass_config *cfg);

/*
 * Create a context on the current CUDA device.
 *   kv_k_device, kv_v_device : caller-allocated device buffers of pass_kv_bytes() each,
 *                              256-byte aligned; layout is private to the library.
 *   workspace_device         : caller-allocated, pass_workspace_bytes(), 256-byte aligned.
 *   cuda_stream              : a cudaStream_t (NULL = default stream).
 * The buffers are borrowed until pass_destroy; the library never frees them.
 * Errors: INVALID_ARG (NULL, misaligned, unsupported shape: d_model != n_heads*d_head,
 * d_head not 64 or 128, k_max out of range), CAPACITY (buffers too small), CUDA.
 */
int pass_create(const pass_config *cfg, void *kv_k_device, void *kv_v_device, size_t kv_bytes,
                void *workspace_device, size_t workspace_bytes, void *cuda_stream,
                pass_ctx **out);

/* Borrow the weights (device memory, unchanged and alive until pass_destroy).
 * Builds the TMA descriptors of the weight-streaming GEMMs.  Errors: INVALID_ARG
 * (NULL or misaligned pointer: every matrix must be 16-byte aligned), CUDA. */
int pass_load_weights(pass_ctx *ctx, const pass_weights *w);

/*
 * Prompt processing for sequence `seq` (Algorithm 1, its input: the prompt the loop
 * starts from).  Caches K/V of tokens[0..n-2]; tokens[n-1] becomes the pending
 * token that the first pass_step feeds; pending drafts are dropped.  n >= 1.
 * Resets the sequence first.  Synchronises the stream.
 * Errors: INVALID_ARG (bad seq, n < 1, id outside [0, vocab)), CAPACITY (n-1 > kv_capacity),
 * STATE (weights not loaded), CUDA.
 */
int pass_prefill(pass_ctx *ctx, int seq, const int32_t *tokens, int n);

/*
 * One PaSS iteration for ALL max_batch sequences (each must have been prefilled).
 * Per sequence, with m in {0, k} pending drafts d_1..d_m drawn from laws Q_dft,1..m:
 *   rows  [pending, d_1..d_m, LA_1..LA_k] (padded to 1+2k rows) at positions len, len+1, ...
 *   P_tgt,j = softmax(logits_j / T) for j = 0..m          (validation phase of Algorithm 1)
 *   draft j is accepted iff u[j-1] < min(1, P_tgt,j-1[d_j] / Q_dft,j[d_j])   (strict <)
 *   first rejection at j: final token y ~ norm(max(0, P_tgt,j-1 - Q_dft,j)) and stop;
 *   no rejection:         final token y ~ P_tgt,m  (the bonus token that ends Algorithm 1's loop body)
 *   emitted tokens = accepted drafts then y; len += number emitted; pending = y
 *   if no draft was rejected the k rows after them give the next drafts
 *   d'_t ~ Q'_t = softmax(logits_{m+t} / T) (drafting phase), else the next call has m = 0.
 * temperature == 0 means greedy (one-hot laws at the first argmax).
 * Sampling y ~ w uses inverse CDF in vocabulary order: smallest i with
 * w_0 + .. + w_i > u * sum(w).  All of this is computed in float64 on the device.
 *
 *   k_lookahead : 0..k_max.  k = 0 is the auto-regressive baseline (one row, one token).
 *   uniforms    : [max_batch][2k+1] floats in [0,1).  Slot j-1 (j=1..k): accept test of
 *                 draft j; slot k: the final token; slot k+t (t=1..k): next draft t.
 *                 May be NULL iff temperature == 0.
 *   out_tokens  : [max_batch][k_max+1] int32, the emitted tokens of each sequence.
 *   n_out       : [max_batch] int32, how many were emitted: 1 .. k+1 (every call adds at
 *                 least one token - section "Parallel Speculative Sampling").
 * Changing k_lookahead or temperature between calls drops pending drafts (they were
 * drawn under other settings).  The step runs as one CUDA graph; the call copies the
 * uniforms in, launches, copies the result out and synchronises the stream.
 * Errors: INVALID_ARG, CAPACITY (len + 1 + 2k > kv_capacity for some sequence, or
 * max_batch*(1+2k) > PASS_MAX_ROWS), STATE, NONFINITE, TIMEOUT, CUDA.
 */
int pass_step(pass_ctx *ctx, int k_lookahead, float temperature, const float *uniforms,
              int32_t *out_tokens, int32_t *n_out);

/*
 * One iteration of Algorithm 1 AS PRINTED (Parallel Speculative Sampling: two model calls per
 * iteration) for all sequences, on the same kernels as pass_step:
 *   drafting call   rows [pending, LA_1..LA_L]: x_{n+1} ~ softmax(logits_0 / T) and the drafts
 *                   d_t ~ Q_t = softmax(logits_t / T); pending drafts of an earlier fused step are dropped;
 *   validation call rows [x_{n+1}, d_1..d_L]: accept tests, residual or extra token as in pass_step;
 *                   the call still carries L look-ahead rows (a step has 1+2L rows whatever it does,
 *                   and its time is set by the weights, not by the rows) whose outputs are not used.
 *   uniforms   : [max_batch][2L+2] floats in [0,1): slot 0 samples x_{n+1}, slots 1..L the drafts,
 *                slots L+1..2L the accept tests, slot 2L+1 the final token.  NULL iff temperature == 0.
 *   out_tokens : [max_batch][k_max+2] int32: x_{n+1}, the accepted drafts, the final token.
 *   n_out      : [max_batch] int32: 2 .. L+2 (each call adds at least one token).
 * Exists so that both schedules can be stated side by side (tokens per model call); pass_step's
 * one-call form is the fast path.  Synchronises the stream twice.  Errors: as pass_step.
 */
int pass_step_two_call(pass_ctx *ctx, int L, float temperature, const float *uniforms,
                       int32_t *out_tokens, int32_t *n_out);

/*
 * The same iteration without host round trip: reads the uniforms from DEVICE memory
 * (same layout, may be NULL iff temperature == 0), enqueues the step and returns at once.
 * Results stay on the device until pass_step_collect.  Capacity is checked against an
 * upper bound of each sequence's length (k+1 tokens per uncollected step).
 */
int pass_step_enqueue(pass_ctx *ctx, int k_lookahead, float temperature,
                      const float *uniforms_device);
/* Synchronise and fetch the LAST enqueued step's result (same meaning as in pass_step).
 * The context keeps one result record per sequence: of several steps enqueued without a collect in
 * between, only the last one's emitted tokens can be read back (the lengths, pending tokens and
 * drafts are right for all of them).  Collect after every step whose tokens are wanted. */
int pass_step_collect(pass_ctx *ctx, int32_t *out_tokens, int32_t *n_out);

/*
 * Multi-token forward for one sequence: n rows appended at positions len .. len+n-1, all
 * scored by one model call (section "Parallel Speculative Sampling").  ids in [0, vocab) are vocabulary
 * tokens; id = vocab + j (0 <= j < k_max) feeds look-ahead embedding j as an input row.
 *   logits_out_device : [n][vocab] float32 on the device, or NULL.
 *   commit            : rows whose K/V are kept, 0..n; len += commit.  Rows after them
 *                       are dead (overwritten by the next call).
 * Drops pending drafts of the sequence; the pending token is left alone.
 * 1 <= n <= PASS_MAX_ROWS.  Synchronises the stream.
 * Errors: INVALID_ARG, CAPACITY (len + n > kv_capacity), STATE, CUDA.
 */
int pass_forward_tokens(pass_ctx *ctx, int seq, const int32_t *tokens, int n,
                        float *logits_out_device, int commit);

/*
 * Arithmetic of long prompts (bf16 models; the paper names no precision).  A prompt of more than
 * PASS_MAX_ROWS tokens runs in chunks of up to 1024 (hi + lo) or 2048 (plain) rows as large tensor-core GEMMs
 * with causal flash attention:
 *   PASS_PROMPT_HI_LO (default): activations as bf16 hi + lo pairs, the arithmetic of pass_step; the cache
 *       it leaves agrees with a float64 computation to about 1e-3 per row.
 *   PASS_PROMPT_BF16: activations, queries and probabilities as single bf16 values - half the tensor-core
 *       work per token; about 5e-3 per row and layer away from a float64 computation (measured, 7B layer
 *       shape), which at full depth uses up the 1e-2 bound stated for the logits of later steps.
 * Host-side setting, applies to later pass_prefill calls.  Errors: INVALID_ARG.
 */
#define PASS_PROMPT_HI_LO 0
#define PASS_PROMPT_BF16  1
int pass_set_prompt_precision(pass_ctx *ctx, int mode);

/*
 * Training of the look-ahead embeddings (Supplementary material, "Training details"; section "Look-ahead
 * embeddings").  The model stays frozen; the only parameters are the first L rows of the look-ahead table.
 * For a training sequence w_0 .. w_{S-1} and a position n the model reads (w_0 .. w_n, LA_1 .. LA_L) in one
 * causal pass; the output at LA_t is the draft of the token t + 1 places after w_n (Algorithm 1, drafting
 * phase), so the loss of the sequence is the mean over t = 1..L of the cross entropy of that output against
 * w_{n+1+t}; a batch averages over its sequences.  The gradient is taken with respect to the L look-ahead input
 * rows only (because of the causal mask no other row depends on them, so the backward pass runs over those rows
 * alone) and applied with AdamW (decoupled weight decay) under a linear warm-up followed by half a cosine down to
 * zero; the paper gives lr 0.01, 2000 warm-up steps, 10000 steps, batches of 8 sequences, and names no other
 * hyper-parameter (betas, eps and weight decay are the caller's; 0.9 / 0.999 / 1e-8 / 0.01 are customary).
 * bf16 models on the tensor-core path only.  float32 master rows, moments and everything the two passes keep live
 * in a training workspace of the caller's (pass_train_workspace_bytes: dominated by a transposed copy of the
 * weights in streaming order, as large as the weights).
 */
typedef struct {
    float lr, beta1, beta2, eps, weight_decay;
    int warmup_steps, total_steps;
} pass_train_config;

/* Bytes of the training workspace for L look-ahead rows and batches of up to max_seqs sequences
 * (L <= k_max, max_seqs <= max_batch, L * max_seqs <= PASS_MAX_ROWS); 0 on a bad argument or a float32 config. */
size_t pass_train_workspace_bytes(const pass_config *cfg, int L, int max_seqs);
/* Set up training: builds the transposed weight copies, copies rows 0..k_max-1 of the context's look-ahead table
 * into float32 master rows, clears the moments and the step count.  train_ws_device: caller-allocated device
 * memory, 256-byte aligned, borrowed until pass_destroy or the next pass_train_init.  Synchronises.
 * Errors: INVALID_ARG, CAPACITY (workspace too small), STATE (weights not loaded, float32 model), CUDA. */
int pass_train_init(pass_ctx *ctx, void *train_ws_device, size_t bytes, const pass_train_config *hp, int L,
                    int max_seqs);
/*
 * One training step on n_seqs sequences (sequence b uses cache slot b, whose contents are replaced).
 *   tokens    : HOST [n_seqs][stride] token ids; of sequence b the entries 0 .. positions[b] + 1 + L are read.
 *   positions : HOST [n_seqs], the index n of the last prompt token of each sequence (n >= 0, n + 1 + L < stride,
 *               n + 1 + L <= kv_capacity).
 *   apply_update : 1 = AdamW update of the master rows and step count + 1; 0 = loss and gradient only.
 *   loss_out  : HOST float, the batch loss (before the update).
 * Runs the prompt parts through pass_prefill's path, then forward and backward over the n_seqs * L look-ahead
 * rows.  Synchronises.  Errors: INVALID_ARG, CAPACITY, STATE (pass_train_init not called), TIMEOUT, CUDA.
 */
int pass_train_step(pass_ctx *ctx, const int32_t *tokens, int stride, const int32_t *positions, int n_seqs,
                    int apply_update, float *loss_out);
/* Read back [L][d_model] float32 rows to HOST memory: the master rows or the gradient of the last step. */
#define PASS_TRAIN_LA    0
#define PASS_TRAIN_GRAD  1
int pass_train_get(pass_ctx *ctx, int what, float *dst_host, size_t bytes);
/* Write the trained rows, rounded to bf16, into rows 0..L-1 of a look-ahead table on the DEVICE (for example the
 * one given to pass_load_weights, which later steps then read). */
int pass_train_export(pass_ctx *ctx, void *la_emb_device);

/* Forget everything about sequence `seq` (len = 0, no pending token, no drafts). */
int pass_reset(pass_ctx *ctx, int seq);

/*
 * Top-k sampling (Experiments, setup: the sampler behind the paper's timings is top-k with a
 * temperature).  top_k > 0: in every later step each law - target rows and look-ahead rows alike -
 * is the temperature softmax over the top_k largest logits of its row, all other tokens have
 * probability 0; among equal logits the lower token id ranks first.  The filter is applied before
 * the acceptance ratio and the residual are formed, so the emitted tokens follow the filtered target
 * law exactly.  top_k = 0 (the default) or top_k >= vocab: no filter.  Greedy steps (temperature 0)
 * are not affected.  Changing top_k drops pending drafts, like a change of k or temperature.
 * Host-side setting, no device work.  Errors: INVALID_ARG (ctx NULL, top_k < 0 or > PASS_MAX_TOP_K).
 */
#define PASS_MAX_TOP_K 1024
int pass_set_top_k(pass_ctx *ctx, int top_k);

/*
 * Restore cached keys/values of one layer (e.g. from a saved session): n positions from
 * pos0, k and v as HOST arrays [n][d_model] in cfg.dtype, keys already rotated.  Does not
 * change len; call pass_set_state afterwards.  Errors: INVALID_ARG, CAPACITY, CUDA.
 */
int pass_set_kv(pass_ctx *ctx, int seq, int layer, int pos0, int n, const void *k, const void *v);
/* Read back cached keys/values of one layer, same layout (for inspection and tests). */
int pass_get_kv(pass_ctx *ctx, int seq, int layer, int pos0, int n, void *k, void *v);
/* Set len and the pending token of a sequence directly; drops pending drafts. */
int pass_set_state(pass_ctx *ctx, int seq, int len, int32_t pending);

/* pass_get_debug selectors.  Each copies to a HOST buffer and synchronises. */
#define PASS_DBG_LOGITS        0  /* float32 [rows][vocab] of the last forward (rows = B*(1+2k)) */
#define PASS_DBG_DRAFT_LOGITS  1  /* float32 [max_batch][k_max][vocab]: logits the pending drafts were drawn from */
#define PASS_DBG_KV_LEN        2  /* int32 [max_batch] */
#define PASS_DBG_N_DRAFT       3  /* int32 [max_batch]: m */
#define PASS_DBG_DRAFTS        4  /* int32 [max_batch][k_max] */
#define PASS_DBG_PENDING       5  /* int32 [max_batch] */
#define PASS_DBG_N_ACCEPTED    6  /* int32 [max_batch]: accepted drafts of the last step */
#define PASS_DBG_STATUS        7  /* int32 [1]: device status word (0 = fine) */
#define PASS_DBG_HIDDEN        8  /* float32 [rows][d_model]: residual stream after the last layer */
#define PASS_DBG_TRACE         9  /* uint64 [launch][4 GEMMs][CTAs][8]: %globaltimer stamps of the GEMM-chain
                                     launches since the last read, when PASS_TRACE is set in the environment:
                                     activations available, first tile ready, last MMA issued, epilogues done */
#define PASS_DBG_FOOTPRINT    10  /* int32 [6] or [9]: shared memory in bytes of the step's GEMM kernel (static, dynamic at up
                                     to 9 rows) and of its attention kernel (static, dynamic), the SM's total and what the
                                     system reserves per block; with room for 9 values also the registers of a CTA of
                                     each and the SM's register file: the two kernels are meant to fit on one SM together */
#define PASS_DBG_ATTN_TRACE   11  /* uint64 [launch][16][16][8]: stamps of the long-cache attention kernel's launches since
                                     the last read (PASS_TRACE set, one sequence): per (head / 4, key slice) of every
                                     fourth head: entry, dependency wait over, first key block in shared memory, last
                                     score product issued, last softmax done, slice stored, head merged (last slice) */
int pass_get_debug(pass_ctx *ctx, int what, void *dst, size_t bytes);

/*
 * One weight-streaming GEMM of the step on its own (bf16 models only): the multi-token model call
 * reduced to a single matrix, y[r][n] = sum_k x[r][k] W[n][k] for R <= PASS_MAX_ROWS rows.
 *   which : 0 wq, 1 wk, 2 wv, 3 wo, 4 wg, 5 wu, 6 wd (K = d_ffn), 7 lm_head (layer ignored),
 *           8 gate|up as the step reads them: output blocks of 128 = 64 gate then 64 up features,
 *           N = ceil(d_ffn/64)*128.
 *   x_device [R][K] float32, y_device [R][N] float32, both on the device.  Synchronises.
 * For tests and for timing the kernel by itself.  Errors: INVALID_ARG, STATE (float32 model),
 * TIMEOUT, CUDA.
 */
int pass_debug_linear(pass_ctx *ctx, int which, int layer, const float *x_device, int R,
                      float *y_device);

/*
 * The work schedule of the weight-streaming GEMM, evaluated on the host (no context, no device):
 * the `it`-th piece of CTA `cta` out of `n_ctas` for a GEMM of n_tiles output tiles with
 * kb_per_tile k-blocks each.  Returns 1 and fills out[7] = {tile, kb0, kb1, n_pieces, index, slot,
 * first_slot} (k-blocks [kb0, kb1) of `tile`; n_pieces CTAs share the tile and this is number
 * `index` of them in k order; slot = which of the CTA's two partial-sum slots the piece uses),
 * or returns 0 when the CTA has no such piece, or -1 on invalid arguments.  It is the same function
 * the kernel runs; the tests check on it what the hand-over of partial sums relies on (every
 * k-block computed exactly once, the CTAs that share a tile are consecutive, ...).
 */
int pass_debug_schedule(int n_tiles, int kb_per_tile, int n_ctas, int cta, int it, int32_t *out);

/*
 * Time that kernel: n_launches launches back to back on the context's stream, cycling over the
 * layers so that every launch streams different weights from HBM (CUDA events; one untimed pass
 * over the layers first).  which as above, except 7; which = 9 times the step's dominant launch, the
 * chain O-projection -> gate|up -> down -> next layer's QKV of layers 0, 1, ... (it overwrites the
 * residual stream and row 0.. of sequence 0's cache: re-run pass_prefill afterwards).  Inputs are
 * whatever the activation buffers hold.  *ms_total receives the elapsed milliseconds.  Synchronises.
 */
int pass_debug_time_linear(pass_ctx *ctx, int which, int R, int n_launches, float *ms_total);

/*
 * pass_debug_linear for callers that must not touch the device allocator.  (The paper has no
 * counterpart: this is a packaging variant of the library's GEMM, not a step of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a region whose memory
 * footprint was fixed up front (a serving process that handed all free HBM to its KV cache and
 * weights), a real-time loop where an allocation could stall or fail, or a host that embeds the
 * library and owns every device byte itself.  The split-K reduction of the GEMM needs scratch
 * (words through which CTAs that share an output tile hand their partial sums to the one that
 * finishes it); here that scratch is a fixed array inside the library image, about 2.6 MB that
 * every GPU loading the library holds until the process exits.  The call itself makes no cudaMalloc /
 * cudaFree and calls no allocating library routine.  Weights and the activation staging rows are still
 * the context's.  Every call, whatever R, runs with the rows padded to 16 so that only the
 * empty-or-value word protocol ever writes to the array (the step's other hand-over protocol, arrival
 * counters with raw partial sums, would leave non-empty words behind).
 *
 * Limit: R <= 16 rows.  More rows return PASS_ERR_CAPACITY (nothing runs).
 * First call on a device: looks up the device address of the built-in array (cudaGetSymbolAddress,
 * with that device current), remembers it and marks every slot empty (a memset on the context's
 * stream); make that first call outside any stream capture.
 * Sharing: all calls, from every context on the device, use the same array.  A slot word is either
 * empty or a partial sum; the CTA that consumes a word marks it empty again, so each call leaves
 * the array as it found it (after a call that returned PASS_ERR_TIMEOUT the whole array is marked
 * empty again).  Two calls that overlap on the GPU (different streams, no ordering) race on it:
 * keep them ordered.
 * Arguments, results and the other errors are those of pass_debug_linear.  Synchronises.
 */
int pass_linear_noalloc(pass_ctx *ctx, int which, int layer, const float *x_device, int R,
                        float *y_device);

/*
 * Switches for the tests of the library's own error handling (no counterpart in the paper).  They are
 * per context, off by default, and are NOT read from the environment, so that nothing outside the
 * process can turn them on.  Setting one synchronises and drops the captured step graphs.
 *   PASS_HOOK_GEMM_STUCK, value 0/1: contributors of the first GEMM of every launch keep their partial
 *       sums to themselves, so the finishers' bounded waits run out (about 0.2 s) and the call returns
 *       PASS_ERR_TIMEOUT with the sequence state untouched.
 *   PASS_HOOK_ATTN_STALE, value n >= 0: the attention kernel's early fetch pretends the cache is n
 *       positions shorter than it is, which forces its re-check and restart path.
 *   PASS_HOOK_ATTN_LONG_FROM, value n >= 0: a step counts as "long" (other attention launch shape; with
 *       d_head 128 and at most 16 rows per sequence the tcgen05 attention kernel) as soon as one sequence
 *       has n cached positions.  Default 3584 (PASS_ATTN_LONG_FROM in the environment at creation); 0
 *       sends every step down the long path, so that small test cases reach it.
 *   PASS_HOOK_ATTN_STUCK, value 0/1: the tcgen05 attention kernel never announces its scores, so its
 *       bounded waits run out; the call returns PASS_ERR_TIMEOUT with the sequence state untouched.
 * Errors: INVALID_ARG.
 */
#define PASS_HOOK_GEMM_STUCK 0
#define PASS_HOOK_ATTN_STALE 1
#define PASS_HOOK_ATTN_LONG_FROM 2
#define PASS_HOOK_ATTN_STUCK 3
int pass_debug_set(pass_ctx *ctx, int hook, int value);

/* Number of kernel launches (graph nodes) of the last pass_step / pass_step_enqueue. */
int pass_last_step_launches(pass_ctx *ctx);
/* Stream of the context (a cudaStream_t), so that callers can time on it. */
void *pass_stream(pass_ctx *ctx);

void pass_destroy(pass_ctx *ctx);
const char *pass_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* PASS_B200_H */
