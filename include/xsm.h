/*
 * xsm: multi-head speculative decoding for cross-attention conditioned
 * auto-regressive mesh transformers on one NVIDIA B200 (sm_100a).
 *
 * C ABI.  Every pointer is marked HOST or DEVICE.  The library allocates no
 * device memory: the caller hands it a weight buffer and a workspace and keeps
 * both alive until xsm_destroy.  All work is enqueued on the stream given to
 * xsm_create.  Functions return XSM_OK or an error code; xsm_last_error gives
 * the text.  Argument and capacity errors are found on the host before any
 * launch.  A device-side wait that runs out of patience ends the kernel
 * cleanly and surfaces as XSM_ERR_TIMEOUT at the next synchronising call.
 *
 * Notation follows the paper: s is the number of committed positions whose
 * keys and values are in the cache, x_s the last committed token (not yet in
 * the cache), x_{s+1..s+K} the drafted tokens, K = n_draft the number of
 * decoding heads (the paper's D), V the vocabulary, c the condition latents.
 */
#ifndef XSM_H
#define XSM_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define XSM_API __attribute__((visibility("default")))
#else
#define XSM_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct xsm_ctx xsm_ctx;

typedef enum {
    XSM_OK = 0,
    XSM_ERR_INVALID_ARG = 1,
    XSM_ERR_STATE = 2,      /* call out of order, e.g. a step before xsm_prefill */
    XSM_ERR_CAPACITY = 3,   /* workspace, page pool or max_seq_len too small */
    XSM_ERR_CUDA = 4,
    XSM_ERR_TIMEOUT = 5     /* a bounded device-side wait expired */
} xsm_status;

#define XSM_MAX_DRAFT 16

/* Model shape.  Weights are one flat DEVICE buffer of `dtype` elements in this
 * order, every matrix row-major [out, in] (y = W x), no biases:
 *   E[V,d]
 *   per layer: g1[d] Wq[d,d] Wk[d,d] Wv[d,d] Wo[d,d]
 *              g2[d] Wqc[d,d] Wkc[d,d_cond] Wvc[d,d_cond] Woc[d,d]
 *              g3[d] Wgate[f,d] Wup[f,d] Wdown[d,f]
 *   gf[d] W0[V,d]
 *   per head i=1..K: W1[head_hidden,d] Wout[V,head_hidden]                        (head_kind 0)
 *                    Wq[d,d] Wk[d,d_cond] Wv[d,d_cond] Wo[d,d] Wout[V,d]          (head_kind 1)
 * Block (Sec. 4.1): pre-norm residual, self-attention (RoPE, causal, cached),
 * cross-attention to c, gated feed-forward network; RMSNorm gains g*.
 * Requirements: n_heads*d_head == d_model, head_hidden == d_model, d_model and d_ff multiples of 128 with rows
 * of at most 16 KB (d_model additionally at most 4 KB per row), d_cond a multiple of 32, d_head 32, 64 or 128,
 * page_size a multiple of 32 with page_size*d_head <= 8192 (bf16) / 16384 (fp32), n_draft <= 15,
 * max_batch*(n_draft+1) <= 128.  fp32 models (the parity configuration): at most 24 token rows per step. */
typedef struct {
    int n_layers, d_model, n_heads, d_head, d_ff, vocab, n_cond, d_cond;
    int n_draft;        /* K; 0 = plain one-token-per-step decoding (Table 3 row A) */
    int head_hidden;
    int head_kind;      /* 0: MLP head, logits = Wout (g + SiLU(W1 g)) (Table 3 rows B, C);
                           1: cross-attention head (Eq. 3), logits = Wout (g + Wo Attn(Wq g, Wk c, Wv c)) */
    int dtype;          /* 0: fp32 weights and cache; 1: bf16 weights, fp16 cache, fp32 arithmetic */
    int page_size;      /* tokens per cache page */
    int max_batch;
    int max_seq_len;    /* largest s; the cache holds max_seq_len + K + 1 positions per sequence */
    float rope_theta, rms_eps;
    int bos_id, eos_id; /* eos_id < 0: no end token */
} xsm_model_config;

/* Verification (Sec. 4.2, Sec. 5.4) and resampling (Appendix, independent sampling). */
typedef struct {
    int verify_mode;    /* 0: strict greedy (top-1); 1: draft within the backbone's top k_accept;
                           2: backbone probability of the draft > delta */
    int k_accept;
    float delta;
    int sample_mode;    /* 0: argmax; 1: every candidate on its own from softmax(top k_sample logits / temperature)
                           (the Appendix's independent sampling); 2: x_{s*} as in mode 1, the K drafts as one path
                           of the Appendix's top-k_sample probability tree over the heads (path weight = product of
                           the tokens' softmax probabilities, paths below 1e-5 pruned) */
    int k_sample;       /* <= 64; mode 2: <= 8 and k_sample ^ n_draft <= 4096 */
    float temperature;
    uint64_t seed;      /* Philox4x32-10 key; sequence b uses (seed_lo ^ b, seed_hi) */
} xsm_decode_config;

typedef struct {
    uint64_t steps;                         /* decoding steps, summed over sequences */
    uint64_t tokens;                        /* committed tokens, summed over sequences */
    uint64_t accept_hist[XSM_MAX_DRAFT + 1];/* steps that accepted a drafts */
    double wall_ms;                         /* device time of the last xsm_generate */
    double scr;                             /* tokens / steps (Sec. 5.1) */
} xsm_stats;

/* Bytes of the flat weight buffer for this shape: the backbone of Sec. 4.1 with its decoder W0 (Eq. 2) and the
 * K decoding heads, in the layout given above. */
XSM_API size_t xsm_weights_bytes(const xsm_model_config *cfg);

/* Bytes of workspace that hold max_batch sequences of max_seq_len positions
 * (page pool, cross-attention cache, activations, decoding state). */
XSM_API size_t xsm_workspace_bytes(const xsm_model_config *cfg);

/* Algorithm 1's inputs other than the condition: the backbone M and the decoding
 * heads {H_i}, as one weight buffer in the layout above.
 * Binds a context to DEVICE weights and DEVICE workspace (both 256-byte
 * aligned, borrowed until xsm_destroy) and a CUDA stream (cudaStream_t passed
 * as void*, may be NULL for the default stream).  A workspace larger than
 * xsm_workspace_bytes adds pages to the shared pool; a smaller one that still
 * holds at least one sequence's pages is accepted and XSM_ERR_CAPACITY is then
 * decided per xsm_prefill.  bf16 models keep cached keys and values as fp16:
 * a key or value element beyond +-65504 is stored as +-65504 without any status
 * (projections of normalised activations by N(0, 0.02) weights stay far below). */
XSM_API xsm_status xsm_create(const xsm_model_config *cfg, const void *d_weights, void *d_workspace,
                      size_t workspace_bytes, void *cuda_stream, xsm_ctx **out);

/* Algorithm 1, line 1, for `batch` independent meshes: computes the cross-
 * attention keys and values of d_cond (DEVICE, [batch, n_cond, d_cond], model
 * dtype), runs prompt tokens 0..prompt_len-2 into the cache, sets x_s to the
 * last prompt token, s = prompt_len-1, draws the K initial drafts uniformly on
 * [0, V) and resets the step counters.  d_prompt: DEVICE int32 [batch,
 * prompt_len].  Synchronises the stream once (the stage tables of the batch
 * are uploaded from host memory of the context); the prefill kernels and the
 * ingestion of the prompt are then enqueued without waiting. */
XSM_API xsm_status xsm_prefill(xsm_ctx *ctx, int batch, const void *d_cond, const int32_t *d_prompt,
                       int prompt_len, const xsm_decode_config *dc);

/* One iteration of Algorithm 1's loop (lines 3-12) for every unfinished
 * sequence: backbone over x_{s..s+K} against the paged cache, heads, verify,
 * resample, commit, roll back.  d_new_tokens: DEVICE int32 [batch, K+1], the
 * tokens committed by this step, padded with -1; d_n_new: DEVICE int32
 * [batch] (0 for a finished sequence).  Either may be NULL.  Asynchronous. */
XSM_API xsm_status xsm_spec_step(xsm_ctx *ctx, int32_t *d_new_tokens, int32_t *d_n_new);

/* The paper has no counterpart of this call; it serves hosts that cannot give the library scratch memory of
 * their own.  xsm_spec_step with one difference: the partial results that the key splits of an attention
 * stage hand to one another (scratch that xsm_spec_step keeps in the caller's workspace) live in a 1 MiB
 * array that is part of the library image, so the call needs no allocation by anyone: not by the library
 * (it calls no allocator) and not by a caller that runs where cudaMalloc is not available, e.g. inside a
 * host process that handed out all device memory at start-up, or on a path that must not synchronise the
 * device.  Every GPU that loads the library holds the 1 MiB until the process exits.  The first call on a
 * device looks up the array's device address; make that call before any stream capture.  A batch whose
 * partials exceed the array (batch * n_heads * splits * (K+1) * (d_head+2) floats, twice) is refused with
 * XSM_ERR_CAPACITY.  The two step calls may alternate freely on one context: when xsm_spec_step, xsm_generate or
 * another call that steps follows this one, the workspace copy of the partials is cleared first.  All contexts of a process share the array and it keeps the last call's contents; the
 * call clears the part it uses first, so calls must not overlap on the GPU (same stream, or otherwise
 * ordered): overlapping calls race.  Arguments and results as xsm_spec_step.  Asynchronous. */
XSM_API xsm_status xsm_spec_step_static(xsm_ctx *ctx, int32_t *d_new_tokens, int32_t *d_n_new);

/* Algorithm 1's loop (line 2: while s < L_max and no EOS is committed) and its
 * output x_{0:i_EOS} (line 14), for every mesh of the batch.
 * Runs steps until every sequence has committed max_new_tokens tokens since
 * xsm_prefill, met EOS, or reached max_seq_len.  d_tokens: DEVICE int32
 * [batch, max_new_tokens] (x_1, x_2, ...; unused tail -1); d_lengths: DEVICE
 * int32 [batch].  host_stats (HOST, may be NULL) is filled before returning.
 * Synchronises the stream. */
XSM_API xsm_status xsm_generate(xsm_ctx *ctx, int max_new_tokens, int32_t *d_tokens, int32_t *d_lengths,
                        xsm_stats *host_stats);

/* The same job from HOST buffers: copies h_cond ([batch, n_cond, d_cond],
 * model dtype) and h_prompt to the device, prefills, generates, and copies
 * tokens and lengths back to h_tokens / h_lengths.  For callers that hold
 * nothing on the device; staging space comes from the workspace. */
XSM_API xsm_status xsm_generate_host(xsm_ctx *ctx, int batch, const void *h_cond, const int32_t *h_prompt,
                             int prompt_len, const xsm_decode_config *dc, int max_new_tokens,
                             int32_t *h_tokens, int32_t *h_lengths, xsm_stats *host_stats);

/* Ends the context (waits for its stream); weights and workspace go back to the caller. */
XSM_API xsm_status xsm_destroy(xsm_ctx *ctx);

/* Text of the last error of this context (or of the last failed xsm_create when ctx is NULL). */
XSM_API const char *xsm_last_error(const xsm_ctx *ctx);

/* Number of kernels this context has launched so far. */
XSM_API uint64_t xsm_kernel_launches(const xsm_ctx *ctx);

/* ---- inspection, for tests and parity checks; all synchronise the stream ---- */

/* Logits of the last step: h_logits0 HOST float [batch, K+1, V] (Eq. 2 before the
 * softmax), h_head_logits HOST float [K, batch, K+1, V].  Either may be NULL. */
XSM_API xsm_status xsm_debug_get_logits(xsm_ctx *ctx, float *h_logits0, float *h_head_logits);

/* Cached keys and values of positions pos0..pos0+n-1 of one sequence and layer,
 * widened to float: h_k, h_v HOST float [n, d_model]. */
XSM_API xsm_status xsm_debug_get_kv(xsm_ctx *ctx, int layer, int seq, int pos0, int n, float *h_k, float *h_v);

/* Replaces the drafted tokens x_{s+1..s+K} of every sequence: h_drafts HOST int32 [batch, K]. */
XSM_API xsm_status xsm_debug_set_drafts(xsm_ctx *ctx, const int32_t *h_drafts);

/* Decoding state: h_len [batch] (s), h_window [batch, K+1] (x_s and drafts), h_finished
 * [batch], h_pages [batch] (pages held), h_free_pages [1].  Any may be NULL. */
XSM_API xsm_status xsm_debug_get_state(xsm_ctx *ctx, int32_t *h_len, int32_t *h_window, int32_t *h_finished,
                               int32_t *h_pages, int32_t *h_free_pages);

/* Runs one decoding step (as xsm_spec_step does, without returning its tokens) and records its timeline:
 * h_times HOST uint64 [n_rows][n_ctas] nanoseconds of the GPU's global timer; row 0 = the step starts, row
 * 1 + 2p = stage p of the step has its inputs in shared memory, row 2 + 2p = stage p has published its
 * outputs; one column per CTA of the persistent kernel; 0 = that CTA had nothing to wait for in that stage.
 * capacity = number of uint64 words h_times can hold.  Synchronises the stream. */
XSM_API xsm_status xsm_debug_trace_step(xsm_ctx *ctx, uint64_t *h_times, size_t capacity, int *n_rows, int *n_ctas);

/* Load generator for Sec. 5.1's speedup = SCR x latency(K = 0) / latency(K): from the next step on, the drafts of
 * every sequence are taken from h_tokens (HOST int32 [batch, n], token of every absolute position 0..n-1) instead
 * of from the decoding heads; at step t the first floor((t+1) a) - floor(t a) drafts are left intact and the others
 * are made wrong (a = mean_accept in [0, K]); the token resampled at the first rejected position is replaced by the
 * script's too.  With a script that the backbone reproduces (its own greedy continuation under strict-greedy
 * verification) the accept length of every step is forced, and SCR = 1 + a; where the backbone's two best logits
 * nearly tie and it disagrees with the script, that one step accepts less and the run stays on the script.
 * h_tokens == NULL or n == 0 turns it off; xsm_prefill turns it off too.  Synchronises the stream. */
XSM_API xsm_status xsm_debug_set_script(xsm_ctx *ctx, const int32_t *h_tokens, int n, float mean_accept);

/* Bounds of the device-side waits: polls of one exchanged word and tries of one shared-memory barrier before a
 * CTA gives up, raises XSM_ERR_TIMEOUT and leaves at the end of the step.  0 restores the default (2^21, 2^22). */
XSM_API xsm_status xsm_debug_set_wait_limits(xsm_ctx *ctx, uint32_t polls, uint32_t barrier_tries);

/* Launches stage `stage` (0-based: eight per layer, then the tail) of the current step alone, without advancing the
 * step counter.  A stage whose inputs no earlier launch has published waits for them until the limit above runs
 * out; the status then shows at the next synchronising call, and xsm_prefill starts afresh. */
XSM_API xsm_status xsm_debug_launch_stage(xsm_ctx *ctx, int stage);

/* Runs the step one stage per launch instead of as one persistent kernel (1) or back (0). */
XSM_API xsm_status xsm_debug_set_phase_launch(xsm_ctx *ctx, int on);

#ifdef __cplusplus
}
#endif
#endif /* XSM_H */
