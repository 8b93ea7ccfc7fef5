/*
 * snlp.h -- C ABI of libsnlp: the layer-parallel Newton sweep of SNLP (Structured Newton Layer
 * Parallelism) for Nanochat-shaped decoder-only Transformers on one NVIDIA B200 (sm_100a).
 *
 * Conventions
 *   - Every function returns 0 (SNLP_OK) or a negative SNLP_ERR_* code; snlp_last_error() gives a
 *     thread-local message for the last failure.  No exception or abort crosses this boundary and
 *     all arguments are validated before anything is launched.  Hidden-state pointers (h0, hL, trace_out)
 *     must be 16-byte aligned and int32 / fp32 scalar arrays 4-byte aligned (whole cudaMalloc'd buffers are); a misaligned pointer is rejected with SNLP_ERR_ARG.
 *   - "host" pointers are read during the call only (the caller keeps ownership and may free them
 *     on return).  "device" pointers are CUDA device memory owned by the caller; the library owns
 *     only its handles, weights, workspace and KV caches.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Unless stated
 *     otherwise calls only enqueue work on that stream and return; results are valid once the
 *     stream has been synchronised.  Calls on one model handle must not overlap on the GPU (they
 *     share the handle's workspace): issue them on one stream, or order them yourself.
 *   - All tensors are row-major with the feature axis innermost.  Hidden states are fp32:
 *     a state is [B*T rows][n_streams][d_model]; a trace is [n_layer+1] such states, index 0 being
 *     the block input h_0 and index l+1 the output of block l.
 *   - 0-based layers: block l maps h_l -> h_{l+1} = F_l(h_l), l = 0 .. n_layer-1.
 *
 * The block (fixed by this library; the paper names only the model family, Sec. 5):
 *   x = RMSNorm(h) (no weights, eps inside the square root); q,k,v = x Wq^T, x Wk^T, x Wv^T;
 *   rotary on q,k (pairs (i, i+head_dim/2), angle pos * rope_base^(-2i/head_dim));
 *   q,k <- RMSNorm over head_dim; causal softmax(q k^T / sqrt(head_dim)) v over the layer's own
 *   keys/values; a = o Wo^T; u = h + a; m = relu(RMSNorm(u) Wup^T)^2 Wdn^T; F(h) = u + m.
 *   With n_streams > 1 the block is the mHC block of App. C.2: each branch reads
 *   RMSNorm(H_pre . x), and x' = H_res x + H_post * branch for the attention and then the MLP wrapper.
 */
#ifndef SNLP_H_
#define SNLP_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SNLP_OK 0
#define SNLP_ERR_ARG (-1)         /* NULL pointer, bad K / mode / flag                      */
#define SNLP_ERR_SHAPE (-2)       /* size beyond what the handle was created for            */
#define SNLP_ERR_STATE (-3)       /* call out of order (e.g. weights not loaded)            */
#define SNLP_ERR_OOM (-4)         /* device or host allocation failed                       */
#define SNLP_ERR_CUDA (-5)        /* a CUDA runtime call failed; see snlp_last_error()      */
#define SNLP_ERR_TIMEOUT (-6)     /* a bounded device-side wait gave up                     */
#define SNLP_ERR_UNSUPPORTED (-7) /* configuration outside what the kernels cover           */

#define SNLP_DTYPE_FP32 0 /* fp32 operands, FFMA arithmetic (no TF32)                       */
#define SNLP_DTYPE_BF16 1 /* bf16 weights / GEMM inputs / KV cache, fp32 accumulate & trace */

#define SNLP_MODE_IDN 0    /* A_l = I                      (Identity Newton, Eqs. 6-7)      */
#define SNLP_MODE_HCN 1    /* A_l = Hres_mlp,l Hres_attn,l (HC Newton, Eq. 8); = IDN if n=1 */
#define SNLP_MODE_NOCORR 2 /* A_l = 0: naive fixed-point update (Sec. 3.2); for tests       */

typedef struct snlp_model snlp_model; /* opaque: weights + workspace                        */
typedef struct snlp_kv snlp_kv;       /* opaque: per-layer KV cache of one batch            */

typedef struct {
  int32_t n_layer, d_model, n_head, head_dim, d_ff, vocab;
  int32_t n_streams; /* 1 = residual blocks, >1 (<= 8) = mHC residual streams               */
  int32_t dtype;     /* SNLP_DTYPE_*                                                        */
  int32_t max_rows;  /* largest B*T of one forward call (sizes the workspace)               */
  int32_t max_batch; /* largest B                                                           */
  int32_t max_ctx;   /* largest position + 1 (sizes the rotary table)                       */
  float rms_eps;     /* e.g. 1e-6                                                           */
  float rope_base;   /* e.g. 10000                                                          */
} snlp_config;

/* Host pointers to the layer-stacked weights ("batched form" of Sec. 3.5: one array per kind, layer
 * axis outermost).  Element type follows config.dtype: float for FP32, uint16 bf16 bit patterns for
 * BF16.  Linear weights are [out][in].  wqkv rows are Wq (d), then Wk (d), then Wv (d).
 * The hc_* arrays are float and may be NULL when n_streams == 1:
 *   hc_res_*  [L][n][n]  residual mixing,  hc_pre_* [L][n] (1 x n row),  hc_post_* [L][n] (n x 1 column). */
typedef struct {
  const void *embed;   /* [vocab][d]      */
  const void *lm_head; /* [vocab][d]      */
  const void *wqkv;    /* [L][3d][d]      */
  const void *wo;      /* [L][d][d]       */
  const void *wup;     /* [L][d_ff][d]    */
  const void *wdn;     /* [L][d][d_ff]    */
  const float *hc_res_attn, *hc_res_mlp, *hc_pre_attn, *hc_pre_mlp, *hc_post_attn, *hc_post_mlp;
} snlp_weights;

/* Create / destroy a model handle.  Allocates device weights and the workspace for max_rows rows.
 * Errors: ARG (NULL, non-positive sizes, n_head*head_dim != d_model, odd head_dim, unknown dtype),
 * OOM, CUDA.  Uses the current CUDA device; the handle stays bound to it. */
int snlp_create(const snlp_config *cfg, snlp_model **out);
int snlp_destroy(snlp_model *m);

/* Copy the weights to the device (synchronous; `host` arrays may be freed on return).  The "stacked"
 * layout is kept as is, so one sweep streams every layer's weights exactly once (Sec. 3.5).
 * Errors: ARG (NULL arrays; n_streams > 1 with a NULL hc_* array), CUDA. */
int snlp_load_weights(snlp_model *m, const snlp_weights *host);

/* h_0 = Embed(x) (Alg. 1 line 1): ids (device, int32 [B*T]) -> h0 (device, fp32 [B*T][n][d]); the
 * embedding row is copied into each of the n streams.  Errors: ARG, SHAPE (B*T > max_rows), STATE. */
int snlp_embed(snlp_model *m, const int32_t *ids, int B, int T, float *h0, void *stream);

/* Algorithm 1: sequential layer execution from h0 (device fp32 [B*T][n][d]), positions 0..T-1 of B
 * independent sequences, attention over the keys/values computed in this call.
 * trace_out (device fp32 [L+1][B*T][n][d], nullable) receives every state.
 * Errors: ARG (NULL h0, B,T < 1), SHAPE (B*T > max_rows, B > max_batch, T > max_ctx), STATE. */
int snlp_forward_sequential(snlp_model *m, const float *h0, int B, int T, float *trace_out, void *stream);

/* Algorithm 2 with prefix length S = 0 and "h0" initialisation: every state starts at h0, then K
 * sweeps; each sweep evaluates all L blocks on their own current input states (independent across
 * layers, executed as layer-batched kernels) and applies the structured correction of Eq. (5)
 * along the layer axis with the surrogate selected by `mode`.
 *   trace_out   (nullable) [L+1][B*T][n][d]: the trace after the last sweep.
 *   resnorm_out (nullable) [K][L][2] fp32: for the trace ENTERING sweep k, per layer
 *               (sum |F_l(h_l) - h_{l+1}|^2, sum |h_{l+1}|^2) over all rows, streams and features,
 *               i.e. the squared residual of Eq. (2) and the normaliser for a relative residual.
 * K > L is allowed (the trace no longer changes after L sweeps).
 * Sweep k evaluates only blocks k .. L-1: by finite-step exactness the states 0..k already equal the sequential
 * trace, so blocks 0..k-1 would reproduce the branch outputs of the previous sweep bit for bit; the correction
 * and the residual norms still cover every layer.  The result is identical to evaluating all L blocks.
 * Errors: ARG (K < 1, unknown mode, NULL h0, B,T < 1), SHAPE, STATE. */
int snlp_forward_parallel(snlp_model *m, const float *h0, int B, int T, int K, int mode,
                          float *trace_out, float *resnorm_out, void *stream);

/* General form of Algorithm 2 (Sec. 3.2, 3.5).
 *   prefix  S: the first S blocks run sequentially (Alg. 2 lines 2-4); the K sweeps cover blocks S .. L-1, with
 *              h_S held fixed.  0 <= S <= L; S = L is Algorithm 1.
 *   init      : SNLP_INIT_H0  -- every suffix state starts at the prefix state h_S (Alg. 2 line 5);
 *               SNLP_INIT_FWD -- suffix state l+1 starts at F_l(h_S): one extra batched evaluation of all suffix
 *               blocks on the prefix state ("fwd" initialisation of Sec. 3.5 / Sec. 5).
 *   fuse    M: chunkwise execution with M fused layers per chunk ("NxFM", Sec. 3.5, App. C.3): the M layers of a
 *              chunk read the chunk input; their attention outputs are summed before the MLPs, which all read
 *              u_C = h + a_C; the correction of Eq. (11) runs between chunk outputs with the identity surrogate.
 *              Needs n_streams == 1, (L - S) % M == 0 and mode IDN or NOCORR; M = 1 is the unfused algorithm.
 *              Only the chunk-boundary states S, S+M, .., L of a trace are defined.
 *   K       : number of sweeps, >= 0 (0 = prefix and initialisation only).
 *   mode    : SNLP_MODE_IDN / HCN / NOCORR, or SNLP_MODE_SEQUENTIAL: run the (fused) chunks one after the other,
 *             the exact forward of the fused model (K and init are ignored).
 * resnorm_out: [K][L][2]; rows of prefix layers and of layers that are not chunk heads are zero. */
#define SNLP_INIT_H0 0
#define SNLP_INIT_FWD 1
#define SNLP_MODE_SEQUENTIAL 3
typedef struct {
  int32_t K, mode, prefix, init, fuse;
} snlp_solver;
/* snlp_forward_parallel with a solver description.  Errors as snlp_forward_parallel, plus ARG for an invalid solver
 * and UNSUPPORTED for fuse > 1 on a multi-stream model. */
int snlp_forward_solver(snlp_model *m, const float *h0, int B, int T, const snlp_solver *solver, float *trace_out,
                        float *resnorm_out, void *stream);
/* snlp_decode_step with a solver description (K = 0 with prefix = L is the sequential step). */
int snlp_decode_step_solver(snlp_model *m, snlp_kv *kv, const int32_t *tok_in, const snlp_solver *solver, int32_t *tok_out,
                            float *resnorm_out, void *stream);

/* Copy the states the handle's last forward left behind (introspection; Alg. 1 / Alg. 2 define the trace, this call
 * only exposes it where the entry point has no trace_out of its own).  Every forward, prefill, decode step and
 * draft-and-verify round runs on the handle's internal trace [L+1][rows][n][d]; after
 *   snlp_decode_step*          rows = batch size: the states of the new position of every sequence,
 *   snlp_prefill               rows = B * (tokens of the last chunk), sequence-major,
 *   snlp_draft_and_verify*     rows = block + 1: the verifier's sequential forward over [last_tok, x_1..x_block],
 *   snlp_forward_*             rows = B * T
 * this copies it to trace_out (device fp32, (L+1)*rows*n*d values).  With fused chunks only chunk-boundary states are
 * defined.  Errors: ARG, STATE (nothing has run yet), SHAPE (rows differs from the last call's row count). */
int snlp_copy_trace(snlp_model *m, int rows, float *trace_out, void *stream);

/* LMHead (Alg. 1 line 5 / Alg. 2 line 14): sum the streams of hL (device fp32 [rows][n][d]), RMSNorm,
 * project with lm_head.  logits (device fp32 [rows][vocab], nullable) and argmax (device int32 [rows],
 * nullable; ties -> lowest index); at least one of them must be given.
 * Errors: ARG, SHAPE (rows > max_rows), STATE. */
int snlp_lm_head(snlp_model *m, const float *hL, int rows, float *logits, int32_t *argmax, void *stream);

/* KV cache for B sequences of up to max_ctx positions: per layer K and V [B][max_ctx][d] in the
 * model's dtype; keys are stored after rotary and QK-norm.  All sequences share one length.
 * A cache may outlive its model (snlp_destroy leaves it valid for snlp_kv_destroy only).
 * Errors: ARG, SHAPE (B > max_batch, max_ctx > config.max_ctx), OOM. */
int snlp_kv_create(snlp_model *m, int B, int max_ctx, snlp_kv **out);
int snlp_kv_destroy(snlp_kv *kv);
/* The length is kept on the device and mirrored on the host.  After snlp_draft_and_verify_async the host knows only an
 * upper bound; snlp_kv_len (and snlp_kv_truncate) then wait for the device (cudaDeviceSynchronize) and read the length
 * back.  In every other situation they return at once. */
int snlp_kv_len(snlp_kv *kv, int32_t *len);                   /* host out                          */
int snlp_kv_truncate(snlp_kv *kv, int new_len, void *stream); /* 0 <= new_len <= len, else ARG     */

/* Sequential forward (Alg. 1) over ids (device int32 [B][T]) at positions len .. len+T-1; fills the
 * cache and advances len by T.  Long prompts are processed in chunks of at most max_rows/B tokens.
 * last_argmax (device int32 [B], nullable) receives the greedy next token after the last position.
 * Errors: ARG, SHAPE (len + T > kv max_ctx, B != kv batch), STATE. */
int snlp_prefill(snlp_model *m, snlp_kv *kv, const int32_t *ids, int B, int T, int32_t *last_argmax,
                 void *stream);

/* One greedy decode step at position len for every sequence: embed tok_in (device int32 [B]), run
 * the layer stack at T = 1 against the cache -- K = 0: sequentially (Alg. 1); K >= 1: K layer-parallel
 * sweeps (Alg. 2) -- then LMHead + argmax into tok_out (device int32 [B]); len advances by 1.
 * Each sweep recomputes the new position's keys/values from its current iterate and overwrites the
 * cache slot, so the cache keeps the last sweep's values.  resnorm_out as in snlp_forward_parallel
 * (ignored for K = 0).  tok_in and tok_out may alias.
 * With CUDA graphs on (the default) a step is captured once per (batch, solver, attention grid size, resnorm_out, cache)
 * and replayed; the token buffers are not baked into the graph (the step's kernels find them through a device slot
 * that a one-thread kernel re-points when a call brings other buffers than the previous call did), so callers may
 * pass fresh buffers every step.
 * Errors: ARG (K < 0, mode), SHAPE (len + 1 > max_ctx), STATE. */
int snlp_decode_step(snlp_model *m, snlp_kv *kv, const int32_t *tok_in, int K, int mode, int32_t *tok_out,
                     float *resnorm_out, void *stream);

/* snlp_decode_step for a caller that keeps its tokens on the host: tok_in_host and tok_out_host are HOST int32 [B]
 * (pageable or pinned; they may alias).  The tokens go through the library's own mapped pinned staging buffer, which
 * the step's kernels read and write across the bus; the call returns once every output token has arrived in host memory
 * (it watches the staging buffer; should the tokens not arrive within 50 ms it synchronises `stream` instead), so
 * tok_out_host is valid on return.  The step's last kernel may still be retiring at that moment; later calls on the same
 * stream are ordered behind it as usual.  One staging buffer per model: calls on the same model must not overlap.  Errors as
 * snlp_decode_step, plus CUDA. */
int snlp_decode_step_host(snlp_model *m, snlp_kv *kv, const int32_t *tok_in_host, int K, int mode, int32_t *tok_out_host,
                          void *stream);

/* One round of greedy self-speculative decoding (Sec. 5.1), batch 1: the SNLP(K, mode) drafter proposes
 * `block` tokens x_1..x_block from *last_tok by decode steps; one sequential forward over
 * [last_tok, x_1..x_block] (block+1 rows) verifies them and overwrites the drafter's cache entries;
 * the longest prefix with x_i == verifier token y_{i-1} is accepted.  Writes emitted (device int32
 * [block+1]) = x_1..x_n, y_n; n_emitted = n+1; n_accepted = n (device int32 each); *last_tok <- y_n;
 * cache length = len_before + n + 1.  This form synchronises `stream` before returning and brings the
 * cache length back to the host.  The emitted stream equals the model's sequential greedy stream.
 * Errors: ARG (block < 1, K < 1, mode, NULLs), SHAPE (kv batch != 1, len + block + 1 > max_ctx,
 * block + 1 > max_rows), STATE. */
int snlp_draft_and_verify(snlp_model *m, snlp_kv *kv, int32_t *last_tok, int block, int K, int mode,
                          int32_t *emitted, int32_t *n_emitted, int32_t *n_accepted, void *stream);
/* The same round (Sec. 5.1) without any host synchronisation: everything is enqueued on `stream`; n_accepted,
 * n_emitted, the emitted tokens, *last_tok and the new cache length stay on the device, so rounds can be issued
 * back to back.  Until snlp_kv_len is called the host tracks the cache length by its upper bound (every draft
 * accepted): capacity checks use that bound -- a call that would not fit under it first fetches the true length --
 * and the decode attention sizes its grid by it (chunks beyond the true length add exact zeros, so no result bit
 * changes).  Errors as snlp_draft_and_verify. */
int snlp_draft_and_verify_async(snlp_model *m, snlp_kv *kv, int32_t *last_tok, int block, int K, int mode,
                                int32_t *emitted, int32_t *n_emitted, int32_t *n_accepted, void *stream);

/* Tuning / introspection (no effect on results).  flag 0: use CUDA graphs for decode steps (default 1).
 * flag 1: force the generic SIMT kernels even where a specialised kernel exists (default 0; testing).
 * flag 2: time every launch with CUDA events on its stream, accumulated per kernel class (default 0;
 *         while on, decode steps are launched directly instead of replaying graphs).
 * flag 4: programmatic dependent launch between the kernels of layer-by-layer execution (sequential forward, sequential
 *         prefix; default 1): a kernel is scheduled while its predecessor finishes and requests its first weight tiles
 *         before it waits for that kernel's results.  The launches of a sweep never use it.
 * flag 5: decode regime: run the three products that follow the attention (out-projection, MLP up, MLP down) as one
 *         cooperative launch with grid barriers between them (default 1); 0 = three launches.  Same results bit for bit.
 *         Under flag 2 the one launch is booked under the MLP-up class.
 * flag 3: failure-detection test hook: waits for the device, then writes `value != 0` into the error word that a
 *         kernel raises when one of its bounded waits expires; snlp_device_status then reports it exactly as it
 *         would report a real expiry (no kernel is made to wait). */
int snlp_set_flag(snlp_model *m, int flag, int value);

/* Kernel classes of snlp_kernel_times, in order: QKV projection, attention, out-projection, MLP up,
 * MLP down, correction, lm head (+argmax), everything else (embed, casts, bookkeeping). */
#define SNLP_NUM_KERNEL_CLASSES 8
/* Waits for the timed launches recorded so far and returns, per class, the summed device time in
 * milliseconds (host double[8]) and the number of launches (host int64[8]); reset != 0 clears them. */
int snlp_kernel_times(snlp_model *m, double *ms, int64_t *launches, int reset);
/* Synchronises `stream` and reports whether any kernel of this handle gave up on one of its bounded
 * device-side waits since the last check (SNLP_ERR_TIMEOUT, flag cleared) or not (SNLP_OK). */
int snlp_device_status(snlp_model *m, void *stream);

/* Number of kernel launches this handle has enqueued since creation (graph replays count their nodes). */
int snlp_launch_count(const snlp_model *m, int64_t *count);
/* Number of decode-step graphs this handle has captured since creation. */
int snlp_graph_count(const snlp_model *m, int64_t *captured);

/* Greedy LM head that allocates nothing (the paper has no counterpart: this entry point exists for
 * callers that cannot obtain device memory at call time -- for example a serving loop whose memory budget
 * has been handed entirely to another allocator, a plug-in running inside a host application that forbids
 * allocation after start-up, or a latency-critical path where the implicit device synchronisation of an
 * allocation is not acceptable).  Same computation as snlp_lm_head restricted to the argmax:
 *     argmax[r] = argmax_v  lm_head[v] . RMSNorm(sum_s hL[r][s][:])        (ties -> lowest index)
 * by a kernel of its own (the two entry points add a logit's terms in different orders, so they can disagree
 * where two logits are closer than bf16 rounding noise), without a model handle and without a cudaMalloc'd
 * workspace: the per-tile argmax partials go to a fixed 256 KiB array inside the library image (each GPU that
 * loads the library holds one copy until the process exits).
 *   hL           device fp32 [rows][n_streams][d_model]
 *   lm_head_bf16 device bf16 bit patterns [vocab][d_model], caller-owned (inputs and outputs are still yours)
 *   argmax       device int32 [rows]
 * Limits: rows <= 16, vocab <= SNLP_STATIC_LM_HEAD_MAX_VOCAB (multiple of 128), d_model <=
 * SNLP_STATIC_LM_HEAD_MAX_D_MODEL (multiple of 32); larger sizes return SNLP_ERR_SHAPE before anything
 * is launched.  Neither this call nor anything it uses calls cudaMalloc/cudaFree.
 * The first call on a device looks up the array's device address and sets two kernel attributes; make
 * that first call during set-up, with the device current.
 * All calls on a device share the one array, which keeps whatever the previous call left in it (nothing
 * needs to start at zero: every slot a call reads, it has written first).  Two calls that overlap on the
 * GPU -- different streams without ordering, or two host threads -- race on it: serialise them.
 * hL and lm_head_bf16 must be 16-byte aligned, argmax 4-byte aligned.
 * Errors: ARG (NULL, misaligned pointer, non-positive sizes), SHAPE (beyond the limits), UNSUPPORTED (vocab % 128,
 * d_model % 32), CUDA. */
#define SNLP_STATIC_LM_HEAD_MAX_VOCAB 262144
#define SNLP_STATIC_LM_HEAD_MAX_D_MODEL 4096
int snlp_lm_head_greedy_static(const float *hL, const void *lm_head_bf16, int rows, int n_streams, int d_model, int vocab,
                               float rms_eps, int32_t *argmax, void *stream);

const char *snlp_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SNLP_H_ */
