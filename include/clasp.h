/*
 * clasp.h -- C ABI of the B200 (sm_100a) layer-skip search library.
 *
 * The library implements the "layer optimisation" stage of CLaSp's three-stage
 * self-speculative decoding loop (Sec. 3.1): after each verification it searches,
 * by the approximate dynamic programme of Eq. 2 / Algorithm 1, for the set of M
 * decoder layers whose removal keeps the last verified token's top hidden state
 * closest (cosine) to the full model's, and it provides the full-model (verify)
 * and layer-skipped (draft) forwards that share its kernels.
 *
 * Conventions
 *   - "device" pointers are CUDA device memory of the current device, allocated
 *     and owned by the caller; the library never allocates or frees device
 *     memory.  "host" pointers are ordinary host memory.
 *   - All work is enqueued on the stream given to clasp_create; results are
 *     valid after the caller synchronises that stream.  No call synchronises
 *     unless its comment says so.
 *   - Matrices are row-major [out_features, in_features] in the model dtype
 *     (CLASP_BF16: bfloat16, CLASP_FP32: float).  Norm weights are float.
 *   - The KV cache of one layer is two arrays [max_ctx, n_kv_heads, head_dim] in
 *     the model dtype; keys are stored AFTER rotary embedding.
 *   - Hidden states / residual stream are float everywhere.
 *   - Layers are f_0..f_{L-1};  h_0 = embedding,  h_{l+1} = f_l(h_l)  (Sec. 3.4).
 *   - Every function returns CLASP_OK (0) or a negative CLASP_ERR_*; nothing
 *     throws, aborts or traps on the device.  Every device-side wait is bounded;
 *     one that runs out records a code readable by clasp_last_device_status.
 *   - Alignment: weight matrices, float buffers (hidden states, layer inputs and
 *     outputs, g_final) and K/V arrays are 16-byte aligned and float strides are
 *     multiples of 4 elements (the kernels use 16-byte accesses); a call that is
 *     given anything else returns CLASP_ERR_INVALID_ARG before it launches.
 *   - No environment variable changes what the library computes or how.
 */
#ifndef CLASP_H_
#define CLASP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CLASP_OK 0
#define CLASP_ERR_INVALID_ARG (-1)  /* null pointer, negative size, M > L ...            */
#define CLASP_ERR_SHAPE (-2)        /* a shape the kernels do not support                 */
#define CLASP_ERR_CAPACITY (-3)     /* exceeds max_ctx / max_rows / workspace size        */
#define CLASP_ERR_DTYPE (-4)        /* unknown dtype                                      */
#define CLASP_ERR_CUDA (-5)         /* a CUDA runtime / driver call failed                */
#define CLASP_ERR_TIMEOUT (-6)      /* a bounded device-side wait gave up                 */
#define CLASP_ERR_NOT_LOADED (-7)   /* a layer or the head has not been loaded            */

#define CLASP_FP32 0
#define CLASP_BF16 1

/* choice table entries (Algorithm 1: which parent g[i][j] was copied from) */
#define CLASP_CHOICE_APPLY 0   /* g[i][j] = f_{i-1}(g[i-1][j])   */
#define CLASP_CHOICE_SKIP 1    /* g[i][j] = g[i-1][j-1]          */
#define CLASP_CHOICE_NONE 255  /* cell not defined (j > i) or "not forced" */

typedef struct clasp_ctx clasp_ctx;

typedef struct clasp_config {
  int32_t L;            /* decoder layers                                         */
  int32_t d_model;      /* multiple of 8                                          */
  int32_t n_q_heads;    /* multiple of n_kv_heads                                 */
  int32_t n_kv_heads;
  int32_t head_dim;     /* 64 or 128                                              */
  int32_t d_ffn;        /* multiple of 8                                          */
  int32_t vocab;
  int32_t dtype;        /* CLASP_FP32 | CLASP_BF16: weights, KV cache             */
  float rms_eps;
  float rope_theta;
  int32_t max_ctx;      /* KV cache capacity in positions                         */
  int32_t max_rows;     /* most rows any call pushes through a layer:
                           clasp_verify n, clasp_dp_search M*T                    */
  int32_t max_M;        /* most skipped layers a search is asked for              */
  int32_t max_T;        /* most objective positions of a search                   */
  int32_t max_head_rows;/* most rows sent through the LM head in one call         */
  int32_t flags;        /* CLASP_FLAG_*                                           */
} clasp_config;

#define CLASP_FLAG_FORCE_SIMT 1 /* bf16 model: use the CUDA-core GEMM instead of the
                                   tcgen05 one (diagnostics; both are device code) */
#define CLASP_FLAG_NO_DEFER 2   /* diagnostics: the search lets every layer wait for the
                                   Eq. 2 decision of the step before it, instead of sending
                                   both candidates of a state through the layer's q/k/v
                                   product and keeping the chosen one.  Same operand bytes
                                   either way, so the results agree. */
#define CLASP_FLAG_PRUNE 8      /* the search leaves out the states from which (L, M) can no longer be
                                   reached, j < M - (L - i): Algorithm 1 computes them, but the backtrack
                                   can never visit them.  Skip mask, g[L][M] and every reachable cell are
                                   unchanged; the cells left out read NaN in `scores` and `margins`. */
#define CLASP_FLAG_MULTI_KERNEL 4 /* diagnostics, bf16 model: one kernel per step (tcgen05
                                   GEMM, attention, norm, Eq. 2 select ...) instead of the
                                   persistent kernel that runs a whole call in one launch */

#define CLASP_FLAG_NO_ATT_TC 16 /* diagnostics: searches over long contexts (about 4000 visible positions or
                                   more; 2500 when a kv head serves at most 64 (row, query head) pairs, 1000
                                   when it serves 256 or more) keep the attention over the cache keys on the warp-level multiply
                                   instead of tcgen05 (the two sum a row's keys in different orders:
                                   results agree to rounding, not bit for bit) */

/* Device pointers to the nine tensors of one decoder layer (borrowed). */
typedef struct clasp_layer_weights {
  const float* attn_norm; /* [d_model]                    */
  const void* wq;         /* [n_q_heads*head_dim, d_model] */
  const void* wk;         /* [n_kv_heads*head_dim, d_model] */
  const void* wv;         /* [n_kv_heads*head_dim, d_model] */
  const void* wo;         /* [d_model, n_q_heads*head_dim] */
  const float* mlp_norm;  /* [d_model]                    */
  const void* w_gate;     /* [d_ffn, d_model]             */
  const void* w_up;       /* [d_ffn, d_model]             */
  const void* w_down;     /* [d_model, d_ffn]             */
} clasp_layer_weights;

/* Device pointers to one layer's KV cache (borrowed). */
typedef struct clasp_kv_layer {
  void* k; /* [max_ctx, n_kv_heads, head_dim], after RoPE */
  void* v; /* [max_ctx, n_kv_heads, head_dim]             */
} clasp_kv_layer;

/* Bytes of device workspace clasp_create needs for this configuration (0 on a
 * bad configuration).  Host-only; launches nothing. */
size_t clasp_workspace_bytes(const clasp_config* cfg);

/* Create a context.  `workspace` is device memory of at least
 * clasp_workspace_bytes(cfg) bytes, 256-byte aligned, owned by the caller and
 * kept alive until clasp_destroy; the library zeroes the parts that need it
 * (on `cuda_stream`).  `cuda_stream` is a cudaStream_t (may be NULL = default
 * stream).  The context keeps host-side descriptors only. */
int clasp_create(const clasp_config* cfg, void* workspace, size_t workspace_bytes,
                 void* cuda_stream, clasp_ctx** out);
void clasp_destroy(clasp_ctx* ctx);

/* 1 when the context runs its searches and forwards in the persistent layer kernel (one
 * cooperative launch per call), 0 when it uses one kernel per step: an fp32 model, the two
 * diagnostic flags above, or a bf16 shape the persistent kernel does not take (vocab not a
 * multiple of 8; more than 128 d_model features per SM; a weight matrix whose per-SM row
 * ranges need more than four distinct heights; no cooperative launch on the device).  Both
 * paths compute the same thing; the second is several times slower, so a caller that sized
 * its deployment for the first should check.  Per call, a search with M*T > 128 candidate
 * rows and a forward over more than 128 rows also take the one-kernel-per-step path.
 * Negative: CLASP_ERR_INVALID_ARG. */
int clasp_engine_active(const clasp_ctx* ctx);

/* Limit of every device-side wait in the context's kernels, in polls (a poll is about
 * 100 ns once a wait has started to sleep between polls); 0 restores the default (about
 * half a second).  A wait that reaches the limit makes its kernel wind down -- copies in
 * flight are awaited, tensor memory is freed -- and clasp_last_device_status reports
 * CLASP_ERR_TIMEOUT; the outputs of that call are unspecified, the context stays usable.
 * A limit of a few polls makes healthy kernels give up: that is how the tests reach the
 * wind-down path without a kernel that would wait forever. */
int clasp_set_wait_limit(clasp_ctx* ctx, uint32_t polls);

/* Register the weights of layers first..first+count-1 (Sec. 3.4: the decoder
 * layers f_l the search and the forwards apply).  `w` is a HOST array of
 * `count` structs holding DEVICE pointers; the tensors are borrowed, must stay
 * alive and unchanged while the context uses them, and must be 16-byte aligned. */
int clasp_load_layers(clasp_ctx* ctx, int32_t first, int32_t count, const clasp_layer_weights* w);

/* Register the embedding table [vocab, d_model], the final norm weight
 * [d_model] (float) and the LM head [vocab, d_model]; device, borrowed. */
int clasp_load_head(clasp_ctx* ctx, const void* embed, const float* final_norm, const void* lm_head);

/* Layer-skip search (Eq. 2, Algorithm 1; j-loop batched as in Sec. 3.6).
 *
 *   hidden_states  device, float: the full model's states x_0..x_L of the T
 *                  objective positions; element (l, t, c) is at
 *                  hidden_states[l*layer_stride + t*token_stride + c].
 *   kv             HOST array of L structs of DEVICE pointers; read-only here.
 *   ctx_len        C: cache positions [0, C) are visible to every state.
 *   pos0           absolute position of the first objective row (normally C).
 *   T, M           objective rows (paper: 1) and number of layers to skip.
 *   skip_mask      device, uint8[L], out: 1 = layer skipped by the draft model.
 *   scores         device, float[(L+1)*(M+1)], out: D(i, j) of Eq. 2, NaN where
 *                  j > i.  For T > 1 the mean of the T per-row cosines.
 *   margins        device or NULL, same shape: cosine(apply) - cosine(skip)
 *                  where both candidates exist, NaN elsewhere.
 *   g_final        device or NULL, float[T*d_model], out: g[L][M].
 *   forced_choice  device or NULL, uint8[(L+1)*(M+1)]: where an entry is not
 *                  CLASP_CHOICE_NONE the search takes that decision instead of
 *                  comparing cosines (test hook: follow an oracle's path).
 *
 * Step i pushes the states g[i-1][1..min(i-1,M)] through layer i-1 in one batch,
 * so each layer's weights are read from HBM once; each state attends to the
 * cache plus its own freshly computed keys, never to another state, and the
 * cache is not written.  M == 0 writes an all-zero mask and D(i,0) = 1 only.
 * Errors: INVALID_ARG (null, M > L, T < 1), CAPACITY (M > max_M, T > max_T,
 * M*T > max_rows, ctx_len + T > max_ctx), NOT_LOADED. */
int clasp_dp_search(clasp_ctx* ctx, const float* hidden_states, int64_t layer_stride,
                    int64_t token_stride, const clasp_kv_layer* kv, int32_t ctx_len, int32_t pos0,
                    int32_t T, int32_t M, uint8_t* skip_mask, float* scores, float* margins,
                    float* g_final, const uint8_t* forced_choice);

/* Full-model forward over n tokens at positions pos0..pos0+n-1 (the verify
 * model of Sec. 3.1; also the prompt prefill and plain autoregressive steps).
 *
 *   tokens       device, int32[n].
 *   kv           HOST array of L structs; K/V of the n positions are WRITTEN for
 *                every layer, positions [0, pos0) are read.
 *   n_head_rows  the last n_head_rows rows go through final norm + LM head.
 *   argmax_out   device, int32[n_head_rows]: greedy token per row, lowest
 *                index on ties.  May be NULL when n_head_rows == 0.
 *   hidden_out   device or NULL, float[n*(L+1)*d_model]: element (t, l, c) at
 *                hidden_out[(t*(L+1) + l)*d_model + c] = residual stream
 *                entering layer l (l = L: after the last layer, before the
 *                final norm) -- the objective the search needs (Sec. 3.4).
 * Errors: CAPACITY (n > max_rows, pos0 + n > max_ctx, n_head_rows > max_head_rows). */
int clasp_verify(clasp_ctx* ctx, const int32_t* tokens, int32_t n, int32_t pos0,
                 const clasp_kv_layer* kv, int32_t n_head_rows, int32_t* argmax_out,
                 float* hidden_out);

/* One token through the layer-skipped draft model (Sec. 3.1, Sec. 3.3).
 *
 *   skip_mask_host  HOST uint8[L], 1 = skip the layer entirely (no weights read,
 *                   no K/V written).
 *   token_in        device, int32[1] (may be the previous call's token_out).
 *   token_out       device, int32[1]: greedy next token.
 *   top1_prob_out   device or NULL, float[1]: softmax probability of token_out. */
int clasp_draft_forward(clasp_ctx* ctx, const uint8_t* skip_mask_host, const int32_t* token_in,
                        int32_t pos, const clasp_kv_layer* kv, int32_t* token_out,
                        float* top1_prob_out);

/* Non-greedy decoding (Sec. 4 and Table 1, "Temperature = 1"; the accept / resample rule is the one of
 * speculative sampling, which the paper cites for losslessness).  Random numbers are Philox4x32-10
 * draws keyed by `seed` and counted by (index, position, purpose, round): a call is a pure function of
 * its arguments, there is no generator state.
 *
 * clasp_draft_sample: one token through the layer-skipped model as clasp_draft_forward, but the next
 * token is a draw of softmax(logits / temperature) (arg-max of logits / T + Gumbel noise, lowest index
 * on ties) instead of the arg-max.
 *   logits_out   device, float[vocab], 16-byte aligned, out: the draft model's logits for the drafted
 *                position (the verification needs them)
 *   round        >= 0: distinguishes the draws of different rounds at the same position
 * clasp_verify_sample: full-model forward over n tokens at pos0.. as clasp_verify; the last
 * n_drafts tokens are drafts (tokens[n - n_drafts + k] sampled from draft_logits[k]).  Draft k is
 * accepted with probability min(1, p_k(x) / q_k(x)); the first rejected position gets a draw of
 * norm(max(0, p_k - q_k)) and ends the walk; if all are accepted the position after the last draft gets
 * a draw of the full model's distribution.  n_drafts == 0 just samples the token after the n rows
 * (prompt prefill, plain ancestral sampling).
 *   draft_logits   device, float[n_drafts * vocab] (may be NULL when n_drafts == 0)
 *   logits_ws      device, float[(n_drafts + 1) * vocab], 16-byte aligned: receives the full model's
 *                  logits of the head rows (caller-owned scratch, readable afterwards)
 *   n_accepted_out device, int32[1]; committed_out device, int32[n_drafts + 1]: the accepted drafts
 *                  followed by the sampled token; must not overlap `tokens`
 * Errors: INVALID_ARG (temperature <= 0, null or misaligned buffers, n_drafts >= n), CAPACITY
 * (n_drafts > 63 or as clasp_verify with n_head_rows = n_drafts + 1). */
int clasp_draft_sample(clasp_ctx* ctx, const uint8_t* skip_mask_host, const int32_t* token_in,
                       int32_t pos, const clasp_kv_layer* kv, float temperature, uint64_t seed,
                       int32_t round, int32_t* token_out, float* logits_out);
int clasp_verify_sample(clasp_ctx* ctx, const int32_t* tokens, int32_t n, int32_t pos0,
                        const clasp_kv_layer* kv, int32_t n_drafts, const float* draft_logits,
                        float temperature, uint64_t seed, int32_t round, float* logits_ws,
                        int32_t* n_accepted_out, int32_t* committed_out, float* hidden_out);

/* Greedy acceptance (Sec. 3.1, verification stage).  HOST pointers, no GPU
 * work: draft[K] are the drafted tokens, full_argmax[K+1] the full model's
 * greedy tokens for the rows [pending, draft_1..draft_K].  Writes the number a
 * of leading drafts that match and the a+1 committed tokens (the accepted
 * drafts followed by the full model's own token). */
int clasp_accept(const int32_t* draft, const int32_t* full_argmax, int32_t K,
                 int32_t* n_accepted, int32_t* committed /* [K+1] */);

/* One decoder layer applied to S independent states of T rows each (the batch
 * of Sec. 3.6).  x_in/x_out: device float, row (s*T+t) at x + row*stride.
 * Row t of a state sits at position pos0+t, sees cache [0, ctx_len) and rows
 * 0..t of its own state.  write_kv != 0 requires S == 1 and stores the rows'
 * K/V into the cache at pos0..pos0+T-1 (they are also what the rows attend to).
 * Exposed so that a single layer can be checked against the oracle. */
int clasp_layer_forward(clasp_ctx* ctx, int32_t layer, const float* x_in, int64_t in_stride,
                        int32_t S, int32_t T, int32_t ctx_len, int32_t pos0,
                        const clasp_kv_layer* kv_layer, int32_t write_kv, float* x_out,
                        int64_t out_stride);

/* y[r, n] = sum_k x[r, k] * w[n, k]  (float out) through the same weight-
 * streaming GEMM the layers use; x: device, model dtype, [R, K] contiguous;
 * w: device, model dtype, [N, K]; y: device float [R, N].  Test hook. */
int clasp_gemm_xwT(clasp_ctx* ctx, const void* x, const void* w, int32_t R, int32_t N, int32_t K,
                   float* y);

/* Allocation-free variant of clasp_gemm_xwT for bf16 operands (the paper has no
 * counterpart; it exists for callers that must not allocate).
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- an inference
 * plug-in's enqueue hook, or a serving loop that handed the whole device to a memory
 * pool at start-up, so that a fresh allocation would fail or force a device-wide
 * synchronisation in the middle of decoding.  Such a caller cannot create a clasp_ctx
 * (whose workspace somebody has to allocate) just to run one product.
 *
 * What it does: y[r, n] = sum_k x[r, k] * w[n, k] with the same tensor-core kernel and
 * the same split-K schedule as clasp_gemm_xwT, so the two agree bit for bit.  The
 * split-K partial sums, the per-tile arrival counters and a status word live in a
 * fixed array of CLASP_NOALLOC_SCRATCH_BYTES that is part of the library image: every
 * GPU that loads the library carries it until the process exits.  The call makes no
 * cudaMalloc, cudaFree or other allocating call; the caller passes inputs and outputs.
 *
 *   x  device, bf16 [R, K] contiguous, 16-byte aligned;  1 <= R <= CLASP_NOALLOC_MAX_ROWS
 *   w  device, bf16 [N, K] contiguous, 16-byte aligned;  K a multiple of 8
 *   y  device, float [R, N]
 *   cuda_stream  the cudaStream_t to launch on (NULL = default stream)
 *   status_out   device int32 or NULL: set to 1 by the kernel if one of its bounded
 *                waits gave up (y is then unspecified); the caller zeroes it beforehand.
 *                With NULL a wait that gave up is NOT reported anywhere (the flag goes to
 *                a word of the scratch array that the next call clears): pass a word if
 *                the result matters.
 *
 * Limits: shapes whose partial sums (splits * R * N floats) exceed the array, or with
 * more than 4096 output tiles under split-K, are refused with CLASP_ERR_CAPACITY;
 * R > CLASP_NOALLOC_MAX_ROWS likewise.  Devices other than sm_100 give CLASP_ERR_CUDA.
 * First use on each device: the first call made with that device current looks up the
 * array's device address and the driver's tensor-map encoder and raises the kernel's
 * shared-memory limit.  Make that first call before any stream capture begins.
 * Sharing: all calls on a device use the one array and it keeps the previous call's
 * contents; each call re-zeroes the counters on its stream before launching.  Two
 * calls that overlap on the GPU (different streams, or different host threads without
 * ordering) race on it: serialise them. */
#define CLASP_NOALLOC_SCRATCH_BYTES (4u * 1024u * 1024u + 16u * 1024u + 256u)
#define CLASP_NOALLOC_MAX_ROWS 256
int clasp_gemm_xwT_noalloc(const void* x, const void* w, int32_t R, int32_t N, int32_t K, float* y,
                           void* cuda_stream, int32_t* status_out);

/* Synchronises the context's stream and returns the device status word:
 * CLASP_OK, or CLASP_ERR_TIMEOUT if a bounded wait inside a kernel gave up
 * since the last call (the word is then cleared), or CLASP_ERR_CUDA. */
int clasp_last_device_status(clasp_ctx* ctx);

/* Per-launch timing of the weight-streaming kernels (measurement aid; no counterpart in
 * the paper).  enable != 0 starts bracketing every launch of the persistent layer kernel
 * (one launch = one search / verify / draft call) and of the stand-alone tensor-core GEMM
 * with a pair of CUDA events on the context's stream.  enable == 0 synchronises the
 * stream, stops, and reports through the non-NULL HOST pointers the number of launches
 * bracketed, the sum of their durations in milliseconds and the bytes those launches had
 * to move (every weight matrix once, N*K*2 bytes, plus the visible K/V of each layer
 * pass).  Returns CLASP_ERR_CUDA if an event call fails. */
int clasp_profile_gemm(clasp_ctx* ctx, int32_t enable, int64_t* n_launches, double* total_ms,
                       double* weight_bytes);

/* Number of kernel launches the context has enqueued so far (host counter). */
int64_t clasp_launch_count(const clasp_ctx* ctx);

/* Step tracing of the persistent layer kernel (measurement aid; no counterpart in the
 * paper).  `stamps` is DEVICE memory of n_ctas * cap_per_cta uint64 (borrowed until it is
 * replaced or cleared with NULL): during every following search / verify / draft call the
 * kernel's CTA c writes %globaltimer values (ns) to stamps[c * cap_per_cta + 64 * j + s]
 * when it reaches step boundary s of job j of the call (jobs: one per decoder layer pass or
 * Eq. 2 step, then the LM head; s: 0 job start, 1 q/k/v done, 2-5 attention partials, 6
 * attention merged, 7 o, 8 gate/up, 9 down, 10-13 Eq. 2 step, 14 head; for product p = 0..3
 * (q/k/v, o, gate/up, down) 16+p first operands ready for the tensor core, 20+p last
 * multiply issued, 24+p first accumulator complete; 28 Eq. 2 step published the next operand;
 * 29-31 operand of q/k/v, o, gate/up seen complete by the operand loader; 32-63 free for finer
 * stamps; entries a CTA does not reach stay as the caller left them, entries beyond
 * cap_per_cta are not recorded).  *n_ctas (HOST, may be NULL) receives the grid size, 0 when
 * the context does not use the persistent kernel.  cap_per_cta < 0 only queries *n_ctas and
 * leaves a trace buffer in use as it is. */
int clasp_engine_trace(clasp_ctx* ctx, uint64_t* stamps, int32_t cap_per_cta, int32_t* n_ctas);

const char* clasp_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* CLASP_H_ */
