/*
 * hispec.h -- C ABI of the B200 (sm_100a) HiSpec verification library.
 *
 * HiSpec (hierarchical speculative decoding) runs on ONE early-exit transformer
 * with exits L_d < L_i < L_f (Sec. 3.1 of the paper): layers [0,L_d) draft
 * tokens, layers [L_d,L_i) verify them first ("intermediate verification"),
 * layers [L_i,L_f) validate the tentatively accepted tokens periodically
 * (Algorithm 2).  The three stages share one KV cache and the hidden states
 * already computed (Sec. 3.2): a stage never recomputes the layers below it.
 *
 * Conventions for every entry point
 *  - Pointers marked "device" are device memory owned by the caller; the
 *    library never frees or reallocates them.  Pointers marked "host" are
 *    read during the call only.  The library allocates its fixed workspace in
 *    hispec_create() and nothing per call.
 *  - All work is enqueued on the caller's CUDA stream (`stream` is a
 *    cudaStream_t passed as void*); no call synchronises.  Outputs are valid
 *    once the caller has synchronised the stream.
 *  - Return value: 0 on success, a negative HISPEC_E* code on a host-detected
 *    error (nothing is enqueued in that case).  Faults only the device can see
 *    (a block-table entry out of range, inconsistent lengths, a bounded wait
 *    that ran out) never trap or hang: the kernel skips the access, ORs a bit
 *    into the context's status word and the call completes;
 *    hispec_device_status() returns and clears that word.
 *  - Positions are 0-based.  A sequence with n committed tokens has KV length
 *    n-1 in every layer group and token x_{n-1} "pending" (it has been through
 *    no layer).  Row j of a call sits at position p0 + j, where p0 is the
 *    valid KV length, on entry, of the layer group the call starts in.
 *  - One context may be used from one host thread at a time.
 */
#ifndef HISPEC_H
#define HISPEC_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HISPEC_OK 0
#define HISPEC_EINVAL (-1)    /* bad argument: NULL, layer range, exits not increasing, batch/k over capacity */
#define HISPEC_ECAPACITY (-2) /* workspace or caller buffer too small for the request */
#define HISPEC_ECUDA (-3)     /* a CUDA runtime/driver call failed (cudaGetLastError is left set) */
#define HISPEC_ENOMEM (-4)    /* workspace allocation failed in hispec_create */

/* bits of the device status word */
#define HISPEC_ST_BOUNDS 1u  /* page id / position / token id outside its table: access skipped */
#define HISPEC_ST_STATE 2u   /* length counters inconsistent with the call (rows not buffered, groups out of step) */
#define HISPEC_ST_TIMEOUT 4u /* a bounded device-side wait gave up */

/* hispec_model_desc.flags */
#define HISPEC_FLAG_SIMT_GEMM 1u  /* debug: run the projections on the plain CUDA-core kernel instead of tcgen05 */
#define HISPEC_FLAG_PLAIN_ACT 2u  /* feed bf16-rounded activations to the tensor cores (default: hi+lo split,
                                     x = bf16(x) + bf16(x - bf16(x)), which costs no extra HBM traffic) */
#define HISPEC_FLAG_NO_PDL 4u     /* debug: launch kernels without programmatic dependent launch */
#define HISPEC_FLAG_MULTI_KERNEL 16u /* run a call as a sequence of kernels instead of the single persistent kernel
                                       (also taken when a call has more than 128 padded rows) */
#define HISPEC_FLAG_ROWWARP_ATTN 8u /* debug: one-warp-per-row attention instead of the tiled kernel (the tiled
                                       kernel needs page_size == 16; other page sizes always take this path) */

typedef struct hispec_ctx hispec_ctx; /* opaque */

typedef struct {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
    float rope_base; /* rotary base; pair (i, i + head_dim/2) rotates by pos * base^(-2i/head_dim) */
    float rms_eps;
    int32_t page_size;         /* tokens per KV page */
    int32_t max_batch;         /* sequences per call */
    int32_t max_rows_per_seq;  /* rows per sequence per call, and row capacity of h_draft / h_inter */
    int32_t max_pages_per_seq; /* width of the block table */
    uint32_t flags;
} hispec_model_desc;

/* Weights: immutable, caller-owned.  Matrices are bf16, row-major [out_features][in_features].
 * The per-layer arrays are HOST arrays of n_layers DEVICE pointers; the entry of a layer no
 * call ever touches may be NULL. */
typedef struct {
    const void *tok_emb;        /* device bf16 [vocab][d_model] */
    const void *const *wqkv;    /* [(n_q_heads + 2 n_kv_heads) * head_dim][d_model]: q heads, k heads, v heads */
    const void *const *wo;      /* [d_model][n_q_heads * head_dim] */
    const void *const *wgu;     /* [2 * d_ffn][d_model]: gate rows, then up rows */
    const void *const *wdown;   /* [d_model][d_ffn] */
    const float *const *attn_norm, *const *ffn_norm; /* device fp32 [d_model] RMSNorm gains */
    const float *final_norm;    /* device fp32 [d_model]: norm in front of every exit head */
} hispec_weights;

/* The three exits of Sec. 3.1 and the LM head each one projects through ("shared or
 * auxiliary LM head": pass the same pointer three times for a shared head).
 * Heads are device bf16 [vocab][d_model]. */
typedef struct {
    int32_t L_d, L_i, L_f; /* 0 < L_d < L_i < L_f <= n_layers; exit L = after L layers */
    const void *head_d, *head_i, *head_f;
} hispec_exits;

/* Paged KV cache with block tables (Sec. 5.4) and the valid length of each layer group. */
typedef struct {
    void *k_pages, *v_pages;    /* device bf16 [n_pool_layers][n_pages][n_kv_heads][page_size][head_dim];
                                   pool layer i holds model layer first_layer + i */
    const int32_t *block_table; /* device [batch][max_pages_per_seq]: physical page of logical page */
    int32_t *len_draft;         /* device [batch], in/out: valid KV length of layers [0, L_d) */
    int32_t *len_inter;         /* ... of [L_d, L_i) */
    int32_t *len_target;        /* ... of [L_i, L_f) */
    int64_t n_pages;
    int32_t first_layer, n_pool_layers;
} hispec_kv;

/* Hidden-state buffers of Sec. 3.2, device fp32 [batch][max_rows_per_seq][d_model], in/out.
 * h_draft row r = exit-L_d hidden state of position len_inter + r (filled by hispec_draft,
 * consumed by hispec_verify_intermediate); h_inter row r = exit-L_i hidden state of position
 * len_target + r (appended by hispec_verify_intermediate over several rounds, consumed by
 * hispec_verify_target). */
typedef struct {
    float *h_draft, *h_inter;
} hispec_hidden;

/* Outputs of a call.  Row strides use max_rows_per_seq.  Optional pointers may be NULL. */
typedef struct {
    int32_t *n_accepted; /* device [batch]: a_b = number of leading block tokens equal to the verifier's */
    int32_t *next_token; /* device [batch]: verifier's token v_{a_b+1} if that row was computed, else -1 */
    int32_t *argmax_ids; /* optional device [batch][max_rows_per_seq] */
    float *top2;         /* optional device [batch][max_rows_per_seq][2]: largest, second largest logit */
    float *logits;       /* optional device [batch][max_rows_per_seq][vocab] (parity/debug; costs HBM writes) */
    float *hidden_out;   /* optional device [batch][max_rows_per_seq][d_model]: residual stream at the exit */
    int32_t *tentative;  /* optional device [batch][max_rows_per_seq], in/out: the list V (see
                            hispec_verify_intermediate) */
    int32_t *pending;    /* optional device [batch]: the token that is pending after a verify call, i.e. the
                            last element of its result list: v_{a_b+1} if that row was computed, else the last
                            accepted block token; untouched for a sequence with no rows */
    int32_t defer_accept; /* verify calls only.  Non-zero: compute the rows (KV appended, exit rows buffered,
                            argmax_ids / top2 / logits written) but decide nothing -- n_accepted, next_token,
                            tentative, pending and the three length counters stay as they were, for
                            hispec_accept_rejection to decide on the same stream */
} hispec_result;

/* Create a context: validates the shape, copies the pointer tables, builds TMA descriptors for
 * every weight matrix and allocates the fixed workspace on the current device. */
int hispec_create(const hispec_model_desc *desc, const hispec_weights *weights, hispec_ctx **out);
int hispec_destroy(hispec_ctx *ctx);

/*
 * One step of Generate(L_d, ., N_d) (Algorithm 2, inner loop; Sec. 3.2 "expanding"): for every
 * sequence b, token in_tokens[b] enters at position p = len_draft[b], runs through layers
 * [layer_begin, layer_end) -- layer_begin must be 0, layer_end one of L_d, L_i, L_f -- appending its
 * K,V to the sequence's pages; the hidden row at the exit is buffered (layer_end == L_d: h_draft
 * row p - len_inter[b]; layer_end == L_i: h_inter row p - len_target[b]); the exit head's greedy
 * token goes to out_tokens[b * out_stride] (device, may be NULL).  The input token of sequence b is
 * in_tokens[b * in_stride] (device); a negative id makes the sequence sit the call out.  With
 * the strides, successive draft steps can read and write the columns of one [batch][k] block
 * of draft ids in place, with no host round trip.  The length of every layer group inside the
 * range grows by 1.  layer_end == L_f gives one plain auto-regressive decoding step.
 * `res` may be NULL; if given, its optional outputs are filled for row 0 and n_accepted /
 * next_token are ignored.
 */
int hispec_draft(hispec_ctx *ctx, void *stream, int layer_begin, int layer_end, const hispec_exits *exits,
                 const hispec_kv *kv, const hispec_hidden *hidden, int batch, const int32_t *in_tokens,
                 int in_stride, int32_t *out_tokens, int out_stride, const hispec_result *res);

/*
 * Generate(L_d, ., N_d) (Algorithm 2) as ONE call: n_steps successive hispec_draft steps, plus one more if
 * `bonus` is non-zero (its token is dropped: the step only pushes S_{N_d} through the draft layers so that the
 * verifier can emit v_{N_d+1}).  Step 0 reads in_tokens[b * in_stride]; step s > 0 reads block[b * block_stride +
 * s - 1]; step s < n_steps writes its greedy token to block[b * block_stride + s] (device int32, block_stride >=
 * n_steps).  State, hidden rows and lengths change exactly as by the separate calls.  Where the persistent kernel
 * takes the call, all steps run inside one launch (the weight stream continues from one step's exit head into
 * the next step's first projection); otherwise the library issues the separate calls itself.  `res`, if given,
 * holds the optional outputs of the last step.  The paper states Generate (Algorithm 2); fusing its steps into one
 * launch is this library's.
 */
int hispec_draft_block(hispec_ctx *ctx, void *stream, int layer_begin, int layer_end, const hispec_exits *exits,
                       const hispec_kv *kv, const hispec_hidden *hidden, int batch, const int32_t *in_tokens,
                       int in_stride, int32_t *block, int block_stride, int n_steps, int bonus,
                       const hispec_result *res);

/*
 * LeadingSubstringVerify(S, L_i, x || V) (Algorithm 2): the n_rows[b] buffered exit-L_d rows of each
 * sequence run through layers [layer_begin, layer_end) (layer_begin == L_d; layer_end == L_i, or L_f
 * for single-stage speculation as in Algorithm 1) with causal attention inside the block and over
 * the sequence's cached pages; v_{j+1} = argmax of the exit head on row j; a_b = number of leading j
 * with draft_tokens[b][j] == v_{j+1}.  Exit rows are appended to h_inter (layer_end == L_i).  Then
 * the state of rejected tokens is dropped ("pruning", Sec. 3.2): every layer group up to layer_end
 * gets length p0 + min(a_b + 1, n_rows[b]).
 *   draft_tokens device: token j of sequence b at draft_tokens[b * token_stride + j], j < k;
 *   n_draft device [batch], 0 <= n_draft[b] <= k; n_rows device [batch], n_draft[b] <= n_rows[b] <=
 *   n_draft[b] + 1 (the extra row yields the bonus token v_{|S|+1}); n_rows[b] == 0 skips the
 *   sequence.  k + 1 <= max_rows_per_seq.  n_rows == NULL and n_draft == NULL together mean "every
 *   buffered row": n_rows[b] = rows buffered by the stage below (at most k + 1), n_draft[b] =
 *   min(k, n_rows[b]) -- this keeps a whole decoding round on the device.
 *   If res->tentative is given, the call's result list [S_1..S_a, v_{a+1}] is appended to it at
 *   row len_inter[b] - len_target[b] (entry values): the list V of Algorithm 2, built on the device.
 */
int hispec_verify_intermediate(hispec_ctx *ctx, void *stream, int layer_begin, int layer_end,
                               const hispec_exits *exits, const hispec_kv *kv, const hispec_hidden *hidden,
                               int batch, const int32_t *draft_tokens, int token_stride, const int32_t *n_draft,
                               const int32_t *n_rows, int k, const hispec_result *res);

/*
 * LeadingSubstringVerify(V, L_f, x) (Algorithm 2): same contract over layers [L_i, L_f) on the
 * accumulated h_inter rows; draft_tokens holds V.  Afterwards all three layer groups have length
 * p0 + min(a_b + 1, n_rows[b]): everything of V from the first mismatch on is flushed.  With
 * n_rows == n_draft == NULL, n_rows[b] = n_draft[b] = len_inter[b] - len_target[b] (all of V, no
 * bonus row; at most k).
 */
int hispec_verify_target(hispec_ctx *ctx, void *stream, int layer_begin, int layer_end,
                         const hispec_exits *exits, const hispec_kv *kv, const hispec_hidden *hidden,
                         int batch, const int32_t *draft_tokens, int token_stride, const int32_t *n_draft,
                         const int32_t *n_rows, int k, const hispec_result *res);

/*
 * Prompt processing (not part of the hot path; the same kernels over [0, L_f) fed from the
 * embedding in chunks of max_rows_per_seq rows).  tokens device [batch][max_tokens] (row b holds
 * n_tokens[b] ids); n_tokens device [batch].  All three lengths must be 0 on entry and equal
 * n_tokens[b] on exit; first_token[b] (device) = greedy token of exit L_f at the last prompt
 * position, i.e. the first pending token.
 */
int hispec_prefill(hispec_ctx *ctx, void *stream, const hispec_exits *exits, const hispec_kv *kv, int batch,
                   const int32_t *tokens, const int32_t *n_tokens, int max_tokens, int32_t *first_token);

/*
 * Rejection-sampling acceptance (App. G) for a verify call that ran with res->defer_accept: per sequence,
 * for j = 0..n_draft-1 in order the block token S_{j+1} = draft_tokens[b * token_stride + j] is kept while
 * u_accept[b * max_rows_per_seq + j] < min(1, q_j(S_{j+1}) / p_j(S_{j+1})); at the first failure the rest of
 * the block is dropped and the next token is drawn from max(0, q_j - p_j) normalised; if every token is kept
 * and the verifier computed one more row, the next token is drawn from that row's q.  Draws use inversion in
 * vocabulary order with u_sample[b].  p_j = softmax(p_logits[b][j] / temperature) (the exit that proposed the
 * block: rows written by the draft steps for stage 1, the rows kept by stage 1 for stage 2), q_j likewise
 * from q_logits (the deferred call's res->logits); both device fp32 [batch][max_rows_per_seq][vocab].
 * stage 1 = intermediate verification over [L_d, L_i), stage 2 = target verification over [L_i, L_f);
 * n_rows / n_draft are taken from the length counters exactly as the verify calls do with NULL n_rows
 * (k = the verify call's k).  Then the state transition of the verify call is applied with the sampled
 * outcome: n_accepted, next_token, tentative, pending and the length counters as documented for
 * hispec_verify_intermediate / hispec_verify_target.  Stage 1 also appends the q rows of the kept tokens and
 * of the next token (rows 0..min(a, n_rows - 1)) to stage_logits [batch][max_rows_per_seq][vocab] at row
 * len_inter - len_target (entry values): the proposal rows stage 2 needs.  stage_logits may be NULL.
 * Probabilities are formed in fp32.  The paper has the rule (App. G); the entry point, its arguments and the
 * uniforms-as-inputs convention are this library's.  Returns HISPEC_EINVAL on bad arguments; state errors go
 * to the status word.
 */
int hispec_accept_rejection(hispec_ctx *ctx, void *stream, int stage, const hispec_exits *exits,
                            const hispec_kv *kv, int batch, const int32_t *draft_tokens, int token_stride, int k,
                            const float *p_logits, const float *q_logits, const float *u_accept,
                            const float *u_sample, float temperature, float *stage_logits,
                            const hispec_result *res);

/*
 * Draw one token per sequence from softmax(logits[b * row_stride ...] / temperature) by inversion in
 * vocabulary order with u[b] (device fp32 [batch], in [0,1)); the token goes to out_tokens[b * out_stride].
 * Used to sample draft tokens from the logits a draft step wrote (App. G: drafts are sampled from p_{L_d}).
 */
int hispec_sample(hispec_ctx *ctx, void *stream, int batch, const float *logits, int64_t row_stride,
                  const float *u, float temperature, int32_t *out_tokens, int out_stride);

/* Synchronises `stream`, copies the device status word to *host_out and clears it. */
int hispec_device_status(hispec_ctx *ctx, void *stream, uint32_t *host_out);

/* Number of kernel launches the library has enqueued through this context since creation. */
int64_t hispec_launch_count(const hispec_ctx *ctx);

/*
 * Measurement aid.  While profiling is enabled every projection (kind 0 = all projections; kinds
 * 10..14 = QKV, O, gate/up, down, exit head separately), attention (kind 1) and persistent whole-call
 * (kind 20; bytes = weights of the layer range + exit head) launch is bracketed by a pair of CUDA events on the call's stream, which also keeps neighbouring
 * launches from overlapping.  hispec_profile_read() synchronises `stream`, adds up the event times
 * recorded since the last read into *ms, the weight bytes those projections streamed into *bytes
 * (0 for attention: the library does not know the context lengths on the host) and their number
 * into *launches, and forgets them.  Not for use inside stream capture.
 */
int hispec_profile_enable(hispec_ctx *ctx, int on);
int hispec_profile_read(hispec_ctx *ctx, void *stream, int kind, double *ms, double *bytes, int64_t *launches);

/*
 * Exit head + greedy token without any allocation (the paper has no counterpart; this is a
 * service entry point for callers that cannot allocate device memory: a process whose free HBM was
 * all given to its KV-page pool, a thread running while the allocator is held elsewhere, a plug-in
 * that only receives raw pointers and a stream).  No hispec context is needed.
 * For each of the n_rows hidden rows: z = head . RMSNorm(hidden[t]; final_norm); argmax_ids[t] = greedy
 * token (lowest id on an exact tie), top2[t] = {largest, second largest logit} (top2 may be NULL).
 *   head device bf16 [vocab][d_model]; final_norm device fp32 [d_model]; hidden device fp32
 *   [n_rows][d_model]; argmax_ids device int32 [n_rows]; top2 device fp32 [n_rows][2].
 * Limits: n_rows <= HISPEC_NOALLOC_MAX_ROWS, d_model <= HISPEC_NOALLOC_MAX_D, vocab <=
 * HISPEC_NOALLOC_MAX_VOCAB; anything larger returns HISPEC_ECAPACITY and enqueues nothing.
 * Scratch is a 1 MiB array compiled into the library, resident on every GPU that loads it, shared by
 * all calls: calls whose kernels overlap on the GPU race with each other -- order them on one stream
 * or with events.  The array keeps the previous call's contents; every element a call reads it has
 * written first.  The first call on a device looks the array's address up
 * (cudaGetSymbolAddress); make that first call outside stream capture.  Asynchronous on `stream`.
 * The call uses no cudaMalloc / cudaFree and no allocating library routine.
 */
#define HISPEC_NOALLOC_MAX_ROWS 16
#define HISPEC_NOALLOC_MAX_D 8192
#define HISPEC_NOALLOC_MAX_VOCAB 262144
int hispec_exit_argmax_noalloc(void *stream, const void *head, const float *final_norm, float rms_eps,
                               int d_model, int vocab, const float *hidden, int n_rows, int32_t *argmax_ids,
                               float *top2);

/* Debug aid: with HISPEC_TRACE=1 in the environment at hispec_create(), the persistent kernel stamps the
 * global timer after each of its grid barriers (block 0); this synchronises the device and copies the 1024
 * stamp slots of the last call into `out` (slot 1023 = kernel start).  Returns the number of slots copied, 0
 * when tracing is off or cap < 1024. */
int hispec_debug_trace(hispec_ctx *ctx, unsigned long long *out, int cap);

/* Text of the most recent CUDA failure behind a HISPEC_ECUDA return (process-wide, not thread-safe). */
const char *hispec_last_error(void);

/* Static text for an error code. */
const char *hispec_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* HISPEC_H */
