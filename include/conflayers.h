/*
 * conflayers.h -- C ABI of libconflayers.so: the hot path of ConfLayers self-speculative decoding
 * on one NVIDIA B200 (sm_100a).
 *
 * The calls follow the paper's statement of the problem (Section 3, Figure 2): load a Llama-style
 * decoder, compute per-layer confidences, set the skip set, draft K tokens with the draft model
 * (= the same model without the skipped layers), verify them with the full model in one pass,
 * accept greedily.
 *
 * Conventions
 *   - Every call returns an int status (CL_OK = 0).  Nothing throws across this boundary.
 *     cl_last_error() returns a description of the context's last failure.
 *   - "host" / "device" on a pointer says where the memory lives.  Output buffers are caller-owned
 *     HOST memory unless stated otherwise.  Sizes are in elements.
 *   - A context owns every byte of device memory it allocates (weights copy, KV cache, scratch)
 *     and frees it in cl_destroy().  Pointers passed to cl_load() are borrowed for the call.
 *   - One context = one CUDA stream (given at creation; may be NULL for the default stream).
 *     A context is not thread-safe.  Calls that return host values synchronise the stream.
 *   - There is no CPU fallback: without a CUDA device every compute call fails with CL_ECUDA.
 *   - Matrices are row-major (out_features, in_features), as Llama checkpoints store them.
 *     weight_dtype selects the storage type of weights, KV cache and hidden-state taps:
 *     0 = fp32, 1 = bf16, 2 = fp16 (the type the paper's models run in, Section 4.1.1).  Norm gains are always
 *     fp32.  Arithmetic accumulates in fp32.
 *   - Requirements: d_model = n_heads * head_dim, n_kv_heads divides n_heads (n_kv_heads < n_heads: grouped-query
 *     attention, query head h reads key/value head h / (n_heads / n_kv_heads)),
 *     head_dim in {64, 128}, d_model and d_ffn multiples of 8, 1 <= K <= CL_MAX_K.
 *   - Which kernels run: single-token steps (draft, vanilla) run in one persistent cooperative kernel when d_model and
 *     d_ffn are at most 16384 (bf16) / 8192 (fp32).  Passes of up to CL_MAX_K + 1 rows (verify, short prompt chunks) of
 *     bf16 and fp16 models run in one persistent cooperative launch on the tensor cores (tcgen05, both operands in the
 *     model's 16-bit type) when d_model and d_ffn are multiples of 64 and d_model <= 31968; for it cl_load keeps a
 *     second copy of every matrix in the order that kernel streams it (device memory for weights doubles).  The
 *     confidence scoring of 16-bit models runs on the tensor cores too; fp32 models and the remaining cases use
 *     per-matrix CUDA-core kernels.
 *     A prompt of more than 16 tokens (bf16 / fp16 models) runs all rows but the last through wide tensor-core GEMMs, up to
 *     512 rows at a time, and the last row through the pass of several rows, which has the LM head.
 *     Environment switches read by cl_load (diagnostics): CL_DISABLE_STEP_KERNEL=1, CL_DISABLE_ROWS_KERNEL=1,
 *     CL_DISABLE_WIDE_PREFILL=1, CL_DISABLE_ROW_SHARES=1, CL_L2_AHEAD_KB=<n>, CL_ROWS_SPLIT=<1|2|4>, CL_ROWS_CHAIN=<k-blocks
 *     of 64 elements per tensor-memory accumulation chain>, CL_ROWS_ENTRY_KB=<size of a ring entry of that pass>.
 */
#ifndef CONFLAYERS_H
#define CONFLAYERS_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CL_MAX_K 8          /* longest draft; a verify pass has at most CL_MAX_K + 1 rows */

enum {
    CL_OK = 0,
    CL_EINVAL = 1,   /* bad argument */
    CL_ENOMEM = 2,   /* device or host allocation failed */
    CL_ECUDA = 3,    /* a CUDA call failed (no device, launch error, ...) */
    CL_ESTATE = 4,   /* call made in the wrong order (e.g. draft before prefill) */
    CL_ERANGE = 5,   /* sequence would exceed max_seq, or K / rows out of range */
    CL_ETIMEOUT = 6  /* a bounded device-side wait expired */
};

typedef struct cl_ctx cl_ctx;

typedef struct {
    int n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab, max_seq;
    float rms_eps, rope_theta;
    int weight_dtype;    /* 0 fp32, 1 bf16, 2 fp16 */
    int tap_positions;   /* P: ring of the last P positions' per-layer hidden states (0 = no ring) */
    int tap_modules;     /* 0 or 1: record each layer's output (after the FFN add); 2: also the stream after the attention add
                            (Section 3.1 scores "FFNN and Attention" hidden states); a layer's confidence = mean over its taps */
} cl_model_cfg;

typedef struct {
    const void *embed;                /* [vocab, d_model] */
    const void *lm_head;              /* [vocab, d_model] (shared by all early exits) */
    const float *final_norm;          /* [d_model] */
    const void *const *wq, *const *wk, *const *wv, *const *wo;   /* n_layers pointers; wq, wo [d_model, d_model], wk, wv [n_kv_heads * head_dim, d_model] */
    const void *const *wg, *const *wu;                           /* each [d_ffn, d_model] */
    const void *const *wd;                                       /* each [d_model, d_ffn] */
    const float *const *norm1, *const *norm2;                    /* each [d_model] */
    int on_device;                    /* 1: the matrices above are device pointers, 0: host (the pointer arrays themselves are host) */
    int head_only;                    /* 1: only embed may be NULL and per-layer arrays are ignored; the context
                                         then serves cl_layer_confidences / cl_select_skip_set / cl_score_loop only */
} cl_weights;

/* Parameters of the adaptive-window selection (Section 3.2, Eq. 5-10). */
typedef struct {
    double w_base;       /* Eq. 7 base window (paper: 2) */
    double lambda;       /* Eq. 10 threshold sensitivity (paper: 0.25 < lambda < 0.5) */
    double eps;          /* epsilon of Eq. 5 and of the min-max rescaling of Eq. 6 */
    double flat_tol;     /* tolerance for "same confidence value" when counting w_max */
    double w_max;        /* <= 0: number of leading eligible layers that share the first one's confidence */
    int lo, hi;          /* eligible layers, inclusive (the paper leaves out the first and last layer) */
    int n_skip;          /* >= 0: exactly this many layers (smallest margins); < 0: Eq. 10, then min_ratio */
    double min_ratio;    /* minimum skip ratio over the eligible layers (paper: 0.4) */
    int fixed_window;    /* > 0: constant window instead of Eq. 7 (the paper's ablation) */
} cl_select_cfg;

typedef struct {
    uint64_t cycles;     /* draft/verify/accept cycles run */
    uint64_t drafted;    /* candidate tokens drafted */
    uint64_t accepted;   /* candidate tokens accepted (alpha = accepted / drafted, M = accepted / cycles) */
    uint64_t emitted;    /* tokens emitted by cycles (accepted + one target token per cycle) */
    int ctx_len;         /* committed KV-cache length */
    int n_skipped;       /* |S|: layers skipped as a whole (beta = n_skipped / n_layers) */
    uint64_t kernel_launches;  /* kernels launched by this context so far */
} cl_stats;

/* ---- life cycle ------------------------------------------------------------------------- */

/* Create a context for a model shape on the current CUDA device.  `cuda_stream` is a cudaStream_t
 * (or NULL).  No large allocation happens before cl_load().  (Section 4.1.1: Llama-family target.) */
int cl_create(const cl_model_cfg *cfg, void *cuda_stream, cl_ctx **out);

/* Copy the weights into the context's own arena (concatenating Q/K/V and interleaving gate/up rows
 * for streaming; one copy, in execution order), allocate the KV cache [n_layers][2][n_heads][max_seq][head_dim] and scratch.  Borrowed
 * pointers may be released after the call returns.  CL_ENOMEM if the device cannot hold it.  With the persistent
 * step kernel the call also runs a few token steps on an empty cache to measure each SM's streaming rate (fixed row
 * shares afterwards); it synchronises the stream. */
int cl_load(cl_ctx *ctx, const cl_weights *w);

int cl_destroy(cl_ctx *ctx);

/* ---- generation step (Section 3: draft with the non-skip layer set, verify, accept) -------- */

/* Reset the cache and run the full model over `n` prompt tokens (host int32), filling the KV
 * cache of every layer; *first_token = greedy token after the prompt, which becomes the pending
 * token of the first cycle.  tap_hidden != 0 records the hidden-state ring while doing so. */
int cl_prefill(cl_ctx *ctx, const int32_t *tokens, int n, int tap_hidden, int32_t *first_token);

/* Skip set S as a byte per layer: bit 0 = skip the attention half, bit 1 = skip the FFN half, 3 = the whole
 * layer (Section 3.1 scores both modules of a layer; the paper's own sets are whole layers).  A skipped half
 * streams no weights in draft steps; a skipped attention half leaves the layer's KV entries untouched. */
int cl_set_skip_set(cl_ctx *ctx, const uint8_t *mask /* host [n_layers] */);
int cl_get_skip_set(cl_ctx *ctx, uint8_t *mask /* host [n_layers] */);

/* Draft up to K candidate tokens with the draft model, feeding each greedy token back on the
 * device.  stop_p > 0 stops early once a draft's top-1 probability falls below it (the
 * confidence-aware drafting the paper takes from SWIFT); 0 = always K.  Outputs (host, may be
 * NULL): toks[K], p_max[K], conf[K] (entropy confidence of the draft distribution, Eq. 1-4),
 * logits [K, vocab], *n_drafted. */
int cl_draft(cl_ctx *ctx, int K, float stop_p, int32_t *toks, float *p_max, float *conf, float *logits,
             int *n_drafted);

/* One full-model pass over [pending, d_1 .. d_n] (n = tokens drafted in this cycle; 0 is allowed),
 * causal among themselves and over the cache; rewrites every layer's KV for those positions.
 * target_toks[i] (i = 0..n) = greedy token after row i.  logits (host, [n+1, vocab]) may be NULL.
 * tap_hidden != 0 also stores each layer's residual stream into the hidden-state ring. */
int cl_verify(cl_ctx *ctx, int tap_hidden, int32_t *target_toks, float *logits);

/* Greedy acceptance: n = longest prefix of drafts equal to the target's tokens; emitted = those n
 * drafts plus the target's next token; the cache length grows by n + 1 and the last emitted token
 * becomes the pending token. */
int cl_accept(cl_ctx *ctx, int *n_accepted, int32_t *emitted /* host [n_accepted + 1], room for CL_MAX_K + 1 */);

/* Plain autoregressive step with the full model (the lossless reference): consumes the pending
 * token, returns the next one. */
int cl_step_vanilla(cl_ctx *ctx, int32_t *tok);

/* Run cycles (draft K, verify, accept) back to back on the device until max_new tokens have been
 * emitted; no host synchronisation inside a cycle.  out: host [max_new].  K = 0 runs vanilla
 * decoding with the same kernels.  stats may be NULL. */
int cl_generate(cl_ctx *ctx, int K, int max_new, int32_t *out, int *n_out, cl_stats *stats);

/* Set the committed cache length and the pending token (rollback after a rejected run, or
 * re-synchronisation of a parity harness).  0 <= ctx_len <= the number of positions full-model passes (prefill,
 * verify, vanilla steps) have written so far; CL_ERANGE beyond that. */
int cl_rollback(cl_ctx *ctx, int ctx_len, int32_t pending_token);

/* Overwrite this cycle's drafted tokens (host int32[n], n <= CL_MAX_K) before cl_verify. */
int cl_force_tokens(cl_ctx *ctx, const int32_t *toks, int n);

/* ---- layer optimisation search step (Sections 3.1-3.3) ------------------------------------- */

/* Early-exit confidence of hidden states (Section 3.1, Eq. 1-4): each row goes through the final
 * RMSNorm and the shared LM head; logits are clamped in fp32; per row the entropy confidence
 * 1 - H/log(vocab), the top-1 probability and the greedy token are reduced on the fly (logits are
 * never stored).  hidden: DEVICE pointer [rows, P, d_model] in the model's storage type (16-byte aligned for
 * 16-bit models, CL_EINVAL otherwise; cl_score_loop's tensors likewise), or NULL to
 * score the context's own ring (rows = n_layers, P = taps * tap_positions with taps = 1 or 2, see tap_modules).
 * Outputs (host, may be NULL): conf_rows, p_max, argmax [rows, P]; c_layer [rows] = mean over P. */
int cl_layer_confidences(cl_ctx *ctx, const void *hidden, int rows, int P, float *conf_rows, float *p_max,
                         int32_t *argmax, float *c_layer);

/* Adaptive-window selection (Section 3.2, Eq. 5-10) on the device, in double precision.
 * c_layer: host float[n_layers], or NULL to use the result of the last cl_layer_confidences.
 * mask: host [n_layers] (3 = skip); margins: host double[n_layers] (Eq. 10's left minus right side,
 * 0 outside lo..hi), may be NULL.  Does not install the set: call cl_set_skip_set. */
int cl_select_skip_set(cl_ctx *ctx, const cl_select_cfg *cfg, const float *c_layer, uint8_t *mask, double *margins);

/* Search rounds (Section 3.3, Appendix D): for each of `iters` hidden-state tensors (DEVICE pointers,
 * each [n_layers, P, d_model]) score all layers, select a skip set, and keep the set of the round
 * with the best score (host float[iters], earliest wins ties).  masks_all (host, [iters, n_layers])
 * may be NULL.  One host synchronisation, at the end. */
int cl_score_loop(cl_ctx *ctx, const cl_select_cfg *cfg, const void *const *hidden_iters, int iters, int P,
                  const float *scores, uint8_t *best_mask, int *best_iter, uint8_t *masks_all, float *c_layers_all);

/* Interval-based periodic search (Section 3.3, Figure 2) around the generation loop.  The skip set installed
 * when the call is made (the paper starts from uniformly skipped layers) is round 0.  Every set drafts for
 * `interval` cycles (Opt_Interval); the round's score is the mean number of accepted candidates per cycle; the
 * best-scoring set is remembered (the earlier one on ties).  After a round whose score reaches score_goal, or after
 * max_rounds searched sets, the search ends and the best set drafts for the rest of the call (it stays installed).
 * Otherwise the layers are scored on the hidden-state ring (Section 3.1), a new set is selected with *sel
 * (Section 3.2) and installed.  Needs tap_positions > 0 and a cl_prefill with tap_hidden = 1 (which clears the
 * ring); while the search is on the verify passes of the last tap_positions cycles of an interval record the ring (earlier
 * ones would be overwritten before the search check).  The emitted tokens do not depend on the search.
 * out: host [max_new].  rep (may be NULL): scores[i] of round i, i < n_scored; masks (host, may be NULL):
 * [(max_rounds + 1), n_layers], row i = the set of round i. */
#define CL_MAX_ROUNDS 32
typedef struct {
    int K, interval, max_rounds;   /* draft length, cycles per interval, searched sets after the initial one */
    float score_goal;              /* the paper halts at 4 accepted tokens */
} cl_search_cfg;
typedef struct {
    int n_scored, best_round, searching;   /* rounds scored, index of the best, 1 if the search was still on at the end */
    float scores[CL_MAX_ROUNDS + 1];
} cl_search_report;
int cl_generate_search(cl_ctx *ctx, const cl_search_cfg *cfg, const cl_select_cfg *sel, int max_new, int32_t *out,
                       int *n_out, cl_search_report *rep, uint8_t *masks);

/* Copy the hidden-state ring to the host: out is [n_layers, taps, tap_positions, d_model] in the storage type
 * (taps = 2: index 0 after the attention add, 1 after the FFN add), position slot = absolute position modulo
 * tap_positions. */
int cl_read_hidden_ring(cl_ctx *ctx, void *out);

/* Confidence scoring for callers that cannot allocate device memory.  The paper has no counterpart of
 * this call: it is cl_layer_confidences() (final RMSNorm -> shared LM head -> clamp -> entropy confidence,
 * top-1 probability, greedy token per row) without a context and without a single cudaMalloc / cudaFree.
 * It is meant for processes in which this library may not allocate: a server whose framework has already
 * reserved the whole GPU for its own caching allocator (a cudaMalloc here would fail or eat into that
 * pool), or a latency-critical loop in which cudaMalloc's device-wide synchronisation is not acceptable.
 *
 * All working memory (normalised rows, per-block softmax partials, the completion ticket, the result
 * staging) lives in one fixed array compiled into the library: about 0.5 MB that every GPU which loads the
 * library holds until the process exits.  Hence the fixed limits below; larger sizes return CL_ERANGE.
 *   lm_head    DEVICE [vocab, d_model] row-major, weight_dtype 0 = fp32 / 1 = bf16
 *   final_norm DEVICE float[d_model]
 *   hidden     DEVICE [n_rows, d_model] in the same storage type as lm_head
 *   (all three 16-byte aligned: the kernels read them with vector loads; CL_EINVAL otherwise.  fp16 is not
 *   supported by this call: weight_dtype 2 is rejected with CL_EINVAL.)
 *   conf, p_max, argmax   HOST [n_rows], caller-owned, each may be NULL
 * The call enqueues on cuda_stream (a cudaStream_t or NULL) and synchronises it before returning.
 * The first call on each device looks up the array's device address; make that first call outside any
 * stream capture.  Every call on a device uses the same array, which keeps whatever the previous call
 * left (the call clears the part that must start at zero itself): two calls whose kernels overlap on the
 * GPU, from different streams or threads, race and give wrong results.  Serialise them.
 * Errors: CL_EINVAL (null input, bad dtype or shape), CL_ERANGE (beyond the limits), CL_ECUDA;
 * the message is read with cl_last_error(NULL). */
#define CL_STATIC_MAX_ROWS 4096
#define CL_STATIC_MAX_D 8192
int cl_layer_confidences_static(const void *lm_head, const float *final_norm, int vocab, int d_model, int weight_dtype,
                                float rms_eps, const void *hidden, int n_rows, void *cuda_stream, float *conf,
                                float *p_max, int32_t *argmax);

/* ---- diagnostics ------------------------------------------------------------------------------ */

/* Every device-side wait in the kernels (a shared-memory barrier, a grid barrier of a persistent kernel) is bounded:
 * when the bound runs out the kernel raises a flag, lets its remaining waits fall through, drains its copies in
 * flight and returns; the host call that finds the flag returns CL_ETIMEOUT, clears it, commits nothing of the
 * call, and the context stays usable (re-run cl_prefill).  The paper has no counterpart; these settings exist so
 * that this path can be exercised without faulting or hanging anything:
 *   CL_DEBUG_WAIT_LIMIT_US   bound of a single wait of the persistent kernels (token steps, T-row pass) in microseconds
 *                            (default 2 000 000)
 *   CL_DEBUG_BARRIER_EXTRA   extra arrivals their grid barriers wait for (default 0); with 1 no barrier can complete,
 *                            so the first one runs into the bound
 *   CL_DEBUG_DEVICE_ERR      sets the device-side error flags to `value`, as an expired wait would */
enum { CL_DEBUG_WAIT_LIMIT_US = 1, CL_DEBUG_BARRIER_EXTRA = 2, CL_DEBUG_DEVICE_ERR = 3 };
int cl_debug_set(cl_ctx *ctx, int what, long long value);

/* Reads a diagnostic record into host memory.  CL_DEBUG_ROWS_PHASE_NS: out = uint64[n_SMs * 8], for every CTA of the
 * persistent T-row pass (verify, short prompt chunks of 16-bit models) the nanoseconds its first thread spent, during
 * the last pass, in: 0 embedding, 1 QKV, 2 attention, 3 output projection, 4 gate/up, 5 down projection, 6 LM head,
 * 7 grid barriers.  The first call switches the recording on (and returns zeros). */
enum { CL_DEBUG_ROWS_PHASE_NS = 1 };
int cl_debug_read(cl_ctx *ctx, int what, void *out, int n);

/* ---- bookkeeping ----------------------------------------------------------------------------- */

int cl_get_stats(cl_ctx *ctx, cl_stats *out);      /* alpha, beta, M of Section 4.1.2 derive from these */
const char *cl_last_error(cl_ctx *ctx);            /* never NULL; ctx may be NULL (global message) */

#ifdef __cplusplus
}
#endif
#endif /* CONFLAYERS_H */
