/*
 * hbsjd.h -- C ABI of the batched speculative-Jacobi rollout library for NVIDIA B200 (sm_100a).
 *
 * The library replaces the token-by-token student rollout of visual on-policy
 * distillation: given a real prefix x_1..x_k per image and its class, it samples
 * x_{k+1}..x_T from the student (Eq. 2), using independent per-image Jacobi
 * windows verified in batched forwards (Sec. 4.2) with Full / Compact execution
 * switching as images finish (Sec. 4.3, Eq. 6).
 *
 * General conventions
 *   - Every function returns 0 (HBSJD_OK) or a negative error code; nothing
 *     aborts or throws across this boundary.  hbsjd_strerror() names a code and
 *     hbsjd_last_error(ctx) gives a one-line detail of the last failure.
 *   - "device" pointers are CUDA global-memory addresses of the context's GPU;
 *     "host" pointers are ordinary process memory.  The caller owns every
 *     argument buffer; the context owns weights, KV pages, rollout state and
 *     all scratch, allocated in hbsjd_create and freed in hbsjd_destroy.
 *   - All GPU work is enqueued on the stream given to hbsjd_create (a
 *     cudaStream_t passed as void*, NULL = the legacy default stream).  Calls
 *     that report a live count synchronise that stream before returning.
 *   - A context is not thread-safe; use one context per host thread / stream.
 *   - There is no CPU path: if no CUDA device is usable the calls fail with
 *     HBSJD_ECUDA.
 */
#ifndef HBSJD_H_
#define HBSJD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    HBSJD_OK = 0,
    HBSJD_EINVAL = -1,   /* bad argument; no kernel was launched */
    HBSJD_ENOMEM = -2,   /* device or host allocation failed */
    HBSJD_ECUDA = -3,    /* a CUDA call failed (detail in hbsjd_last_error) */
    HBSJD_ESTATE = -4,   /* call not valid in the context's current state */
    HBSJD_ETIMEOUT = -5  /* a bounded device-side wait gave up; the context stays usable */
};

enum { HBSJD_DTYPE_FP32 = 0, HBSJD_DTYPE_BF16 = 1 };
enum { HBSJD_VERIFY_PROB = 0, HBSJD_VERIFY_GREEDY = 1 };              /* Eq. 5 / Eq. 4 */
enum { HBSJD_EXEC_FULL = 0, HBSJD_EXEC_COMPACT = 1, HBSJD_EXEC_HYBRID = 2,  /* Sec. 4.3 */
       /* Full execution with batch-synchronous progress: every live image advances by the smallest commit of
        * the batch (an image that verified more keeps only that many of its accepted drafts).  The baseline of
        * the ablation "Is independent progress necessary for batched SJD?" (Sec. 5.3, Table 2); not a mode to
        * use for speed. */
       HBSJD_EXEC_SYNC = 3 };

typedef struct hbsjd_ctx hbsjd_ctx;

/* Decoder description.  Pre-norm blocks: h += Wo Attn(rope(Wq a), rope(Wk a), Wv a), a = rmsnorm(h) g_attn;
 * h += W2 (silu(W1 m) * (W3 m)), m = rmsnorm(h) g_ffn; logits = W_head rmsnorm(h) g_out.
 * Sequence index 0 is the class token, index s >= 1 is image token x_s on a grid_h x grid_w raster;
 * T = grid_h * grid_w tokens per image.  The paper names the model family only (Sec. 5.1). */
typedef struct {
    int32_t n_layers, dim, n_heads, ffn_hidden, vocab, grid_h, grid_w, n_classes;
    int32_t dtype;      /* HBSJD_DTYPE_*: element type of the weight image and of activations */
    float rms_eps;
    float rope_base;
} hbsjd_model_desc;

/* Rollout parameters. */
typedef struct {
    int32_t window;          /* W: inputs per image per round = last committed token + W-1 drafts (Sec. 4.2) */
    int32_t history_offset;  /* H: new draft slots copy the token H positions back (Sec. 4.2) */
    float cfg_scale;         /* 1 = no guidance; otherwise logits = l_u + s (l_c - l_u) (Sec. 4.2) */
    float temperature;       /* > 0 */
    int32_t top_k;           /* 0 or >= vocab: off; ties at the k-th value are kept */
    int32_t verify_mode;     /* HBSJD_VERIFY_* */
    int32_t exec_mode;       /* HBSJD_EXEC_* */
    int32_t gamma;           /* HYBRID: Full iff live images > gamma, else Compact (Eq. 6) */
    uint64_t seed;           /* key of the counter-based generator; counter = (image, position, round) */
    int32_t max_rounds;      /* < 0: run to completion; 0: init + prefill only; > 0: at most that many rounds */
    int32_t reserved;
} hbsjd_params;

typedef struct {
    int64_t rounds;            /* verification rounds run with at least one live image */
    int64_t image_forwards;    /* sum over rounds of live images */
    int64_t committed;         /* tokens committed (accepted drafts + replacement / bonus tokens) */
    int64_t rejects;           /* image-rounds that ended in a rejection */
    int64_t full_rounds;       /* rounds executed in Full form */
    int64_t compact_rounds;    /* rounds executed in Compact form */
    int64_t prefill_forwards;  /* batched forwards spent on prefix pre-filling */
    int64_t kernel_launches;   /* kernels of this library launched by the call */
    float ms_total;            /* GPU time of the call (CUDA events on the context's stream) */
    float ms_prefill;          /* of which state init + prefix pre-filling */
} hbsjd_stats;

/* Creates a context on the current CUDA device.
 *   m            model description
 *   weights      HOST pointer to the flat weight image: tok_emb[V,D], cls_emb[C+1,D] (row C = null
 *                class), per layer g_attn[D], w_qkv[3D,D], w_o[D,D], g_ffn[D], w_13[2F,D], w_2[D,F],
 *                then g_out[D], w_head[V,D]; matrices row-major [out,in]; each tensor starts on a
 *                256-byte boundary.  The image is copied; the caller keeps ownership.
 *   weight_bytes size of the image; must match the description exactly
 *   max_batch    largest batch of hbsjd_rollout; max_window largest params.window (<= 64)
 *   cuda_stream  cudaStream_t as void*
 * Constraints: dim % n_heads == 0; head size 16/32/64/128 for fp32 models, 32 or 64 for bf16 models (64 runs
 * the tensor-core attention kernel, 32 a plain one); dim, ffn_hidden, vocab multiples of 64 for bf16;
 * vocab <= 32768 (a position's probabilities stay in one CTA's shared memory).
 * Errors: HBSJD_EINVAL, HBSJD_ENOMEM, HBSJD_ECUDA. */
int hbsjd_create(hbsjd_ctx **out, const hbsjd_model_desc *m, const void *weights, size_t weight_bytes,
                 int max_batch, int max_window, void *cuda_stream);

/* Student rollout of Eq. 2 for `batch` images (Sec. 4.2-4.3).
 *   prefix_tokens DEVICE int32 [batch, T]; only the first prefix_len[b] entries of row b are read
 *   prefix_len    DEVICE int32 [batch], 0..T
 *   class_labels  DEVICE int32 [batch], 0..n_classes-1 (n_classes selects the null class)
 *   p             HOST parameters
 *   out_tokens    DEVICE int32 [batch, T]; row b receives x_1..x_T, the prefix copied through.
 *                 With max_rounds >= 0 positions not yet committed hold drafts / zeros.
 *   stats         HOST, may be NULL
 * Runs state init, prefix pre-filling, the initial history windows, then rounds until every image
 * is complete or max_rounds is reached; returns after the stream has finished that work.
 * Errors: HBSJD_EINVAL for batch/window beyond the context's limits, prefix_len > T, label or
 * prefix token out of range, non-positive temperature; HBSJD_ECUDA; HBSJD_ETIMEOUT. */
int hbsjd_rollout(hbsjd_ctx *c, int batch, const int32_t *prefix_tokens, const int32_t *prefix_len,
                  const int32_t *class_labels, const hbsjd_params *p, int32_t *out_tokens, hbsjd_stats *stats);

/* hbsjd_rollout for callers whose buffers live in HOST memory (pinned memory makes the copies
 * asynchronous): copies the three inputs to staging buffers of the context, runs the rollout, and copies
 * the tokens back, all on the context's stream; returns after the result has arrived.
 *   prefix_tokens HOST int32 [batch, T];  prefix_len, class_labels HOST int32 [batch];  out_tokens HOST int32 [batch, T] */
int hbsjd_rollout_host(hbsjd_ctx *c, int batch, const int32_t *prefix_tokens, const int32_t *prefix_len,
                       const int32_t *class_labels, const hbsjd_params *p, int32_t *out_tokens, hbsjd_stats *stats);

/* Threshold calibration of Sec. 4.3 ("a lightweight, data-independent latency test with a few verifier
 * forwards"): times the verifier forward of a `batch`-image rollout (window, guidance on/off) with A live
 * images, once in Full form (all `batch` slots) and once in Compact form (A slots), for
 * A = batch, 3/4, 1/2, 1/4 and 1/8 of the batch, on a synthetic state (cursors at T/2).  *gamma_out (HOST) =
 * the largest tested A at which Compact is not slower than Full beyond 1 % timing noise (Eq. 6 keeps Full for
 * A > gamma); 0 if Compact
 * is slower everywhere.  ms_full / ms_compact: HOST float[5] or NULL, the measured milliseconds in that order.
 * Discards the context's rollout state.  Errors: HBSJD_EINVAL, HBSJD_ECUDA, HBSJD_ETIMEOUT. */
int hbsjd_calibrate_gamma(hbsjd_ctx *c, int batch, int window, int guidance, int *gamma_out, float *ms_full,
                          float *ms_compact);

/* One verification round (Sec. 4.2 "Batched verification" .. "Independent progress") on the state left
 * by hbsjd_rollout or a previous hbsjd_round.  *live_out (HOST) = images still incomplete afterwards.
 * A sequence of hbsjd_rollout(max_rounds = 0) and hbsjd_round calls yields the same tokens as one
 * monolithic hbsjd_rollout.  Errors: HBSJD_ESTATE without a preceding hbsjd_rollout. */
int hbsjd_round(hbsjd_ctx *c, int *live_out);

/* Copies the current token rows (committed tokens, then drafts) to DEVICE int32 [batch, T]. */
int hbsjd_tokens(hbsjd_ctx *c, int32_t *out_tokens);

/* Frees every resource of the context.  NULL is allowed. */
void hbsjd_destroy(hbsjd_ctx *c);

/* ---- state export / import (debugging, parity tests, resuming a rollout); HOST buffers ----
 * cursor int32[batch]: committed tokens per image (Sec. 4.2 "committed cursor")
 * seq    int32[batch, T+1]: seq[b][t] = token at position t (1-based; entry 0 unused); t <= cursor committed,
 *        cursor < t < cursor+window: drafts
 * delta  uint8[batch, T+1]: 1 where the draft is a history / fallback draft (point-mass proposal)
 * qbase  int32[batch]: cursor at the start of the previous round (row t-qbase-1 of the previous
 *        round's probabilities is the proposal of draft t)
 * round  next round index.
 * hbsjd_set_state leaves the KV pages and the stored probabilities untouched. */
int hbsjd_get_state(hbsjd_ctx *c, int32_t *cursor, int32_t *seq, uint8_t *delta, int32_t *qbase, int32_t *round);
int hbsjd_set_state(hbsjd_ctx *c, const int32_t *cursor, const int32_t *seq, const uint8_t *delta,
                    const int32_t *qbase, int32_t round);

/* Reads intermediate results of the last round into a HOST buffer.
 *   HBSJD_DBG_PROBS   index = image: fp32 [window, V] probabilities of the last round
 *   HBSJD_DBG_LOGITS  index = 2*image + branch (0 conditional, 1 unconditional): fp32 [window, V]
 *   HBSJD_DBG_SLOTS   index ignored: int32 [3, n_slots] = image, cursor, n of each physical slot; returns n_slots
 *   After hbsjd_debug_forward (index = 2*image + branch; elements of the context's type unless stated):
 *   HBSJD_DBG_ACT_A   [n, dim]  operand of the next projection: fp32 models, the normed rows of the last norm that ran;
 *                     bf16 models (RMSNorm folded into the GEMMs), the bf16 copy of the residual stream
 *   HBSJD_DBG_ACT_Q   [n, dim]  rotated queries        HBSJD_DBG_ACT_O  [n, dim]  attention output
 *   HBSJD_DBG_ACT_FFN [n, ffn_hidden]  silu(gate) * up  HBSJD_DBG_ACT_H  fp32 [n, dim]  residual stream
 *   HBSJD_DBG_KV_K / HBSJD_DBG_KV_V  [cursor + n, dim]  cache rows of sequence indices 0..cursor+n-1 of that layer;
 *                     returns cursor + n
 * Returns the number of leading rows that are valid (or n_slots), or a negative error. */
enum { HBSJD_DBG_PROBS = 0, HBSJD_DBG_LOGITS = 1, HBSJD_DBG_SLOTS = 2, HBSJD_DBG_ACT_A = 3, HBSJD_DBG_ACT_Q = 4,
       HBSJD_DBG_ACT_O = 5, HBSJD_DBG_ACT_FFN = 6, HBSJD_DBG_ACT_H = 7, HBSJD_DBG_KV_K = 8, HBSJD_DBG_KV_V = 9 };
int hbsjd_debug_read(hbsjd_ctx *c, int what, int index, void *host_dst, size_t max_bytes);

/* Component-parity aid: runs the verifier forward of the current rollout state (Full layout, Sec. 4.2 "Batched
 * verification") up to and including layer `layer` -- stage 0: through the attention sub-block (norm, QKV + RoPE +
 * KV write, attention, output projection into the residual stream); stage 1: the whole block -- and stops, so
 * that hbsjd_debug_read can fetch that layer's intermediates.  No logits, no verification; the rollout state
 * is untouched (the KV rows written are the ones the next round rewrites with the same values).
 * Errors: HBSJD_ESTATE without a preceding hbsjd_rollout; HBSJD_EINVAL for layer / stage out of range. */
int hbsjd_debug_forward(hbsjd_ctx *c, int layer, int stage);

/* Decoder GEMM as used by the round (Sec. 4.2 verifier forward): C[M,N] (+)= A[M,K] . W[N,K]^T on the
 * context's stream.  A, W: DEVICE, element type of the context (bf16: tcgen05 tensor cores, fp32
 * accumulation; fp32: CUDA cores).  C: DEVICE fp32 [M,N]; accumulate != 0 adds into C.
 * M may be any size; bf16 needs N % 64 == 0 and K % 64 == 0; A, W 16-byte aligned.  A, W and C are ordered
 * like any other kernel argument behind earlier work of the stream. */
int hbsjd_gemm(hbsjd_ctx *c, const void *A, const void *W, float *C, int M, int N, int K, int accumulate);

/* accumulate = 2 (bf16 contexts, N = dim, M within the context's activation rows): the residual-update form the
 * forward itself uses, C += A W^T together with the bf16 copy and the per-row partial sums of squares of the new C
 * (written to buffers of the context), so that it can be timed and checked alone.
 * hbsjd_gemm `reps` times back to back before the one synchronisation (micro-benchmarks time the decoder's GEMM
 * shapes the way a forward issues them), and -- acc_wait_ns > 0, bf16 contexts -- with the bounded wait of the
 * epilogue warps on their accumulator shortened to that many nanoseconds (Sec. 4.2 verifier forward; the paper has
 * no counterpart of the failure path).  A limit shorter than the main loop makes a healthy pipeline take the
 * time-out path: every role leaves its loop, copies and MMAs in flight are drained, TMEM is freed, the call
 * returns HBSJD_ETIMEOUT with C partly written, and the context stays usable.  Tests use it to exercise that path.
 * tile (bf16 contexts, accumulate 0 or 1): 0 = the library's own choice for the shape; 32, 64, 128, 256 = one CTA
 * per 128 x tile block of C; 512 / 640 = 256 x 256 / 256 x 128 blocks on CTA pairs (N a multiple of 256 / 128).  Every choice gives the
 * same bits (each element's products are summed in the same order); HBSJD_EINVAL for any other value. */
int hbsjd_debug_gemm(hbsjd_ctx *c, const void *A, const void *W, float *C, int M, int N, int K, int accumulate,
                     int reps, unsigned int acc_wait_ns, int tile);

/* Chooses the form of RMSNorm of a bf16 context (Sec. 4.2 verifier forward; the paper does not go below the model):
 * on = 1 folds it into the GEMM epilogues (bf16 copy of the unnormalised residual stream as the operand, gain in the
 * weights, row factor in the next epilogue), on = 0 runs it as a kernel of its own in front of the projections.
 * hbsjd_create picks the folded form for contexts of at most 2048 activation rows (2 x max_batch x max_window) and the
 * separate one above; this call lets tests run either form at any size.  The two forms round the GEMM operand at
 * different points (x r g against x), so their results differ at bf16-noise level; one context always uses one form,
 * so Full and Compact execution stay bit-identical.  Only before the first rollout, and only for models whose norm
 * gains are all 1 (nothing to re-fold): HBSJD_ESTATE otherwise. */
int hbsjd_debug_fold_norm(hbsjd_ctx *c, int on);

/* Scatters the context's KV pages over the page pool (a seeded permutation of the page table) so that tests can
 * check that results do not depend on where a row's pages lie (Sec. 4.2: per-image KV-cache locations).  Only
 * before the first rollout of the context; HBSJD_ESTATE afterwards. */
int hbsjd_debug_shuffle_pages(hbsjd_ctx *c, uint64_t seed);

/* Probability pipeline of the verification step on caller-supplied logits (Sec. 4.2: "verification uses the
 * fused guided logits"): p = softmax(top_k((l_u + s (l_c - l_u)) / temperature)), ties at the k-th value kept.
 * logits_c, logits_u: DEVICE fp32 [rows, V] (logits_u may be NULL: no guidance); probs: DEVICE fp32 [rows, V].
 * V is the context's vocabulary.  Runs on the context's stream and waits for completion. */
int hbsjd_probs(hbsjd_ctx *c, const float *logits_c, const float *logits_u, int rows, float cfg_scale,
                float temperature, int top_k, float *probs);

/* Verification step of one round on caller-supplied logits (Sec. 4.2, Eq. 5 / Eq. 4): probability pipeline,
 * accept test of every draft left to right, residual resampling at the first reject (or the bonus token),
 * commit, cursor advance and draft refresh, for `batch` images in Full layout.  All pointers DEVICE.
 *   logits  fp32 [branches, batch, window, V]  branch 0 conditional, branch 1 unconditional (branches = 1 or 2)
 *   q_prev  fp32 [batch, window, V]  previous round's probabilities (row t - qbase - 1 = proposal of draft t)
 *   p_out   fp32 [batch, window, V]  this round's probabilities (rows 0..n-1 of each live image written)
 *   cursor int32 [batch], seq int32 [batch, T+1], delta uint8 [batch, T+1], qbase int32 [batch]: rollout
 *           state as in hbsjd_get_state, updated in place;  m_out int32 [batch]: tokens committed (images
 *           with cursor == T are skipped and keep their m_out entry)
 * The random words are Philox(seed; image, position, round).  Uses scratch buffers of the context; runs on
 * the context's stream and waits for completion.  Limits: batch <= max_batch and window <= max_window of the
 * context, V % 4 == 0, V <= 32768. */
typedef struct {
    int32_t batch, window, T, V, branches, history_offset, greedy, top_k;
    float cfg_scale, temperature;
    uint64_t seed;
    uint32_t round;
    uint32_t reserved;
} hbsjd_verify_desc;
int hbsjd_verify(hbsjd_ctx *c, const hbsjd_verify_desc *d, const float *logits, const float *q_prev, float *p_out,
                 int32_t *cursor, int32_t *seq, uint8_t *delta, int32_t *qbase, int32_t *m_out);

/* hbsjd_verify for callers that must not allocate device memory.  (The paper has no counterpart of this
 * entry point; it exists for deployment reasons only.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a training process whose framework has
 * handed the whole device to its own caching allocator (a raw allocation there can fail or fragment the
 * pool), a latency-critical loop in which an allocation would synchronise the device, or a plug-in called
 * from inside another runtime that owns all device memory.  Such a caller cannot create an hbsjd_ctx either,
 * so this function takes no context: it needs only the stream, the descriptor and the same input / output
 * buffers as hbsjd_verify.
 *
 * How: the scratch of the verification kernels (slot tables, accept flags, candidate tokens, counters) lives
 * in a fixed array of 192 KiB that is part of the library image; every GPU that loads the library holds it
 * until the process exits.  The function calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - Limits: batch <= 1024, batch * window <= 16384, window <= 64, V % 4 == 0, V <= 32768; larger requests
 *     are refused with HBSJD_EINVAL and nothing is launched.
 *   - The first call on each device looks up the array's device address and raises the kernels' shared-
 *     memory limit; make that first call before any stream capture begins.
 *   - Every call uses the same array and finds the previous call's contents in it; the function clears
 *     what has to start at zero.  Calls that overlap on the GPU (other streams, other host threads) race on
 *     the array: serialise them.
 *   - cuda_stream is a cudaStream_t passed as void*; the call returns after the stream has finished the work.
 * Results are identical to hbsjd_verify on the same inputs. */
int hbsjd_verify_static(void *cuda_stream, const hbsjd_verify_desc *d, const float *logits, const float *q_prev,
                        float *p_out, int32_t *cursor, int32_t *seq, uint8_t *delta, int32_t *qbase,
                        int32_t *m_out);

/* Bidirectional KL of Eq. 3 per row: out[r] = 1/2 KL(p || q) + 1/2 KL(q || p) with p = softmax(logits_s[r]),
 * q = softmax(logits_t[r]).  logits_s, logits_t: DEVICE fp32 [rows, V], V the context's vocabulary; out: DEVICE
 * fp32 [rows].  fp32 arithmetic with running maxima (no overflow for any finite logits).  Runs on the context's
 * stream and waits for completion. */
int hbsjd_bikl(hbsjd_ctx *c, const float *logits_s, const float *logits_t, int rows, float *out);

/* Distillation score of completed trajectories (Eq. 3): for image b with real prefix k_b, the mean over the
 * generated positions t = k_b+1..T of D_biKL(p_S(. | x_<t), p_T(. | x_<t)), where both models read the same
 * tokens and class label (no guidance, temperature 1, no top-k), then the mean over the images of the batch that
 * generated anything (k_b < T).  This is the step that follows the rollout in the on-policy distillation loop.
 *   student, teacher  two contexts with the same grid (T) and vocabulary; batch <= max_batch of both.  Both
 *                     models run full-sequence causal forwards in chunks of min(64, 2 min(max_window)) inputs per image
 *                     through the same kernels as the rollout; their rollout state and KV caches are
 *                     overwritten (a stepped rollout cannot be continued afterwards).
 *   tokens        DEVICE int32 [batch, T]   completed trajectories (e.g. hbsjd_rollout's out_tokens)
 *   prefix_len    DEVICE int32 [batch]      k_b in 0..T
 *   class_labels  DEVICE int32 [batch]
 *   bikl_pos      DEVICE fp32 [batch, T] or NULL: entry t-1 = the term of position t (0 for t <= k_b)
 *   per_image     DEVICE fp32 [batch] or NULL: the per-image means (0 where k_b = T)
 *   loss          HOST float: the batch mean
 * Work is enqueued on each context's own stream with event dependencies between them; the call returns after
 * both streams finished.  Errors as hbsjd_rollout (arguments are validated on the host before any launch). */
int hbsjd_score(hbsjd_ctx *student, hbsjd_ctx *teacher, int batch, const int32_t *tokens, const int32_t *prefix_len,
                const int32_t *class_labels, float *bikl_pos, float *per_image, float *loss);

/* Per-kernel-class timing with CUDA events on the context's stream (off by default).  While enabled,
 * every launch of a timed class is bracketed by an event pair; totals accumulate until the next
 * hbsjd_profile(c, 1), which also resets them.  work = algorithmic FLOPs (GEMM: 2 M N K per launch) or
 * algorithmic bytes (attention: K,V rows read + q read + output written; accept: logits read + probabilities
 * written) of the launches that were timed. */
enum { HBSJD_PROF_GEMM = 0, HBSJD_PROF_ATTENTION = 1, HBSJD_PROF_ACCEPT = 2, HBSJD_PROF_OTHER = 3 };
typedef struct {
    double ms[4];
    double work[4];
    int64_t launches[4];
    int64_t dropped;   /* launches not timed because the event pool was exhausted */
    /* the GEMM class again, split by the number of activation rows M of the launch:
     * M <= 512, 512 < M <= 2048, 2048 < M <= 6144, M > 6144 */
    double gemm_ms_by_rows[4];
    double gemm_work_by_rows[4];
    int64_t gemm_launches_by_rows[4];
    double gemm_bytes_by_rows[4];   /* algorithmic bytes: operands read once, outputs written (residual: read + written) */
} hbsjd_kernel_profile;
int hbsjd_profile(hbsjd_ctx *c, int enable);
int hbsjd_profile_read(hbsjd_ctx *c, hbsjd_kernel_profile *out);
/* What an event pair adds to a timed launch: an event between two kernels makes the second one start only after
 * the first has completed, so its launch latency lies inside the bracket (in normal operation the library's
 * kernels are launched programmatically dependent and that latency overlaps the previous kernel).  This call
 * brackets `reps` launches of an empty kernel in the same way and returns the median bracket in microseconds;
 * benchmarks report it beside the per-class times so that a reader can net it out. */
int hbsjd_profile_launch_floor(hbsjd_ctx *c, int reps, float *us_out);

const char *hbsjd_strerror(int code);
const char *hbsjd_last_error(const hbsjd_ctx *c);

#ifdef __cplusplus
}
#endif
#endif /* HBSJD_H_ */
