/*
 * scd.h - C ABI of the B200 (sm_100a) Speculative Coupled Decoding library.
 *
 * One SCD iteration = one window-parallel forward of a Llama-style decoder over L draft tokens
 * (Algorithm 6, "Evaluate": p_j^{t+1} <- p_theta(. | X^t_{0:j-1}) for every window position in
 * parallel) followed by one fused verify-and-redraft pass over the vocabulary (Algorithm 6,
 * "Verify & Drafting with vectorised MRS"; Algorithm 1 for the accept rule and the residual
 * distribution; Sec. 4.3 for logit post-processing; Sec. 5.1 for the CFG mix).
 *
 * General conventions
 *   - Every function returns an int status: SCD_OK (0) or a negative SCD_ERR_* code. Nothing
 *     throws, aborts or prints. scd_strerror() names a code; scd_last_error() gives the detail
 *     of the most recent failure on the calling thread.
 *   - Pointers marked [dev] are device memory owned by the CALLER (for example the data_ptr()
 *     of a PyTorch tensor); the library borrows them for the lifetime stated and never frees
 *     them. Pointers marked [host] are ordinary host memory. Handles are opaque and owned by
 *     the library (create / free pairs).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream). Calls are
 *     asynchronous with respect to the host unless stated; a session must be driven from one
 *     stream at a time and is not thread-safe.
 *   - Row-major everywhere. Weight matrices are [out_features, in_features].
 *   - Sequence layout: a decode batch has B sequences and S streams per sequence (S = 2 with
 *     classifier-free guidance: stream 0 conditional, stream 1 unconditional; else S = 1).
 *     Stream-sequence index q = s * B + b; window rows of one stream-sequence are contiguous:
 *     row = q * L + k.
 *   - Arguments are validated on the host before anything is launched; a call that fails
 *     validation leaves all state unchanged.
 */
#ifndef SCD_H_
#define SCD_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    SCD_OK = 0,
    SCD_ERR_ARG = -1,         /* null pointer, non-positive size, bad enum */
    SCD_ERR_SHAPE = -2,       /* shape not supported (see each call) */
    SCD_ERR_CAPACITY = -3,    /* would exceed max_seq / window / scratch capacity */
    SCD_ERR_STATE = -4,       /* call out of order (e.g. step before prefill) */
    SCD_ERR_CUDA = -5,        /* a CUDA runtime/driver call failed; see scd_last_error() */
    SCD_ERR_TIMEOUT = -6,     /* a bounded device-side wait gave up; the session's error word stays set
                                 until the next scd_prefill, which clears it: re-prefill or recreate */
    SCD_ERR_UNSUPPORTED = -7  /* valid request that the library does not implement */
};

enum { SCD_F32 = 0, SCD_BF16 = 1 };

/* Decode modes. SCD_MODE_AR: vanilla autoregressive sampling, one token per forward (Sec. 2.1,
 * the baseline "A"). SCD_MODE_SCD_MC: Speculative Coupled Decoding with the maximal coupling
 * (the "Maximal Coupling" branch of Algorithm 3, efficient form Algorithm 6). SCD_MODE_SJD:
 * Speculative Jacobi Decoding, independent redraft (Algorithm 2). SCD_MODE_ALPHA: the
 * alpha-coupling of the two (Algorithm 5): every row beyond the committed prefix keeps its
 * maximal-coupling redraft with probability alpha and is redrawn independently from p otherwise
 * (alpha = 1 is SCD_MODE_SCD_MC, alpha = 0 is SCD_MODE_SJD, both up to the extra coin).
 * SCD_MODE_SCD_GS: SCD with the Gumbel-sharing coupling (Algorithm 4 inside Algorithm 7): rows
 * beyond the committed prefix are redrafted as argmax(log p + g) with Gumbel noise g that depends
 * on (seed, sequence, position, id) only - not on the iteration - and fresh rows start from the
 * same race under the uniform draft distribution. The race is decided in integers (race times
 * -log2 u in 40-bit fixed point, compared by cross-multiplication; ties to the smaller id). */
enum { SCD_MODE_AR = 0, SCD_MODE_SJD = 1, SCD_MODE_SCD_MC = 2, SCD_MODE_SCD_GS = 3, SCD_MODE_ALPHA = 4 };

typedef struct scd_model scd_model_t;
typedef struct scd_session scd_session_t;

/* Shape of the decoder p_theta. head_dim must be even; n_heads % n_kv_heads == 0. */
typedef struct {
    int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn;
    int32_t vocab_out;      /* V: rows of the LM head = size of the sampled vocabulary */
    int32_t vocab_in;       /* rows of the token embedding (>= any id ever fed) */
    float   rope_base;      /* RoPE: angle = pos * rope_base^(-2i/head_dim), pairs (i, i+head_dim/2) */
    float   rms_eps;
    int32_t dtype;          /* SCD_F32 or SCD_BF16: type of all weights, activations and KV cache;
                               the residual stream and the logits are always fp32 */
    int32_t max_seq;        /* KV capacity per stream-sequence, in tokens */
    int32_t kv_page_tokens; /* tokens per KV page (power of two, >= 16) */
} scd_model_config_t;

/* Weights. The nine per-layer members are [host] arrays of n_layers [dev] pointers. All tensors
 * have the model dtype, are borrowed until scd_free_model, and must be 16-byte aligned. */
typedef struct {
    const void *tok_emb;     /* [vocab_in, d_model] */
    const void *final_norm;  /* [d_model] */
    const void *lm_head;     /* [vocab_out, d_model] */
    const void *const *attn_norm, *const *wq, *const *wk, *const *wv, *const *wo;
    const void *const *ffn_norm, *const *w_gate, *const *w_up, *const *w_down;
} scd_weights_t;

/* Decode settings (Sec. 4.3, Sec. 5.1, App. "Experimental Details"). */
typedef struct {
    int32_t  mode;          /* SCD_MODE_* */
    int32_t  batch;         /* B independent sequences */
    int32_t  window_L;      /* Jacobi window length L, 1..256 (ignored, = 1, in AR mode) */
    float    temperature;   /* > 0 */
    int32_t  top_k;         /* <= 0: off. Threshold form: ids whose logit >= the k-th largest stay */
    float    cfg_lambda;    /* 0: no guidance, one stream. Else logits = (1+lambda) c - lambda u */
    uint64_t seed;          /* Philox key */
    int32_t  allowed_lo, allowed_hi; /* sampled ids are allowed_lo <= v < allowed_hi (0, V = all) */
    int32_t  row_period;    /* > 0: generated position g (0-based) with g % row_period ==
                               row_period-1 is forced to eol_id (end-of-row token of an image grid) */
    int32_t  eol_id;
    float    alpha;         /* SCD_MODE_ALPHA only: probability of keeping the coupled redraft, 0..1 */
    float    top_p;         /* nucleus mass, applied after top-k on the integer weights: with theta the
                               largest weight value whose ids {W_v >= theta} hold at least top_p of the
                               mass (mass * 2^24 >= trunc(top_p * 2^24 + 1/2) * Z), ids below theta are
                               dropped (ties kept). <= 0 or >= 1: off. (The paper's video setting
                               samples with top-p 0.8.) */
} scd_decode_config_t;

typedef struct {
    int64_t forwards;          /* decoder forwards run (= NFE of the paper) */
    int64_t committed;         /* tokens committed, summed over the batch */
    int64_t accept_hist[257];  /* accept_hist[a]: (sequence, iteration) pairs that committed a tokens */
    float   elapsed_ms;        /* device time of the generate call (CUDA events) */
} scd_stats_t;

const char *scd_strerror(int code);
const char *scd_last_error(void);

/* ---- model ------------------------------------------------------------------------------
 * scd_init_model: the model p_theta that Algorithm 6 REQUIREs (a Llama-style decoder; the paper treats it
 * as a black box that yields p_theta(. | X_{0:j-1}) for all window positions in one pass, Sec. 2.2).
 * Validates the shape, records the borrowed weight pointers, builds the RoPE
 * table and the TMA descriptors of the weight matrices on the current CUDA device.
 * Errors: SCD_ERR_ARG (null), SCD_ERR_SHAPE (odd head_dim, heads not divisible, sizes <= 0;
 * bf16 models additionally need d_model, d_ffn and n_heads*head_dim to be multiples of 64),
 * SCD_ERR_CUDA. */
int scd_init_model(const scd_model_config_t *cfg, const scd_weights_t *weights, scd_model_t **out);
int scd_free_model(scd_model_t *model);

/* ---- session ----------------------------------------------------------------------------
 * scd_session_create: the state Algorithm 6 keeps between iterations (REQUIRE: draft length L, maximum
 * sequence length; its loop variables i, t, the drafts X and the draft distributions p^(t)).
 * A session holds the KV cache (paged), the window state (drafts, draft distributions, position
 * and iteration counters - all resident on the device) and scratch activations for one decode
 * batch. Allocates device memory (cudaMalloc); free with scd_session_free. bf16 models: a forward
 * carries S*B*L window rows; the weight GEMMs take them in blocks of 256 (one pass over the weights
 * per block), and at most 1024 rows are accepted (SCD_ERR_CAPACITY beyond). */
int scd_session_create(scd_model_t *model, const scd_decode_config_t *cfg, scd_session_t **out);
int scd_session_free(scd_session_t *session);

/* scd_prefill: feeds the prompts. prompt_ids [host] int32 [S*B, P] (stream-sequence major).
 * Tokens 0..P-2 of every stream enter the KV cache; token P-1 is the "last committed token"
 * that the first iteration feeds. Afterwards n = P, kv_len = P-1, t = 0 and the window holds
 * L fresh rows (draft distribution uniform over the allowed ids, draft X ~ it: the
 * initialisation of Algorithm 6). n_total = P + n_new is the final sequence length (window rows beyond it stay
 * inert). Errors: SCD_ERR_CAPACITY if P + n_new > max_seq. Synchronises the stream. */
int scd_prefill(scd_session_t *session, const int32_t *prompt_ids, int32_t P, int32_t n_new,
                void *stream);

/* scd_step: ONE iteration (the loop body of Algorithm 6): window forward, KV write, fused
 * post-process / verify / residual sample / first-rejection / commit / coupled redraft.
 * Fully asynchronous; all state stays on the device. */
int scd_step(scd_session_t *session, void *stream);

/* scd_step_result: the loop variables of Algorithm 6 after an iteration (i <- Accept + 1): waits for
 * the stream, then copies out per-sequence counters.
 * n_committed[b] = tokens committed by the LAST step, n_known[b] = prompt + committed tokens,
 * kv_len[b] = committed KV entries (always n_known - 1). Any pointer may be NULL. [host][B] */
int scd_step_result(scd_session_t *session, int32_t *n_committed, int32_t *n_known,
                    int32_t *kv_len, void *stream);

/* scd_generate: the While loop of Algorithm 6 ("while i < N"; Algorithm 7 in SCD_MODE_SCD_GS, Algorithm 2
 * in SCD_MODE_SJD): runs iterations until every sequence holds n_total tokens (set by prefill),
 * then copies the generated tokens to out_tokens [host] int32 [B, n_new] and fills stats
 * [host] (may be NULL). Blocking. */
int scd_generate(scd_session_t *session, int32_t *out_tokens, scd_stats_t *stats, void *stream);

/* scd_read_tokens: copies tokens [first, first+count) of every sequence's conditional stream
 * (prompt included) to out [host] int32 [B, count]. Blocking. */
int scd_read_tokens(scd_session_t *session, int32_t first, int32_t count, int32_t *out,
                    void *stream);

/* ---- test and benchmark hooks -------------------------------------------------------------
 * scd_verify: the fused verify-and-redraft kernel alone on caller-supplied logits
 * (the verify-and-drafting part of Algorithm 6 for one window per sequence; Algorithm 1 per row).
 *   p_logits      [dev] f32 [S, B, L, V]  target logits (S = 2 iff cfg_lambda != 0)
 *   q_logits      [dev] f32 [B, L, V]     draft logits, post-processed with the same temperature
 *                                         and top-k (no guidance); NULL = every row is fresh
 *                                         (uniform over the allowed ids)
 *   draft_ids     [dev] i32 [B, L]        X_j, drawn from q_j: inside the allowed range with q_j(X_j) > 0.
 *                                         (A draft without mass under p_j is rejected whatever q_j says,
 *                                         so no id outside the support of p is ever committed.)
 *   positions     [dev] i64 [B]           global position of window row 0 of each sequence
 *   iteration                              t (noise key)
 *   n_commit      [dev] i32 [B]           out: a = tokens committed (1..L)
 *   committed_ids [dev] i32 [B, L]        out: first a entries valid
 *   next_draft_ids[dev] i32 [B, L]        out: drafts of the next window (row k <- old row k+a;
 *                                         rows entering the window get a fresh uniform draft)
 *   accept_flags  [dev] u8  [B, L]        out: k_j of every row (all rows are evaluated)
 *   workspace     [dev] scratch of scd_verify_workspace_bytes(cfg, V) bytes, 256-byte aligned
 * Uses cfg->mode (AR: draws one token per sequence from p, L treated as 1), batch, window_L,
 * temperature, top_k, cfg_lambda, seed, allowed range, row_period/eol_id (positions are
 * "generated positions": prompt length 0). */
int64_t scd_verify_workspace_bytes(const scd_decode_config_t *cfg, int32_t V);
int scd_verify(const scd_decode_config_t *cfg, int32_t V, const float *p_logits,
               const float *q_logits, const int32_t *draft_ids, const int64_t *positions,
               int64_t iteration, int32_t *n_commit, int32_t *committed_ids,
               int32_t *next_draft_ids, uint8_t *accept_flags, void *workspace, void *stream);

/* scd_verify_noalloc: scd_verify for callers that must not allocate device memory. (The paper has
 * no counterpart; this is a deployment convenience.) Some hosts of this library cannot call
 * cudaMalloc at the point where they verify a window: a serving loop that has handed all device
 * memory to its own pool at start-up, or code running where an allocation would synchronise the
 * device or fail (inside a latency-critical section, under a memory cap, between captured
 * regions). For them the scratch that scd_verify takes as `workspace` is a buffer built into the
 * library: a file-scope device array of scd_verify_noalloc_max_bytes() bytes (16 MiB) that
 * every GPU context loading the library holds until the process exits.
 *   - Arguments, outputs and results are exactly those of scd_verify, minus `workspace`.
 *   - The call issues no cudaMalloc / cudaFree and no allocating library routine; the caller still
 *     supplies all inputs and outputs.
 *   - A request whose scratch (scd_verify_workspace_bytes) exceeds the built-in buffer returns
 *     SCD_ERR_CAPACITY and launches nothing; e.g. B = 1 or 2 with L = 32, V = 16384 fit,
 *     B = 8 does not: use scd_verify with your own workspace there.
 *   - The FIRST call on each device is a warm-up and belongs to start-up: it looks up the buffer's
 *     device address (one cudaGetSymbolAddress with that device current), and with CUDA's lazy module
 *     loading it is also the moment the runtime loads the kernels on that device and gives the 16 MiB
 *     array its memory - so that first call may synchronise, take memory, or fail where memory is
 *     already short. Make it (any small problem will do) before device memory is handed to your own
 *     pool and outside any stream capture; from the second call on nothing is allocated. The address
 *     is cached per device ordinal for the life of the process (cudaDeviceReset invalidates it).
 *   - All calls on a device share the one buffer, which keeps whatever the previous call left
 *     in it; the part that must start at zero is cleared on `stream` before the kernel. Two
 *     calls that can overlap on the GPU (different streams, no ordering between them) race on
 *     the buffer: order them, or give one of them scd_verify with its own workspace. */
int64_t scd_verify_noalloc_max_bytes(void);
int scd_verify_noalloc(const scd_decode_config_t *cfg, int32_t V, const float *p_logits,
                       const float *q_logits, const int32_t *draft_ids, const int64_t *positions,
                       int64_t iteration, int32_t *n_commit, int32_t *committed_ids,
                       int32_t *next_draft_ids, uint8_t *accept_flags, void *stream);

/* scd_forward_window: the window forward alone, teacher-forced. ids [dev] i32 [S*B, M] are fed
 * at positions kv_len .. kv_len+M-1 of each stream-sequence (M <= max(L, prefill chunk) of the
 * session); ids[.,0] must be the last known token (the one at position kv_len = n-1). Writes
 * logits [dev] f32 [S*B, M, V] and, if not NULL, the final-layer residual stream
 * hidden [dev] f32 [S*B, M, d_model]. KV entries of the M inputs are written. With
 * commit != 0 the ids[., 1..M) of the conditional streams are appended to the token record
 * and n, kv_len advance by M-1 (the invariant kv_len = n-1 is kept; the last input's KV entry
 * is recomputed by the next forward). Positions beyond max_seq are neither written nor read. */
int scd_forward_window(scd_session_t *session, const int32_t *ids, int32_t M, float *logits,
                       float *hidden, int32_t commit, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* SCD_H_ */
