// C-ABI entry points around a model and a decode session: scd_init_model, scd_session_create,
// scd_prefill, scd_step, scd_generate and the teacher-forced forward hook.
#include <algorithm>
#include <atomic>
#include <cstring>
#include <new>

#include "model.cuh"
#include "gemm.cuh"

using namespace scd;

namespace scd {
static std::atomic<long long> g_launches{0};
void count_launches(long long n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
}  // namespace scd

namespace {

constexpr int GENERATE_BLOCK = 64;      // iterations scd_generate enqueues between two looks at the counters

inline bool is_pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }
inline size_t elem_size(int dtype) { return dtype == SCD_F32 ? 4 : 2; }

template <class T>
int dev_alloc(T **p, size_t count)
{
    *p = nullptr;
    SCD_CUDA_TRY(cudaMalloc((void **)p, std::max<size_t>(count, 1) * sizeof(T)));
    return SCD_OK;
}

__global__ void identity_pages_kernel(int *table, int n)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) table[i] = i;
}

__global__ void set_state_kernel(int *n_known, int *n_total, int B, int n, int total)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B) { n_known[b] = n; n_total[b] = total; }
}

// Teacher-forced commit of the forward hook: ids[1..M) are appended to the token record of the
// conditional stream and n advances by M - 1 (ids[0] is the already known last token).
__global__ void commit_ids_kernel(const int *ids, int M, int B, int *n_known, int *tokens, int token_stride)
{
    const int b = blockIdx.x;
    const int n = n_known[b];
    for (int i = 1 + threadIdx.x; i < M; i += blockDim.x)
        if (n + i - 1 < token_stride) tokens[(size_t)b * token_stride + n + i - 1] = ids[(size_t)b * M + i];
    __syncthreads();
    if (threadIdx.x == 0) n_known[b] = n + M - 1;
}

void session_verify_params(scd_session *s, VerifyParams &p)
{
    fill_verify_params(p, &s->cfg, s->model->cfg.vocab_out);
    p.p_logits = s->logits;
    p.xbuf[0] = s->xbuf[0]; p.xbuf[1] = s->xbuf[1];
    p.stats[0] = s->stats[0]; p.stats[1] = s->stats[1];
    p.q_is_raw = 0; p.q_present = 1; p.keep_x = 1;
    p.positions = nullptr;
    p.n_known = s->n_known; p.n_total = s->n_total;
    p.prompt_len = s->prompt_len;
    p.iter = s->iter; p.iteration = 0;
    p.shift = s->shift; p.prev_lw = s->prev_lw;
    p.draft_in = s->drafts; p.draft_out = s->drafts;
    p.n_commit = s->n_commit; p.committed_ids = nullptr;
    p.tokens = s->tokens; p.token_stride = s->model->cfg.max_seq;
    p.accept_flags = s->accept_flags;
    p.row_y = s->row_y; p.row_y_indep = s->row_y_indep;
    p.done_count = s->done_count;
    p.dev_stats = s->dev_stats;
    p.finished = s->finished;
}

int enqueue_step(scd_session *s, cudaStream_t st, StepProfiler *prof = nullptr)
{
    ForwardArgs a;
    a.ids = nullptr; a.Mq = s->L; a.pos_override = -1; a.want_logits = true;
    a.logits = s->logits; a.hidden = nullptr; a.prof = prof;
    a.skip = s->finished + 1;                            // an iteration enqueued after the last token costs only its launches
    // the sampler reads only the ids it may draw: the allowed range and the end-of-row id
    a.lm_lo = s->cfg.allowed_lo; a.lm_hi = s->cfg.allowed_hi;
    a.lm_eol = s->cfg.row_period > 0 ? s->cfg.eol_id : -1;
    int rc = run_forward(s, a, st);
    if (rc != SCD_OK) return rc;
    VerifyParams p;
    session_verify_params(s, p);
    if (prof) prof->mark(PROF_VERIFY);
    count_launches(1);
    return launch_verify(p, st);
}

void drop_step_graph(scd_session *s)
{
    if (s->step_graph) cudaGraphExecDestroy(s->step_graph);
    s->step_graph = nullptr;
    s->step_graph_nodes = 0;
}

// One iteration as one graph launch. The first call after a prefill captures enqueue_step (all
// kernel arguments are device pointers and constants of the session, so one graph serves every
// iteration); programmatic-dependent-launch edges and cluster launches are kept by the capture.
// The host then submits one node list instead of ~160 launches per iteration.
int launch_step(scd_session *s, cudaStream_t st)
{
    // the captured launches carry the attention variant: capture again when it changes (once per generation)
    const int variant = s->attn_plan ? attention_tc_variant(s, s->L, s->ctx_floor) : 0;
    if (variant != s->att_variant) { s->att_variant = variant; drop_step_graph(s); }
    struct Advance { scd_session *s; ~Advance() { s->ctx_floor += 1; } } advance{s};   // every iteration commits >= 1 token
    if (s->step_graph_off) return enqueue_step(s, st);
    if (!s->step_graph) {
        cudaGraph_t graph = nullptr;
        const long long before = scd_kernel_launches();
        if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
            cudaGetLastError();
            s->step_graph_off = true;
            return enqueue_step(s, st);
        }
        const int rc = enqueue_step(s, st);
        const cudaError_t e = cudaStreamEndCapture(st, &graph);
        const long long nodes = scd_kernel_launches() - before;
        count_launches(-nodes);                          // nothing ran yet
        if (rc != SCD_OK || e != cudaSuccess || !graph) {
            cudaGetLastError();
            if (graph) cudaGraphDestroy(graph);
            s->step_graph_off = true;
            if (rc != SCD_OK) return rc;
            return enqueue_step(s, st);
        }
        const cudaError_t ei = cudaGraphInstantiate(&s->step_graph, graph, 0);
        cudaGraphDestroy(graph);
        if (ei != cudaSuccess) {
            cudaGetLastError();
            s->step_graph = nullptr;
            s->step_graph_off = true;
            return enqueue_step(s, st);
        }
        s->step_graph_nodes = nodes;
    }
    SCD_CUDA_TRY(cudaGraphLaunch(s->step_graph, st));
    count_launches(s->step_graph_nodes);
    return SCD_OK;
}

void free_session_memory(scd_session *s)
{
    if (s->step_graph) cudaGraphExecDestroy(s->step_graph);
    void *ptrs[] = {s->kv_pool, s->page_table, s->n_known, s->n_total, s->shift, s->prev_lw, s->drafts,
                    s->n_commit, s->tokens, s->tokens_u, s->row_y, s->row_y_indep, s->ids_buf, s->iter,
                    s->done_count, s->accept_flags, s->xbuf[0], s->xbuf[1], s->stats[0], s->stats[1],
                    s->dev_stats, s->finished, s->h, s->ss, s->xn, s->qkv, s->att, s->gu, s->act, s->logits, s->gemm_ws, s->stamps};
    for (void *p : ptrs) if (p) cudaFree(p);
    if (s->host_pinned) cudaFreeHost(s->host_pinned);
    if (s->gemm_state) gemm_session_release(s);
    if (s->attn_plan) attention_session_release(s);
}

// A bounded device-side wait that gave up leaves a non-zero error word (sticky until the next prefill:
// the GEMM kernels skip their output operation while it is set).
int check_device_health(scd_session *s, cudaStream_t st)
{
    int word = 0;
    int rc = gemm_error_word(s, &word, st);
    if (rc != SCD_OK) return rc;
    static const char *const who[] = {"", "GEMM: producer waiting for a free ring slot", "GEMM: MMA issuer waiting for operands",
                                      "GEMM: epilogue waiting for the accumulator", "attention: waiting for a free ring slot",
                                      "attention: waiting for a K/V tile", "attention: shared memory base not 1024-byte aligned",
                                      "attention: softmax waiting for the scores", "attention: waiting for the probabilities",
                                      "attention: waiting for the product P V", "attention: waiting for a free score buffer"};
    SCD_REQUIRE(word == 0, SCD_ERR_TIMEOUT, "a bounded device-side wait gave up (%s, code %d); prefill the session again",
                word > 0 && word < 11 ? who[word] : "unknown", word);
    return SCD_OK;
}

}  // namespace

extern "C" {

int scd_init_model(const scd_model_config_t *cfg, const scd_weights_t *w, scd_model_t **out)
{
    SCD_REQUIRE(cfg && w && out, SCD_ERR_ARG, "scd_init_model: NULL argument");
    *out = nullptr;
    SCD_REQUIRE(cfg->n_layers > 0 && cfg->d_model > 0 && cfg->n_heads > 0 && cfg->n_kv_heads > 0 &&
                cfg->head_dim > 0 && cfg->d_ffn > 0 && cfg->vocab_out > 0 && cfg->vocab_in > 0 &&
                cfg->max_seq > 1, SCD_ERR_SHAPE, "model sizes must be positive");
    SCD_REQUIRE(cfg->head_dim % 32 == 0 && cfg->head_dim <= 128, SCD_ERR_SHAPE,
                "head_dim %d: must be a multiple of 32, at most 128", cfg->head_dim);
    SCD_REQUIRE(cfg->n_heads % cfg->n_kv_heads == 0, SCD_ERR_SHAPE, "n_heads %% n_kv_heads != 0");
    SCD_REQUIRE(cfg->dtype == SCD_F32 || cfg->dtype == SCD_BF16, SCD_ERR_ARG, "unknown dtype %d", cfg->dtype);
    SCD_REQUIRE(is_pow2(cfg->kv_page_tokens) && cfg->kv_page_tokens >= 16, SCD_ERR_SHAPE,
                "kv_page_tokens %d: power of two >= 16", cfg->kv_page_tokens);
    SCD_REQUIRE(cfg->rms_eps > 0.f && cfg->rope_base > 1.f, SCD_ERR_ARG, "rms_eps / rope_base");
    if (cfg->dtype == SCD_BF16)
        SCD_REQUIRE(cfg->d_model % 64 == 0 && cfg->d_ffn % 64 == 0 && (cfg->n_heads * cfg->head_dim) % 64 == 0,
                    SCD_ERR_SHAPE, "bf16 models need d_model, d_ffn and n_heads*head_dim multiples of 64");
    SCD_REQUIRE(w->tok_emb && w->final_norm && w->lm_head && w->attn_norm && w->wq && w->wk && w->wv &&
                w->wo && w->ffn_norm && w->w_gate && w->w_up && w->w_down, SCD_ERR_ARG, "NULL weight table");
    const void *const *tabs[9] = {w->attn_norm, w->wq, w->wk, w->wv, w->wo, w->ffn_norm, w->w_gate, w->w_up, w->w_down};
    for (int t = 0; t < 9; ++t)
        for (int l = 0; l < cfg->n_layers; ++l)
            SCD_REQUIRE(tabs[t][l] && ((uintptr_t)tabs[t][l] & 15) == 0, SCD_ERR_ARG,
                        "weight table %d layer %d: NULL or not 16-byte aligned", t, l);
    SCD_REQUIRE((((uintptr_t)w->tok_emb | (uintptr_t)w->final_norm | (uintptr_t)w->lm_head) & 15) == 0,
                SCD_ERR_ARG, "weights must be 16-byte aligned");

    scd_model *m = new (std::nothrow) scd_model();
    SCD_REQUIRE(m, SCD_ERR_CUDA, "out of host memory");
    m->cfg = *cfg;
    m->rope_table = nullptr;
    m->gemm_plan = nullptr;
    cudaError_t e = cudaGetDevice(&m->device);
    if (e != cudaSuccess) { delete m; return cuda_fail(e, "cudaGetDevice"); }
    m->tok_emb = w->tok_emb; m->final_norm = w->final_norm; m->lm_head = w->lm_head;
    std::vector<const void *> *dst[9] = {&m->attn_norm, &m->wq, &m->wk, &m->wv, &m->wo, &m->ffn_norm,
                                         &m->w_gate, &m->w_up, &m->w_down};
    for (int t = 0; t < 9; ++t) dst[t]->assign(tabs[t], tabs[t] + cfg->n_layers);
    int rc = build_rope_table(m);
    if (rc == SCD_OK && cfg->dtype == SCD_BF16) rc = gemm_plan_create(m);
    if (rc != SCD_OK) { scd_free_model(m); return rc; }
    *out = m;
    return SCD_OK;
}

int scd_free_model(scd_model_t *m)
{
    if (!m) return SCD_OK;
    gemm_plan_destroy(m);
    if (m->rope_table) cudaFree(m->rope_table);
    delete m;
    return SCD_OK;
}

int scd_session_create(scd_model_t *m, const scd_decode_config_t *cfg, scd_session_t **out)
{
    SCD_REQUIRE(m && cfg && out, SCD_ERR_ARG, "scd_session_create: NULL argument");
    *out = nullptr;
    const scd_model_config_t &c = m->cfg;
    int rc = validate_decode_config(cfg, c.vocab_out);
    if (rc != SCD_OK) return rc;
    scd_session *s = new (std::nothrow) scd_session();
    SCD_REQUIRE(s, SCD_ERR_CUDA, "out of host memory");
    std::memset((void *)s, 0, sizeof(*s));
    s->model = m;
    s->cfg = *cfg;
    s->B = cfg->batch;
    s->S = cfg->cfg_lambda != 0.0f ? 2 : 1;
    s->Q = s->B * s->S;
    s->L = cfg->mode == SCD_MODE_AR ? 1 : cfg->window_L;
    s->cfg.window_L = s->L;
    s->att_t5_min_ctx = 512;
    // rows one forward may carry per stream-sequence: the window, or a prefill chunk
    s->chunk = std::max(s->L, std::max(1, std::min(128, 256 / s->Q)));
    s->rows_cap = s->Q * s->chunk;
    if (c.dtype == SCD_BF16 && s->rows_cap > 1024) {
        set_last_error("bf16 sessions carry at most 1024 rows per forward (S*B*L = %d)", s->Q * s->L);
        delete s;
        return SCD_ERR_CAPACITY;
    }
    s->pages_per_seq = (c.max_seq + c.kv_page_tokens - 1) / c.kv_page_tokens;
    const size_t es = elem_size(c.dtype);
    const int d = c.d_model, dq = c.n_heads * c.head_dim, dkv = c.n_kv_heads * c.head_dim, F = c.d_ffn, V = c.vocab_out;
    const size_t page_elems = (size_t)c.n_kv_heads * c.kv_page_tokens * c.head_dim;
    s->kv_kind_stride = (size_t)s->Q * s->pages_per_seq * page_elems;
    s->kv_layer_stride = 2 * s->kv_kind_stride;
    const size_t rows = (size_t)s->rows_cap, wrows = (size_t)s->B * s->L;

#define TRY_ALLOC(expr) do { rc = (expr); if (rc != SCD_OK) { free_session_memory(s); delete s; return rc; } } while (0)
    {
        char *p = nullptr;
        TRY_ALLOC(dev_alloc(&p, s->kv_layer_stride * c.n_layers * es));
        s->kv_pool = p;
    }
    TRY_ALLOC(dev_alloc(&s->page_table, (size_t)s->Q * s->pages_per_seq));
    TRY_ALLOC(dev_alloc(&s->n_known, s->B));
    TRY_ALLOC(dev_alloc(&s->n_total, s->B));
    TRY_ALLOC(dev_alloc(&s->shift, s->B));
    TRY_ALLOC(dev_alloc(&s->prev_lw, s->B));
    TRY_ALLOC(dev_alloc(&s->n_commit, s->B));
    TRY_ALLOC(dev_alloc(&s->iter, s->B));
    TRY_ALLOC(dev_alloc(&s->done_count, s->B));
    TRY_ALLOC(dev_alloc(&s->drafts, wrows));
    TRY_ALLOC(dev_alloc(&s->row_y, wrows));
    TRY_ALLOC(dev_alloc(&s->row_y_indep, 2 * wrows));
    TRY_ALLOC(dev_alloc(&s->accept_flags, wrows));
    TRY_ALLOC(dev_alloc(&s->tokens, (size_t)s->B * c.max_seq));
    TRY_ALLOC(dev_alloc(&s->tokens_u, (size_t)s->B * c.max_seq));
    TRY_ALLOC(dev_alloc(&s->ids_buf, rows));
    TRY_ALLOC(dev_alloc(&s->xbuf[0], wrows * V));
    TRY_ALLOC(dev_alloc(&s->xbuf[1], wrows * V));
    TRY_ALLOC(dev_alloc(&s->stats[0], wrows));
    TRY_ALLOC(dev_alloc(&s->stats[1], wrows));
    TRY_ALLOC(dev_alloc(&s->dev_stats, 1));
    TRY_ALLOC(dev_alloc(&s->finished, 2));
    TRY_ALLOC(dev_alloc(&s->h, rows * d));
    // bf16 sessions: GEMM inputs (xn, att, act) in two bf16 planes [2][rows][K], projections (qkv) in fp32
    const size_t wide = c.dtype == SCD_BF16 ? 2 : 1;
    { char *p; TRY_ALLOC(dev_alloc(&p, wide * rows * d * es)); s->xn = p; }
    { char *p; TRY_ALLOC(dev_alloc(&p, wide * rows * (dq + 2 * dkv) * es)); s->qkv = p; }
    { char *p; TRY_ALLOC(dev_alloc(&p, wide * rows * dq * es)); s->att = p; }
    { char *p; TRY_ALLOC(dev_alloc(&p, rows * 2 * F * es)); s->gu = p; }
    { char *p; TRY_ALLOC(dev_alloc(&p, wide * rows * F * es)); s->act = p; }
    s->ss_parts_cap = c.dtype == SCD_BF16 && m->gemm_plan ? gemm_norm_parts_cap(s) : 1;
    TRY_ALLOC(dev_alloc(&s->ss, (size_t)s->ss_parts_cap * rows));
    TRY_ALLOC(dev_alloc(&s->logits, (size_t)s->Q * s->L * V));
    s->host_pinned_ints = std::max<size_t>((size_t)s->Q * c.max_seq, 4096);
    {
        cudaError_t e = cudaMallocHost((void **)&s->host_pinned, s->host_pinned_ints * sizeof(int));
        if (e != cudaSuccess) { free_session_memory(s); delete s; return cuda_fail(e, "cudaMallocHost"); }
    }
    if (c.dtype == SCD_BF16 && m->gemm_plan) {
        TRY_ALLOC(gemm_session_prepare(s));
        TRY_ALLOC(attention_session_prepare(s));
    }
#undef TRY_ALLOC
    const int np = s->Q * s->pages_per_seq;
    identity_pages_kernel<<<(np + 255) / 256, 256>>>(s->page_table, np);
    cudaMemset(s->done_count, 0, s->B * sizeof(unsigned));
    cudaMemset(s->dev_stats, 0, sizeof(VerifyStatsDev));
    cudaMemset(s->kv_pool, 0, s->kv_layer_stride * c.n_layers * es);
    cudaMemset(s->logits, 0, (size_t)s->Q * s->L * V * sizeof(float));
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { free_session_memory(s); delete s; return cuda_fail(e, "session init"); }
    *out = s;
    return SCD_OK;
}

int scd_session_free(scd_session_t *s)
{
    if (!s) return SCD_OK;
    cudaDeviceSynchronize();
    free_session_memory(s);
    delete s;
    return SCD_OK;
}

int scd_prefill(scd_session_t *s, const int32_t *prompt_ids, int32_t P, int32_t n_new, void *stream)
{
    SCD_REQUIRE(s && prompt_ids, SCD_ERR_ARG, "scd_prefill: NULL argument");
    SCD_REQUIRE(P >= 1 && n_new >= 0, SCD_ERR_ARG, "scd_prefill: P %d, n_new %d", P, n_new);
    const scd_model_config_t &c = s->model->cfg;
    SCD_REQUIRE((long long)P + n_new <= c.max_seq, SCD_ERR_CAPACITY,
                "P + n_new = %lld exceeds max_seq %d", (long long)P + n_new, c.max_seq);
    for (long long i = 0; i < (long long)s->Q * P; ++i)
        SCD_REQUIRE(prompt_ids[i] >= 0 && prompt_ids[i] < c.vocab_in, SCD_ERR_ARG,
                    "prompt id %d outside [0, %d)", prompt_ids[i], c.vocab_in);
    cudaStream_t st = (cudaStream_t)stream;
    s->prompt_len = P;
    s->n_new = n_new;
    s->prefilled = false;
    drop_step_graph(s);                                  // the prompt length is baked into the captured launches
    if (s->gemm_ws) SCD_CUDA_TRY(cudaMemsetAsync(s->gemm_ws, 0, s->gemm_ws_bytes, st));   // a fresh start clears the error word
    // token records: conditional prompts -> tokens, unconditional prompts -> tokens_u
    std::memcpy(s->host_pinned, prompt_ids, (size_t)s->Q * P * sizeof(int));
    SCD_CUDA_TRY(cudaMemcpy2DAsync(s->tokens, (size_t)c.max_seq * sizeof(int), s->host_pinned,
                                   (size_t)P * sizeof(int), (size_t)P * sizeof(int), s->B,
                                   cudaMemcpyHostToDevice, st));
    if (s->S == 2)
        SCD_CUDA_TRY(cudaMemcpy2DAsync(s->tokens_u, (size_t)c.max_seq * sizeof(int),
                                       s->host_pinned + (size_t)s->B * P, (size_t)P * sizeof(int),
                                       (size_t)P * sizeof(int), s->B, cudaMemcpyHostToDevice, st));
    // chunks of the prompt (all but its last token) through the forward, no logits; the kernels read the
    // prompt from the token records just copied, so the chunks are enqueued back to back
    for (int p0 = 0; p0 < P - 1; p0 += s->chunk) {
        const int len = std::min(s->chunk, P - 1 - p0);
        ForwardArgs a;
        a.ids = nullptr; a.Mq = len; a.pos_override = p0; a.want_logits = false; a.skip = nullptr;
        a.logits = nullptr; a.hidden = nullptr; a.prof = nullptr; a.lm_lo = 0; a.lm_hi = 0; a.lm_eol = -1;
        int rc = run_forward(s, a, st);
        if (rc != SCD_OK) return rc;
    }
    set_state_kernel<<<(s->B + 63) / 64, 64, 0, st>>>(s->n_known, s->n_total, s->B, P, P + n_new);
    SCD_CUDA_TRY(cudaMemsetAsync(s->dev_stats, 0, sizeof(VerifyStatsDev), st));
    SCD_CUDA_TRY(cudaMemsetAsync(s->finished, 0, 2 * sizeof(int), st));
    VerifyParams p;
    session_verify_params(s, p);
    int rc = launch_init_window(p, st);
    if (rc != SCD_OK) return rc;
    SCD_CUDA_TRY(cudaStreamSynchronize(st));
    rc = check_device_health(s, st);
    if (rc != SCD_OK) return rc;
    s->ctx_floor = (long long)P - 1;                   // kv_len after the prefill
    s->att_variant = 0;
    s->prefilled = true;
    return SCD_OK;
}

int scd_step(scd_session_t *s, void *stream)
{
    SCD_REQUIRE(s, SCD_ERR_ARG, "scd_step: NULL session");
    SCD_REQUIRE(s->prefilled, SCD_ERR_STATE, "scd_step before scd_prefill");
    return launch_step(s, (cudaStream_t)stream);
}

int scd_session_attention_min_ctx(scd_session_t *s, int64_t min_ctx)
{
    SCD_REQUIRE(s, SCD_ERR_ARG, "scd_session_attention_min_ctx: NULL session");
    s->att_t5_min_ctx = (long long)min_ctx;
    return SCD_OK;
}

int scd_step_profile(scd_session_t *s, float *ms_by_class, int32_t *launches_by_class, void *stream)
{
    SCD_REQUIRE(s && ms_by_class && launches_by_class, SCD_ERR_ARG, "scd_step_profile: NULL argument");
    SCD_REQUIRE(s->prefilled, SCD_ERR_STATE, "scd_step_profile before scd_prefill");
    StepProfiler prof;
    prof.st = (cudaStream_t)stream;
    int rc = enqueue_step(s, prof.st, &prof);
    s->ctx_floor += 1;
    if (rc != SCD_OK) return rc;
    return prof.finish(ms_by_class, launches_by_class);
}

int scd_autotune(scd_session_t *s, int32_t *k_splits_out, void *stream)
{
    SCD_REQUIRE(s, SCD_ERR_ARG, "scd_autotune: NULL session");
    SCD_REQUIRE(s->prefilled, SCD_ERR_STATE, "scd_autotune before scd_prefill");
    const scd_model_config_t &c = s->model->cfg;
    if (k_splits_out) for (int k = 0; k < 4; ++k) k_splits_out[k] = 0;
    if (c.dtype != SCD_BF16 || !s->model->gemm_plan) return SCD_OK;      // nothing to tune on the fp32 path
    cudaStream_t st = (cudaStream_t)stream;
    drop_step_graph(s);                                  // the captured launches carry the old shapes
    ForwardArgs a;
    a.ids = nullptr; a.Mq = s->L; a.pos_override = -1; a.want_logits = true;
    a.logits = s->logits; a.hidden = nullptr; a.prof = nullptr; a.skip = nullptr;
    a.lm_lo = s->cfg.allowed_lo; a.lm_hi = s->cfg.allowed_hi;
    a.lm_eol = s->cfg.row_period > 0 ? s->cfg.eol_id : -1;
    cudaEvent_t e0, e1;
    SCD_CUDA_TRY(cudaEventCreate(&e0));
    SCD_CUDA_TRY(cudaEventCreate(&e1));
    int rc = SCD_OK;
    // device time of one window forward (no verify, no commit: the session state does not move)
    auto forward_ms = [&](float *best) -> int {
        *best = 1e30f;
        for (int rep = 0; rep < 4; ++rep) {              // the first repetition warms up
            if (cudaEventRecord(e0, st) != cudaSuccess) return SCD_ERR_CUDA;
            const int r = run_forward(s, a, st);
            if (r != SCD_OK) return r;
            if (cudaEventRecord(e1, st) != cudaSuccess || cudaEventSynchronize(e1) != cudaSuccess) return SCD_ERR_CUDA;
            float ms = 0.f;
            if (cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) return SCD_ERR_CUDA;
            if (rep > 0 && ms < *best) *best = ms;
        }
        return SCD_OK;
    };
    const int kinds[4] = {GEMM_QKV, GEMM_O, GEMM_GATE_UP, GEMM_DOWN};
    const int kblocks[4] = {c.d_model / 64, c.n_heads * c.head_dim / 64, c.d_model / 64, c.d_ffn / 64};
    for (int k = 0; k < 4 && rc == SCD_OK; ++k) {
        float best_ms = 0.f;
        int best = 0;                                    // 0: the built-in rule
        gemm_set_kind_splits(s->model, kinds[k], 0);
        rc = forward_ms(&best_ms);
        for (int C = 1; C <= 8 && rc == SCD_OK; ++C) {
            if (C > 1 && kblocks[k] / C < 2) break;
            gemm_set_kind_splits(s->model, kinds[k], C);
            float ms = 0.f;
            rc = forward_ms(&ms);
            if (rc == SCD_OK && ms < best_ms * 0.995f) { best_ms = ms; best = C; }   // (a tie keeps the rule)
        }
        gemm_set_kind_splits(s->model, kinds[k], rc == SCD_OK ? best : 0);
        if (k_splits_out) k_splits_out[k] = best;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (rc != SCD_OK) return rc;
    return check_device_health(s, st);
}

int scd_step_timeline(scd_session_t *s, float *ms_by_class, int32_t *launches_by_class, void *stream)
{
    SCD_REQUIRE(s && ms_by_class && launches_by_class, SCD_ERR_ARG, "scd_step_timeline: NULL argument");
    SCD_REQUIRE(s->prefilled, SCD_ERR_STATE, "scd_step_timeline before scd_prefill");
    const size_t launches = (size_t)s->model->cfg.n_layers * 8 + 16;
    const size_t bytes = launches * 2 * STAMP_CTAS * sizeof(unsigned long long);
    if (!s->stamps) SCD_CUDA_TRY(cudaMalloc(&s->stamps, bytes));
    cudaStream_t st = (cudaStream_t)stream;
    SCD_CUDA_TRY(cudaMemsetAsync(s->stamps, 0, bytes, st));
    SCD_CUDA_TRY(cudaStreamSynchronize(st));           // the memset must not sit between two kernels
    StepProfiler prof;
    prof.st = st;
    prof.stamps = (unsigned long long *)s->stamps;
    prof.stamp_launches = launches;
    int rc = enqueue_step(s, st, &prof);
    s->ctx_floor += 1;
    take_stamp_slot();
    if (rc != SCD_OK) return rc;
    return prof.finish(ms_by_class, launches_by_class);
}

int64_t scd_kernel_launches(void) { return (int64_t)g_launches.load(std::memory_order_relaxed); }

int scd_step_result(scd_session_t *s, int32_t *n_committed, int32_t *n_known, int32_t *kv_len, void *stream)
{
    SCD_REQUIRE(s, SCD_ERR_ARG, "scd_step_result: NULL session");
    SCD_REQUIRE(s->prefilled, SCD_ERR_STATE, "scd_step_result before scd_prefill");
    cudaStream_t st = (cudaStream_t)stream;
    int *hp = s->host_pinned;
    SCD_CUDA_TRY(cudaMemcpyAsync(hp, s->n_commit, s->B * sizeof(int), cudaMemcpyDeviceToHost, st));
    SCD_CUDA_TRY(cudaMemcpyAsync(hp + s->B, s->n_known, s->B * sizeof(int), cudaMemcpyDeviceToHost, st));
    SCD_CUDA_TRY(cudaStreamSynchronize(st));
    int rc = check_device_health(s, st);
    if (rc != SCD_OK) return rc;
    for (int b = 0; b < s->B; ++b) {
        if (n_committed) n_committed[b] = hp[b];
        if (n_known) n_known[b] = hp[s->B + b];
        if (kv_len) kv_len[b] = hp[s->B + b] - 1;
    }
    return SCD_OK;
}

int scd_read_tokens(scd_session_t *s, int32_t first, int32_t count, int32_t *out, void *stream)
{
    SCD_REQUIRE(s && out, SCD_ERR_ARG, "scd_read_tokens: NULL argument");
    const int max_seq = s->model->cfg.max_seq;
    SCD_REQUIRE(first >= 0 && count >= 0 && (long long)first + count <= max_seq, SCD_ERR_ARG,
                "token range [%d, %d) outside [0, %d)", first, first + count, max_seq);
    if (count == 0) return SCD_OK;
    cudaStream_t st = (cudaStream_t)stream;
    SCD_CUDA_TRY(cudaMemcpy2DAsync(s->host_pinned, (size_t)count * sizeof(int), s->tokens + first,
                                   (size_t)max_seq * sizeof(int), (size_t)count * sizeof(int), s->B,
                                   cudaMemcpyDeviceToHost, st));
    SCD_CUDA_TRY(cudaStreamSynchronize(st));
    std::memcpy(out, s->host_pinned, (size_t)s->B * count * sizeof(int));
    return SCD_OK;
}

int scd_generate(scd_session_t *s, int32_t *out_tokens, scd_stats_t *stats, void *stream)
{
    SCD_REQUIRE(s && out_tokens, SCD_ERR_ARG, "scd_generate: NULL argument");
    SCD_REQUIRE(s->prefilled, SCD_ERR_STATE, "scd_generate before scd_prefill");
    cudaStream_t st = (cudaStream_t)stream;
    cudaEvent_t e0, e1;
    SCD_CUDA_TRY(cudaEventCreate(&e0));
    SCD_CUDA_TRY(cudaEventCreate(&e1));
    SCD_CUDA_TRY(cudaEventRecord(e0, st));
    const int total = s->prompt_len + s->n_new;
    int *hp = s->host_pinned;
    int rc = SCD_OK;
    long long launched = 0;
    for (;;) {
        // Every iteration commits between 1 and L tokens per unfinished sequence: `remaining` iterations
        // always suffice and ceil(remaining / L) are always needed. Iterations are enqueued in blocks of
        // up to GENERATE_BLOCK without a host round trip; the host looks at the counters once per block.
        // An iteration that runs after the last token costs only its (empty) launches: the verify kernel
        // raises a device flag when every sequence is complete and the forward kernels return on it.
        SCD_CUDA_TRY(cudaMemcpyAsync(hp, s->n_known, s->B * sizeof(int), cudaMemcpyDeviceToHost, st));
        SCD_CUDA_TRY(cudaStreamSynchronize(st));
        int remaining = 0;
        for (int b = 0; b < s->B; ++b) remaining = std::max(remaining, total - hp[b]);
        if (remaining <= 0) break;
        const int steps = std::max((remaining + s->L - 1) / s->L, std::min(remaining, GENERATE_BLOCK));
        launched += steps;
        if (launched > (long long)s->n_new + 8 + GENERATE_BLOCK) {      // each live iteration commits >= 1 token
            set_last_error("scd_generate: no progress after %lld iterations", launched);
            rc = SCD_ERR_TIMEOUT;
            break;
        }
        for (int i = 0; i < steps && rc == SCD_OK; ++i) rc = launch_step(s, st);
        if (rc != SCD_OK) break;
    }
    cudaEventRecord(e1, st);
    cudaEventSynchronize(e1);
    float ms = 0.f;
    cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (rc != SCD_OK) return rc;
    rc = check_device_health(s, st);
    if (rc != SCD_OK) return rc;
    rc = scd_read_tokens(s, s->prompt_len, s->n_new, out_tokens, stream);
    if (rc != SCD_OK) return rc;
    if (stats) {
        VerifyStatsDev hs;
        SCD_CUDA_TRY(cudaMemcpy(&hs, s->dev_stats, sizeof(hs), cudaMemcpyDeviceToHost));
        stats->forwards = (int64_t)hs.forwards;
        stats->committed = (int64_t)hs.committed;
        for (int i = 0; i < 257; ++i) stats->accept_hist[i] = (int64_t)hs.accept_hist[i];
        stats->elapsed_ms = ms;
    }
    return SCD_OK;
}

int scd_forward_window(scd_session_t *s, const int32_t *ids, int32_t M, float *logits, float *hidden,
                       int32_t commit, void *stream)
{
    SCD_REQUIRE(s && ids && logits, SCD_ERR_ARG, "scd_forward_window: NULL argument");
    SCD_REQUIRE(s->prefilled, SCD_ERR_STATE, "scd_forward_window before scd_prefill");
    SCD_REQUIRE(M >= 1 && M <= s->chunk, SCD_ERR_CAPACITY, "M %d outside 1..%d", M, s->chunk);
    cudaStream_t st = (cudaStream_t)stream;
    ForwardArgs a;
    a.ids = ids; a.Mq = M; a.pos_override = -1; a.want_logits = true; a.logits = logits; a.hidden = hidden;
    a.prof = nullptr; a.skip = nullptr; a.lm_lo = 0; a.lm_hi = 0; a.lm_eol = -1;
    int rc = run_forward(s, a, st);
    if (rc != SCD_OK) return rc;
    if (commit) {
        commit_ids_kernel<<<s->B, 64, 0, st>>>(ids, M, s->B, s->n_known, s->tokens, s->model->cfg.max_seq);
        SCD_CUDA_TRY(cudaGetLastError());
    }
    return SCD_OK;
}

int scd_debug_read(scd_session_t *s, int32_t what, void *out, int64_t bytes, void *stream)
{
    SCD_REQUIRE(s && out, SCD_ERR_ARG, "scd_debug_read: NULL argument");
    const void *src = nullptr;
    int64_t want = 0;
    if (what == 0) { src = s->logits; want = (int64_t)s->Q * s->L * s->model->cfg.vocab_out * 4; }
    else if (what == 1) { src = s->drafts; want = (int64_t)s->B * s->L * 4; }
    SCD_REQUIRE(src, SCD_ERR_ARG, "scd_debug_read: unknown item %d", what);
    SCD_REQUIRE(bytes == want, SCD_ERR_ARG, "scd_debug_read: %lld bytes given, %lld needed",
                (long long)bytes, (long long)want);
    cudaStream_t st = (cudaStream_t)stream;
    SCD_CUDA_TRY(cudaMemcpyAsync(out, src, (size_t)bytes, cudaMemcpyDeviceToHost, st));
    SCD_CUDA_TRY(cudaStreamSynchronize(st));
    return SCD_OK;
}

}  // extern "C"
