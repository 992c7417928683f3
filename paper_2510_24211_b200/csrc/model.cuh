// Host-side model / session objects and the launch interface of the window-forward kernels.
#pragma once
#include <vector>

#include "common.cuh"
#include "verify.cuh"

struct scd_model {
    scd_model_config_t cfg;
    int device;
    const void *tok_emb, *final_norm, *lm_head;
    std::vector<const void *> attn_norm, wq, wk, wv, wo, ffn_norm, w_gate, w_up, w_down;
    float2 *rope_table;       // [max_seq][head_dim/2] (cos, sin), built in fp64 on the device
    void *gemm_plan;          // tcgen05 GEMM descriptors of the weight matrices (bf16 models)
};

struct scd_session {
    scd_model *model;
    scd_decode_config_t cfg;
    int B, S, Q, L;           // sequences, streams per sequence, stream-sequences, window rows
    int chunk;                // rows per stream-sequence that one forward may carry
    int rows_cap;             // Q * chunk
    int pages_per_seq;
    int prompt_len, n_new;
    bool prefilled;

    // KV cache: pool[layer][K|V][physical page][kv head][token in page][head_dim]
    void *kv_pool;
    int *page_table;          // [Q][pages_per_seq] -> physical page
    size_t kv_layer_stride;   // elements between layers (covers K and V)
    size_t kv_kind_stride;    // elements between the K and the V pool of a layer

    // window state (device)
    int *n_known, *n_total, *shift, *prev_lw, *drafts, *n_commit, *tokens, *tokens_u;
    int *row_y, *row_y_indep, *ids_buf;
    unsigned *iter, *done_count;
    unsigned char *accept_flags;
    float *xbuf[2];
    scd::RowStats *stats[2];
    scd::VerifyStatsDev *dev_stats;
    int *finished;            // device: [0] finished sequences, [1] all finished (see VerifyParams::finished)
    const int *skip_now;      // what the forward being enqueued hands its kernels as skip flag (NULL or finished + 1)

    // activations (device)
    float *h;                 // residual stream [rows][d]
    void *xn, *qkv, *att, *gu, *act;
    float *ss;                // bf16 sessions: partial sums of squares of h, [ss_parts_cap][rows_cap]
    int ss_parts_cap;
    float *logits;            // [rows_cap_logits][V]
    long long ctx_floor;      // host-side floor of the committed context of every live sequence (P - 1 + iterations)
    int att_variant;          // attention variant the captured iteration was built with
    long long att_t5_min_ctx; // known context from which the tcgen05 attention kernel is used (< 0: never)
    void *stamps;             // device time stamps of scd_step_timeline (allocated on first use)
    void *gemm_ws;            // device error word of the tcgen05 GEMM
    size_t gemm_ws_bytes;
    void *gemm_state;         // activation-side tensor maps
    void *attn_plan;          // tensor map of the KV pool for the tensor-core attention (bf16 sessions)

    int *host_pinned;         // staging for prompt ids and counters
    size_t host_pinned_ints;
    cudaGraphExec_t step_graph;   // one iteration as a CUDA graph (captured on the first step after a prefill)
    long long step_graph_nodes;   // kernels in it
    bool step_graph_off;          // capture failed once: stay on plain launches
};

namespace scd {

// Kernel classes of one iteration, for the per-class device timing of scd_step_profile.
enum { PROF_EMBED = 0, PROF_RMSNORM, PROF_GEMM_QKV, PROF_ROPE_KV, PROF_ATTENTION, PROF_GEMM_O,
       PROF_GEMM_GATE_UP, PROF_GEMM_DOWN, PROF_GEMM_LM_HEAD, PROF_VERIFY, PROF_OTHER, PROF_CLASSES };

// Records one CUDA event in front of every kernel of a step; the time between two consecutive
// events is charged to the class of the kernel launched between them.
// Two ways to split an iteration's device time over the kernel classes:
//  - events: a CUDA event in front of every kernel (switches the programmatic overlap between
//    neighbouring kernels off: each launch is timed on its own);
//  - stamps: the GEMM and attention kernels write %globaltimer at CTA entry and exit into `stamps`
//    ([launch][2][STAMP_CTAS]); nothing else changes, so the kernels overlap as in production. The
//    time from the end of the previous stamped kernel to the end of kernel i is charged to i's class.
constexpr int STAMP_CTAS = 512;      // CTAs per launch that leave a stamp (grids here are <= 444)
struct StepProfiler {
    std::vector<cudaEvent_t> events;
    std::vector<int> cls;
    size_t used = 0;
    cudaStream_t st = nullptr;
    bool failed = false;
    unsigned long long *stamps = nullptr;              // device buffer: stamp mode
    size_t stamp_launches = 0;                         // launches it has room for
    void mark(int c);                                  // call right before launching a kernel of class c
    int finish(float *ms_by_class, int *launches_by_class);   // sync, accumulate; blocking
    ~StepProfiler();
};
// The slot of the launch that mark() announced (stamp mode), handed to the next GEMM / attention
// launch of this thread; nullptr otherwise.
unsigned long long *take_stamp_slot();

struct ForwardArgs {
    const int *ids;           // explicit input ids [Q][Mq] (device) or NULL: window inputs from state, or - with
                              // pos_override >= 0 - the recorded tokens at positions pos_override .. + Mq - 1 (prefill)
    const int *skip;          // device flag: the kernels return at once when it is set (NULL: never)
    int Mq;                   // rows per stream-sequence
    int pos_override;         // >= 0: position of row 0 for every stream-sequence; < 0: n_known - 1
    bool want_logits;
    float *logits;            // [Q*Mq][V]
    float *hidden;            // optional [Q*Mq][d] copy of the final residual stream
    StepProfiler *prof;       // optional per-kernel event marks
    int lm_lo, lm_hi, lm_eol; // logits wanted: ids [lm_lo, lm_hi) and, if >= 0, id lm_eol (lm_hi <= 0: all)
};

int run_forward(scd_session *s, const ForwardArgs &a, cudaStream_t st);
int build_rope_table(scd_model *m);

// tcgen05 GEMM plan (bf16 models); implemented in gemm_tcgen05.cu
int gemm_plan_create(scd_model *m);
void gemm_plan_destroy(scd_model *m);

int validate_decode_config(const scd_decode_config_t *cfg, int V);
void fill_verify_params(VerifyParams &p, const scd_decode_config_t *cfg, int V);

}  // namespace scd
