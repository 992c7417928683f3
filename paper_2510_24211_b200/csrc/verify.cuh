// Parameters of the fused verify-and-redraft kernel (shared by the stand-alone entry point and
// the in-session step).
#pragma once
#include "common.cuh"

namespace scd {

struct RowStats {          // one post-processed distribution: p(v) = W_v / Z,
    float m;               //   W_v = [x_v >= tau] * trunc(scd_exp(x_v - m) * 2^30)
    float tau;
    unsigned long long Z;  //   ... and, with top-p, W_v = 0 below the nucleus threshold theta
    unsigned theta;
    unsigned pad_;
};

struct VerifyStatsDev {    // device-resident counters of a session
    unsigned long long forwards;
    unsigned long long committed;
    unsigned long long accept_hist[257];
};

struct VerifyParams {
    int mode;              // SCD_MODE_*
    float alpha;           // SCD_MODE_ALPHA: probability of keeping the coupled redraft (Algorithm 5)
    int B, L, V, S;
    float temperature, lam, one_plus_lam;
    int top_k;
    unsigned top_p24;      // trunc(top_p * 2^24 + 1/2); 0: no nucleus truncation
    unsigned long long seed;
    int allowed_lo, allowed_hi, row_period, eol_id;

    // target logits of this iteration: row (s, b, k) at p_logits + ((s*B + b)*L + k) * V
    const float *p_logits;

    // integer weights W (uint32 in the float-typed cells) of the window rows' target distributions,
    // two buffers [B][L][V] used in ping-pong by iteration parity: this iteration writes
    // xbuf[t & 1] and reads the drafts' distributions from xbuf[(t & 1) ^ 1]. Stand-alone use:
    // xbuf[0] = scratch (rows that do not fit in shared memory), xbuf[1] = raw draft logits.
    float *xbuf[2];
    RowStats *stats[2];    // [B][L] each; stats of xbuf[i] rows
    int keep_x;            // 1: write the target row's weights to xbuf[t & 1] (the next iteration reads them)
    int q_is_raw;          // 1: xbuf[1] holds raw draft logits whose stats must be computed here
    int q_present;         // stand-alone: 0 = every row fresh

    // window state, per sequence
    const long long *positions;   // stand-alone: position of row 0            (or NULL)
    int *n_known;                 // session: n[b] = prompt + committed tokens  (or NULL)
    const int *n_total;           // session: final length                      (or NULL)
    int prompt_len;               // generated position g = position - prompt_len
    unsigned int *iter;           // session: t[b] (updated here)               (or NULL)
    long long iteration;          // stand-alone t
    int *shift;                   // session: tokens committed by the previous iteration
    int *prev_lw;                 // session: live rows of the previous iteration (0: all fresh)

    const int *draft_in;          // [B][L]
    int *draft_out;               // [B][L] (may alias draft_in)
    int *n_commit;                // [B] out: a
    int *committed_ids;           // stand-alone [B][L] out                      (or NULL)
    int *tokens;                  // session: token record [B][token_stride]     (or NULL)
    int token_stride;
    unsigned char *accept_flags;  // [B][L] out (k_j of every row)
    int *row_y;                   // [B][L] scratch: per-row output token Y_j
    int *row_y_indep;             // [2][B][L] scratch: redraft beyond the prefix (SJD, alpha, Gumbel); fresh rows (Gumbel)
    unsigned int *done_count;     // [B] scratch, zero on entry, zero again on exit
    VerifyStatsDev *dev_stats;    // session counters (or NULL)
    int *finished;                // session: [0] sequences that reached their final length, [1] = 1 once all B have
                                  // (the forward kernels of an iteration enqueued after that return at once)   (or NULL)
};

// ---- device helpers shared by the two verify kernels -----------------------------------------------
// ids a position may take: the allowed range, or the single end-of-row id at forced positions
__device__ __forceinline__ void allowed_range(const VerifyParams &p, long long pos, int &lo, int &hi)
{
    const long long g = pos - p.prompt_len;
    if (p.row_period > 0 && g >= 0 && (g % p.row_period) == p.row_period - 1) {
        lo = p.eol_id; hi = p.eol_id + 1;
    } else {
        lo = p.allowed_lo; hi = p.allowed_hi;
    }
}

// w * z for a 32-bit weight and a 64-bit normaliser as a 128-bit value, from two 32 x 32 -> 64
// products (the general 128-bit multiply costs several times more).
__device__ __forceinline__ u128 mul_32x64(unsigned w, unsigned long long z)
{
    const unsigned long long p0 = (unsigned long long)w * (unsigned)z;
    const unsigned long long p1 = (unsigned long long)w * (unsigned)(z >> 32);
    const unsigned long long lo = p0 + (p1 << 32);
    const unsigned long long hi = (p1 >> 32) + (lo < p0 ? 1ull : 0ull);
    return ((u128)hi << 64) | lo;
}

// Draft of a row that enters the window: X ~ uniform over the allowed ids of its position
// (the initialisation of Algorithm 6: "p <- Random(); X ~ p").
__device__ __forceinline__ int fresh_draft(const VerifyParams &p, int b, long long pos, unsigned first_iter)
{
    int lo, hi;
    allowed_range(p, pos, lo, hi);
    const unsigned U = noise_u24(p.seed, NOISE_INIT, (unsigned)b, pos, first_iter, 0);
    return lo + (int)(((unsigned long long)U * (unsigned long long)(hi - lo)) >> 24);
}

// Window of one sequence at this iteration (session: device-resident counters; stand-alone: arguments)
struct WindowState {
    long long pos0;
    int Lw, shift, prev_lw, parity;
    unsigned t;
};

__device__ __forceinline__ WindowState load_state(const VerifyParams &p, int b)
{
    WindowState w;
    if (p.n_known) {
        const int n = p.n_known[b];
        w.pos0 = n;
        w.Lw = max(0, min(p.L, p.n_total[b] - n));
        w.t = p.iter[b];
        w.parity = (int)(w.t & 1u);
        w.shift = p.shift[b];
        w.prev_lw = p.prev_lw[b];
    } else {
        w.pos0 = p.positions[b];
        w.Lw = p.L;
        w.t = (unsigned)p.iteration;
        w.parity = 0;
        w.shift = 0;
        w.prev_lw = p.q_present ? p.L : 0;
    }
    if (p.mode == SCD_MODE_AR) w.Lw = min(w.Lw, 1);
    return w;
}

int launch_verify(const VerifyParams &p, cudaStream_t stream);
// the kernel that gives every window row a thread-block cluster (verify_cluster.cu)
bool verify_cluster_supported(const VerifyParams &p);
int launch_verify_cluster(const VerifyParams &p, cudaStream_t stream);
int launch_init_window(const VerifyParams &p, cudaStream_t stream);

}  // namespace scd
