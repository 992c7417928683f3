/*
 * CPU oracle for Speculative Coupled Decoding (SCD), Speculative Jacobi Decoding (SJD) and
 * vanilla autoregressive (AR) sampling.
 *
 * THIS FILE IS TEST INFRASTRUCTURE. It is a plain, slow, single-purpose restatement of the
 * algorithms of the paper, used only to check the CUDA library and to serve as a timed CPU
 * baseline. It shares no code with the CUDA library and must never be called by it.
 *
 * What follows the paper:
 *   - Modified Rejection Sampling, Algorithm 1 (accept rule u <= min(1, P(X)/Q(X)), residual
 *     norm(max(0, P - Q))).
 *   - Speculative Jacobi Decoding, Algorithm 2 (independent redraft, sequential verify).
 *   - SCD with the maximal coupling, Algorithm 3 (its "Maximal Coupling" branch) / Algorithm 6 (vectorised MRS over the
 *     whole window, first rejection index, i <- Accept + 1).
 *   - Gumbel-sharing coupling, Algorithm 4, and its use in Algorithm 7.
 *   - alpha-coupling, Algorithm 5 (Bernoulli mixture of a coupling and the independent one).
 *   - Logit post-processing (Sec. 4.3 "Implementation Details", Sec. 5.1 "Effect on CFG"):
 *     classifier-free-guidance mix (1+lambda)*c - lambda*u, temperature, top-k.
 *
 * What the paper leaves open and is fixed here (the same conventions are restated,
 * independently, by the CUDA library so that both can be compared bit for bit):
 *   - noise: Philox4x32-10 (Salmon et al., SC'11), key = 64-bit seed,
 *     counter = (sub-index, position, iteration, stream-id | batch << 8); the top 24 bits of
 *     output word 0 are the uniform variate.
 *   - a distribution is a vector of integer weights W_v = trunc(scd_exp(x_v - max x) * 2^30)
 *     with normaliser Z = sum W_v; p(v) = W_v / Z exactly. All tests (accept, residual,
 *     inverse CDF) are integer inequalities on 128-bit products, hence independent of the
 *     order in which a parallel implementation sums.
 *   - scd_exp is a fixed sequence of correctly rounded fp32 operations (below).
 *   - the Gumbel race of Algorithm 4 compares E_v / W_v with E_v = -log2 u_v in fixed point
 *     (40 fraction bits from the digit-by-digit squaring recurrence, stated below) by 128-bit
 *     cross-multiplication: an integer decision, so the argmax does not depend on a library's
 *     logarithm or on the order of a parallel reduction. Ties go to the smaller id.
 *
 * Floating point: the sampling core follows the fp32 sequence stated above (it decides
 * integers, so both sides must take the same steps). The transformer forward keeps values in
 * fp32 and accumulates every dot product, norm and softmax in fp64.
 *
 * Parity pins (tests/, -m "not gpu"): Philox known-answer vectors; MRS marginal = p,
 * acceptance = 1 - TV, residual = norm(max(0,p-q)) by exact counting over all 2^24 noise
 * values; coupling costs by brute-force enumeration on V <= 8; chi-square losslessness of the
 * AR / SJD / SCD loops against the exact AR joint; greedy and L = 1 degenerate cases; the
 * forward against PyTorch CPU ops and against token-by-token evaluation. The exact token
 * values of a full generation are "parity unpinned" against the paper (it prints no worked
 * example); they are pinned only between this oracle and the CUDA library.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef unsigned __int128 u128;

/* ------------------------------------------------------------------------------------------
 * Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3").
 * ---------------------------------------------------------------------------------------- */
void oracle_philox4x32_10(const uint32_t key[2], const uint32_t ctr[4], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Noise streams. */
enum { NOISE_ACCEPT = 1, NOISE_RESIDUAL = 2, NOISE_INIT = 3, NOISE_INDEP = 4, NOISE_ALPHA = 5,
       NOISE_GUMBEL = 6 };

/* 24-bit uniform integer keyed by (seed, stream, batch, position, iteration, sub). */
uint32_t oracle_noise_u24(uint64_t seed, uint32_t stream, uint32_t batch, uint64_t position,
                          uint32_t iteration, uint32_t sub)
{
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t ctr[4] = { sub, (uint32_t)position, iteration, stream | (batch << 8) };
    uint32_t out[4];
    oracle_philox4x32_10(key, ctr, out);
    return out[0] >> 8;
}

/* ------------------------------------------------------------------------------------------
 * scd_exp: e^x for x <= 0 as a fixed sequence of fp32 operations.
 *   x < -22            -> 0   (e^-22 * 2^30 < 1, the weight truncates to 0 anyway)
 *   n = rint(x * log2e); r = x - n*ln2 (two fused steps, hi/lo split)
 *   e^r by the degree-6 Taylor polynomial in Horner form with fused multiply-adds
 *   result = poly * 2^n
 * Compiled with -ffp-contract=off so that only the explicit fmaf calls fuse.
 * ---------------------------------------------------------------------------------------- */
float oracle_scd_exp(float x)
{
    if (!(x >= -22.0f)) return 0.0f;
    if (x > 0.0f) x = 0.0f;
    float t = x * 0x1.715476p+0f;
    float n = rintf(t);
    float r = fmaf(n, -0x1.62e400p-1f, x);
    r = fmaf(n, -0x1.7f7d1cp-20f, r);
    float p = 0x1.6c16c2p-10f;
    p = fmaf(p, r, 0x1.111112p-7f);
    p = fmaf(p, r, 0x1.555556p-5f);
    p = fmaf(p, r, 0x1.555556p-3f);
    p = fmaf(p, r, 0.5f);
    p = fmaf(p, r, 1.0f);
    p = fmaf(p, r, 1.0f);
    int32_t e = (int32_t)n + 127;
    uint32_t bits = (uint32_t)e << 23;
    float scale;
    memcpy(&scale, &bits, 4);
    return p * scale;
}

/* ------------------------------------------------------------------------------------------
 * Logit post-processing: allowed-id range -> CFG mix -> temperature -> top-k (threshold form,
 * ties kept) -> integer weights. "p^(t) is the final distribution after all logit
 * post-processing (top-k, CFG)" (Sec. 4.3); CFG mix (1+lambda)*c - lambda*u (Sec. 5.1).
 *   c, u    : conditional / unconditional logits [V]; u may be NULL when lam == 0
 *   lo, hi  : allowed ids are lo <= v < hi
 *   x_out   : optional [V], the post-processed logits (ids outside the range get -inf)
 *   W       : [V] integer weights, 0 outside the kept set
 * returns the number of kept ids.
 * ---------------------------------------------------------------------------------------- */
static int cmp_float_desc(const void *a, const void *b)
{
    float fa = *(const float *)a, fb = *(const float *)b;
    return (fa < fb) - (fa > fb);
}

int oracle_postprocess(const float *c, const float *u, int V, int lo, int hi, float T, int top_k,
                       float lam, float *x_out, uint32_t *W, uint64_t *Z_out)
{
    int n = hi - lo;
    float *x = (float *)malloc(sizeof(float) * (size_t)(n > 0 ? n : 1));
    float one_plus = 1.0f + lam;
    for (int i = 0; i < n; ++i) {
        float v = c[lo + i];
        if (lam != 0.0f) {
            float a = one_plus * v;
            float b = lam * u[lo + i];
            v = a - b;
        }
        if (T != 1.0f) v = v / T;
        x[i] = v;
    }
    float m = -INFINITY;
    for (int i = 0; i < n; ++i) if (x[i] > m) m = x[i];
    float tau = -INFINITY;
    if (top_k > 0 && top_k < n) {
        float *s = (float *)malloc(sizeof(float) * (size_t)n);
        memcpy(s, x, sizeof(float) * (size_t)n);
        qsort(s, (size_t)n, sizeof(float), cmp_float_desc);
        tau = s[top_k - 1];
        free(s);
    }
    uint64_t Z = 0;
    int kept = 0;
    for (int v = 0; v < V; ++v) { W[v] = 0; if (x_out) x_out[v] = -INFINITY; }
    for (int i = 0; i < n; ++i) {
        if (x_out) x_out[lo + i] = x[i];
        if (x[i] >= tau) {
            float e = oracle_scd_exp(x[i] - m);
            uint32_t w = (uint32_t)(e * 1073741824.0f);
            W[lo + i] = w;
            Z += w;
            ++kept;
        }
    }
    free(x);
    *Z_out = Z;
    return kept;
}

/* ------------------------------------------------------------------------------------------
 * Nucleus (top-p) truncation of a distribution given by integer weights (the video setting of the
 * experiments samples with top-p 0.8): keep the most probable ids until their mass reaches top_p.
 * In threshold form, so that ties need no order: theta = the largest weight value for which the
 * mass of {v : W_v >= theta} is at least top_p * Z; every id with W_v >= theta is kept, the
 * others get weight 0. top_p enters as P24 = trunc(top_p * 2^24 + 1/2) and the test is the
 * integer inequality mass * 2^24 >= P24 * Z. top_p <= 0 or >= 1: nothing happens.
 * ---------------------------------------------------------------------------------------- */
static int cmp_u32_desc(const void *a, const void *b)
{
    uint32_t ua = *(const uint32_t *)a, ub = *(const uint32_t *)b;
    return (ua < ub) - (ua > ub);
}

void oracle_top_p(uint32_t *W, int V, float top_p, uint64_t *Z_io)
{
    if (!(top_p > 0.0f && top_p < 1.0f)) return;
    const uint32_t P24 = (uint32_t)((double)top_p * 16777216.0 + 0.5);
    const uint64_t Z = *Z_io;
    uint32_t *s = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)V);
    memcpy(s, W, sizeof(uint32_t) * (size_t)V);
    qsort(s, (size_t)V, sizeof(uint32_t), cmp_u32_desc);
    uint64_t mass = 0;
    uint32_t theta = 0;
    for (int i = 0; i < V; ++i) {
        mass += s[i];
        if (((u128)mass << 24) >= (u128)P24 * Z) { theta = s[i]; break; }
    }
    free(s);
    if (theta == 0) theta = 1;                 /* (an all-zero row stays all zero) */
    uint64_t kept = 0;
    for (int v = 0; v < V; ++v) {
        if (W[v] < theta) W[v] = 0;
        kept += W[v];
    }
    *Z_io = kept;
}

/* Initial draft distribution (the "p <- Random()" initialisation of Alg. 2/3/6): uniform on the allowed ids. */
void oracle_uniform_weights(int V, int lo, int hi, uint32_t *W, uint64_t *Z_out)
{
    for (int v = 0; v < V; ++v) W[v] = (v >= lo && v < hi) ? 1u : 0u;
    *Z_out = (uint64_t)(hi - lo);
}

/* Inverse-CDF sample from integer weights: Y = min{ v : sum_{v'<=v} W_v' > (U * Z) >> 24 }. */
int oracle_sample(const uint32_t *W, uint64_t Z, int V, uint32_t U)
{
    u128 target = ((u128)U * Z) >> 24;
    u128 acc = 0;
    for (int v = 0; v < V; ++v) {
        acc += W[v];
        if (acc > target) return v;
    }
    return V - 1;
}

/* ------------------------------------------------------------------------------------------
 * Algorithm 1, MRS(p, q, X). p = Wp/Zp, q = Wq/Zq, X ~ q.
 *   accept  iff  u <= min(1, p(X)/q(X))  with u = (U_acc + 1) / 2^24 in (0, 1]
 *           <=>  (U_acc + 1) * Wq[X] * Zp <= Wp[X] * Zq * 2^24          (exact integers)
 *   reject  ->   Y ~ norm(max(0, p - q)):  R_v = max(0, Wp[v]*Zq - Wq[v]*Zp),
 *                Y = min{ v : sum_{v'<=v} R_v' > (U_res * sum R) >> 24 }
 * returns k (1 = accepted); *Y receives the output token.
 * ---------------------------------------------------------------------------------------- */
int oracle_mrs(const uint32_t *Wp, uint64_t Zp, const uint32_t *Wq, uint64_t Zq, int V, int X,
               uint32_t U_acc, uint32_t U_res, int *Y)
{
    u128 lhs = (u128)(U_acc + 1u) * Wq[X] * Zp;
    u128 rhs = ((u128)Wp[X] * Zq) << 24;
    /* p(X) = 0 is never accepted (u > 0); this also covers p(X) = q(X) = 0, which X ~ q excludes and
     * where the inequality would read 0 <= 0: a sampler of p must not emit an id without mass. */
    if (Wp[X] != 0 && lhs <= rhs) { *Y = X; return 1; }
    u128 R = 0;
    for (int v = 0; v < V; ++v) {
        u128 a = (u128)Wp[v] * Zq, b = (u128)Wq[v] * Zp;
        if (a > b) R += a - b;
    }
    if (R == 0) { *Y = X; return 0; }
    u128 target = ((u128)U_res * R) >> 24;
    u128 acc = 0;
    int y = V - 1;
    for (int v = 0; v < V; ++v) {
        u128 a = (u128)Wp[v] * Zq, b = (u128)Wq[v] * Zp;
        if (a > b) {
            acc += a - b;
            if (acc > target) { y = v; break; }
        }
    }
    *Y = y;
    return 0;
}

/* Total variation numerator: sum_v max(0, Wp*Zq - Wq*Zp) = D_TV(p,q) * Zp * Zq
 * (appendix, proof of Prop. 2.1). Returned as a double ratio. */
double oracle_tv(const uint32_t *Wp, uint64_t Zp, const uint32_t *Wq, uint64_t Zq, int V)
{
    u128 R = 0;
    for (int v = 0; v < V; ++v) {
        u128 a = (u128)Wp[v] * Zq, b = (u128)Wq[v] * Zp;
        if (a > b) R += a - b;
    }
    return (double)R / ((double)Zp * (double)Zq);
}

/* ------------------------------------------------------------------------------------------
 * Algorithm 4, GS(P, Q, G): X = argmax(log P_i + g_i), Y = argmax(log Q_i + g_i) with shared
 * Gumbel noise. Written as the exponential race of the appendix (proof of the Gumbel coupling
 * theorem): argmax(log P_i + g_i) = argmin(E_i / P_i), E_i = -log(u_i) ~ Exp(1). The noise of
 * vocabulary entry v is the 24-bit Philox variate with sub-index v.
 * ---------------------------------------------------------------------------------------- */
/* -log2(u) for u = (U + 1/2) / 2^24 = n / 2^25, n = 2U + 1, as an integer with 40 fraction bits:
 * 25 - log2(n). log2 of the mantissa m = n / 2^e in [1, 2) comes one binary digit at a time from
 * the squaring recurrence (m <- m^2; digit 1 and m <- m / 2 when m >= 2), with m held as a 64-bit
 * fixed-point number and every square truncated to its upper 64 bits. The result is > 0 for all
 * 24-bit U and falls strictly as U grows past a change of the leading digits. (The common factor
 * ln 2 between log2 and the natural logarithm of Algorithm 4 does not change an argmin.) */
uint64_t oracle_neglog2_q40(uint32_t U)
{
    uint32_t n = 2u * (U & 0xFFFFFFu) + 1u;           /* odd, 1 .. 2^25 - 1 */
    int e = 0;
    while ((n >> (e + 1)) != 0) ++e;                  /* floor(log2 n) */
    uint64_t x = (uint64_t)n << (63 - e);             /* m * 2^63, in [2^63, 2^64) */
    uint64_t frac = 0;
    for (int i = 0; i < 40; ++i) {
        uint64_t y = (uint64_t)(((u128)x * x) >> 64); /* m^2 * 2^62 */
        frac <<= 1;
        if (y >> 63) { frac |= 1u; x = y; }           /* m^2 >= 2: digit 1, m <- m^2 / 2 */
        else x = y << 1;                              /* digit 0, m <- m^2 */
    }
    return ((uint64_t)25 << 40) - (((uint64_t)e << 40) | frac);
}

int oracle_gumbel_argmax(const uint32_t *W, int V, uint64_t seed, uint32_t batch,
                         uint64_t position, uint32_t iteration)
{
    int best = -1;
    uint64_t best_T = 0;
    uint32_t best_W = 0;
    for (int v = 0; v < V; ++v) {
        if (W[v] == 0) continue;
        uint32_t U = oracle_noise_u24(seed, NOISE_GUMBEL, batch, position, iteration, (uint32_t)v);
        uint64_t T = oracle_neglog2_q40(U);
        /* T / W[v] < best_T / best_W  <=>  T * best_W < best_T * W[v] */
        if (best < 0 || (u128)T * best_W < (u128)best_T * W[v]) { best = v; best_T = T; best_W = W[v]; }
    }
    return best;
}

/* ------------------------------------------------------------------------------------------
 * One vectorised "Verify & Drafting" step over a window (Algorithm 6, the two parallel-for
 * bodies and the first-rejection index), for one sequence.
 *   Lw          : live window rows (C: window clamped at the end of the sequence)
 *   Wp, Zp      : target distributions  [Lw][V], [Lw]
 *   Wq, Zq      : draft distributions   [Lw][V], [Lw]
 *   X           : drafts [Lw];  pos0 : global position of row 0
 *   mode        : 0 = SCD pi_MC (all rows evaluated), 1 = SJD (rows after the first rejection
 *                 are redrawn independently from p), 2 = alpha-coupling of the two
 * outputs: acc[Lw] flags, Y[Lw] per-row outputs, returns a = tokens committed.
 * ---------------------------------------------------------------------------------------- */
int oracle_verify_window(int Lw, int V, const uint32_t *Wp, const uint64_t *Zp, const uint32_t *Wq,
                         const uint64_t *Zq, const int32_t *X, int64_t pos0, uint32_t iteration,
                         uint64_t seed, uint32_t batch, int mode, float alpha, uint8_t *acc,
                         int32_t *Y)
{
    int first_reject = Lw;
    for (int k = 0; k < Lw; ++k) {
        uint64_t pos = (uint64_t)(pos0 + k);
        uint32_t Ua = oracle_noise_u24(seed, NOISE_ACCEPT, batch, pos, iteration, 0);
        uint32_t Ur = oracle_noise_u24(seed, NOISE_RESIDUAL, batch, pos, iteration, 0);
        int y;
        int kflag = oracle_mrs(Wp + (size_t)k * V, Zp[k], Wq + (size_t)k * V, Zq[k], V, X[k], Ua,
                               Ur, &y);
        acc[k] = (uint8_t)kflag;
        Y[k] = y;
        if (!kflag && first_reject == Lw) first_reject = k;
    }
    int a = first_reject < Lw ? first_reject + 1 : Lw;
    if (mode != 0) {
        /* rows beyond the committed prefix: independent redraft from p (the redraw step of Alg. 2), always
         * (SJD) or with probability 1 - alpha (Alg. 5). */
        for (int k = a; k < Lw; ++k) {
            uint64_t pos = (uint64_t)(pos0 + k);
            int indep = 1;
            if (mode == 2) {
                uint32_t Ub = oracle_noise_u24(seed, NOISE_ALPHA, batch, pos, iteration, 0);
                indep = !((double)(Ub + 1u) <= (double)alpha * 16777216.0);
            }
            if (indep) {
                uint32_t Ui = oracle_noise_u24(seed, NOISE_INDEP, batch, pos, iteration, 0);
                Y[k] = oracle_sample(Wp + (size_t)k * V, Zp[k], V, Ui);
            }
        }
    }
    return a;
}

/* ------------------------------------------------------------------------------------------
 * Decode loops over an abstract model.
 *   forward(ctx, stream, ids, n_in, pos0, logits): evaluate n_in input tokens placed at
 *   positions pos0 .. pos0+n_in-1 of the given stream, conditioned on that stream's cached
 *   prefix [0, pos0); logits[k] is the next-token logit vector after input k. Cache entries at
 *   those positions are overwritten.
 * ---------------------------------------------------------------------------------------- */
typedef void (*oracle_forward_fn)(void *ctx, int stream, const int32_t *ids, int n_in,
                                  int64_t pos0, float *logits);

typedef struct {
    int32_t mode;        /* 0 AR, 1 SJD, 2 SCD pi_MC, 3 SCD pi_GS, 4 alpha-coupling (of pi_MC) */
    int32_t window_L;
    int32_t vocab;       /* V */
    float   temperature;
    int32_t top_k;
    float   cfg_lambda;  /* 0 -> one stream */
    float   alpha;
    uint64_t seed;
    int32_t batch_index; /* b in the noise key */
    int32_t allowed_lo, allowed_hi;   /* allowed id range of ordinary positions */
    int32_t row_period;  /* > 0: every row_period-th generated position is forced to eol_id */
    int32_t eol_id;
    float   top_p;       /* nucleus mass, applied after top-k; <= 0 or >= 1: off */
} oracle_decode_config;

typedef struct {
    int64_t forwards;
    int64_t committed;
    int64_t accept_hist[257];    /* accept_hist[a] = iterations that committed a tokens */
} oracle_stats;

static void allowed_range(const oracle_decode_config *cfg, int64_t pos, int64_t prompt_len,
                          int *lo, int *hi)
{
    if (cfg->row_period > 0 && ((pos - prompt_len) % cfg->row_period) == cfg->row_period - 1) {
        *lo = cfg->eol_id; *hi = cfg->eol_id + 1;
    } else {
        *lo = cfg->allowed_lo; *hi = cfg->allowed_hi;
    }
}

/* Fresh window row: q = uniform over the allowed set, X ~ q (the initialisation of Alg. 6). */
static int fresh_draft(const oracle_decode_config *cfg, int64_t pos, int64_t prompt_len,
                       uint32_t first_iter)
{
    int lo, hi;
    allowed_range(cfg, pos, prompt_len, &lo, &hi);
    uint32_t U = oracle_noise_u24(cfg->seed, NOISE_INIT, (uint32_t)cfg->batch_index, (uint64_t)pos,
                                  first_iter, 0);
    return lo + (int)(((uint64_t)U * (uint64_t)(hi - lo)) >> 24);
}

/*
 * tokens      : [n_total]; the first prompt_len entries hold the conditional prompt
 * uncond      : [prompt_len] prompt of the unconditional stream (used when cfg_lambda != 0)
 * trace_a     : optional [n_total] tokens committed by each iteration (for parity tests)
 * returns 0, or -1 on a bad argument.
 */
int oracle_generate(oracle_forward_fn forward, void *ctx, const oracle_decode_config *cfg,
                    int32_t *tokens, const int32_t *uncond, int64_t prompt_len, int64_t n_total,
                    oracle_stats *stats, int32_t *trace_a)
{
    const int V = cfg->vocab;
    const int L = cfg->mode == 0 ? 1 : cfg->window_L;
    const int S = cfg->cfg_lambda != 0.0f ? 2 : 1;
    if (prompt_len < 1 || n_total < prompt_len || L < 1 || L > 256) return -1;
    memset(stats, 0, sizeof(*stats));

    /* prefill: inputs 0 .. prompt_len-2 enter the cache; token prompt_len-1 is fed by the
     * first iteration. */
    if (prompt_len > 1) {
        float *scratch = (float *)malloc(sizeof(float) * (size_t)(prompt_len - 1) * V);
        forward(ctx, 0, tokens, (int)(prompt_len - 1), 0, scratch);
        if (S == 2) forward(ctx, 1, uncond, (int)(prompt_len - 1), 0, scratch);
        free(scratch);
    }

    float *logits = (float *)malloc(sizeof(float) * (size_t)S * L * V);
    uint32_t *Wp = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)L * V);
    uint32_t *Wq = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)L * V);
    uint32_t *Wtmp = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)L * V);
    uint64_t Zp[256], Zq[256], Ztmp[256];
    int32_t D[256], Y[256], in_c[256], in_u[256];
    uint8_t acc[256];

    int64_t n = prompt_len;
    uint32_t t = 0;

    if (cfg->mode != 0) {
        for (int k = 0; k < L && n + k < n_total; ++k) {
            int lo, hi;
            allowed_range(cfg, n + k, prompt_len, &lo, &hi);
            oracle_uniform_weights(V, lo, hi, Wq + (size_t)k * V, &Zq[k]);
            if (cfg->mode == 3)
                D[k] = oracle_gumbel_argmax(Wq + (size_t)k * V, V, cfg->seed,
                                            (uint32_t)cfg->batch_index, (uint64_t)(n + k), 0);
            else
                D[k] = fresh_draft(cfg, n + k, prompt_len, 0);
        }
    }

    while (n < n_total) {
        int Lw = (int)((n_total - n) < L ? (n_total - n) : L);
        /* inputs [x_{n-1}, D_0 .. D_{Lw-2}] at positions n-1 .. n+Lw-2 */
        in_c[0] = tokens[n - 1];
        in_u[0] = (n - 1 < prompt_len) ? (uncond ? uncond[n - 1] : 0) : tokens[n - 1];
        for (int k = 1; k < Lw; ++k) { in_c[k] = D[k - 1]; in_u[k] = D[k - 1]; }
        forward(ctx, 0, in_c, Lw, n - 1, logits);
        if (S == 2) forward(ctx, 1, in_u, Lw, n - 1, logits + (size_t)L * V);
        stats->forwards += 1;

        for (int k = 0; k < Lw; ++k) {
            int lo, hi;
            allowed_range(cfg, n + k, prompt_len, &lo, &hi);
            oracle_postprocess(logits + (size_t)k * V,
                               S == 2 ? logits + (size_t)(L + k) * V : NULL, V, lo, hi,
                               cfg->temperature, cfg->top_k, cfg->cfg_lambda, NULL,
                               Wp + (size_t)k * V, &Zp[k]);
            oracle_top_p(Wp + (size_t)k * V, V, cfg->top_p, &Zp[k]);
        }

        int a;
        if (cfg->mode == 0) {
            /* vanilla AR: x_n ~ p(. | x_<n) */
            uint32_t U = oracle_noise_u24(cfg->seed, NOISE_INDEP, (uint32_t)cfg->batch_index,
                                          (uint64_t)n, 0, 0);
            Y[0] = oracle_sample(Wp, Zp[0], V, U);
            a = 1;
        } else if (cfg->mode == 3) {
            /* Algorithm 7: sequential MRS verify with break; redraft by shared Gumbel noise
             * (fixed per position, independent of the iteration). */
            int first_reject = Lw;
            for (int k = 0; k < Lw; ++k) {
                uint64_t pos = (uint64_t)(n + k);
                uint32_t Ua = oracle_noise_u24(cfg->seed, NOISE_ACCEPT, (uint32_t)cfg->batch_index, pos, t, 0);
                uint32_t Ur = oracle_noise_u24(cfg->seed, NOISE_RESIDUAL, (uint32_t)cfg->batch_index, pos, t, 0);
                int y;
                int kf = oracle_mrs(Wp + (size_t)k * V, Zp[k], Wq + (size_t)k * V, Zq[k], V, D[k], Ua, Ur, &y);
                acc[k] = (uint8_t)kf; Y[k] = y;
                if (!kf) { first_reject = k; break; }
            }
            a = first_reject < Lw ? first_reject + 1 : Lw;
            for (int k = a; k < Lw; ++k)
                Y[k] = oracle_gumbel_argmax(Wp + (size_t)k * V, V, cfg->seed,
                                            (uint32_t)cfg->batch_index, (uint64_t)(n + k), 0);
        } else {
            int vmode = cfg->mode == 2 ? 0 : (cfg->mode == 1 ? 1 : 2);
            a = oracle_verify_window(Lw, V, Wp, Zp, Wq, Zq, D, n, t, cfg->seed,
                                     (uint32_t)cfg->batch_index, vmode, cfg->alpha, acc, Y);
        }

        for (int k = 0; k < a; ++k) tokens[n + k] = Y[k];
        if (trace_a) trace_a[stats->forwards - 1] = a;
        stats->committed += a;
        stats->accept_hist[a] += 1;
        n += a;
        t += 1;

        if (cfg->mode != 0) {
            /* slide the window: new row k' <- old row k'+a (draft Y, draft distribution p);
             * rows entering the window are fresh. */
            for (int k = 0; k < L; ++k) {
                if (n + k >= n_total) break;
                if (k + a < Lw) {
                    D[k] = Y[k + a];
                    memcpy(Wtmp + (size_t)k * V, Wp + (size_t)(k + a) * V, sizeof(uint32_t) * (size_t)V);
                    Ztmp[k] = Zp[k + a];
                } else {
                    int lo, hi;
                    allowed_range(cfg, n + k, prompt_len, &lo, &hi);
                    oracle_uniform_weights(V, lo, hi, Wtmp + (size_t)k * V, &Ztmp[k]);
                    if (cfg->mode == 3)
                        D[k] = oracle_gumbel_argmax(Wtmp + (size_t)k * V, V, cfg->seed,
                                                    (uint32_t)cfg->batch_index, (uint64_t)(n + k), 0);
                    else
                        D[k] = fresh_draft(cfg, n + k, prompt_len, t);
                }
            }
            uint32_t *sw = Wq; Wq = Wtmp; Wtmp = sw;
            memcpy(Zq, Ztmp, sizeof(Zq));
        }
    }
    free(logits); free(Wp); free(Wq); free(Wtmp);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Table model for the losslessness tests: logits are a fixed pseudo-random function of the
 * whole prefix (so every conditional differs), with no transformer involved.
 * ---------------------------------------------------------------------------------------- */
typedef struct {
    int32_t vocab;
    int32_t max_seq;
    uint64_t salt;
    float   scale;
    int32_t *ids;        /* [2][max_seq] tokens seen per stream */
} oracle_table_model;

oracle_table_model *oracle_table_model_new(int vocab, int max_seq, uint64_t salt, float scale)
{
    oracle_table_model *m = (oracle_table_model *)calloc(1, sizeof(*m));
    m->vocab = vocab; m->max_seq = max_seq; m->salt = salt; m->scale = scale;
    m->ids = (int32_t *)calloc((size_t)2 * max_seq, sizeof(int32_t));
    return m;
}

void oracle_table_model_free(oracle_table_model *m) { if (m) { free(m->ids); free(m); } }

void oracle_table_model_forward(void *ctx, int stream, const int32_t *ids, int n_in, int64_t pos0,
                                float *logits)
{
    oracle_table_model *m = (oracle_table_model *)ctx;
    int32_t *seen = m->ids + (size_t)stream * m->max_seq;
    for (int k = 0; k < n_in; ++k) seen[pos0 + k] = ids[k];
    for (int k = 0; k < n_in; ++k) {
        uint64_t h = m->salt ^ 0x9E3779B97F4A7C15ull ^ ((uint64_t)stream << 56);
        for (int64_t j = 0; j <= pos0 + k; ++j) {
            h ^= (uint64_t)(uint32_t)seen[j] + 0x9E3779B97F4A7C15ull + (h << 6) + (h >> 2);
            h *= 0xD6E8FEB86659FD93ull;
            h ^= h >> 32;
        }
        for (int v = 0; v < m->vocab; ++v) {
            uint64_t g = h + (uint64_t)v * 0xBF58476D1CE4E5B9ull;
            g ^= g >> 30; g *= 0x94D049BB133111EBull; g ^= g >> 31;
            double unit = (double)(g >> 11) / 9007199254740992.0;   /* [0,1) */
            logits[(size_t)k * m->vocab + v] = (float)((unit * 2.0 - 1.0) * m->scale);
        }
    }
}

int oracle_generate_table(oracle_table_model *m, const oracle_decode_config *cfg, int32_t *tokens,
                          const int32_t *uncond, int64_t prompt_len, int64_t n_total,
                          oracle_stats *stats, int32_t *trace_a)
{
    return oracle_generate(oracle_table_model_forward, m, cfg, tokens, uncond, prompt_len, n_total,
                           stats, trace_a);
}

/* ------------------------------------------------------------------------------------------
 * Llama-style decoder (the black-box p_theta of the paper; the architecture comes from the
 * workload definitions): pre-norm blocks,
 *   h += Wo * Attn(RoPE(Wq n1), RoPE(Wk n1), Wv n1),  n1 = RMSNorm(h) * g1
 *   h += Wdown * (silu(Wgate n2) * (Wup n2)),          n2 = RMSNorm(h) * g2
 *   logits = Wlm * (RMSNorm(h) * gf)
 * RoPE pairs element i with i + head_dim/2, angle = pos * base^(-2i/head_dim); softmax scale
 * 1/sqrt(head_dim); grouped-query attention maps query head h to kv head h / (H / Hkv).
 * Weights are row-major [out, in], fp32 (wtype 0) or bf16 bit patterns (wtype 1, widened
 * exactly to fp32). Values are stored in fp32; sums run in fp64.
 * ---------------------------------------------------------------------------------------- */
typedef struct {
    int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab_out, vocab_in;
    int32_t max_seq, wtype, n_streams;
    float   rope_base, rms_eps;
    const void *tok_emb, *final_norm, *lm_head;
    const void **attn_norm, **wq, **wk, **wv, **wo, **ffn_norm, **w_gate, **w_up, **w_down;
    float *k_cache, *v_cache;  /* [stream][layer][max_seq][n_kv_heads*head_dim] */
    float *last_hidden;        /* [n_in][d_model] of the most recent forward (after all layers) */
    int    last_hidden_cap;
} oracle_model;

static inline float wload(const void *w, size_t i, int wtype)
{
    if (wtype == 0) return ((const float *)w)[i];
    uint32_t bits = (uint32_t)((const uint16_t *)w)[i] << 16;
    float f;
    memcpy(&f, &bits, 4);
    return f;
}

/* y[m][n] = sum_k x[m][k] * W[n][k] */
static void matmul_nt(const float *x, int M, int K, const void *W, int N, int wtype, float *y)
{
    #pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int m = 0; m < M; ++m) {
            const float *xr = x + (size_t)m * K;
            double acc = 0.0;
            if (wtype == 0) {
                const float *wr = (const float *)W + (size_t)n * K;
                #pragma omp simd reduction(+:acc)
                for (int k = 0; k < K; ++k) acc += (double)xr[k] * (double)wr[k];
            } else {
                const uint16_t *wr = (const uint16_t *)W + (size_t)n * K;
                #pragma omp simd reduction(+:acc)
                for (int k = 0; k < K; ++k) {
                    uint32_t bits = (uint32_t)wr[k] << 16;
                    float wf;
                    memcpy(&wf, &bits, 4);
                    acc += (double)xr[k] * (double)wf;
                }
            }
            y[(size_t)m * N + n] = (float)acc;
        }
    }
}

static void rmsnorm_rows(const float *x, int M, int d, const void *g, int wtype, float eps, float *y)
{
    for (int m = 0; m < M; ++m) {
        const float *xr = x + (size_t)m * d;
        double ss = 0.0;
        for (int i = 0; i < d; ++i) ss += (double)xr[i] * (double)xr[i];
        double inv = 1.0 / sqrt(ss / d + (double)eps);
        for (int i = 0; i < d; ++i)
            y[(size_t)m * d + i] = (float)((double)xr[i] * inv * (double)wload(g, (size_t)i, wtype));
    }
}

oracle_model *oracle_model_new(const int32_t *icfg /*11 ints*/, float rope_base, float rms_eps,
                               const void *tok_emb, const void *final_norm, const void *lm_head,
                               const void **attn_norm, const void **wq, const void **wk,
                               const void **wv, const void **wo, const void **ffn_norm,
                               const void **w_gate, const void **w_up, const void **w_down)
{
    oracle_model *m = (oracle_model *)calloc(1, sizeof(*m));
    m->n_layers = icfg[0]; m->d_model = icfg[1]; m->n_heads = icfg[2]; m->n_kv_heads = icfg[3];
    m->head_dim = icfg[4]; m->d_ffn = icfg[5]; m->vocab_out = icfg[6]; m->vocab_in = icfg[7];
    m->max_seq = icfg[8]; m->wtype = icfg[9]; m->n_streams = icfg[10];
    m->rope_base = rope_base; m->rms_eps = rms_eps;
    m->tok_emb = tok_emb; m->final_norm = final_norm; m->lm_head = lm_head;
    size_t nl = (size_t)m->n_layers;
    const void ***dst[9] = { &m->attn_norm, &m->wq, &m->wk, &m->wv, &m->wo, &m->ffn_norm,
                             &m->w_gate, &m->w_up, &m->w_down };
    const void **src[9] = { attn_norm, wq, wk, wv, wo, ffn_norm, w_gate, w_up, w_down };
    for (int i = 0; i < 9; ++i) {
        *dst[i] = (const void **)malloc(sizeof(void *) * nl);
        memcpy(*dst[i], src[i], sizeof(void *) * nl);
    }
    size_t kv = (size_t)m->n_streams * nl * m->max_seq * m->n_kv_heads * m->head_dim;
    m->k_cache = (float *)calloc(kv, sizeof(float));
    m->v_cache = (float *)calloc(kv, sizeof(float));
    return m;
}

void oracle_model_free(oracle_model *m)
{
    if (!m) return;
    free(m->attn_norm); free(m->wq); free(m->wk); free(m->wv); free(m->wo); free(m->ffn_norm);
    free(m->w_gate); free(m->w_up); free(m->w_down);
    free(m->k_cache); free(m->v_cache); free(m->last_hidden);
    free(m);
}

static void rope_rows(float *x, int M, int n_heads, int dh, int64_t pos0, float base)
{
    int half = dh / 2;
    for (int m = 0; m < M; ++m) {
        double pos = (double)(pos0 + m);
        for (int h = 0; h < n_heads; ++h) {
            float *v = x + ((size_t)m * n_heads + h) * dh;
            for (int i = 0; i < half; ++i) {
                double theta = pow((double)base, -2.0 * (double)i / (double)dh);
                double c = cos(pos * theta), s = sin(pos * theta);
                double a = v[i], b = v[i + half];
                v[i] = (float)(a * c - b * s);
                v[i + half] = (float)(b * c + a * s);
            }
        }
    }
}

void oracle_model_forward(void *ctx, int stream, const int32_t *ids, int M, int64_t pos0,
                          float *logits)
{
    oracle_model *md = (oracle_model *)ctx;
    const int d = md->d_model, H = md->n_heads, Hkv = md->n_kv_heads, dh = md->head_dim;
    const int F = md->d_ffn, V = md->vocab_out, wt = md->wtype;
    const int dq = H * dh, dkv = Hkv * dh, group = H / Hkv;
    float *h = (float *)malloc(sizeof(float) * (size_t)M * d);
    float *xn = (float *)malloc(sizeof(float) * (size_t)M * d);
    float *q = (float *)malloc(sizeof(float) * (size_t)M * dq);
    float *k = (float *)malloc(sizeof(float) * (size_t)M * dkv);
    float *v = (float *)malloc(sizeof(float) * (size_t)M * dkv);
    float *att = (float *)malloc(sizeof(float) * (size_t)M * dq);
    float *proj = (float *)malloc(sizeof(float) * (size_t)M * d);
    float *gate = (float *)malloc(sizeof(float) * (size_t)M * F);
    float *up = (float *)malloc(sizeof(float) * (size_t)M * F);

    for (int m = 0; m < M; ++m)
        for (int i = 0; i < d; ++i)
            h[(size_t)m * d + i] = wload(md->tok_emb, (size_t)ids[m] * d + i, wt);

    for (int l = 0; l < md->n_layers; ++l) {
        float *kc = md->k_cache + (((size_t)stream * md->n_layers + l) * md->max_seq) * dkv;
        float *vc = md->v_cache + (((size_t)stream * md->n_layers + l) * md->max_seq) * dkv;
        rmsnorm_rows(h, M, d, md->attn_norm[l], wt, md->rms_eps, xn);
        matmul_nt(xn, M, d, md->wq[l], dq, wt, q);
        matmul_nt(xn, M, d, md->wk[l], dkv, wt, k);
        matmul_nt(xn, M, d, md->wv[l], dkv, wt, v);
        rope_rows(q, M, H, dh, pos0, md->rope_base);
        rope_rows(k, M, Hkv, dh, pos0, md->rope_base);
        memcpy(kc + (size_t)pos0 * dkv, k, sizeof(float) * (size_t)M * dkv);
        memcpy(vc + (size_t)pos0 * dkv, v, sizeof(float) * (size_t)M * dkv);

        const double scale = 1.0 / sqrt((double)dh);
        #pragma omp parallel for collapse(2) schedule(static)
        for (int m = 0; m < M; ++m) {
            for (int hh = 0; hh < H; ++hh) {
                int64_t n_keys = pos0 + m + 1;     /* causal: keys 0 .. own position */
                const float *qv = q + ((size_t)m * H + hh) * dh;
                int kvh = hh / group;
                double *sc = (double *)malloc(sizeof(double) * (size_t)n_keys);
                double mx = -INFINITY;
                for (int64_t j = 0; j < n_keys; ++j) {
                    const float *kv_ = kc + (size_t)j * dkv + (size_t)kvh * dh;
                    double dot = 0.0;
                    for (int i = 0; i < dh; ++i) dot += (double)qv[i] * (double)kv_[i];
                    sc[j] = dot * scale;
                    if (sc[j] > mx) mx = sc[j];
                }
                double den = 0.0;
                for (int64_t j = 0; j < n_keys; ++j) { sc[j] = exp(sc[j] - mx); den += sc[j]; }
                float *o = att + ((size_t)m * H + hh) * dh;
                for (int i = 0; i < dh; ++i) {
                    double accv = 0.0;
                    for (int64_t j = 0; j < n_keys; ++j)
                        accv += sc[j] * (double)vc[(size_t)j * dkv + (size_t)kvh * dh + i];
                    o[i] = (float)(accv / den);
                }
                free(sc);
            }
        }
        matmul_nt(att, M, dq, md->wo[l], d, wt, proj);
        for (size_t i = 0; i < (size_t)M * d; ++i) h[i] += proj[i];

        rmsnorm_rows(h, M, d, md->ffn_norm[l], wt, md->rms_eps, xn);
        matmul_nt(xn, M, d, md->w_gate[l], F, wt, gate);
        matmul_nt(xn, M, d, md->w_up[l], F, wt, up);
        for (size_t i = 0; i < (size_t)M * F; ++i) {
            double g = gate[i];
            gate[i] = (float)(g / (1.0 + exp(-g)) * (double)up[i]);
        }
        matmul_nt(gate, M, F, md->w_down[l], d, wt, proj);
        for (size_t i = 0; i < (size_t)M * d; ++i) h[i] += proj[i];
    }

    if (md->last_hidden_cap < M) {
        free(md->last_hidden);
        md->last_hidden = (float *)malloc(sizeof(float) * (size_t)M * d);
        md->last_hidden_cap = M;
    }
    memcpy(md->last_hidden, h, sizeof(float) * (size_t)M * d);

    rmsnorm_rows(h, M, d, md->final_norm, wt, md->rms_eps, xn);
    matmul_nt(xn, M, d, md->lm_head, V, wt, logits);

    free(h); free(xn); free(q); free(k); free(v); free(att); free(proj); free(gate); free(up);
}

const float *oracle_model_last_hidden(const oracle_model *m) { return m->last_hidden; }

int oracle_generate_model(oracle_model *m, const oracle_decode_config *cfg, int32_t *tokens,
                          const int32_t *uncond, int64_t prompt_len, int64_t n_total,
                          oracle_stats *stats, int32_t *trace_a)
{
    return oracle_generate(oracle_model_forward, m, cfg, tokens, uncond, prompt_len, n_total, stats,
                           trace_a);
}
