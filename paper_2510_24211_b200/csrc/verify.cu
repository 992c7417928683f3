// Fused verify-and-redraft kernel: logits -> CFG mix -> temperature -> top-k -> integer weights
// -> accept / reject -> residual sample -> first rejection -> commit -> coupled redraft.
//
// One CTA per window row (Algorithm 6 evaluates ALL rows, with no break; Algorithm 1 per row).
// The CTA that finishes last for a sequence ("last block done" ticket, no spinning) runs the
// only serial part, the first-rejection index (the Accept step of Algorithm 6), commits the accepted
// prefix and builds the next window: a row that survives keeps its MRS output as draft and its
// target distribution as draft distribution, which is the maximal coupling of Algorithm 3
// at no extra cost (Sec. 4.3).
//
// Redraft rules besides the maximal coupling: the independent redraw of Algorithm 2 (SJD), its
// alpha-mixture with the coupling (Algorithm 5), and the Gumbel-sharing coupling (Algorithms 4
// and 7) as an integer exponential race with noise keyed by position and id only. Top-p after
// top-k as a threshold on the integer weights.
//
// Data flow of a row: logits -> x (registers when the row has at most 16 ids per thread, else the
// row's cells) -> radix selection of the top-k threshold -> integer weights W, written once into
// the row's cells (shared memory when the row fits, else global memory); every later pass (sum,
// accept test, residual search, race) reads integers. A session stores W as the next iteration's
// draft distribution.
//
// Exactness: a distribution is the integer vector W_v = trunc(scd_exp(x_v - max x) * 2^30) over
// the ids whose post-processed logit x_v reaches the top-k threshold; every decision is an
// inequality between exact 128-bit integer expressions, so the result does not depend on the
// order in which threads sum.
#include "verify.cuh"

namespace scd {

namespace {

constexpr int VT = 1024;       // threads per CTA
constexpr int NW = VT / 32;    // warps per CTA
constexpr unsigned FULL = 0xffffffffu;

struct Smem {
    float red_f[NW];
    unsigned long long red_lo[NW], red_hi[NW];
    unsigned long long base_lo[NW], base_hi[NW], tot_lo, tot_hi;   // block_search: prefix of the warp sums
    unsigned int hist[256];
    unsigned long long mass[256];
    unsigned int sel_bin, sel_k;
    int result;
    int flag;
};

// Post-processed logit of id v of a stored row; raw draft logits still need the temperature.
struct XRow {
    const float *row;      // global row (off = 0) or its copy in shared memory (off = first allowed id)
    int off;
    float T;
    bool div;
    __device__ __forceinline__ float operator()(int v) const
    {
        const float x = row[v - off];
        return div ? __fdiv_rn(x, T) : x;
    }
};

__device__ __forceinline__ float block_max(float v, Smem &sm)
{
    v = warp_max(v);
    if ((threadIdx.x & 31) == 0) sm.red_f[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = sm.red_f[0];
#pragma unroll
    for (int i = 1; i < NW; ++i) r = fmaxf(r, sm.red_f[i]);
    __syncthreads();
    return r;
}

__device__ __forceinline__ unsigned long long block_sum_u64(unsigned long long v, Smem &sm)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
    if ((threadIdx.x & 31) == 0) sm.red_lo[threadIdx.x >> 5] = v;
    __syncthreads();
    unsigned long long r = 0;
#pragma unroll
    for (int i = 0; i < NW; ++i) r += sm.red_lo[i];
    __syncthreads();
    return r;
}

// After a histogram pass: the bin (from the top) in which the kk-th largest element falls, and its
// rank inside that bin. Warp 0 scans the 256 counters; the caller synchronises afterwards.
__device__ __forceinline__ void select_bin(Smem &sm, unsigned kk)
{
    const int tid = threadIdx.x, lane = tid & 31;
    if (tid < 32) {
        unsigned c[8], s = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { c[j] = sm.hist[8 * lane + j]; s += c[j]; }
        unsigned incl = s;                       // suffix sum over lanes >= lane
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned t = __shfl_down_sync(FULL, incl, o);
            if (lane + o < 32) incl += t;
        }
        const unsigned above = incl - s;
        if (above < kk && kk <= above + s) {
            unsigned acc = above;
#pragma unroll
            for (int j = 7; j >= 0; --j) {
                if (acc + c[j] >= kk) { sm.sel_bin = 8u * lane + j; sm.sel_k = kk - acc; break; }
                acc += c[j];
            }
        }
    }
}

// k-th largest post-processed logit of ids [lo, hi) by radix selection on order-preserving
// keys, 8 bits per pass. Exact; ties are resolved by the caller's ">= tau" test.
__device__ float kth_largest(const XRow &x, int lo, int hi, int k, Smem &sm)
{
    const int tid = threadIdx.x, lane = tid & 31;
    unsigned prefix = 0, mask = 0;
    unsigned kk = (unsigned)k;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = tid; i < 256; i += VT) sm.hist[i] = 0;
        __syncthreads();
        for (int base = lo; base < hi; base += 4 * VT) {     // (uniform trip count: warp-wide votes inside)
            float xv[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) xv[j] = base + j * VT + tid < hi ? x(base + j * VT + tid) : 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int v = base + j * VT + tid;
                unsigned key = 0;
                bool match = false;
                if (v < hi) {
                    key = float_key(xv[j]);
                    match = (key & mask) == prefix;
                }
                const unsigned bin = (key >> shift) & 255u;
                if (shift == 24) {
                    // sign and high exponent bits: a handful of distinct bins per warp, so count the
                    // lanes of each bin once (match.any costs one round per distinct value)
                    const unsigned active = __ballot_sync(FULL, match);
                    if (match) {
                        const unsigned peers = __match_any_sync(active, bin);
                        if (lane == __ffs(peers) - 1) atomicAdd(&sm.hist[bin], (unsigned)__popc(peers));
                    }
                } else if (match) {
                    atomicAdd(&sm.hist[bin], 1u);          // lower bytes are spread out: few collisions
                }
            }
        }
        __syncthreads();
        select_bin(sm, kk);
        __syncthreads();
        prefix |= sm.sel_bin << shift;
        mask |= 0xFFu << shift;
        kk = sm.sel_k;
    }
    __syncthreads();
    return key_float(prefix);
}

// A row whose ids fit EPT per thread, kept in registers from the logits to the weights: thread t
// owns ids lo + t + i VT. Loads are issued as a batch; the radix selection works on the registers
// (a bit per element says whether it still matches the selected prefix) and the exponential runs
// once per id. Writes the integer weights to wcell[v - lo] (and to wglob[v] when given) and returns
// the row maximum, the top-k threshold and the sum of the weights.
template <int EPT>
__device__ __forceinline__ void row_in_registers(const float *c, const float *u, float one_plus_lam, float lam,
                                                 bool div, float T, int lo, int hi, int top_k, unsigned *wcell,
                                                 unsigned *wglob, unsigned *scratch, int scratch_words, Smem &sm,
                                                 float &m_out, float &tau_out, unsigned long long &Z_out)
{
    const int tid = threadIdx.x, lane = tid & 31;
    float x[EPT];
    {
        float a[EPT], bu[EPT];
#pragma unroll
        for (int i = 0; i < EPT; ++i) {
            const int v = lo + tid + i * VT;
            a[i] = v < hi ? c[v] : 0.f;
            bu[i] = (u && v < hi) ? u[v] : 0.f;
        }
#pragma unroll
        for (int i = 0; i < EPT; ++i) {
            float t = a[i];
            if (u) t = __fsub_rn(__fmul_rn(one_plus_lam, t), __fmul_rn(lam, bu[i]));
            if (div) t = __fdiv_rn(t, T);
            x[i] = t;
        }
    }
    unsigned mine = 0;                             // bit i: element i exists
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < EPT; ++i)
        if (lo + tid + i * VT < hi) { mine |= 1u << i; mx = fmaxf(mx, x[i]); }
    const bool ragged = (hi - lo) != EPT * VT;     // (uniform) some threads own fewer than EPT ids
    const float m = block_max(mx, sm);
    float tau = -INFINITY;
    if (top_k > 0 && top_k < hi - lo) {
        // radix selection, 8 bits per pass, on order-preserving keys held in the registers of x
        unsigned key[EPT];
#pragma unroll
        for (int i = 0; i < EPT; ++i) key[i] = float_key(x[i]);
        unsigned prefix = 0, mask = 0, kk = (unsigned)top_k;
        bool any = true;                           // this thread still owns a candidate
        for (int shift = 24; shift >= 0; shift -= 8) {
            for (int i = tid; i < 256; i += VT) sm.hist[i] = 0;
            __syncthreads();
            if (shift == 24 && scratch_words >= 256 * 32) {
                // sign and high exponent bits: a handful of bins take almost every element. One
                // histogram per lane (scratch[bin][lane]) keeps a warp's atomics apart; a warp
                // then adds the 32 copies of a bin with one reduction.
                for (int i = tid; i < 256 * 32; i += VT) scratch[i] = 0u;
                __syncthreads();
#pragma unroll
                for (int i = 0; i < EPT; ++i)
                    if (!ragged || ((mine >> i) & 1u)) atomicAdd(&scratch[(key[i] >> 24) * 32u + lane], 1u);
                __syncthreads();
                for (int bin = tid >> 5; bin < 256; bin += NW) {
                    const unsigned cnt = __reduce_add_sync(FULL, scratch[bin * 32 + lane]);
                    if (lane == 0) sm.hist[bin] = cnt;
                }
            } else if (shift == 24) {
                // (no scratch: count the lanes of each bin once; every thread takes part in the votes)
#pragma unroll
                for (int i = 0; i < EPT; ++i) {
                    const bool on = !ragged || ((mine >> i) & 1u);
                    const unsigned bin = key[i] >> 24;
                    const unsigned active = __ballot_sync(FULL, on);
                    if (on) {
                        const unsigned peers = __match_any_sync(active, bin);
                        if (lane == __ffs(peers) - 1) atomicAdd(&sm.hist[bin], (unsigned)__popc(peers));
                    }
                }
            } else if (any) {
                // the candidates thin out by a factor of the bin count per pass: most threads skip
                any = false;
#pragma unroll
                for (int i = 0; i < EPT; ++i) {
                    if ((key[i] & mask) == prefix && (!ragged || ((mine >> i) & 1u))) {
                        atomicAdd(&sm.hist[(key[i] >> shift) & 255u], 1u);
                        any = true;
                    }
                }
            }
            __syncthreads();
            select_bin(sm, kk);
            __syncthreads();
            prefix |= sm.sel_bin << shift;
            mask |= 0xFFu << shift;
            kk = sm.sel_k;
        }
        __syncthreads();
        tau = key_float(prefix);
    }
    unsigned long long z = 0;
#pragma unroll
    for (int i = 0; i < EPT; ++i) {
        if ((mine >> i) & 1u) {
            const int v = lo + tid + i * VT;
            const unsigned wv = weight_of(x[i], m, tau);
            wcell[v - lo] = wv;
            if (wglob) wglob[v] = wv;
            z += wv;
        }
    }
    Z_out = block_sum_u64(z, sm);
    m_out = m;
    tau_out = tau;
}

// Nucleus (top-p) threshold on the integer weights of ids [lo, hi): the largest weight value theta
// for which the ids with W_v >= theta hold at least P24 / 2^24 of the mass Z (integer test
// mass * 2^24 >= P24 * Z). Radix descent over the weight value, 8 bits per pass, with per-bin MASS
// instead of counts. Returns theta; *kept = mass of {W_v >= theta}.
template <class F>
__device__ unsigned nucleus_threshold(const F &weight, int lo, int hi, unsigned long long Z, unsigned P24,
                                      Smem &sm, unsigned long long *kept)
{
    const int tid = threadIdx.x;
    unsigned prefix = 0, mask = 0;
    unsigned long long above = 0;                 // mass of the weights above the current prefix range
    const u128 need = (u128)P24 * Z;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = tid; i < 256; i += VT) sm.mass[i] = 0ull;
        __syncthreads();
        unsigned long long mine0 = 0;             // bin 0 of the top byte holds almost every id: keep it in a register
        for (int v = lo + tid; v < hi; v += VT) {
            const unsigned w = weight(v);
            if (w == 0u || (w & mask) != prefix) continue;
            const unsigned bin = (w >> shift) & 255u;
            if (shift == 24 && bin == 0u) mine0 += w;
            else atomicAdd(&sm.mass[bin], (unsigned long long)w);
        }
        if (shift == 24) {
            const unsigned long long all0 = block_sum_u64(mine0, sm);
            if (tid == 0) sm.mass[0] = all0;
        }
        __syncthreads();
        if (tid == 0) {
            unsigned long long cum = above;
            int sel = 0;
            for (int bin = 255; bin >= 0; --bin) {
                const unsigned long long mb = sm.mass[bin];
                if (mb == 0ull) continue;
                sel = bin;
                if (((u128)(cum + mb) << 24) >= need) break;
                cum += mb;
            }
            sm.sel_bin = (unsigned)sel;
            sm.red_lo[0] = cum;
            sm.red_hi[0] = cum + sm.mass[sel];
        }
        __syncthreads();
        prefix |= sm.sel_bin << shift;
        mask |= 0xFFu << shift;
        above = sm.red_lo[0];
        *kept = sm.red_hi[0];
        __syncthreads();
    }
    return prefix;
}

// Inverse-CDF search: smallest id v in [lo, hi) with sum_{v' <= v} f(v') > (U * total) >> 24,
// ids in increasing order. Warps own contiguous id ranges; the warp whose range holds the
// target walks it 32 ids at a time. Returns -1 when the total is zero.
template <class F>
__device__ int block_search(const F &f, int lo, int hi, unsigned U, Smem &sm)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = hi - lo;
    const int chunk = (((n + NW - 1) / NW) + 31) & ~31;
    const int w_lo = min(hi, lo + warp * chunk);
    const int w_hi = min(hi, w_lo + chunk);
    Limbs s = {0ull, 0ull};
#pragma unroll 4
    for (int v = w_lo + lane; v < w_hi; v += 32) s.add(f(v));
    s = warp_sum(s);
    if (lane == 0) { sm.red_lo[warp] = s.lo; sm.red_hi[warp] = s.hi; }
    if (tid == 0) sm.result = -1;
    __syncthreads();
    if (warp == 0) {
        // exclusive prefix of the warp sums, in warp (= id) order, and their total
        const Limbs t = {sm.red_lo[lane], sm.red_hi[lane]};
        const Limbs inc = warp_scan_inclusive(t, lane);
        sm.base_lo[lane] = inc.lo - t.lo;
        sm.base_hi[lane] = inc.hi - t.hi;
        if (lane == 31) { sm.tot_lo = inc.lo; sm.tot_hi = inc.hi; }
    }
    __syncthreads();
    const u128 base = ((u128)sm.base_hi[warp] << 40) + sm.base_lo[warp];
    const u128 total = ((u128)sm.tot_hi << 40) + sm.tot_lo;
    const u128 mine = s.value();
    const u128 target = ((u128)U * total) >> 24;
    if (total != 0 && base <= target && target < base + mine) {
        u128 run = base;
        for (int i = w_lo; i < w_hi; i += 32) {
            const int v = i + lane;
            Limbs r = {0ull, 0ull};
            if (v < w_hi) r.add(f(v));
            const Limbs inc = warp_scan_inclusive(r, lane);
            const unsigned hit = __ballot_sync(FULL, run + inc.value() > target);
            if (hit) {
                if (lane == 0) sm.result = i + __ffs(hit) - 1;
                break;
            }
            Limbs tot;
            tot.lo = __shfl_sync(FULL, inc.lo, 31);
            tot.hi = __shfl_sync(FULL, inc.hi, 31);
            run += tot.value();
        }
    }
    __syncthreads();
    const int res = sm.result;
    __syncthreads();
    return res;
}

// ---- Gumbel race (Algorithm 4, in the exponential-race form of its proof) ----------------------
// Candidate v finishes at E_v / W_v, E_v = -log2 u_v in fixed point; the earliest wins. Times are
// compared by cross-multiplication in 128 bits and ties go to the smaller id: a strict total
// order, so the winner does not depend on how the candidates are dealt to threads.
struct Racer { unsigned long long T; unsigned W; int v; };       // v < 0: nobody yet
__device__ __forceinline__ bool race_before(const Racer &a, const Racer &b)
{
    if (a.v < 0) return false;
    if (b.v < 0) return true;
    const u128 l = (u128)a.T * b.W, r = (u128)b.T * a.W;
    return l < r || (l == r && a.v < b.v);
}
// argmin over ids [lo, hi) with weight(v) > 0; the noise of id v at a position is the same in
// every iteration (the coupling shares it between the draft and the target distribution).
template <class F>
__device__ int block_race(const F &weight, int lo, int hi, const VerifyParams &p, int b, long long pos, Smem &sm)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    Racer best = {0ull, 0u, -1};
    for (int v = lo + (int)threadIdx.x; v < hi; v += VT) {
        const unsigned W = weight(v);
        if (W == 0u) continue;
        const Racer c = {neglog2_q40(noise_u24(p.seed, NOISE_GUMBEL, (unsigned)b, pos, 0u, (unsigned)v)), W, v};
        if (race_before(c, best)) best = c;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Racer other;
        other.T = __shfl_xor_sync(FULL, best.T, o);
        other.W = __shfl_xor_sync(FULL, best.W, o);
        other.v = __shfl_xor_sync(FULL, best.v, o);
        if (race_before(other, best)) best = other;
    }
    if (lane == 0) { sm.red_lo[warp] = best.T; sm.red_hi[warp] = ((unsigned long long)best.W << 32) | (unsigned)best.v; }
    __syncthreads();
    Racer r = {0ull, 0u, -1};
    for (int i = 0; i < NW; ++i) {
        const Racer c = {sm.red_lo[i], (unsigned)(sm.red_hi[i] >> 32), (int)(unsigned)sm.red_hi[i]};
        if (race_before(c, r)) r = c;
    }
    __syncthreads();
    return r.v;
}

// Rows are staged in shared memory when they fit (stage_cap floats per row; stage_q: a second
// buffer for the draft row), so that the selection, sum and search passes read HBM only once.
__global__ void __launch_bounds__(VT, 1) verify_kernel(const VerifyParams p, int stage_cap, int stage_q)
{
    extern __shared__ float staged[];
    __shared__ Smem sm;
    const int tid = threadIdx.x;
    const int k = blockIdx.x, b = blockIdx.y;
    const WindowState w = load_state(p, b);
    const int L = p.L, V = p.V;

    if (k < w.Lw) {
        const long long pos = w.pos0 + k;
        int lo, hi;
        allowed_range(p, pos, lo, hi);
        const size_t row = (size_t)b * L + k;

        // ---- target distribution p = post-process(logits) ------------------------------------
        // The row's cells (shared memory when the row fits, else its row of xbuf in global memory)
        // first hold the post-processed logits x and then, in place, the integer weights W: the
        // exponential is evaluated once per id and every later pass reads integers. In a session
        // the weights also go to xbuf[t & 1]: they are the next iteration's draft distribution.
        float *xp = p.xbuf[w.parity] + row * V;
        const bool in_smem = hi - lo <= stage_cap;           // this row fits the staging buffer
        float *xs_q = in_smem && stage_q ? staged + stage_cap : nullptr;
        float *prow = in_smem ? staged : xp;
        const int poff = in_smem ? lo : 0;
        unsigned *wp = (unsigned *)prow;
        const bool store_w = p.keep_x && in_smem;            // (cells in global memory are xbuf itself)
        const float *c = p.p_logits + row * V;
        const float *u = p.S == 2 ? p.p_logits + ((size_t)(p.B + b) * L + k) * V : nullptr;
        const bool mix = (p.S == 2);
        const bool div = (p.temperature != 1.0f);
        const bool use_topk = p.top_k > 0 && p.top_k < hi - lo;
        float m_p, tau_p;
        unsigned long long Zp;
        unsigned *const wstore = (store_w && !p.top_p24) ? (unsigned *)xp : nullptr;
        if (in_smem && hi - lo <= 8 * VT) {
            row_in_registers<8>(c, mix ? u : nullptr, p.one_plus_lam, p.lam, div, p.temperature, lo, hi, p.top_k,
                                wp, wstore, (unsigned *)xs_q, xs_q ? stage_cap : 0, sm, m_p, tau_p, Zp);
        } else if (in_smem && hi - lo <= 16 * VT) {
            row_in_registers<16>(c, mix ? u : nullptr, p.one_plus_lam, p.lam, div, p.temperature, lo, hi, p.top_k,
                                 wp, wstore, (unsigned *)xs_q, xs_q ? stage_cap : 0, sm, m_p, tau_p, Zp);
        } else {
            // long rows: the cells live in global memory; loads go out four at a time
            float mx = -INFINITY;
            for (int v0 = lo + tid; v0 < hi; v0 += 4 * VT) {
                float xc[4], xu[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int v = v0 + j * VT;
                    xc[j] = v < hi ? c[v] : 0.f;
                    xu[j] = (mix && v < hi) ? u[v] : 0.f;
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int v = v0 + j * VT;
                    if (v < hi) {
                        float x = xc[j];
                        if (mix) x = __fsub_rn(__fmul_rn(p.one_plus_lam, x), __fmul_rn(p.lam, xu[j]));
                        if (div) x = __fdiv_rn(x, p.temperature);
                        prow[v - poff] = x;
                        mx = fmaxf(mx, x);
                    }
                }
            }
            m_p = block_max(mx, sm);       // barrier inside: the row is visible to the CTA
            tau_p = use_topk ? kth_largest(XRow{prow, poff, 1.0f, false}, lo, hi, p.top_k, sm) : -INFINITY;
            unsigned long long zp = 0;
            for (int v0 = lo + tid; v0 < hi; v0 += 4 * VT) {     // x -> W, each thread on its own cells
                float xv[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) xv[j] = v0 + j * VT < hi ? prow[v0 + j * VT - poff] : -INFINITY;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int v = v0 + j * VT;
                    if (v < hi) {
                        const unsigned wv = weight_of(xv[j], m_p, tau_p);
                        wp[v - poff] = wv;
                        if (wstore) wstore[v] = wv;
                        zp += wv;
                    }
                }
            }
            Zp = block_sum_u64(zp, sm);                          // (barriers inside: the weights are visible)
        }
        unsigned theta_p = 0u;
        if (p.top_p24) {
            auto fw = [&](int v) -> unsigned { return wp[v - poff]; };
            unsigned long long kept;
            theta_p = nucleus_threshold(fw, lo, hi, Zp, p.top_p24, sm, &kept);
            Zp = kept;
            for (int v = lo + tid; v < hi; v += VT) {
                unsigned wv = wp[v - poff];
                if (wv < theta_p) { wv = 0u; wp[v - poff] = 0u; }
                if (store_w) ((unsigned *)xp)[v] = wv;
            }
            __syncthreads();
        }
        if (tid == 0) {
            RowStats st; st.m = m_p; st.tau = tau_p; st.Z = Zp; st.theta = theta_p; st.pad_ = 0u;
            p.stats[w.parity][row] = st;
        }
        auto WP = [&](int v) -> unsigned { return wp[v - poff]; };

        // ---- draft distribution q: the previous iteration's p of the same position -----------
        // session: its integer weights, as stored by that iteration; stand-alone: raw logits that
        // go through the same steps here (cached in shared memory when the row fits, else
        // recomputed per visit); fresh rows: uniform weights 1 on the allowed ids.
        const int qk = k + w.shift;
        const bool fresh = !(qk < w.prev_lw);
        unsigned long long Zq = (unsigned long long)(hi - lo);
        const unsigned *qcache = nullptr;                     // cached integer weights, id v at qcache[v - qoff]
        int qoff = 0;
        bool q_in_smem = false;
        XRow XQ = {nullptr, 0, p.temperature, false};         // recompute path only
        float m_q = 0.f, tau_q = -INFINITY;
        unsigned theta_q = 0u;
        if (!fresh) {
            const size_t qrow = (size_t)b * L + qk;
            if (p.q_is_raw) {
                XQ.row = p.xbuf[w.parity ^ 1] + qrow * V;
                XQ.div = div;
                if (xs_q) {
                    unsigned *wq = (unsigned *)xs_q;
                    if (hi - lo <= 8 * VT) {
                        row_in_registers<8>(XQ.row, nullptr, 0.f, 0.f, div, p.temperature, lo, hi, p.top_k, wq, nullptr,
                                            wq, stage_cap, sm, m_q, tau_q, Zq);
                    } else if (hi - lo <= 16 * VT) {
                        row_in_registers<16>(XQ.row, nullptr, 0.f, 0.f, div, p.temperature, lo, hi, p.top_k, wq, nullptr,
                                             wq, stage_cap, sm, m_q, tau_q, Zq);
                    } else {
                        float mq = -INFINITY;
                        for (int v = lo + tid; v < hi; v += VT) {
                            const float x = XQ(v);
                            xs_q[v - lo] = x;
                            mq = fmaxf(mq, x);
                        }
                        m_q = block_max(mq, sm);
                        tau_q = use_topk ? kth_largest(XRow{xs_q, lo, 1.0f, false}, lo, hi, p.top_k, sm) : -INFINITY;
                        unsigned long long zq = 0;
                        for (int v = lo + tid; v < hi; v += VT) {
                            const unsigned wv = weight_of(xs_q[v - lo], m_q, tau_q);
                            wq[v - lo] = wv;
                            zq += wv;
                        }
                        Zq = block_sum_u64(zq, sm);
                    }
                    if (p.top_p24) {
                        auto fq = [&](int v) -> unsigned { return wq[v - lo]; };
                        unsigned long long kept;
                        theta_q = nucleus_threshold(fq, lo, hi, Zq, p.top_p24, sm, &kept);
                        Zq = kept;
                        for (int v = lo + tid; v < hi; v += VT)
                            if (wq[v - lo] < theta_q) wq[v - lo] = 0u;
                        __syncthreads();
                    }
                    qcache = wq; qoff = lo; q_in_smem = true;
                } else {
                    float mq = -INFINITY;
                    for (int v = lo + tid; v < hi; v += VT) mq = fmaxf(mq, XQ(v));
                    m_q = block_max(mq, sm);
                    tau_q = use_topk ? kth_largest(XQ, lo, hi, p.top_k, sm) : -INFINITY;
                    unsigned long long zq = 0;
                    for (int v = lo + tid; v < hi; v += VT) zq += weight_of(XQ(v), m_q, tau_q);
                    Zq = block_sum_u64(zq, sm);
                    if (p.top_p24) {
                        auto fq = [&](int v) -> unsigned { return weight_of(XQ(v), m_q, tau_q); };
                        unsigned long long kept;
                        theta_q = nucleus_threshold(fq, lo, hi, Zq, p.top_p24, sm, &kept);
                        Zq = kept;
                    }
                }
            } else {
                Zq = p.stats[w.parity ^ 1][qrow].Z;
                qcache = (const unsigned *)(p.xbuf[w.parity ^ 1] + qrow * V);
                qoff = 0;
            }
        }
        auto WQ = [&](int v) -> unsigned {
            if (fresh) return 1u;
            if (qcache) return qcache[v - qoff];
            return weight_of(XQ(v), m_q, tau_q, theta_q);
        };

        // ---- Algorithm 1 on (p, q, X) ----------------------------------------------------------
        const int X = p.draft_in[row];
        int Y = X, Yi = X, Yf = X;
        int accept = 1;
        if (p.mode == SCD_MODE_AR) {
            // vanilla AR: x ~ p by inverse CDF (Sec. 2.1)
            const unsigned U = noise_u24(p.seed, NOISE_INDEP, (unsigned)b, pos, 0u, 0);
            auto fw = [&](int v) -> u128 { return (u128)WP(v); };
            Y = block_search(fw, lo, hi, U, sm);
            if (Y < 0) Y = lo;
        } else {
            if (tid == 0) {
                unsigned WpX = 0, WqX = 0;
                if (X >= lo && X < hi) {
                    WpX = WP(X);
                    WqX = WQ(X);
                }
                const unsigned Ua = noise_u24(p.seed, NOISE_ACCEPT, (unsigned)b, pos, w.t, 0);
                // u <= min(1, p(X)/q(X)) with u = (Ua+1)/2^24  <=>  (Ua+1) Wq[X] Zp <= Wp[X] Zq 2^24
                // (a draft without mass under p - possible only when X was not drawn from q - is rejected)
                const u128 lhs = (u128)(Ua + 1u) * WqX * Zp;
                const u128 rhs = ((u128)WpX * Zq) << 24;
                sm.flag = (WpX != 0u && lhs <= rhs) ? 1 : 0;
            }
            __syncthreads();
            accept = sm.flag;
            __syncthreads();
            if (!accept) {
                // Y ~ norm(max(0, p - q)): R_v = max(0, Wp_v Zq - Wq_v Zp)
                const unsigned Ur = noise_u24(p.seed, NOISE_RESIDUAL, (unsigned)b, pos, w.t, 0);
                if (!fresh && !q_in_smem && qcache && xs_q) {
                    // rejected: the residual needs the whole draft row, twice; read it from HBM once
                    unsigned *wq = (unsigned *)xs_q;
                    for (int v0 = lo + tid; v0 < hi; v0 += 8 * VT) {        // loads issued as a batch
                        unsigned t[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) t[j] = v0 + j * VT < hi ? qcache[v0 + j * VT - qoff] : 0u;
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            if (v0 + j * VT < hi) wq[v0 + j * VT - lo] = t[j];
                    }
                    __syncthreads();
                    qcache = wq; qoff = lo; q_in_smem = true;
                }
                auto fr = [&](int v) -> u128 {
                    const u128 a = mul_32x64(WP(v), Zq);
                    const u128 bq = mul_32x64(WQ(v), Zp);
                    return a > bq ? a - bq : (u128)0;
                };
                Y = block_search(fr, lo, hi, Ur, sm);
                if (Y < 0) Y = X;
            }
            bool indep = p.mode == SCD_MODE_SJD;
            if (p.mode == SCD_MODE_ALPHA) {
                // Algorithm 5: keep the coupled redraft with probability alpha, b = (Ub + 1) / 2^24
                const unsigned Ub = noise_u24(p.seed, NOISE_ALPHA, (unsigned)b, pos, w.t, 0);
                indep = !((double)(Ub + 1u) <= (double)p.alpha * 16777216.0);
                Yi = Y;
            }
            if (p.mode == SCD_MODE_SCD_GS) {
                // Algorithm 7: beyond the committed prefix the next draft is the Gumbel-max sample
                // of p under this position's shared noise ...
                auto fw = [&](int v) -> unsigned { return WP(v); };
                Yi = block_race(fw, lo, hi, p, b, pos, sm);
                if (Yi < 0) Yi = lo;
                // ... and the row that may enter the window at position pos0 + L + k starts from the
                // same race under the uniform draft distribution of its allowed ids
                const long long posf = w.pos0 + L + k;
                int flo, fhi;
                allowed_range(p, posf, flo, fhi);
                Yf = block_race([](int) -> unsigned { return 1u; }, flo, fhi, p, b, posf, sm);
            }
            if (indep) {
                // Algorithm 2 (its redraw step): the next draft is an independent draw from p
                const unsigned Ui = noise_u24(p.seed, NOISE_INDEP, (unsigned)b, pos, w.t, 0);
                auto fw = [&](int v) -> u128 { return (u128)WP(v); };
                Yi = block_search(fw, lo, hi, Ui, sm);
                if (Yi < 0) Yi = lo;
            }
        }
        if (tid == 0) {
            p.accept_flags[row] = (unsigned char)accept;
            p.row_y[row] = Y;
            p.row_y_indep[row] = Yi;
            if (p.mode == SCD_MODE_SCD_GS) p.row_y_indep[(size_t)p.B * L + row] = Yf;
        }
    }

    // ---- last CTA of the sequence: first rejection, commit, next window ----------------------
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned ticket = atomicAdd(&p.done_count[b], 1u);
        sm.flag = (ticket == gridDim.x - 1) ? 1 : 0;
    }
    __syncthreads();
    if (!sm.flag) return;
    __threadfence();

    if (w.Lw == 0) {
        if (tid == 0) { p.n_commit[b] = 0; p.done_count[b] = 0; }
        return;
    }
    if (tid == 0) sm.result = w.Lw;
    __syncthreads();
    if (tid < w.Lw && __ldcg(&p.accept_flags[(size_t)b * L + tid]) == 0) atomicMin(&sm.result, tid);
    __syncthreads();
    const int kstar = sm.result;
    const int a = kstar < w.Lw ? kstar + 1 : w.Lw;     // the rejected row's residual sample is committed

    for (int kk = tid; kk < L; kk += VT) {
        const size_t row = (size_t)b * L + kk;
        if (kk < a) {
            const int y = __ldcg(&p.row_y[row]);
            if (p.committed_ids) p.committed_ids[row] = y;
            if (p.tokens) p.tokens[(size_t)b * p.token_stride + w.pos0 + kk] = y;
        }
        if (p.mode != SCD_MODE_AR) {
            const int src = kk + a;
            int nd;
            if (src < w.Lw)
                nd = p.mode != SCD_MODE_SCD_MC ? __ldcg(&p.row_y_indep[(size_t)b * L + src])
                                               : __ldcg(&p.row_y[(size_t)b * L + src]);
            else if (p.mode == SCD_MODE_SCD_GS && src >= L)
                nd = __ldcg(&p.row_y_indep[(size_t)p.B * L + (size_t)b * L + (src - L)]);   // position pos0 + src
            else
                nd = fresh_draft(p, b, w.pos0 + a + kk, w.t + 1u);
            // every row CTA of this sequence has passed its ticket, so draft_in is no longer read
            p.draft_out[row] = nd;
        }
    }
    if (tid == 0) {
        p.n_commit[b] = a;
        if (p.n_known) {
            p.n_known[b] = (int)w.pos0 + a;
            p.iter[b] = w.t + 1u;
            p.shift[b] = a;
            p.prev_lw[b] = w.Lw;
            // this iteration completed the sequence (it was live: Lw > 0): the last of the batch raises the flag
            if (p.finished && (int)w.pos0 + a >= p.n_total[b] && atomicAdd(&p.finished[0], 1) == p.B - 1) p.finished[1] = 1;
        }
        if (p.dev_stats) {
            atomicMax(&p.dev_stats->forwards, (unsigned long long)w.t + 1ull);   // iterations in which a sequence was live
            atomicAdd(&p.dev_stats->committed, (unsigned long long)a);
            atomicAdd(&p.dev_stats->accept_hist[a], 1ull);
        }
        p.done_count[b] = 0;
    }
}

// Window initialisation after prefill: every row fresh.
__global__ void init_window_kernel(const VerifyParams p)
{
    __shared__ Smem sm;
    const int b = blockIdx.x;
    const long long pos0 = p.n_known[b];
    if (p.mode == SCD_MODE_SCD_GS) {
        for (int k = 0; k < p.L; ++k) {
            int lo, hi;
            allowed_range(p, pos0 + k, lo, hi);
            const int d = block_race([](int) -> unsigned { return 1u; }, lo, hi, p, b, pos0 + k, sm);
            if (threadIdx.x == 0) p.draft_out[(size_t)b * p.L + k] = d;
        }
    } else {
        for (int k = threadIdx.x; k < p.L; k += blockDim.x)
            p.draft_out[(size_t)b * p.L + k] = fresh_draft(p, b, pos0 + k, 0u);
    }
    if (threadIdx.x == 0) {
        p.iter[b] = 0u;
        p.shift[b] = 0;
        p.prev_lw[b] = 0;
        p.n_commit[b] = 0;
        p.done_count[b] = 0u;
    }
}

}  // namespace

int launch_verify(const VerifyParams &p, cudaStream_t stream)
{
    // a cluster per row wherever it applies; this kernel keeps the Gumbel race, the nucleus truncation
    // and rows too long for a cluster's registers
    if (verify_cluster_supported(p)) return launch_verify_cluster(p, stream);
    dim3 grid((unsigned)p.L, (unsigned)p.B);
    // shared-memory staging: both rows if they fit, else the target row alone, else none
    const int n = p.allowed_hi - p.allowed_lo;
    const size_t budget = 200 * 1024;
    int stage_cap = 0, stage_q = 0;
    if ((size_t)n * 8 <= budget) { stage_cap = n; stage_q = 1; }
    else if ((size_t)n * 4 <= budget) { stage_cap = n; }
    const size_t smem = (size_t)stage_cap * 4 * (stage_q ? 2 : 1);
    static DeviceOnce once;
    int dev = 0;
    int rc = current_device(&dev);
    if (rc != SCD_OK) return rc;
    rc = once.run(dev, [&]() -> int {
        SCD_CUDA_TRY(cudaFuncSetAttribute(verify_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)budget));
        return SCD_OK;
    });
    if (rc != SCD_OK) return rc;
    verify_kernel<<<grid, VT, smem, stream>>>(p, stage_cap, stage_q);
    SCD_CUDA_TRY(cudaGetLastError());
    return SCD_OK;
}

int launch_init_window(const VerifyParams &p, cudaStream_t stream)
{
    init_window_kernel<<<p.B, VT, 0, stream>>>(p);
    SCD_CUDA_TRY(cudaGetLastError());
    return SCD_OK;
}

}  // namespace scd
