// Fused verify-and-redraft kernel, one thread-block CLUSTER per window row (Algorithm 6 evaluates all
// rows, Algorithm 1 per row). A row's vocabulary is cut into slices, one per CTA of the cluster; every
// id lives in a register of exactly one thread from the logits to the integer weights, and what the
// row needs as a whole (maximum, top-k threshold, normaliser, residual mass) is merged through
// distributed shared memory after a hardware cluster barrier. With 32 rows of 8192 ids this puts
// 128 CTAs on the GPU instead of 32 and shortens every per-row pass by the cluster size.
//
// Passes over a row (all on registers; the only HBM traffic is the logits in, the draft weights in and,
// in a session, the target weights out):
//   1. x = post-processed logit (guidance mix, temperature); row maximum m                -> barrier 1
//   2. W = trunc(scd_exp(x - m) 2^30) for every LIVE id (x >= m - 22: only they can get a non-zero
//      weight) and a histogram of the live ids over 512 equal steps of m - x; every CTA merges the
//      histograms and finds the step that holds the k-th largest                           -> barrier 2
//   3. mass of the ids above that step, summed per CTA; the ids OF the step go to a short list as
//      (key of x, W); every CTA reads all lists, picks the exact k-th largest by counting (radix
//      selection over the cluster when the lists overflow) and has the normaliser:
//      Z = mass above the step + the candidates that stay; ids below tau lose their weight -> barrier 3
//      accept test of Algorithm 1 in 128-bit integers, computed alike by every CTA (each weighs the draft
//      itself, from the draft's own logits)
//   4. on rejection: residual mass R_v = max(0, Wp_v Zq - Wq_v Zp) per CTA                 -> barrier 4
//      and the inverse-CDF walk inside the one warp that holds the target
// A stand-alone call with raw draft logits runs passes 1-3 on both rows at once. The CTA that finds a
// row's token writes it and takes the sequence's ticket (with two tokens per row - SJD, alpha - rank 0
// does, after the closing barrier); the last ticket of a sequence does the only serial part (first
// rejection, commit, next window), exactly as in the one-CTA-per-row kernel. The closing barrier (nobody
// may leave while a peer still reads its shared memory) is off the critical path: everybody arrives as
// soon as it has finished reading, the ticket's CTA waits only at its very end.
//
// What every thread needs from every peer (maxima, masses, counts) is fetched by ONE lane per peer and
// handed on through local shared memory: distributed shared memory is for few, wide requests.
//
// Fewer than top_k live ids: the k-th largest then has weight 0 and so has everything below it, so
// the threshold is dropped - the weights are those of the definition.
// Exactness: sums are integers, thresholds are exact selections, every decision is an integer
// inequality: nothing depends on how ids are dealt to threads or CTAs.
// No thread ever spins: the only waits are hardware barriers that every CTA of a cluster reaches
// the same number of times (every branch that holds a barrier is taken on values that all CTAs of
// the cluster compute from the same data).
#include "verify.cuh"

namespace scd {

namespace {

constexpr int MAXW = 32;           // warps per CTA at most (512 or 1024 threads)
constexpr int NB = 512;            // steps of the live range in the top-k histogram
constexpr int CAND_CAP = 512;      // candidates one CTA may hand over
constexpr int CAND_ALL = 1024;     // candidates of a whole row that are selected by counting
constexpr int MAXC = 8;
constexpr unsigned FULLM = 0xffffffffu;
constexpr float LIVE_SPAN = 22.0f; // scd_exp(x) = 0 below -22

// Code that runs on the target row and, when the draft row arrives as raw logits, on the draft row too:
// the row index is a compile-time constant inside, so the per-thread values stay in registers.
template <int A> struct RowIndex { static constexpr int value = A; };
#define EACH_ARRAY(...) do { auto fn_ = __VA_ARGS__; fn_(RowIndex<0>{}); if (NA > 1) fn_(RowIndex<1>{}); } while (0)

struct Xchg {                      // read by the peers through distributed shared memory
    unsigned hist[2][NB];          // (first: read with 16-byte loads)
    uint2 cand[2][CAND_CAP];       // (order-preserving key of x, weight) of the ids in the selected step
    unsigned radix[1024];          // overflow path: four passes x 256 counters
    // nucleus threshold: mass per byte value of the weight, one table per pass, as two 32-bit sums (low 15 bits
    // of the weights / the rest: a row has at most 2^16 ids and a weight 30 bits, so neither overflows) -
    // 32-bit shared-memory adds stay fast when a flat distribution sends thousands of ids to one value
    unsigned massh[4][2][256];
    unsigned long long zpart[2];   // mass of this CTA's ids above the selected step (overflow path: above the threshold)
    unsigned long long res_lo, res_hi;   // residual mass of this CTA's slice (two limbs)
    float mx[2];
    unsigned cand_n[2];
};

struct Local {
    float red_f[2][MAXW];
    unsigned long long red_u[2][MAXW];
    unsigned scan_w[2][4];
    int sel_bucket[2];
    unsigned sel_k[2];
    uint2 all_cand[2][CAND_ALL];
    unsigned scratch[256];
    float pm[2][MAXC];                         // what the peers published, fetched by a few lanes for the whole CTA
    unsigned long long pz[2][MAXC], pr[2][MAXC];
    unsigned pc[2][MAXC];
    unsigned tau_key[2];
    unsigned long long w_lo[MAXW], w_hi[MAXW];   // per-warp sums of a search (two limbs)
    unsigned long long merged[256];            // nucleus threshold: the cluster's mass per byte value
    unsigned long long np_above, np_kept;
    unsigned np_sel;
    int last;
    int result;
};

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_sync() { cluster_arrive(); cluster_wait(); }
__device__ __forceinline__ uint32_t peer_addr(uint32_t local, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
    return r;
}
__device__ __forceinline__ unsigned ld_peer_u32(const void *local, uint32_t rank)
{
    unsigned v;
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(peer_addr(smem_addr(local), rank)) : "memory");
    return v;
}
__device__ __forceinline__ float ld_peer_f32(const void *local, uint32_t rank)
{
    return __uint_as_float(ld_peer_u32(local, rank));
}
__device__ __forceinline__ unsigned long long ld_peer_u64(const void *local, uint32_t rank)
{
    unsigned long long v;
    asm volatile("ld.shared::cluster.u64 %0, [%1];" : "=l"(v) : "r"(peer_addr(smem_addr(local), rank)) : "memory");
    return v;
}
__device__ __forceinline__ uint4 ld_peer_u32x4(const void *local, uint32_t rank)
{
    uint4 v;
    asm volatile("ld.shared::cluster.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(peer_addr(smem_addr(local), rank)) : "memory");
    return v;
}

// step of the live range an id falls into: 0 at the maximum, NB - 1 at m - 22; -1: not live
__device__ __forceinline__ int live_step(float x, float m)
{
    const float dlt = __fsub_rn(m, x);                 // = -(x - m) exactly
    if (!(dlt <= LIVE_SPAN)) return -1;
    const int b = __float2int_rd(__fmul_rn(dlt, (float)NB / 22.5f));
    return min(max(b, 0), NB - 1);
}

// residual mass of one id: max(0, Wp Zq - Wq Zp)
__device__ __forceinline__ u128 residual_of(unsigned wp, unsigned wq, unsigned long long Zp, unsigned long long Zq)
{
    if (wp == 0u) return (u128)0;
    const u128 a = mul_32x64(wp, Zq), b = mul_32x64(wq, Zp);
    return a > b ? a - b : (u128)0;
}

// Whether row (b, pos) of iteration t is redrawn independently (Algorithm 2 always, Algorithm 5 by its coin).
__device__ __forceinline__ bool redraw_independent(const VerifyParams &p, int b, long long pos, unsigned t)
{
    if (p.mode == SCD_MODE_SJD) return true;
    if (p.mode != SCD_MODE_ALPHA) return false;
    const unsigned Ub = noise_u24(p.seed, NOISE_ALPHA, (unsigned)b, pos, t, 0);
    return !((double)(Ub + 1u) <= (double)p.alpha * 16777216.0);
}

// Inverse CDF over the ids of this CTA in id order. The mass of this thread's i-th id is its residual
// max(0, wp Zq - wq Zp) (RESIDUAL) or its weight wp. `base` = mass of the slices in front, `target` the
// searched prefix value. The caller has stored the per-warp sums in lc.w_lo / w_hi (and synchronised).
// Returns the id (in every lane of the one warp that finds it), else -1.
template <int EPT, bool RESIDUAL>
__device__ __forceinline__ int walk_slice(const unsigned (&wp)[EPT], const unsigned (&wq)[EPT], unsigned long long Zp,
                                          unsigned long long Zq, u128 base, u128 target, int wbase, int hi, Local &lc)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    u128 run = base;
    for (int w = 0; w < warp; ++w) run += ((u128)lc.w_hi[w] << 40) + lc.w_lo[w];
    const u128 mine = ((u128)lc.w_hi[warp] << 40) + lc.w_lo[warp];
    if (!(run <= target && target < run + mine)) return -1;
    int found = -1;
#pragma unroll
    for (int i = 0; i < EPT; ++i) {
        Limbs r = {0ull, 0ull};
        r.add(RESIDUAL ? residual_of(wp[i], wq[i], Zp, Zq) : (u128)wp[i]);
        if (found < 0) {                                   // (warp-uniform)
            const Limbs inc = warp_scan_inclusive(r, lane);
            const unsigned hit = __ballot_sync(FULLM, run + inc.value() > target);
            if (hit) {
                found = wbase + 32 * i + (__ffs(hit) - 1);
            } else {
                Limbs tot;
                tot.lo = __shfl_sync(FULLM, inc.lo, 31);
                tot.hi = __shfl_sync(FULLM, inc.hi, 31);
                run += tot.value();
            }
        }
    }
    return found < hi ? found : -1;
}

template <int EPT, int CT>
__global__ void __launch_bounds__(CT, (CT == 512 && EPT <= 8) ? 2 : 1) verify_cluster_kernel(const VerifyParams p, int C)
{
    constexpr int CNW = CT / 32;
    __shared__ __align__(16) Xchg xc;
    __shared__ Local lc;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rank = blockIdx.x % C;                       // = rank in the cluster (cluster dims (C, 1, 1))
    const int k = blockIdx.x / C, b = blockIdx.y;
    pdl_trigger();
    // (launched with programmatic stream serialisation: everything up to pdl_wait() below reads only what
    // earlier iterations left behind - the window counters, the draft ids, the drafts' stored weights)
    const WindowState w = load_state(p, b);
    const int L = p.L, V = p.V;
    const size_t row = (size_t)b * L + k;
    bool takes_ticket = rank == 0;                         // the CTA that reports this row to the sequence

    if (k < w.Lw) {
        const long long pos = w.pos0 + k;
        int lo, hi;
        allowed_range(p, pos, lo, hi);
        const int wbase = lo + rank * (EPT * CT) + warp * (32 * EPT);   // this warp's ids: wbase + 32 i + lane
        const bool mix = p.S == 2, div = p.temperature != 1.0f;
        const bool use_topk = p.top_k > 0 && p.top_k < hi - lo;
        const int qk = k + w.shift;
        const bool fresh = !(qk < w.prev_lw);
        const bool rawq = !fresh && p.q_is_raw;              // draft distribution from raw logits, built here
        const int NA = rawq ? 2 : 1;
        const size_t qrow = (size_t)b * L + qk;
        const bool mrs = p.mode != SCD_MODE_AR;
        // SJD and the alpha-coupling report two tokens per row, possibly found by two CTAs: there the
        // ticket waits for the closing barrier; otherwise the CTA that finds the row's token takes it
        const bool late_ticket = p.mode == SCD_MODE_SJD || p.mode == SCD_MODE_ALPHA;

        // ---- pass 1: loads, post-processing, maximum ---------------------------------------------------
        float xv[2][EPT];                                    // [0] target, [1] draft (raw logits)
        unsigned wt[2][EPT];                                 // integer weights
        const int X = p.draft_in[row];
        const bool x_in = X >= lo && X < hi;
        float xX, xqX = 0.f;                                 // the draft's own logits: every CTA weighs X itself
        unsigned long long Zq_stored = 0ull;
        {
            const float *c = p.p_logits + row * V;
            const float *u = mix ? p.p_logits + ((size_t)(p.B + b) * L + k) * V : nullptr;
            const float *qr = fresh ? nullptr : p.xbuf[w.parity ^ 1] + qrow * V;
            float a[EPT], bu[EPT];
#pragma unroll
            for (int i = 0; i < EPT; ++i) {
                const int v = wbase + 32 * i + lane;
                xv[1][i] = (qr && v < hi) ? qr[v] : 0.f;     // raw logits, or stored integer weights (bit pattern)
            }
            xqX = (qr && x_in) ? qr[X] : 0.f;
            if (!fresh && !rawq) Zq_stored = p.stats[w.parity ^ 1][qrow].Z;
            for (int i = tid; i < 2 * NB; i += CT) (&xc.hist[0][0])[i] = 0u;
            if (tid < 2) { xc.cand_n[tid] = 0u; lc.sel_bucket[tid] = -1; }
            pdl_wait();                                      // the target logits come from the kernel in front
            // (read through L2: this kernel may have started before that kernel wrote them, and the
            // non-coherent load path then served stale lines of the previous iteration)
#pragma unroll
            for (int i = 0; i < EPT; ++i) {
                const int v = wbase + 32 * i + lane;
                const bool in = v < hi;
                a[i] = in ? __ldcg(c + v) : 0.f;
                bu[i] = (mix && in) ? __ldcg(u + v) : 0.f;
            }
            const float cX = x_in ? __ldcg(c + X) : 0.f, uX = (mix && x_in) ? __ldcg(u + X) : 0.f;
#pragma unroll
            for (int i = 0; i < EPT; ++i) {
                float t = a[i];
                if (mix) t = __fsub_rn(__fmul_rn(p.one_plus_lam, t), __fmul_rn(p.lam, bu[i]));
                if (div) t = __fdiv_rn(t, p.temperature);
                xv[0][i] = t;
                if (rawq && div) xv[1][i] = __fdiv_rn(xv[1][i], p.temperature);
            }
            xX = cX;
            if (mix) xX = __fsub_rn(__fmul_rn(p.one_plus_lam, cX), __fmul_rn(p.lam, uX));
            if (div) xX = __fdiv_rn(xX, p.temperature);
            if (rawq && div) xqX = __fdiv_rn(xqX, p.temperature);
        }
        float mloc[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int i = 0; i < EPT; ++i) {
            if (wbase + 32 * i + lane < hi) {
                mloc[0] = fmaxf(mloc[0], xv[0][i]);
                if (rawq) mloc[1] = fmaxf(mloc[1], xv[1][i]);
            }
        }
        EACH_ARRAY([&](auto A_) {
            constexpr int a = decltype(A_)::value;
            const float t = warp_max(mloc[a]);
            if (lane == 0) lc.red_f[a][warp] = t;
        });
        __syncthreads();
        if (tid < NA) {
            float t = lc.red_f[tid][0];
            for (int i = 1; i < CNW; ++i) t = fmaxf(t, lc.red_f[tid][i]);
            xc.mx[tid] = t;
        }
        cluster_sync();                                                               // ---- barrier 1
        // (a value that every thread needs from every peer is fetched once per CTA - one lane per peer -
        // and handed on through local shared memory: 512 threads asking 8 peers each cost microseconds)
        if (warp < NA && lane < MAXC) lc.pm[warp][lane] = lane < C ? ld_peer_f32(&xc.mx[warp], (uint32_t)lane) : -INFINITY;
        __syncthreads();
        float m[2] = {-INFINITY, 0.f};
        EACH_ARRAY([&](auto A_) {
            constexpr int a = decltype(A_)::value;
            float t = lc.pm[a][0];
#pragma unroll
            for (int r = 1; r < MAXC; ++r) t = fmaxf(t, lc.pm[a][r]);
            m[a] = t;
        });

        // ---- pass 2: weights of all live ids (the threshold comes later), histogram of the live range ----
        EACH_ARRAY([&](auto A_) {
            constexpr int a = decltype(A_)::value;
#pragma unroll
            for (int i = 0; i < EPT; ++i) {
                const bool in = wbase + 32 * i + lane < hi;
                wt[a][i] = in ? weight_of(xv[a][i], m[a], -INFINITY) : 0u;
                if (use_topk && in) {
                    const int s = live_step(xv[a][i], m[a]);
                    if (s >= 0) atomicAdd(&xc.hist[a][s], 1u);
                }
            }
        });
        if (!rawq) {
#pragma unroll
            for (int i = 0; i < EPT; ++i) {
                const bool in = wbase + 32 * i + lane < hi;
                wt[1][i] = !in ? 0u : fresh ? 1u : __float_as_uint(xv[1][i]);   // uniform, or stored by the previous iteration
            }
        }
        if (use_topk) {
            cluster_sync();                                                           // ---- barrier 2
            // every CTA merges the C histograms: threads 0..127 take the target row, 128..255 the draft
            // row; each owns four steps
            const int ga = tid >> 7, gt = tid & 127, gw = gt >> 5;
            uint4 s4 = make_uint4(0u, 0u, 0u, 0u);
            unsigned mine = 0, inc = 0;
            if (ga < NA) {
                uint4 t4[MAXC];
#pragma unroll
                for (int r = 0; r < MAXC; ++r)                       // all loads in flight, then the sums
                    t4[r] = r < C ? ld_peer_u32x4(&xc.hist[ga][4 * gt], (uint32_t)r) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                for (int r = 0; r < MAXC; ++r) { s4.x += t4[r].x; s4.y += t4[r].y; s4.z += t4[r].z; s4.w += t4[r].w; }
                mine = s4.x + s4.y + s4.z + s4.w;
                inc = mine;                                          // inclusive scan over the warp's threads
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const unsigned t = __shfl_up_sync(FULLM, inc, o);
                    if (lane >= o) inc += t;
                }
                if (lane == 31) lc.scan_w[ga][gw] = inc;
            }
            __syncthreads();
            if (ga < NA) {
                unsigned before = 0;
                for (int i = 0; i < gw; ++i) before += lc.scan_w[ga][i];
                const unsigned excl = before + inc - mine, kk = (unsigned)p.top_k;
                if (excl < kk && kk <= excl + mine) {                // the k-th largest sits in one of my four steps
                    unsigned acc = excl;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const unsigned cnt = j == 0 ? s4.x : j == 1 ? s4.y : j == 2 ? s4.z : s4.w;
                        if (acc < kk && kk <= acc + cnt) { lc.sel_bucket[ga] = 4 * gt + j; lc.sel_k[ga] = kk - acc; }
                        acc += cnt;
                    }
                }
            }
            __syncthreads();
        }

        // ---- pass 3: mass above the selected step, candidates of the step, exact threshold, normaliser ----
        // (no selected step - top-k off, or fewer than k live ids -: every live id keeps its weight)
        int sb[2] = {-1, -1};
        unsigned long long zab[2] = {0ull, 0ull};
        EACH_ARRAY([&](auto A_) {
            constexpr int a = decltype(A_)::value;
            sb[a] = lc.sel_bucket[a];
#pragma unroll
            for (int i = 0; i < EPT; ++i) {
                if (wbase + 32 * i + lane < hi) {
                    const int s = sb[a] < 0 ? -1 : live_step(xv[a][i], m[a]);
                    if (sb[a] < 0 || (s >= 0 && s < sb[a])) zab[a] += wt[a][i];
                    else if (s == sb[a]) {
                        const unsigned at = atomicAdd(&xc.cand_n[a], 1u);
                        if (at < CAND_CAP) xc.cand[a][at] = make_uint2(float_key(xv[a][i]), wt[a][i]);
                    }
                }
            }
            unsigned long long z = zab[a];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(FULLM, z, o);
            if (lane == 0) lc.red_u[a][warp] = z;
        });
        __syncthreads();
        if (tid < NA) {
            unsigned long long z = 0;
            for (int i = 0; i < CNW; ++i) z += lc.red_u[tid][i];
            xc.zpart[tid] = z;
        }
        cluster_sync();                                                               // ---- barrier 3
        float tau[2] = {-INFINITY, -INFINITY};
        unsigned long long Zall[2] = {0ull, 0ull}, Zbefore[2] = {0ull, 0ull};   // row normaliser; mass of the slices in front of mine
        bool overflow[2] = {false, false};
        unsigned n_all[2] = {0u, 0u}, n_front[2] = {0u, 0u};
        if (warp < 2 * NA && lane < MAXC) {              // warps 0, 1: the target row's masses and counts; 2, 3: the draft row's
            const int a = warp >> 1;
            if (warp & 1) lc.pc[a][lane] = (lane < C && lc.sel_bucket[a] >= 0) ? ld_peer_u32(&xc.cand_n[a], (uint32_t)lane) : 0u;
            else lc.pz[a][lane] = lane < C ? ld_peer_u64(&xc.zpart[a], (uint32_t)lane) : 0ull;
        }
        __syncthreads();
        EACH_ARRAY([&](auto A_) {
            constexpr int a = decltype(A_)::value;
#pragma unroll
            for (int r = 0; r < MAXC; ++r) {
                const unsigned cn = lc.pc[a][r];
                Zall[a] += lc.pz[a][r];
                if (r < rank) { Zbefore[a] += lc.pz[a][r]; n_front[a] += cn; }
                if (cn > CAND_CAP) overflow[a] = true;
                n_all[a] += cn;
            }
            if (n_all[a] > CAND_ALL) overflow[a] = true;
            if (sb[a] < 0 || overflow[a]) return;
            // gather: entry e of the row's list is entry e - off_r of CTA r's list (lists in rank order)
            for (unsigned e = tid; e < n_all[a]; e += CT) {
                unsigned off = 0;
                int rr = 0;
                bool found = false;                              // e < n_all = sum of the counts: found for some rr < C
#pragma unroll
                for (int r = 0; r < MAXC; ++r) {
                    if (!found) {
                        if (e < off + lc.pc[a][r]) { found = true; rr = r; }
                        else off += lc.pc[a][r];
                    }
                }
                if (!found || rr >= C) continue;                 // (cannot happen; never address a rank outside the cluster)
                const unsigned long long kw = ld_peer_u64(&xc.cand[a][e - off], (uint32_t)rr);
                lc.all_cand[a][e] = make_uint2((unsigned)kw, (unsigned)(kw >> 32));
            }
        });
        __syncthreads();
        EACH_ARRAY([&](auto A_) {
            constexpr int a = decltype(A_)::value;
            if (sb[a] < 0 || overflow[a]) return;
            // the sel_k-th largest key of the list, by counting
            const unsigned kk = lc.sel_k[a];
            for (unsigned j = tid; j < n_all[a]; j += CT) {
                const unsigned key = lc.all_cand[a][j].x;
                unsigned gt = 0, ge = 0;
                for (unsigned i = 0; i < n_all[a]; ++i) {
                    const unsigned o = lc.all_cand[a][i].x;
                    gt += o > key ? 1u : 0u;
                    ge += o >= key ? 1u : 0u;
                }
                if (gt < kk && kk <= ge) lc.tau_key[a] = key;    // (equal keys write the same value)
            }
        });
        __syncthreads();
        EACH_ARRAY([&](auto A_) {
            constexpr int a = decltype(A_)::value;
            if (sb[a] < 0 || overflow[a]) return;
            const unsigned tk = lc.tau_key[a];
            tau[a] = key_float(tk);
            // the candidates that stay add to the normaliser (every warp sums the list for itself)
            unsigned long long add_all = 0, add_front = 0;
            for (unsigned i = lane; i < n_all[a]; i += 32) {
                const uint2 kw = lc.all_cand[a][i];
                if (kw.x >= tk) { add_all += kw.y; if (i < n_front[a]) add_front += kw.y; }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                add_all += __shfl_xor_sync(FULLM, add_all, o);
                add_front += __shfl_xor_sync(FULLM, add_front, o);
            }
            Zall[a] += add_all;
            Zbefore[a] += add_front;
        });
        // lists that overflowed (long runs of equal or nearly equal logits): radix selection over the cluster,
        // 8 bits per pass, among the ids of the selected step; then the normaliser from scratch
        EACH_ARRAY([&](auto A_) {
            constexpr int a = decltype(A_)::value;
            if (!overflow[a]) return;
            unsigned prefix = 0, mask = 0, kk = lc.sel_k[a];
            for (int i = tid; i < 1024; i += CT) xc.radix[i] = 0u;            // four passes x 256 counters
            cluster_sync();
            for (int pass = 0; pass < 4; ++pass) {
                const int shift = 24 - 8 * pass;
                unsigned *h = &xc.radix[256 * pass];
#pragma unroll
                for (int i = 0; i < EPT; ++i) {
                    if (wbase + 32 * i + lane < hi && live_step(xv[a][i], m[a]) == sb[a]) {
                        const unsigned key = float_key(xv[a][i]);
                        if ((key & mask) == prefix) atomicAdd(&h[(key >> shift) & 255u], 1u);
                    }
                }
                cluster_sync();
                if (tid < 256) {
                    unsigned s = 0;
                    for (int r = 0; r < C; ++r) s += ld_peer_u32(&h[tid], (uint32_t)r);
                    lc.scratch[tid] = s;
                }
                __syncthreads();
                if (tid == 0) {
                    unsigned acc = 0;
                    int sel = 0;
                    for (int bin = 255; bin >= 0; --bin) {
                        const unsigned cnt = lc.scratch[bin];
                        if (acc + cnt >= kk) { sel = bin; break; }
                        acc += cnt;
                    }
                    lc.sel_bucket[a] = sel;
                    lc.sel_k[a] = kk - acc;
                }
                __syncthreads();
                prefix |= (unsigned)lc.sel_bucket[a] << shift;
                mask |= 0xFFu << shift;
                kk = lc.sel_k[a];
                __syncthreads();
            }
            tau[a] = key_float(prefix);
            unsigned long long z = 0;
#pragma unroll
            for (int i = 0; i < EPT; ++i)
                if (wbase + 32 * i + lane < hi && xv[a][i] >= tau[a]) z += wt[a][i];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(FULLM, z, o);
            if (lane == 0) lc.red_u[a][warp] = z;
            __syncthreads();
            if (tid == 0) {
                unsigned long long t = 0;
                for (int i = 0; i < CNW; ++i) t += lc.red_u[a][i];
                xc.zpart[a] = t;                     // (every peer has read the earlier value: a cluster barrier lies in between)
            }
            cluster_sync();
            Zall[a] = 0; Zbefore[a] = 0;
            for (int r = 0; r < C; ++r) {
                const unsigned long long t = ld_peer_u64(&xc.zpart[a], (uint32_t)r);
                Zall[a] += t;
                if (r < rank) Zbefore[a] += t;
            }
        });
        // the threshold takes effect: ids below it lose their weight (the step is monotone in x, so this
        // removes exactly the ids of later steps and the candidates below tau)
#pragma unroll
        for (int i = 0; i < EPT; ++i) {
            if (!(xv[0][i] >= tau[0])) wt[0][i] = 0u;
            if (rawq && !(xv[1][i] >= tau[1])) wt[1][i] = 0u;
        }
        // ---- nucleus (top-p) on the integer weights: theta = the largest weight value whose ids {W >= theta}
        // hold at least top_p of the mass; radix descent over the weight value, 8 bits per pass, with the
        // MASS per byte value merged over the cluster (integers: the same theta in every CTA)
        unsigned theta[2] = {0u, 0u};
        if (p.top_p24) {
            for (int i = tid; i < 4 * 2 * 256; i += CT) (&xc.massh[0][0][0])[i] = 0u;
            EACH_ARRAY([&](auto A_) {
                constexpr int a = decltype(A_)::value;
                const u128 need = (u128)p.top_p24 * Zall[a];
                unsigned prefix = 0, mask = 0;
                unsigned long long above = 0, kept = 0;
                __syncthreads();         // the tables are zeroed
                for (int pass = 0; pass < 4; ++pass) {
                    const int shift = 24 - 8 * pass;
#pragma unroll
                    for (int i = 0; i < EPT; ++i) {
                        const unsigned wv = wt[a][i];
                        if (wv != 0u && (wv & mask) == prefix) {
                            const unsigned bin = (wv >> shift) & 255u;
                            atomicAdd(&xc.massh[pass][0][bin], wv & 0x7FFFu);
                            atomicAdd(&xc.massh[pass][1][bin], wv >> 15);
                        }
                    }
                    cluster_sync();
                    if (tid < 256) {
                        unsigned long long mm = 0;
                        for (int r = 0; r < C; ++r)
                            mm += ((unsigned long long)ld_peer_u32(&xc.massh[pass][1][tid], (uint32_t)r) << 15) +
                                  ld_peer_u32(&xc.massh[pass][0][tid], (uint32_t)r);
                        lc.merged[tid] = mm;
                    }
                    __syncthreads();
                    if (warp == 0) {
                        // the highest byte value at which the mass from the top reaches `need`: lane l owns the
                        // values 8 l .. 8 l + 7; suffix sums over the lanes, then each lane walks its eight
                        unsigned long long mine8 = 0;
#pragma unroll
                        for (int j = 0; j < 8; ++j) mine8 += lc.merged[8 * lane + j];
                        unsigned long long suf = mine8;              // sum over lanes >= lane
#pragma unroll
                        for (int o = 1; o < 32; o <<= 1) {
                            const unsigned long long t = __shfl_down_sync(FULLM, suf, o);
                            if (lane + o < 32) suf += t;
                        }
                        unsigned long long cum = above + suf - mine8;   // mass above my eight values
                        int sel = -1;
                        unsigned long long cum_at = 0, mass_at = 0;
#pragma unroll
                        for (int j = 7; j >= 0; --j) {
                            const unsigned long long mb = lc.merged[8 * lane + j];
                            if (sel < 0 && mb != 0ull && (((u128)(cum + mb) << 24) >= need)) { sel = 8 * lane + j; cum_at = cum; mass_at = mb; }
                            cum += mb;
                        }
                        const unsigned hit = __ballot_sync(FULLM, sel >= 0);
                        // (the total reaches `need` by construction, so some lane has a hit; the highest one wins)
                        if (hit != 0u && lane == 31 - __clz(hit)) { lc.np_sel = (unsigned)sel; lc.np_above = cum_at; lc.np_kept = cum_at + mass_at; }
                        if (hit == 0u && lane == 0) { lc.np_sel = 0u; lc.np_above = above; lc.np_kept = above; }
                    }
                    __syncthreads();
                    prefix |= lc.np_sel << shift;
                    mask |= 0xFFu << shift;
                    above = lc.np_above;
                    kept = lc.np_kept;
                    __syncthreads();
                }
                theta[a] = prefix;
                Zall[a] = kept;
                unsigned long long z = 0;
#pragma unroll
                for (int i = 0; i < EPT; ++i) {
                    if (wt[a][i] < prefix) wt[a][i] = 0u;
                    z += wt[a][i];
                }
                // the slices' masses after the cut (an independent draw walks them in id order)
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(FULLM, z, o);
                if (lane == 0) lc.red_u[a][warp] = z;
                __syncthreads();
                if (tid == 0) {
                    unsigned long long t = 0;
                    for (int i = 0; i < CNW; ++i) t += lc.red_u[a][i];
                    xc.zpart[a] = t;
                }
                cluster_sync();          // the masses are published; every peer has finished reading my tables
                if (a == 0) {
                    if (warp == 0 && lane < MAXC) lc.pz[0][lane] = lane < C ? ld_peer_u64(&xc.zpart[0], (uint32_t)lane) : 0ull;
                    __syncthreads();
                    Zbefore[0] = 0;
                    for (int r = 0; r < rank; ++r) Zbefore[0] += lc.pz[0][r];
                    if (rawq)            // the draft row uses the tables next
                        for (int i = tid; i < 4 * 2 * 256; i += CT) (&xc.massh[0][0][0])[i] = 0u;
                }
            });
        }
        if (p.keep_x) {
            unsigned *wstore = (unsigned *)(p.xbuf[w.parity] + row * V);
#pragma unroll
            for (int i = 0; i < EPT; ++i) {
                const int v = wbase + 32 * i + lane;
                if (v < hi) wstore[v] = wt[0][i];
            }
        }
        const unsigned long long Zp = Zall[0];
        unsigned long long Zq;
        if (rawq) Zq = Zall[1];
        else if (fresh) Zq = (unsigned long long)(hi - lo);
        else Zq = Zq_stored;
        if (rank == 0 && tid == 0) {
            RowStats st; st.m = m[0]; st.tau = tau[0]; st.Z = Zp; st.theta = theta[0]; st.pad_ = 0u;
            p.stats[w.parity][row] = st;
        }

        // ---- Algorithm 1 on (p, q, X) ------------------------------------------------------------------
        int accept = 1;
        if (mrs) {
            const unsigned WpX = x_in ? weight_of(xX, m[0], tau[0], theta[0]) : 0u;
            const unsigned WqX = !x_in ? 0u : rawq ? weight_of(xqX, m[1], tau[1], theta[1]) : fresh ? 1u : __float_as_uint(xqX);
            const unsigned Ua = noise_u24(p.seed, NOISE_ACCEPT, (unsigned)b, pos, w.t, 0);
            // u <= min(1, p(X)/q(X)) with u = (Ua+1)/2^24  <=>  (Ua+1) Wq[X] Zp <= Wp[X] Zq 2^24;
            // a draft without mass under p is rejected
            const u128 lhs = (u128)(Ua + 1u) * WqX * Zp;
            const u128 rhs = ((u128)WpX * Zq) << 24;
            accept = (WpX != 0u && lhs <= rhs) ? 1 : 0;
            // the flag and the token are written by the CTA that takes the ticket (the order of its own
            // writes and its ticket is what the last CTA of the sequence relies on)
            if (accept) {
                if (rank == 0 && tid == 0) { p.accept_flags[row] = 1; p.row_y[row] = X; }
                takes_ticket = rank == 0;
            } else {
                // Y ~ norm(max(0, p - q)): per-CTA residual mass, then the walk in the CTA that holds the target
                Limbs s = {0ull, 0ull};
#pragma unroll
                for (int i = 0; i < EPT; ++i) s.add(residual_of(wt[0][i], wt[1][i], Zp, Zq));
                s = warp_sum(s);
                if (lane == 0) { lc.w_lo[warp] = s.lo; lc.w_hi[warp] = s.hi; }
                __syncthreads();
                if (tid == 0) {
                    unsigned long long a0 = 0, a1 = 0;
                    for (int i = 0; i < CNW; ++i) { a0 += lc.w_lo[i]; a1 += lc.w_hi[i]; }
                    xc.res_lo = a0; xc.res_hi = a1;
                }
                cluster_sync();                                                       // ---- barrier 4
                u128 total = 0, before = 0, mine = 0;
                if (warp < 2 && lane < MAXC)
                    lc.pr[warp][lane] = lane < C ? ld_peer_u64(warp == 0 ? &xc.res_lo : &xc.res_hi, (uint32_t)lane) : 0ull;
                __syncthreads();
#pragma unroll
                for (int r = 0; r < MAXC; ++r) {
                    const u128 t = ((u128)lc.pr[1][r] << 40) + lc.pr[0][r];
                    if (r < rank) before += t;
                    if (r == rank) mine = t;
                    total += t;
                }
                const unsigned Ur = noise_u24(p.seed, NOISE_RESIDUAL, (unsigned)b, pos, w.t, 0);
                const u128 target = ((u128)Ur * total) >> 24;
                if (total == 0) {
                    if (rank == 0 && tid == 0) { p.accept_flags[row] = 0; p.row_y[row] = X; }
                    takes_ticket = rank == 0;
                } else {
                    takes_ticket = before <= target && target < before + mine;      // (one CTA of the cluster)
                    if (takes_ticket) {
                        const int y = walk_slice<EPT, true>(wt[0], wt[1], Zp, Zq, before, target, wbase, hi, lc);
                        if (y >= 0 && lane == 0) { p.accept_flags[row] = 0; p.row_y[row] = y; __threadfence(); }
                    }
                }
            }
        }
        // ---- an independent draw from p: the token of vanilla AR, the redraft of Algorithm 2 -----------
        const bool indep = !mrs || redraw_independent(p, b, pos, w.t);
        if (indep) {
            const unsigned Ui = noise_u24(p.seed, NOISE_INDEP, (unsigned)b, pos, mrs ? w.t : 0u, 0);
            const u128 target = ((u128)Ui * Zp) >> 24;
            unsigned long long z = 0;
#pragma unroll
            for (int i = 0; i < EPT; ++i) z += wt[0][i];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(FULLM, z, o);
            __syncthreads();                                       // the warp sums of the residual walk are done with
            if (lane == 0) { lc.w_lo[warp] = z & ((1ull << 40) - 1); lc.w_hi[warp] = z >> 40; }
            __syncthreads();
            unsigned long long zmine = 0;
            for (int i = 0; i < CNW; ++i) zmine += (lc.w_hi[i] << 40) + lc.w_lo[i];
            int *dst = mrs ? p.row_y_indep : p.row_y;
            if (Zp == 0) {
                if (rank == 0 && tid == 0) { dst[row] = lo; if (!mrs) p.accept_flags[row] = 1; }
                if (!mrs) takes_ticket = rank == 0;
            } else {
                const bool mine_it = (u128)Zbefore[0] <= target && target < (u128)Zbefore[0] + zmine;
                if (mine_it) {
                    const int y = walk_slice<EPT, false>(wt[0], wt[1], Zp, Zq, (u128)Zbefore[0], target, wbase, hi, lc);
                    if (y >= 0 && lane == 0) { dst[row] = y; if (!mrs) p.accept_flags[row] = 1; __threadfence(); }
                }
                if (!mrs) takes_ticket = mine_it;
            }
        }
        // The CTA that takes the row's ticket has itself written the row's token (or waits, below, for the
        // peers that wrote one); everybody tells the cluster that it has finished reading its peers.
        if (late_ticket) {
            if (rank == 0 && tid == 0) p.accept_flags[row] = (unsigned char)accept;   // (rank 0 takes the ticket)
            __threadfence();                     // a token found here is visible before the barrier completes
            cluster_arrive();
            cluster_wait();
            takes_ticket = rank == 0;
            if (!takes_ticket) return;
        } else {
            cluster_arrive();
        }
        if (!late_ticket && !takes_ticket) {
            cluster_wait();                      // nobody leaves while a peer may still read its shared memory
            return;
        }
    } else {
        pdl_wait();                          // (no kernel may finish before the kernel in front has)
        if (rank != 0) return;               // a row beyond the end of the sequence: only the ticket is taken
    }
    const bool pending_wait = k < w.Lw && !(p.mode == SCD_MODE_SJD || p.mode == SCD_MODE_ALPHA);

    // ---- last CTA of the sequence: first rejection, commit, next window ----------------------------
    __syncthreads();                         // the row's token is written (by a thread of this CTA)
    if (tid == 0) {
        __threadfence();
        const unsigned ticket = atomicAdd(&p.done_count[b], 1u);
        lc.last = (ticket == (unsigned)L - 1u) ? 1 : 0;
        __threadfence();                     // what the other rows wrote before their tickets is read below (from L2)
    }
    __syncthreads();
    if (pending_wait) cluster_wait();        // (the peers arrived long ago: they only had to finish reading)
    if (!lc.last) return;

    if (w.Lw == 0) {
        if (tid == 0) { p.n_commit[b] = 0; p.done_count[b] = 0; }
        return;
    }
    if (tid == 0) lc.result = w.Lw;
    __syncthreads();
    if (tid < w.Lw && __ldcg(&p.accept_flags[(size_t)b * L + tid]) == 0) atomicMin(&lc.result, tid);
    __syncthreads();
    const int kstar = lc.result;
    const int a = kstar < w.Lw ? kstar + 1 : w.Lw;     // the rejected row's residual sample is committed

    for (int kk = tid; kk < L; kk += CT) {
        const size_t r = (size_t)b * L + kk;
        if (kk < a) {
            const int y = __ldcg(&p.row_y[r]);
            if (p.committed_ids) p.committed_ids[r] = y;
            if (p.tokens) p.tokens[(size_t)b * p.token_stride + w.pos0 + kk] = y;
        }
        if (p.mode != SCD_MODE_AR) {
            const int src = kk + a;
            int nd;
            if (src < w.Lw) {
                const bool ind = redraw_independent(p, b, w.pos0 + src, w.t);
                nd = ind ? __ldcg(&p.row_y_indep[(size_t)b * L + src]) : __ldcg(&p.row_y[(size_t)b * L + src]);
            } else {
                nd = fresh_draft(p, b, w.pos0 + a + kk, w.t + 1u);
            }
            // every row of this sequence has taken its ticket, so draft_in is no longer read
            p.draft_out[r] = nd;
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

// cluster size, threads per CTA and ids per thread for rows of at most n ids, `rows` rows in the grid
bool choose_cluster(int n, int rows, int sm_count, int *C_out, int *ept_out, int *ct_out)
{
    int C = 1;
    while (C < MAXC && rows * C * 2 <= sm_count) C *= 2;              // at most one CTA per SM (two would share its issue slots)
    while (C > 1 && (C / 2) * 4 * 512 >= n) C /= 2;                   // no more CTAs than slices of 4 ids per thread
    for (;; C *= 2) {
        for (int ept = 4; ept <= 8; ept *= 2)
            if ((long long)C * ept * 512 >= n) { *C_out = C; *ept_out = ept; *ct_out = 512; return true; }
        // long rows: rather a larger cluster than more ids per thread; at the largest cluster, 1024 threads
        if (C >= MAXC) {
            if ((long long)C * 8 * 1024 >= n) { *C_out = C; *ept_out = 8; *ct_out = 1024; return true; }
            return false;
        }
    }
}

}  // namespace

bool verify_cluster_supported(const VerifyParams &p)
{
    if (p.mode == SCD_MODE_SCD_GS) return false;                      // the Gumbel race: the one-CTA kernel
    if (p.L > 512) return false;
    int C, ept, ct;
    return choose_cluster(p.allowed_hi - p.allowed_lo, p.L * p.B, 148, &C, &ept, &ct);
}

int launch_verify_cluster(const VerifyParams &p, cudaStream_t stream)
{
    int dev = 0, sms = 148;
    int rc = current_device(&dev);
    if (rc != SCD_OK) return rc;
    static int sm_count[DeviceOnce::kSlots];
    static DeviceOnce once;
    rc = once.run(dev, [&]() -> int {
        SCD_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        if (dev >= 0 && dev < DeviceOnce::kSlots) sm_count[dev] = sms;
        return SCD_OK;
    });
    if (rc != SCD_OK) return rc;
    if (dev >= 0 && dev < DeviceOnce::kSlots) sms = sm_count[dev];
    int C = 1, ept = 4, ct = 512;
    SCD_REQUIRE(choose_cluster(p.allowed_hi - p.allowed_lo, p.L * p.B, sms, &C, &ept, &ct), SCD_ERR_SHAPE,
                "verify: rows of %d ids do not fit a cluster", p.allowed_hi - p.allowed_lo);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.L * C), (unsigned)p.B, 1);
    cfg.blockDim = dim3((unsigned)ct, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)C;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (ct == 1024) SCD_CUDA_TRY(cudaLaunchKernelEx(&cfg, verify_cluster_kernel<8, 1024>, p, C));
    else if (ept == 4) SCD_CUDA_TRY(cudaLaunchKernelEx(&cfg, verify_cluster_kernel<4, 512>, p, C));
    else SCD_CUDA_TRY(cudaLaunchKernelEx(&cfg, verify_cluster_kernel<8, 512>, p, C));
    return SCD_OK;
}

}  // namespace scd
