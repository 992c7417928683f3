// Window-parallel forward of the Llama-style decoder p_theta (the parallel forward of Algorithm 6: all window
// positions are evaluated in one pass, causal attention over the KV cache plus the window).
//
// Pre-norm blocks: h += Wo Attn(RoPE(Wq n1), RoPE(Wk n1), Wv n1); h += Wdown(silu(Wgate n2) * Wup n2);
// logits = Wlm RMSNorm(h). The residual stream h and the logits are fp32; GEMM inputs, the KV
// cache and the attention output have the model dtype T (float or bf16).
#include <type_traits>
#include <algorithm>
#include <vector>

#include "model.cuh"
#include "gemm.cuh"

namespace scd {

namespace {

template <class T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <class T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

struct SeqState {             // where window inputs and positions come from
    const int *ids;           // explicit [Q][Mq] or NULL
    const int *n_known;       // [B]
    const int *tokens;        // [B][token_stride] conditional stream record
    const int *tokens_u;      // [B][prompt_cap] unconditional prompt
    const int *drafts;        // [B][L]
    int token_stride, prompt_cap, prompt_len, L, B, Mq, pos_override, vocab_in;
    const int *skip;          // all sequences finished: nothing to do
};

__device__ __forceinline__ int base_position(const SeqState &s, int q)
{
    return s.pos_override >= 0 ? s.pos_override : s.n_known[q % s.B] - 1;
}

// ---- window input assembly + embedding gather ---------------------------------------------
// Inputs of a stream-sequence are [x_{n-1}, D_0 .. D_{L-2}]: the last committed token, then the
// drafts; the unconditional stream sees its own (masked) prompt but the same generated tokens.
// With `gain` (bf16 sessions) the kernel also prepares the first RMSNorm for the GEMM that follows:
// xg = bf16(h * gain) and the row's sum of squares (one "partial").
constexpr int EMBED_THREADS = 512;      // a row of the table is one latency-bound read: many loads in flight
// `lo_plane` > 0: xg is kept as two planes, xg[lo_plane + .] = T(x - T(x)).
template <class T>
__global__ void __launch_bounds__(EMBED_THREADS) embed_kernel(SeqState s, const T *__restrict__ emb, float *__restrict__ h, int d,
                             const T *__restrict__ gain, T *__restrict__ xg, float *__restrict__ ss_out, long long lo_plane)
{
    __shared__ float red[EMBED_THREADS / 32];
    pdl_trigger();
    if (s.skip && *s.skip) return;
    const int r = blockIdx.x, q = r / s.Mq, i = r % s.Mq;
    int id;
    if (s.ids) {
        id = s.ids[r];
    } else if (s.pos_override >= 0) {
        // prefill: the prompt as recorded on the device (the unconditional stream has its own prompt)
        const int b = q % s.B, stream = q / s.B, pos = s.pos_override + i;
        id = stream == 1 ? s.tokens_u[(size_t)b * s.prompt_cap + pos] : s.tokens[(size_t)b * s.token_stride + pos];
    } else {
        const int b = q % s.B, stream = q / s.B;
        if (i == 0) {
            const int last = s.n_known[b] - 1;
            id = (stream == 1 && last < s.prompt_len) ? s.tokens_u[(size_t)b * s.prompt_cap + last]
                                                      : s.tokens[(size_t)b * s.token_stride + last];
        } else {
            id = (i - 1 < s.L) ? s.drafts[(size_t)b * s.L + i - 1] : 0;
        }
    }
    id = min(max(id, 0), s.vocab_in - 1);
    const T *src = emb + (size_t)id * d;
    float *dst = h + (size_t)r * d;
    float ss = 0.f;
    for (int j = threadIdx.x; j < d; j += blockDim.x) {
        const float v = to_f<T>(src[j]);
        dst[j] = v;
        if (gain) {
            const float x = v * to_f<T>(gain[j]);
            const T hi = from_f<T>(x);
            xg[(size_t)r * d + j] = hi;
            if (lo_plane > 0) xg[lo_plane + (size_t)r * d + j] = from_f<T>(x - to_f<T>(hi));
            ss += v * v;
        }
    }
    if (gain) {
        ss = warp_sum_f(ss);
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
        __syncthreads();
        if (threadIdx.x == 0) {
            float t = 0.f;                       // fixed order: the sum does not depend on scheduling
#pragma unroll
            for (int w = 0; w < EMBED_THREADS / 32; ++w) t += red[w];
            ss_out[r] = t;
        }
    }
}

// ---- RMSNorm: y = x / sqrt(mean(x^2) + eps) * g --------------------------------------------
template <class T>
__global__ void rmsnorm_kernel(const float *__restrict__ h, const T *__restrict__ g, T *__restrict__ y,
                               int d, float eps)
{
    __shared__ float red[32];
    pdl_trigger();
    const int r = blockIdx.x;
    const float *x = h + (size_t)r * d;
    float ss = 0.f;
    for (int j = threadIdx.x; j < d; j += blockDim.x) { const float v = x[j]; ss += v * v; }
    ss = warp_sum_f(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) tot += red[i];
    const float inv = 1.0f / sqrtf(tot / (float)d + eps);
    for (int j = threadIdx.x; j < d; j += blockDim.x)
        y[(size_t)r * d + j] = from_f<T>(x[j] * inv * to_f<T>(g[j]));
}

// ---- plain fp32-accumulate GEMM y[M,N] (+)= x[M,K] W[N,K]^T (fp32 models; any shape) --------
enum { EPI_STORE_T = 0, EPI_STORE_F32 = 1, EPI_ADD_F32 = 2 };

template <class T, int EPI>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const T *__restrict__ x, const T *__restrict__ w,
                                                        void *__restrict__ y, int M, int N, int K, int ldy)
{
    __shared__ float xs[32][33], ws[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int m0 = blockIdx.y * 32, n0 = blockIdx.x * 32;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int k0 = 0; k0 < K; k0 += 32) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int rr = ty + 8 * j, kk = k0 + tx;
            xs[rr][tx] = (m0 + rr < M && kk < K) ? to_f<T>(x[(size_t)(m0 + rr) * K + kk]) : 0.f;
            ws[rr][tx] = (n0 + rr < N && kk < K) ? to_f<T>(w[(size_t)(n0 + rr) * K + kk]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 32; ++kk) {
            const float bv = ws[tx][kk];
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[j] = fmaf(xs[ty + 8 * j][kk], bv, acc[j]);
        }
        __syncthreads();
    }
    const int n = n0 + tx;
    if (n >= N) return;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int m = m0 + ty + 8 * j;
        if (m >= M) continue;
        const size_t o = (size_t)m * ldy + n;
        if (EPI == EPI_STORE_T) ((T *)y)[o] = from_f<T>(acc[j]);
        else if (EPI == EPI_STORE_F32) ((float *)y)[o] = acc[j];
        else ((float *)y)[o] += acc[j];
    }
}

template <class T, int EPI>
void gemm_simt(const T *x, const void *w, void *y, int M, int N, int K, int ldy, cudaStream_t st)
{
    dim3 grid((N + 31) / 32, (M + 31) / 32);
    gemm_simt_kernel<T, EPI><<<grid, 256, 0, st>>>(x, (const T *)w, y, M, N, K, ldy);
    count_launches(1);
}

// ---- RoPE on Q and K, KV-cache write --------------------------------------------------------
// Pairs (i, i + dh/2), angle = pos * base^(-2i/dh); K is cached after rotation. The window's K/V
// land in cache slots [kv_len, kv_len + Mq): committing a prefix is then only a counter update.
struct KvLayout {
    void *k_pool, *v_pool;        // this layer's pools
    const int *page_table;        // [Q][pages_per_seq]
    int pages_per_seq, page_tokens, page_shift, n_kv_heads, head_dim, max_seq;
};

template <class T>
__device__ __forceinline__ size_t kv_offset(const KvLayout &kv, int q, int pos, int kvh)
{
    const int page = kv.page_table[(size_t)q * kv.pages_per_seq + (pos >> kv.page_shift)];
    return (((size_t)page * kv.n_kv_heads + kvh) * kv.page_tokens + (pos & (kv.page_tokens - 1))) * kv.head_dim;
}

// TQ: type of the projections in qkv (fp32 when they come from the tensor-core GEMM, else T).
template <class T, class TQ>
__global__ void rope_kv_kernel(SeqState s, TQ *__restrict__ qkv, KvLayout kv, const float2 *__restrict__ rope,
                               int n_heads)
{
    pdl_trigger();
    const int r = blockIdx.x, q = r / s.Mq, i = r % s.Mq;
    const int dh = kv.head_dim, half = dh >> 1, Hkv = kv.n_kv_heads;
    const int pos = base_position(s, q) + i;
    const bool in_range = pos >= 0 && pos < kv.max_seq;
    const int pc = min(max(pos, 0), kv.max_seq - 1);
    const float2 *cs = rope + (size_t)pc * half;
    TQ *row = qkv + (size_t)r * (n_heads + 2 * Hkv) * dh;
    // Q heads: rotate in place
    for (int e = threadIdx.x; e < n_heads * half; e += blockDim.x) {
        const int hh = e / half, j = e % half;
        TQ *v = row + (size_t)hh * dh;
        const float a = to_f<TQ>(v[j]), b = to_f<TQ>(v[j + half]);
        const float2 t = cs[j];
        v[j] = from_f<TQ>(a * t.x - b * t.y);
        v[j + half] = from_f<TQ>(b * t.x + a * t.y);
    }
    if (!in_range) return;
    // K heads: rotate into the cache; V heads: copy into the cache
    const TQ *krow = row + (size_t)n_heads * dh, *vrow = krow + (size_t)Hkv * dh;
    for (int e = threadIdx.x; e < Hkv * half; e += blockDim.x) {
        const int hh = e / half, j = e % half;
        const float a = to_f<TQ>(krow[hh * dh + j]), b = to_f<TQ>(krow[hh * dh + j + half]);
        const float2 t = cs[j];
        const size_t o = kv_offset<T>(kv, q, pos, hh);
        ((T *)kv.k_pool)[o + j] = from_f<T>(a * t.x - b * t.y);
        ((T *)kv.k_pool)[o + j + half] = from_f<T>(b * t.x + a * t.y);
        ((T *)kv.v_pool)[o + j] = from_f<T>(to_f<TQ>(vrow[hh * dh + j]));
        ((T *)kv.v_pool)[o + j + half] = from_f<T>(to_f<TQ>(vrow[hh * dh + j + half]));
    }
}

// ---- causal window attention over the paged KV cache ----------------------------------------
// Query i of a stream-sequence sits at position base + i and attends to cache entries
// 0 .. base + i (its own K/V were just written). One CTA per (stream-sequence, head, tile of
// AQ queries); keys stream through shared memory in tiles of 32; online softmax in fp32.
constexpr int AQ = 16;           // queries per CTA (4 warps x 4 queries)
constexpr int AKT = 32;          // keys per tile

// `lo_plane` > 0: the output is kept as two planes (out[lo_plane + .] = T(o - T(o))).
template <class T, class TQ>
__global__ void __launch_bounds__(128) attention_kernel(SeqState s, const TQ *__restrict__ qkv, KvLayout kv,
                                                        T *__restrict__ out, int n_heads, float scale, long long lo_plane)
{
    extern __shared__ float smem[];
    pdl_trigger();
    const int dh = kv.head_dim, Hkv = kv.n_kv_heads;
    const int dpl = dh / 32;                          // dims per lane (head_dim multiple of 32)
    float *qs = smem;                                 // [AQ][dh]
    float *ks = qs + AQ * dh;                         // [AKT][dh+1]
    float *vs = ks + AKT * (dh + 1);                  // [AKT][dh]
    const int q = blockIdx.x / n_heads, hh = blockIdx.x % n_heads;
    const int kvh = hh / (n_heads / Hkv);
    const int i0 = blockIdx.y * AQ;
    const int nq = min(AQ, s.Mq - i0);
    const int base = base_position(s, q);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const size_t qstride = (size_t)(n_heads + 2 * Hkv) * dh;

    for (int e = tid; e < nq * dh; e += blockDim.x) {
        const int qi = e / dh, j = e % dh;
        qs[qi * dh + j] = to_f<TQ>(qkv[((size_t)q * s.Mq + i0 + qi) * qstride + (size_t)hh * dh + j]) * scale;
    }
    float m[4], l[4], acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        m[a] = -INFINITY; l[a] = 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[a][c] = 0.f;
    }
    const int n_keys = min(base + i0 + nq, kv.max_seq);   // keys 0 .. position of the last query
    for (int k0 = 0; k0 < n_keys; k0 += AKT) {
        __syncthreads();
        for (int e = tid; e < AKT * dh; e += blockDim.x) {
            const int kj = e / dh, j = e % dh;
            const int pos = k0 + kj;
            float kvv = 0.f, vvv = 0.f;
            if (pos < n_keys) {
                const size_t o = kv_offset<T>(kv, q, pos, kvh) + j;
                kvv = to_f<T>(((const T *)kv.k_pool)[o]);
                vvv = to_f<T>(((const T *)kv.v_pool)[o]);
            }
            ks[kj * (dh + 1) + j] = kvv;
            vs[kj * dh + j] = vvv;
        }
        __syncthreads();
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            const int qi = warp * 4 + a;
            if (qi >= nq) continue;                    // warp-uniform
            const int qpos = base + i0 + qi;
            const int kpos = k0 + lane;
            float sc = -INFINITY;
            if (kpos <= qpos && kpos < n_keys) {
                float dot = 0.f;
                const float *qv = qs + qi * dh, *kvp = ks + lane * (dh + 1);
                for (int j = 0; j < dh; ++j) dot = fmaf(qv[j], kvp[j], dot);
                sc = dot;
            }
            const float mt = warp_max(sc);
            if (mt == -INFINITY) continue;             // whole tile masked for this query
            const float m_new = fmaxf(m[a], mt);
            const float corr = expf(m[a] - m_new);
            const float pj = sc == -INFINITY ? 0.f : expf(sc - m_new);
            l[a] = l[a] * corr + warp_sum_f(pj);
            m[a] = m_new;
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[a][c] *= corr;
            for (int j = 0; j < AKT; ++j) {
                const float pb = __shfl_sync(0xffffffffu, pj, j);
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (c < dpl) acc[a][c] = fmaf(pb, vs[j * dh + lane + 32 * c], acc[a][c]);
            }
        }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int qi = warp * 4 + a;
        if (qi >= nq) continue;
        const float inv = l[a] > 0.f ? 1.0f / l[a] : 0.f;
        T *o = out + ((size_t)q * s.Mq + i0 + qi) * (size_t)n_heads * dh + (size_t)hh * dh;
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (c < dpl) {
                const float x = acc[a][c] * inv;
                const T hi = from_f<T>(x);
                o[lane + 32 * c] = hi;
                if (lo_plane > 0) o[lo_plane + lane + 32 * c] = from_f<T>(x - to_f<T>(hi));
            }
    }
}

// ---- SwiGLU: act = silu(gate) * up -----------------------------------------------------------
template <class T>
__global__ void swiglu_kernel(const T *__restrict__ gu, T *__restrict__ act, int F, long long total)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    const long long r = i / F;
    const int j = (int)(i % F);
    const float g = to_f<T>(gu[r * 2 * F + j]), u = to_f<T>(gu[r * 2 * F + F + j]);
    act[i] = from_f<T>(g / (1.0f + expf(-g)) * u);
}

__global__ void rope_table_kernel(float2 *table, int max_seq, int half, int dh, double base)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)max_seq * half) return;
    const int pos = (int)(i / half), j = (int)(i % half);
    const double theta = pow(base, -2.0 * (double)j / (double)dh);
    double sn, cs;
    sincos((double)pos * theta, &sn, &cs);
    table[i] = make_float2((float)cs, (float)sn);
}

template <class T>
int forward_impl(scd_session *s, const ForwardArgs &a, cudaStream_t st)
{
    scd_model *m = s->model;
    const scd_model_config_t &c = m->cfg;
    const int d = c.d_model, H = c.n_heads, Hkv = c.n_kv_heads, dh = c.head_dim, F = c.d_ffn;
    const int dq = H * dh, dkv = Hkv * dh, dqkv = dq + 2 * dkv;
    const int rows = s->Q * a.Mq;
    const bool tc = std::is_same<T, __nv_bfloat16>::value && m->gemm_plan != nullptr;

    SeqState ss;
    ss.ids = a.ids; ss.n_known = s->n_known; ss.tokens = s->tokens; ss.tokens_u = s->tokens_u;
    ss.drafts = s->drafts; ss.token_stride = c.max_seq; ss.prompt_cap = c.max_seq;
    ss.prompt_len = s->prompt_len; ss.L = s->L; ss.B = s->B; ss.Mq = a.Mq;
    ss.pos_override = a.pos_override; ss.vocab_in = c.vocab_in; ss.skip = a.skip;

    T *xn = (T *)s->xn, *qkv = (T *)s->qkv, *att = (T *)s->att, *gu = (T *)s->gu, *act = (T *)s->act;
    StepProfiler *prof = a.prof;
#define MARK(c) do { if (prof) prof->mark(c); } while (0)
    MARK(PROF_EMBED);
    // tensor-core path: the norms are folded into the GEMMs (see gemm.cuh); `parts` = partial sums
    // of squares the producer of xn left per row
    int parts = 1;
    embed_kernel<T><<<rows, EMBED_THREADS, 0, st>>>(ss, (const T *)m->tok_emb, s->h, d,
                                          tc ? (const T *)m->attn_norm[0] : nullptr, xn, s->ss,
                                          tc ? (long long)s->rows_cap * d : 0ll);
    count_launches(1);

    KvLayout kv;
    kv.page_table = s->page_table; kv.pages_per_seq = s->pages_per_seq;
    kv.page_tokens = c.kv_page_tokens; kv.page_shift = __builtin_ctz((unsigned)c.kv_page_tokens);
    kv.n_kv_heads = Hkv; kv.head_dim = dh; kv.max_seq = c.max_seq;
    const size_t att_smem = (size_t)(AQ * dh + AKT * (dh + 1) + AKT * dh) * sizeof(float);
    const float scale = 1.0f / sqrtf((float)dh);

    for (int l = 0; l < c.n_layers; ++l) {
        kv.k_pool = (T *)s->kv_pool + (size_t)l * s->kv_layer_stride;
        kv.v_pool = (T *)kv.k_pool + s->kv_kind_stride;
        if (!tc) {
            MARK(PROF_RMSNORM);
            rmsnorm_kernel<T><<<rows, 256, 0, st>>>(s->h, (const T *)m->attn_norm[l], xn, d, c.rms_eps);
            count_launches(1);
        }
        MARK(PROF_GEMM_QKV);
        if (tc) {
            int rc = gemm_tc_qkv(s, l, rows, parts, st);
            if (rc != SCD_OK) return rc;
        } else {
            gemm_simt<T, EPI_STORE_T>(xn, m->wq[l], qkv, rows, dq, d, dqkv, st);
            gemm_simt<T, EPI_STORE_T>(xn, m->wk[l], qkv + dq, rows, dkv, d, dqkv, st);
            gemm_simt<T, EPI_STORE_T>(xn, m->wv[l], qkv + dq + dkv, rows, dkv, d, dqkv, st);
        }
        if (tc && attention_tc_supported(s, a.Mq)) {
            MARK(PROF_ATTENTION);
            int rc = attention_tc(s, l, a.Mq, a.pos_override, st);
            if (rc != SCD_OK) return rc;
        } else {
            MARK(PROF_ROPE_KV);
            dim3 agrid((unsigned)(s->Q * H), (unsigned)((a.Mq + AQ - 1) / AQ));
            if (tc) {
                // (projections in fp32 from the tensor-core GEMM; the output in two planes for the next one)
                rope_kv_kernel<T, float><<<rows, 128, 0, st>>>(ss, (float *)s->qkv, kv, m->rope_table, H);
                count_launches(1);
                MARK(PROF_ATTENTION);
                attention_kernel<T, float><<<agrid, 128, att_smem, st>>>(ss, (const float *)s->qkv, kv, att, H, scale,
                                                                         (long long)s->rows_cap * dq);
            } else {
                rope_kv_kernel<T, T><<<rows, 128, 0, st>>>(ss, qkv, kv, m->rope_table, H);
                count_launches(1);
                MARK(PROF_ATTENTION);
                attention_kernel<T, T><<<agrid, 128, att_smem, st>>>(ss, qkv, kv, att, H, scale, 0ll);
            }
            count_launches(1);
        }
        MARK(PROF_GEMM_O);
        if (tc) {
            int rc = gemm_tc_residual(s, l, /*which=*/0, rows, m->ffn_norm[l], &parts, st);
            if (rc != SCD_OK) return rc;
        } else {
            gemm_simt<T, EPI_ADD_F32>(att, m->wo[l], s->h, rows, d, dq, d, st);
            MARK(PROF_RMSNORM);
            rmsnorm_kernel<T><<<rows, 256, 0, st>>>(s->h, (const T *)m->ffn_norm[l], xn, d, c.rms_eps);
            count_launches(1);
        }
        MARK(PROF_GEMM_GATE_UP);
        if (tc) {
            int rc = gemm_tc_gate_up(s, l, rows, parts, st);
            if (rc != SCD_OK) return rc;
        } else {
            gemm_simt<T, EPI_STORE_T>(xn, m->w_gate[l], gu, rows, F, d, 2 * F, st);
            gemm_simt<T, EPI_STORE_T>(xn, m->w_up[l], gu + F, rows, F, d, 2 * F, st);
            const long long total = (long long)rows * F;
            swiglu_kernel<T><<<(unsigned)((total + 255) / 256), 256, 0, st>>>(gu, act, F, total);
            count_launches(1);
        }
        MARK(PROF_GEMM_DOWN);
        if (tc) {
            int rc = gemm_tc_residual(s, l, /*which=*/1, rows,
                                      l + 1 < c.n_layers ? m->attn_norm[l + 1] : m->final_norm, &parts, st);
            if (rc != SCD_OK) return rc;
        } else {
            gemm_simt<T, EPI_ADD_F32>(act, m->w_down[l], s->h, rows, d, F, d, st);
        }
    }
    MARK(PROF_OTHER);
    if (a.hidden)
        SCD_CUDA_TRY(cudaMemcpyAsync(a.hidden, s->h, (size_t)rows * d * sizeof(float),
                                     cudaMemcpyDeviceToDevice, st));
    if (a.want_logits) {
        if (!tc) {
            MARK(PROF_RMSNORM);
            rmsnorm_kernel<T><<<rows, 256, 0, st>>>(s->h, (const T *)m->final_norm, xn, d, c.rms_eps);
            count_launches(1);
        }
        MARK(PROF_GEMM_LM_HEAD);
        if (tc) {
            const bool all = a.lm_hi <= 0;
            int rc = gemm_tc_lm_head(s, rows, a.logits, all ? 0 : a.lm_lo, all ? c.vocab_out : a.lm_hi,
                                     all ? -1 : a.lm_eol, parts, st);
            if (rc != SCD_OK) return rc;
        } else {
            gemm_simt<T, EPI_STORE_F32>(xn, m->lm_head, a.logits, rows, c.vocab_out, d, c.vocab_out, st);
        }
    }
    MARK(PROF_OTHER);
#undef MARK
    SCD_CUDA_TRY(cudaGetLastError());
    return SCD_OK;
}

}  // namespace

// ---- per-kernel event marks --------------------------------------------------------------------
namespace { thread_local unsigned long long *g_stamp_slot = nullptr; }

unsigned long long *take_stamp_slot()
{
    unsigned long long *p = g_stamp_slot;
    g_stamp_slot = nullptr;
    return p;
}

void StepProfiler::mark(int c)
{
    if (failed) return;
    if (stamps) {
        if (used == cls.size()) cls.push_back(PROF_OTHER);
        cls[used] = c;
        g_stamp_slot = used < stamp_launches ? stamps + used * 2 * STAMP_CTAS : nullptr;
        ++used;
        return;
    }
    if (used == events.size()) {
        cudaEvent_t e;
        if (cudaEventCreate(&e) != cudaSuccess) { failed = true; return; }
        events.push_back(e);
        cls.push_back(PROF_OTHER);
    }
    cls[used] = c;
    if (cudaEventRecord(events[used], st) != cudaSuccess) { failed = true; return; }
    ++used;
}

int StepProfiler::finish(float *ms_by_class, int *launches_by_class)
{
    if (stamps) {
        g_stamp_slot = nullptr;
        SCD_CUDA_TRY(cudaStreamSynchronize(st));
        const size_t n = std::min(used, stamp_launches);
        std::vector<unsigned long long> h(n * 2 * STAMP_CTAS);
        SCD_CUDA_TRY(cudaMemcpy(h.data(), stamps, h.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
        unsigned long long prev_end = 0;
        for (size_t i = 0; i < n; ++i) {
            unsigned long long first = ~0ull, last = 0;
            for (int c = 0; c < STAMP_CTAS; ++c) {
                const unsigned long long a = h[(i * 2) * STAMP_CTAS + c], b = h[(i * 2 + 1) * STAMP_CTAS + c];
                if (a) first = std::min(first, a);
                last = std::max(last, b);
            }
            if (last == 0) continue;                   // a kernel that leaves no stamps: charged to the next one
            if (prev_end == 0) prev_end = first;       // the first stamped kernel starts the clock
            if (last > prev_end) ms_by_class[cls[i]] += (float)((double)(last - prev_end) * 1e-6);
            launches_by_class[cls[i]] += 1;
            prev_end = std::max(prev_end, last);
        }
        used = 0;
        return SCD_OK;
    }
    mark(PROF_OTHER);
    SCD_REQUIRE(!failed, SCD_ERR_CUDA, "step profiler: event creation or record failed");
    SCD_CUDA_TRY(cudaEventSynchronize(events[used - 1]));
    for (size_t i = 0; i + 1 < used; ++i) {
        float ms = 0.f;
        SCD_CUDA_TRY(cudaEventElapsedTime(&ms, events[i], events[i + 1]));
        ms_by_class[cls[i]] += ms;
        launches_by_class[cls[i]] += 1;
    }
    used = 0;
    return SCD_OK;
}

StepProfiler::~StepProfiler()
{
    for (cudaEvent_t e : events) cudaEventDestroy(e);
}

int run_forward(scd_session *s, const ForwardArgs &a, cudaStream_t st)
{
    s->skip_now = a.skip;
    if (s->model->cfg.dtype == SCD_F32) return forward_impl<float>(s, a, st);
    return forward_impl<__nv_bfloat16>(s, a, st);
}

int build_rope_table(scd_model *m)
{
    const int half = m->cfg.head_dim / 2;
    const long long n = (long long)m->cfg.max_seq * half;
    SCD_CUDA_TRY(cudaMalloc(&m->rope_table, (size_t)n * sizeof(float2)));
    rope_table_kernel<<<(unsigned)((n + 255) / 256), 256>>>(m->rope_table, m->cfg.max_seq, half,
                                                            m->cfg.head_dim, (double)m->cfg.rope_base);
    SCD_CUDA_TRY(cudaGetLastError());
    SCD_CUDA_TRY(cudaDeviceSynchronize());
    return SCD_OK;
}

}  // namespace scd
