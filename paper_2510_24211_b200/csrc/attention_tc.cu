// Window attention over the paged KV cache for bf16 models (the parallel forward of Algorithm 6: every window
// position is evaluated in one pass, "masked attention" over the committed prefix plus the causal
// window), fused with RoPE and the KV-cache write of the window rows.
//
// One thread-block cluster per (stream-sequence, KV head); the committed context [0, base) is cut
// into tiles of 64 keys that are dealt to the CTAs of the cluster (split-KV); the last CTA of
// the cluster also owns the window rows: it rotates their keys, stores K and V into the cache
// slots [base, base + Mq) and attends to them under the causal mask.
//   - K/V tiles come from the cache by TMA (64 keys x 64 dims per box, 128-byte swizzle) through
//     a ring of shared-memory slots with full/empty mbarriers; the first slots are requested
//     before griddepcontrol.wait, because the cache of earlier iterations does not depend on
//     the QKV projection that runs in front of this kernel.
//   - one warp per 16 query rows: S = Q K^T and O += P V on mma.sync m16n8k16 (bf16 in, fp32
//     accumulate), online softmax in fp32 with base-2 exponentials. The rotated, scaled queries are
//     kept as two bf16 planes (value and remainder) and S = Q_hi K^T + Q_lo K^T: the queries are the
//     one operand of the scores that is not bound to the cache's bf16, and their rounding was a
//     measurable part of the distance to an fp32 evaluation at full depth.
//   - each CTA leaves (max, sum, unnormalised O) of its key range in shared memory; after a
//     cluster barrier CTA c merges the query rows [c R / C, (c+1) R / C) over all peers through
//     distributed shared memory in peer order, normalises and stores bf16.
//   - for long contexts a second variant of the kernel puts two warps on every query tile (each
//     takes half of the keys of a tile); the host chooses the variant per launch.
// Every mbarrier wait is bounded; on expiry an error word is raised and the CTA still meets its
// cluster at the barriers.
#include <cuda.h>
#include <cstring>
#include <algorithm>

#include "model.cuh"
#include "gemm.cuh"

namespace scd {

namespace {

constexpr int TK = 64;                 // keys per tile
constexpr int MAX_ATT_STAGES = 8;
constexpr unsigned ATT_SPIN_LIMIT = 1u << 22;

struct AttnParams {
    CUtensorMap kv_map;                // the whole pool as a 2-D bf16 matrix [rows][head_dim]
    const float *qkv;                  // [rows][(H + 2 Hkv) dh] fp32 projections, Q and K not yet rotated
    __nv_bfloat16 *out;                // [rows][H dh], hi plane; the lo plane (bf16 of the remainder) out_plane elements on
    long long out_plane;
    __nv_bfloat16 *pool;               // KV pool base (window rows are stored with plain stores)
    const int *page_table;             // [Q][pages_per_seq]
    const int *n_known;                // [B]
    const float2 *rope;                // [max_seq][dh/2] (cos, sin)
    int *err;
    const int *skip;                   // optional device flag: set = nothing to do, return at once
    long long row0_k, row0_v;          // pool row of (this layer, K | V, page 0, head 0, token 0)
    int B, Mq, H, Hkv, n_rep, pages_per_seq, page_tokens, page_shift, max_seq, pos_override;
    int C, stages, stages_v, n_mtiles;   // (stages_v: the tcgen05 kernel's V ring; its K ring has `stages` slots)
    float qscale;                      // log2(e) / sqrt(dh)
    unsigned long long *stamp;         // optional [2][STAMP_CTAS]: %globaltimer at CTA entry and exit
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, unsigned parity)
{
    const uint32_t a = smem_u32(bar);
    for (unsigned i = 0; i < ATT_SPIN_LIMIT; ++i) {
        unsigned ok;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(a), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}
__device__ __forceinline__ void tma_load_2d(const CUtensorMap *map, uint64_t *bar, void *dst, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes"
                 " [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(smem_u32(dst)), "l"((uint64_t)map), "r"(smem_u32(bar)), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_peer(uint32_t local_smem_addr, uint32_t peer)
{
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_smem_addr), "r"(peer));
    return remote;
}
__device__ __forceinline__ float ld_cluster_f32(uint32_t addr)
{
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
    return v;
}

__device__ __forceinline__ float4 ld_cluster_f32x4(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// Byte offset of element (row, col) in a buffer made of sub-tiles of 64 columns: sub-tile h holds
// `rows` rows of 128 bytes whose 16-byte chunks are XOR-swizzled with the row (the layout TMA
// writes with the 128-byte swizzle when every sub-tile starts on a 1024-byte boundary).
__device__ __forceinline__ uint32_t sw_off(int rows, int row, int col)
{
    const int h = col >> 6, c = (col >> 3) & 7, e = col & 7;
    return (uint32_t)(h * rows * 128 + row * 128 + (((c ^ (row & 7)) << 4)) + e * 2);
}

// RoPE on 8 consecutive pairs (x[j], y[j]) = (dims j0.., dims j0 + dh/2 ..) of an fp32 projection row:
// 16-byte loads of the two halves and of the (cos, sin) table; rotated in fp32, scaled, rounded to bf16 once.
__device__ __forceinline__ uint32_t pack_bf16_rest(float lo, float hi);
// (rest_lo / rest_hi, when given, receive what the rounding dropped, as bf16: the second plane)
struct Rope8 { float4 t0, t1, t2, t3; };                         // (cos, sin) of 8 consecutive pairs
__device__ __forceinline__ Rope8 load_rope8(const float2 *cs)
{
    Rope8 r;
    r.t0 = *(const float4 *)(cs); r.t1 = *(const float4 *)(cs + 2); r.t2 = *(const float4 *)(cs + 4); r.t3 = *(const float4 *)(cs + 6);
    return r;
}
__device__ __forceinline__ void rotate8(const float *xlo, const float *xhi, const Rope8 &rp,
                                        float scale, uint4 &out_lo, uint4 &out_hi, uint4 *rest_lo = nullptr,
                                        uint4 *rest_hi = nullptr)
{
    const float4 a0 = *(const float4 *)xlo, a1 = *(const float4 *)(xlo + 4);
    const float4 b0 = *(const float4 *)xhi, b1 = *(const float4 *)(xhi + 4);
    const float4 t0 = rp.t0, t1 = rp.t1, t2 = rp.t2, t3 = rp.t3;
    const float c[8] = {t0.x, t0.z, t1.x, t1.z, t2.x, t2.z, t3.x, t3.z};
    const float sn[8] = {t0.y, t0.w, t1.y, t1.w, t2.y, t2.w, t3.y, t3.w};
    const float x[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
    const float y[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
    uint32_t lo[4], hi[4], rlo[4], rhi[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float l0 = (x[2 * k] * c[2 * k] - y[2 * k] * sn[2 * k]) * scale;
        const float l1 = (x[2 * k + 1] * c[2 * k + 1] - y[2 * k + 1] * sn[2 * k + 1]) * scale;
        const float h0 = (y[2 * k] * c[2 * k] + x[2 * k] * sn[2 * k]) * scale;
        const float h1 = (y[2 * k + 1] * c[2 * k + 1] + x[2 * k + 1] * sn[2 * k + 1]) * scale;
        lo[k] = pack_bf16(l0, l1);
        hi[k] = pack_bf16(h0, h1);
        rlo[k] = pack_bf16_rest(l0, l1);
        rhi[k] = pack_bf16_rest(h0, h1);
    }
    out_lo = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    out_hi = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    if (rest_lo) { *rest_lo = make_uint4(rlo[0], rlo[1], rlo[2], rlo[3]); *rest_hi = make_uint4(rhi[0], rhi[1], rhi[2], rhi[3]); }
}
__device__ __forceinline__ void rotate8(const float *xlo, const float *xhi, const float2 *cs,
                                        float scale, uint4 &out_lo, uint4 &out_hi, uint4 *rest_lo = nullptr,
                                        uint4 *rest_hi = nullptr)
{
    rotate8(xlo, xhi, load_rope8(cs), scale, out_lo, out_hi, rest_lo, rest_hi);
}
// 8 consecutive fp32 values as bf16
__device__ __forceinline__ uint4 round8(const float *x)
{
    const float4 a = *(const float4 *)x, b = *(const float4 *)(x + 4);
    return make_uint4(pack_bf16(a.x, a.y), pack_bf16(a.z, a.w), pack_bf16(b.x, b.y), pack_bf16(b.z, b.w));
}
// the part of (lo, hi) that bf16 drops, as bf16: the second plane of a two-plane activation
__device__ __forceinline__ uint32_t pack_bf16_rest(float lo, float hi)
{
    return pack_bf16(lo - __bfloat162float(__float2bfloat16_rn(lo)), hi - __bfloat162float(__float2bfloat16_rn(hi)));
}

template <int DH>
struct WarpState {
    uint32_t qf[DH / 16][4];     // Q fragments of this warp's 16 rows
    float o[DH / 8][4];          // unnormalised output
    float m[2], l[2];            // running max / sum of rows g and g + 8
    uint32_t qlo_base;           // shared-memory address of the queries' remainder plane
    int q_rows, q_row;           // its row count (padded) and the row this lane addresses in ldmatrix
};

// One tile of TK keys: S = Q K^T, masking, online softmax, O += P V.
//   kbase / vbase : shared-memory byte addresses of the K and V tiles
//   allowed(row_slot, key) decides the mask; row_slot 0 -> row g, 1 -> row g + 8
//   KEYS keys starting at kbase / vbase (the whole tile, or one warp's half of it); koff = index of
//   the first of them inside the tile, for the mask
template <int DH, int KEYS, class Mask>
__device__ __forceinline__ void process_keys(WarpState<DH> &w, uint32_t kbase, uint32_t vbase, int lane, int koff,
                                             bool need_mask, const Mask &allowed)
{
    float s[KEYS / 8][4];
#pragma unroll
    for (int n = 0; n < KEYS / 8; ++n) { s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f; }
    // ---- S = Q_hi K^T + Q_lo K^T (the remainder fragments come from shared memory, one per K step) ----
#pragma unroll
    for (int ks = 0; ks < DH / 16; ++ks) {
        uint32_t ql[4];
        ldsm_x4(w.qlo_base + sw_off(w.q_rows, w.q_row, ks * 16 + ((lane >> 4) << 3)), ql[0], ql[1], ql[2], ql[3]);
#pragma unroll
        for (int n2 = 0; n2 < KEYS / 16; ++n2) {
            const int key = n2 * 16 + ((lane >> 4) << 3) + (lane & 7);
            const int col = ks * 16 + (((lane >> 3) & 1) << 3);
            uint32_t b0, b1, b2, b3;
            ldsm_x4(kbase + sw_off(TK, key, col), b0, b1, b2, b3);
            mma_bf16(s[2 * n2], w.qf[ks], b0, b1);
            mma_bf16(s[2 * n2 + 1], w.qf[ks], b2, b3);
            mma_bf16(s[2 * n2], ql, b0, b1);
            mma_bf16(s[2 * n2 + 1], ql, b2, b3);
        }
    }
    // ---- mask ----
    if (need_mask) {
#pragma unroll
        for (int n = 0; n < KEYS / 8; ++n) {
            const int key = koff + n * 8 + 2 * (lane & 3);
            if (!allowed(0, key)) s[n][0] = -INFINITY;
            if (!allowed(0, key + 1)) s[n][1] = -INFINITY;
            if (!allowed(1, key)) s[n][2] = -INFINITY;
            if (!allowed(1, key + 1)) s[n][3] = -INFINITY;
        }
    }
    // ---- online softmax (scores are already in units of log2) ----
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int n = 0; n < KEYS / 8; ++n) {
        mx[0] = fmaxf(mx[0], fmaxf(s[n][0], s[n][1]));
        mx[1] = fmaxf(mx[1], fmaxf(s[n][2], s[n][3]));
    }
    float scale[2], msafe[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
        mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
        const float m_new = fmaxf(w.m[h], mx[h]);
        msafe[h] = m_new == -INFINITY ? 0.f : m_new;
        scale[h] = exp2f(w.m[h] - msafe[h]);          // m = -inf -> 0
        w.m[h] = m_new;
    }
    float sum[2] = {0.f, 0.f};
#pragma unroll
    for (int n = 0; n < KEYS / 8; ++n) {
        s[n][0] = exp2f(s[n][0] - msafe[0]);
        s[n][1] = exp2f(s[n][1] - msafe[0]);
        s[n][2] = exp2f(s[n][2] - msafe[1]);
        s[n][3] = exp2f(s[n][3] - msafe[1]);
        sum[0] += s[n][0] + s[n][1];
        sum[1] += s[n][2] + s[n][3];
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        sum[h] += __shfl_xor_sync(0xffffffffu, sum[h], 1);
        sum[h] += __shfl_xor_sync(0xffffffffu, sum[h], 2);
        w.l[h] = w.l[h] * scale[h] + sum[h];
    }
#pragma unroll
    for (int j = 0; j < DH / 8; ++j) {
        w.o[j][0] *= scale[0]; w.o[j][1] *= scale[0];
        w.o[j][2] *= scale[1]; w.o[j][3] *= scale[1];
    }
    // ---- O += P V ----
#pragma unroll
    for (int t = 0; t < KEYS / 16; ++t) {
        uint32_t a[4];
        a[0] = pack_bf16(s[2 * t][0], s[2 * t][1]);
        a[1] = pack_bf16(s[2 * t][2], s[2 * t][3]);
        a[2] = pack_bf16(s[2 * t + 1][0], s[2 * t + 1][1]);
        a[3] = pack_bf16(s[2 * t + 1][2], s[2 * t + 1][3]);
        const int key = t * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
#pragma unroll
        for (int j2 = 0; j2 < DH / 16; ++j2) {
            const int col = j2 * 16 + ((lane >> 4) << 3);
            uint32_t b0, b1, b2, b3;
            ldsm_x4_t(vbase + sw_off(TK, key, col), b0, b1, b2, b3);
            mma_bf16(w.o[2 * j2], a, b0, b1);
            mma_bf16(w.o[2 * j2 + 1], a, b2, b3);
        }
    }
}

// One tile for a warp: all TK keys, or - with two warps per query tile - the half `kh` of them.
template <int DH, int KS, class Mask>
__device__ __forceinline__ void process_tile(WarpState<DH> &w, uint32_t kbase, uint32_t vbase, int lane, int kh,
                                             bool need_mask, const Mask &allowed)
{
    // (a half starts TK / 2 rows = TK / 2 * 128 bytes into the swizzled tiles; the swizzle pattern
    // repeats every 8 rows, so the offset goes into the base addresses and the index arithmetic
    // inside stays compile-time)
    if (KS == 2) {
        const uint32_t off = (uint32_t)kh * (TK / 2) * 128u;
        process_keys<DH, TK / 2>(w, kbase + off, vbase + off, lane, kh * (TK / 2), need_mask, allowed);
    } else {
        process_keys<DH, TK>(w, kbase, vbase, lane, 0, need_mask, allowed);
    }
}

// KS = 1: one warp per 16-row query tile. KS = 2 (long contexts, at most two query tiles): two warps
// per query tile, each taking half of the keys of every tile; the two are folded together before
// the cluster merge. That halves the tile loop; it pays from about four key tiles per CTA on
// (measured on the 7B-shaped model: -0.12 ms per iteration at 2200 tokens of context, +0.03 ms at 120).
template <int DH, int KS>
__global__ void __launch_bounds__(256) attention_tc_kernel(const __grid_constant__ AttnParams p)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];          // 128-byte swizzle: tiles start on 1024-byte boundaries
    __shared__ uint64_t full_bar[MAX_ATT_STAGES], empty_bar[MAX_ATT_STAGES];
    __shared__ int abort_flag;

    pdl_trigger();                     // the GEMM behind may take the SM slots this grid leaves free
    if (p.skip && *p.skip) return;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (p.stamp && tid == 0 && blockIdx.x < STAMP_CTAS) p.stamp[blockIdx.x] = global_timer_ns();
    const int C = p.C, rank = blockIdx.x % C, unit = blockIdx.x / C;
    const int q = unit / p.Hkv, kvh = unit % p.Hkv;
    const int b = q % p.B;
    const int Mq = p.Mq, rows = Mq * p.n_rep, qrows_pad = p.n_mtiles * 16;
    constexpr int half = DH / 2;
    constexpr uint32_t tile_bytes = TK * DH * 2;                  // one K (or V) tile
    constexpr uint32_t stage_bytes = 2 * tile_bytes;

    if ((smem_u32(smem_raw) & 1023u) != 0u) {                     // (the launch asks for no slack to align by hand)
        if (tid == 0) atomicExch(p.err, 6);
        return;
    }
    uint8_t *q_s = smem_raw;                                      // [DH/64][qrows_pad][128 B]: the queries as bf16 ...
    const size_t q_plane = ((size_t)qrows_pad * DH * 2 + 1023) & ~(size_t)1023;
    uint8_t *q_lo_s = q_s + q_plane;                              // ... and what bf16 dropped, same layout
    uint8_t *stages = q_lo_s + q_plane;

    if (tid == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], (unsigned)(p.n_mtiles * KS)); }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // n_known was written by the previous iteration, which is complete before any kernel of this
    // one starts; the cache entries below `base` are older still.
    const int base = p.pos_override >= 0 ? p.pos_override : p.n_known[b] - 1;
    const int ctx = min(max(base, 0), p.max_seq);
    const int n_tiles = (ctx + TK - 1) / TK;
    // The last CTA of the cluster also rotates, stores and attends to the window rows, which costs
    // about as much as three context tiles: it takes that many fewer context tiles.
    const bool has_window = rank == C - 1;
    const int per = (n_tiles + 3 + C - 1) / C;                     // context tiles of the other CTAs
    const int t0 = min(n_tiles, rank * per);
    const int t1 = has_window ? n_tiles : min(n_tiles, (rank + 1) * per);
    const int my_tiles = t1 - t0;

    // warp w < n_mtiles * KS owns query tile w % n_mtiles (and, with KS = 2, the half w / n_mtiles of
    // every key tile); any further warps only help with staging and merging
    const int mt = warp % p.n_mtiles, kh = warp / p.n_mtiles;
    const bool compute = warp < p.n_mtiles * KS;

    const int *pt = p.page_table + (size_t)q * p.pages_per_seq;

    auto issue = [&](int t) {                                     // thread 0 only: request ctx tile t0 + t
        const int s = t % p.stages;
        const int pos = (t0 + t) * TK;
        const int page = pt[pos >> p.page_shift];
        const long long r = ((long long)page * p.Hkv + kvh) * p.page_tokens + (pos & (p.page_tokens - 1));
        uint8_t *dst = stages + (size_t)s * stage_bytes;
        mbar_expect_tx(&full_bar[s], stage_bytes);
#pragma unroll
        for (int h = 0; h < DH / 64; ++h) {
            tma_load_2d(&p.kv_map, &full_bar[s], dst + h * (TK * 128), h * 64, (int)(p.row0_k + r));
            tma_load_2d(&p.kv_map, &full_bar[s], dst + tile_bytes + h * (TK * 128), h * 64, (int)(p.row0_v + r));
        }
    };
    if (tid == 0) {
        const int pre = min(p.stages - 1, my_tiles);
        for (int t = 0; t < pre; ++t) issue(t);
    }

    pdl_wait();                                                   // Q, K, V of the window come from the GEMM in front

    // ---- Q: rotate, scale, stage in shared memory (8 dims of both halves per item, 16-byte accesses) ---
    const size_t qstride = (size_t)(p.H + 2 * p.Hkv) * DH;
    constexpr int CH = half / 8;                                  // 16-byte chunks per half row
#pragma unroll 4
    for (int e = tid; e < qrows_pad * CH; e += blockDim.x) {
        const int rr = e / CH, j0 = (e % CH) * 8;
        uint4 lo = make_uint4(0u, 0u, 0u, 0u), hi = lo, rlo = lo, rhi = lo;
        if (rr < rows) {
            const int i = rr % Mq, g = rr / Mq;
            const int pos = min(max(base + i, 0), p.max_seq - 1);
            const float *src = p.qkv + ((size_t)q * Mq + i) * qstride + (size_t)(kvh * p.n_rep + g) * DH;
            rotate8(src + j0, src + j0 + half, p.rope + (size_t)pos * half + j0, p.qscale, lo, hi, &rlo, &rhi);
        }
        *(uint4 *)(q_s + sw_off(qrows_pad, rr, j0)) = lo;
        *(uint4 *)(q_s + sw_off(qrows_pad, rr, j0 + half)) = hi;
        *(uint4 *)(q_lo_s + sw_off(qrows_pad, rr, j0)) = rlo;
        *(uint4 *)(q_lo_s + sw_off(qrows_pad, rr, j0 + half)) = rhi;
    }
    __syncthreads();

    WarpState<DH> w;
    w.qlo_base = smem_u32(q_lo_s);
    w.q_rows = qrows_pad;
    w.q_row = mt * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
    if (compute) {
        const int row = mt * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks) {
            const int col = ks * 16 + ((lane >> 4) << 3);
            ldsm_x4(smem_u32(q_s) + sw_off(qrows_pad, row, col), w.qf[ks][0], w.qf[ks][1], w.qf[ks][2], w.qf[ks][3]);
        }
    }
#pragma unroll
    for (int j = 0; j < DH / 8; ++j) { w.o[j][0] = w.o[j][1] = w.o[j][2] = w.o[j][3] = 0.f; }
    w.m[0] = w.m[1] = -INFINITY;
    w.l[0] = w.l[1] = 0.f;
    const int g = lane >> 2;
    // query index (inside the window) of this thread's two rows; padding rows behave like row 0
    int qi[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int rr = mt * 16 + g + 8 * h;
        qi[h] = rr < rows ? rr % Mq : 0;
    }

    // ---- committed context --------------------------------------------------------------------------
    bool ok = true;
    for (int t = 0; compute && t < my_tiles; ++t) {
        if (tid == 0 && t + p.stages - 1 < my_tiles) {
            const int tn = t + p.stages - 1, s = tn % p.stages;
            // the slot held tile tn - stages: every warp must have released it
            if (tn >= p.stages && !mbar_wait(&empty_bar[s], ((tn / p.stages) - 1) & 1)) {
                atomicExch(p.err, 4); abort_flag = 1;
            } else {
                issue(tn);
            }
        }
        const int s = t % p.stages;
        if (ok) {
            ok = mbar_wait(&full_bar[s], (t / p.stages) & 1);
            if (!ok) atomicExch(p.err, 5);
        }
        if (ok) {
            const uint32_t kb = smem_u32(stages + (size_t)s * stage_bytes);
            const int valid = ctx - (t0 + t) * TK;                // keys of this tile below the context end
            process_tile<DH, KS>(w, kb, kb + tile_bytes, lane, kh, valid < TK,
                             [&](int, int key) { return key < valid; });
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[s]);
    }

    // ---- the window rows: rotate K, store K and V into the cache, attend under the causal mask -------
    if (has_window) {
        for (int wt = 0; wt * TK < Mq; ++wt) {
            __syncthreads();                                      // every warp is done with the ring
            uint8_t *kt = stages, *vt = stages + tile_bytes;
#pragma unroll 4
            for (int e = tid; e < TK * CH; e += blockDim.x) {
                const int jr = e / CH, j0 = (e % CH) * 8;
                const int i = wt * TK + jr;
                uint4 klo = make_uint4(0u, 0u, 0u, 0u), khi = klo, vlo = klo, vhi = klo;
                const int pos = base + i;
                if (i < Mq && pos >= 0 && pos < p.max_seq) {
                    const float *src = p.qkv + ((size_t)q * Mq + i) * qstride + (size_t)(p.H + kvh) * DH;
                    const float *vs = src + (size_t)p.Hkv * DH;
                    vlo = round8(vs + j0);
                    vhi = round8(vs + j0 + half);
                    rotate8(src + j0, src + j0 + half, p.rope + (size_t)pos * half + j0, 1.0f, klo, khi);
                    const int page = pt[pos >> p.page_shift];
                    const long long r = ((long long)page * p.Hkv + kvh) * p.page_tokens + (pos & (p.page_tokens - 1));
                    __nv_bfloat16 *kd = p.pool + (size_t)(p.row0_k + r) * DH, *vd = p.pool + (size_t)(p.row0_v + r) * DH;
                    *(uint4 *)(kd + j0) = klo; *(uint4 *)(kd + j0 + half) = khi;
                    *(uint4 *)(vd + j0) = vlo; *(uint4 *)(vd + j0 + half) = vhi;
                }
                *(uint4 *)(kt + sw_off(TK, jr, j0)) = klo;
                *(uint4 *)(kt + sw_off(TK, jr, j0 + half)) = khi;
                *(uint4 *)(vt + sw_off(TK, jr, j0)) = vlo;
                *(uint4 *)(vt + sw_off(TK, jr, j0 + half)) = vhi;
            }
            __syncthreads();
            const int klim = min(Mq, p.max_seq - base) - wt * TK; // window keys that exist
            const uint32_t kb = smem_u32(kt);
            if (compute)
                process_tile<DH, KS>(w, kb, kb + tile_bytes, lane, kh, true,
                                 [&](int h, int key) { return key < klim && wt * TK + key <= qi[h]; });
        }
    }

    // ---- two warps per query tile: fold the keys of the second warp into the first ----------------------
    const bool fin = compute && kh == 0;                          // the warps that carry the result on
    if (KS == 2) {
        __syncthreads();                                          // the ring is free
        float *o2 = (float *)stages;                              // [qrows_pad][DH], then max and sum per row
        float *m2 = o2 + (size_t)qrows_pad * DH, *l2 = m2 + qrows_pad;
        if (compute && kh == 1) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int rr = mt * 16 + g + 8 * h;
#pragma unroll
                for (int j = 0; j < DH / 8; ++j)
                    *(float2 *)(o2 + (size_t)rr * DH + j * 8 + 2 * (lane & 3)) = make_float2(w.o[j][2 * h], w.o[j][2 * h + 1]);
                if ((lane & 3) == 0) { m2[rr] = w.m[h]; l2[rr] = w.l[h]; }
            }
        }
        __syncthreads();
        if (fin) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int rr = mt * 16 + g + 8 * h;
                const float m1 = m2[rr], l1 = l2[rr];
                const float M = fmaxf(w.m[h], m1), Ms = M == -INFINITY ? 0.f : M;
                const float a0 = exp2f(w.m[h] - Ms), a1 = exp2f(m1 - Ms);       // exp2(-inf) = 0: an empty side drops out
                w.m[h] = M;
                w.l[h] = w.l[h] * a0 + l1 * a1;
#pragma unroll
                for (int j = 0; j < DH / 8; ++j) {
                    const float2 t = *(const float2 *)(o2 + (size_t)rr * DH + j * 8 + 2 * (lane & 3));
                    w.o[j][2 * h] = w.o[j][2 * h] * a0 + t.x * a1;
                    w.o[j][2 * h + 1] = w.o[j][2 * h + 1] * a0 + t.y * a1;
                }
            }
        }
        // (each of these warps reads and, below, rewrites only its own rows of this area)
    }

    // ---- finish: normalise (one CTA) or merge over the cluster -----------------------------------------
    const size_t ostride = (size_t)p.H * DH;
    if (C == 1) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int rr = mt * 16 + g + 8 * h;
            if (fin && rr < rows) {
                const int i = rr % Mq, gq = rr / Mq;
                const float inv = w.l[h] > 0.f ? 1.0f / w.l[h] : 0.f;
                __nv_bfloat16 *dst = p.out + ((size_t)q * Mq + i) * ostride + (size_t)(kvh * p.n_rep + gq) * DH;
#pragma unroll
                for (int j = 0; j < DH / 8; ++j) {
                    const int col = j * 8 + 2 * (lane & 3);
                    const float o0 = w.o[j][2 * h] * inv, o1 = w.o[j][2 * h + 1] * inv;
                    *(__nv_bfloat162 *)(dst + col) = __floats2bfloat162_rn(o0, o1);
                    *(uint32_t *)(dst + p.out_plane + col) = pack_bf16_rest(o0, o1);
                }
            }
        }
        if (p.stamp && tid == 0 && blockIdx.x < STAMP_CTAS) p.stamp[STAMP_CTAS + blockIdx.x] = global_timer_ns();
        return;
    }
    __syncthreads();                                              // the ring is free: reuse it for the partials
    float *o_st = (float *)stages;                                // [qrows_pad][DH]
    float *m_st = o_st + (size_t)qrows_pad * DH;                  // [qrows_pad]
    float *l_st = m_st + qrows_pad;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int rr = mt * 16 + g + 8 * h;
        if (!fin) break;
#pragma unroll
        for (int j = 0; j < DH / 8; ++j) {
            const int col = j * 8 + 2 * (lane & 3);
            *(float2 *)(o_st + (size_t)rr * DH + col) = make_float2(w.o[j][2 * h], w.o[j][2 * h + 1]);
        }
        if ((lane & 3) == 0) { m_st[rr] = w.m[h]; l_st[rr] = w.l[h]; }
    }
    __syncwarp();
    cluster_sync_all();
    {
        const int r_lo = (int)(((long long)rank * rows) / C), r_hi = (int)(((long long)(rank + 1) * rows) / C);
        const int nr = r_hi - r_lo;                                // <= 64 because C >= 2
        const uint32_t o_addr = smem_u32(o_st), m_addr = smem_u32(m_st), l_addr = smem_u32(l_st);
        // four dims per item; the loads of all peers - the partial outputs and the row's max and sum -
        // are in flight together, then every thread works out its row's weights exp2(m_p - M) / L
        for (int e = tid; e < nr * (DH / 4); e += blockDim.x) {
            const int rl = e / (DH / 4), rr = r_lo + rl, col = (e % (DH / 4)) * 4;
            float4 part[8];
            float mp[8], lp[8];
#pragma unroll
            for (int peer = 0; peer < 8; ++peer) {
                part[peer] = make_float4(0.f, 0.f, 0.f, 0.f);
                mp[peer] = -INFINITY;
                lp[peer] = 0.f;
                if (peer < C) {
                    part[peer] = ld_cluster_f32x4(map_peer(o_addr + (uint32_t)(rr * DH + col) * 4u, (uint32_t)peer));
                    mp[peer] = ld_cluster_f32(map_peer(m_addr + rr * 4u, (uint32_t)peer));
                    lp[peer] = ld_cluster_f32(map_peer(l_addr + rr * 4u, (uint32_t)peer));
                }
            }
            float M = -INFINITY;
#pragma unroll
            for (int peer = 0; peer < 8; ++peer) M = fmaxf(M, mp[peer]);
            float L = 0.f;
#pragma unroll
            for (int peer = 0; peer < 8; ++peer) {
                mp[peer] = mp[peer] == -INFINITY ? 0.f : exp2f(mp[peer] - M);
                L += mp[peer] * lp[peer];
            }
            const float inv = L > 0.f ? 1.0f / L : 0.f;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int peer = 0; peer < 8; ++peer) {
                const float wp = mp[peer] * inv;
                acc.x += wp * part[peer].x; acc.y += wp * part[peer].y;
                acc.z += wp * part[peer].z; acc.w += wp * part[peer].w;
            }
            const int i = rr % Mq, gq = rr / Mq;
            __nv_bfloat16 *dst = p.out + ((size_t)q * Mq + i) * ostride + (size_t)(kvh * p.n_rep + gq) * DH + col;
            uint2 packed;
            packed.x = pack_bf16(acc.x, acc.y);
            packed.y = pack_bf16(acc.z, acc.w);
            *(uint2 *)dst = packed;
            packed.x = pack_bf16_rest(acc.x, acc.y);
            packed.y = pack_bf16_rest(acc.z, acc.w);
            *(uint2 *)(dst + p.out_plane) = packed;
        }
    }
    __syncwarp();
    cluster_sync_all();
    if (p.stamp && tid == 0 && blockIdx.x < STAMP_CTAS) p.stamp[STAMP_CTAS + blockIdx.x] = global_timer_ns();
}


// ================================================================================================
// Long contexts: the same attention with S = Q K^T and O = P V on tcgen05.mma.
//
// One CTA = (stream-sequence, KV head, cluster rank) as above, one CTA per SM. 256 threads: warps 0-3 are
// the softmax - thread t owns tensor-memory lane t (no shuffles) - and one lane each of warps 4-7 issues
// the S MMAs, the O MMAs, the K copies and the V copies: four instruction streams that only meet at
// mbarriers (one lane doing all four in turn spends about 0.4 us on each: 2.2 us per tile). Per key tile t
// of 64 keys:
//   S[t & 1][128 x 64] = Q_hi K^T + Q_lo K^T   A = the queries, B = the K tile (shared memory, K-major)
//   the thread reads its row of S from tensor memory, masks it and writes P = exp2(S - m) as bf16
//   O[128 x dh] += P[t & 1] V                   A = P, B = the V tile as it lies in the cache ([key][dh]: MN-major)
// The A operands - both bf16 planes of the rotated queries and the two P tiles - live in tensor memory next
// to S and O, written with tcgen05.st by the thread that owns the row. With A in shared memory the kernel
// is bound by shared-memory bandwidth (measured: every MMA re-reads its 4 KB of A; 176 KB per tile and
// 0.73 us, with the TMA writes into the rings starved meanwhile); so the rings are all the shared memory
// the kernel uses, and a tile costs two reads of K, one of V and the TMA writes: 80 KB.
// O stays in tensor memory over all tiles. m is the maximum the row has met, but it is raised - and the
// row of O multiplied by exp2(m_old - m_new) - only when a score exceeds it by more than 8: until then
// P <= 2^8, which bf16 and the fp32 row sum hold without loss, and the final O / l does not depend on m.
// S and P are double-buffered: S(t + 1) is computed while the threads work on S(t), and they write P(t + 1)
// while O += P(t) V(t) runs. The K tiles and the V tiles have rings of their own: a K slot is free as soon
// as S is complete, long before the V slot of the same tile.
// With R = 128 / G query rows or fewer (G = 2, 4) lane g R + r holds query row r again, and its thread
// takes only the keys [g 64/G, (g + 1) 64/G) of every tile: it writes those columns of its row of P (the
// others stay zero), so lane g R + r of O accumulates the part of row r's output that these keys give,
// with a maximum and a sum of its own; the G parts of a row are merged at the end like the parts of the
// cluster's CTAs. All 128 threads then share the exponentials. Rows beyond the live queries are zero.
// The CTA holds all 512 columns of tensor memory. It asks for nearly all of the SM's shared memory, so
// no CTA of another kernel (the GEMMs around it allocate tensor memory too) is ever resident beside it.
constexpr int T5_THREADS = 256;
constexpr float T5_RAISE = 8.0f;
constexpr int T5_MAX_TILES = 1024;          // key tiles one CTA may take (the host checks max_seq against it)

__device__ __forceinline__ uint64_t t5_desc_k(uint32_t smem_addr)      // K-major, 128-byte swizzle: 8-row groups 1024 B apart
{
    return (uint64_t)((smem_addr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// MN-major, 128-byte swizzle: 64 consecutive MN elements per 128-byte row, one row per K index, 8-row groups
// 1024 B apart (stride offset), the next 64 MN elements `lbo_bytes` on (leading offset)
__device__ __forceinline__ uint64_t t5_desc_mn(uint32_t smem_addr, uint32_t lbo_bytes)
{
    return (uint64_t)((smem_addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) | (64ull << 32) |
           (1ull << 46) | (2ull << 61);
}
// A bounded wait that gives up early when another thread of the CTA already has (`failed`).
__device__ __forceinline__ bool t5_wait(uint64_t *bar, unsigned parity, volatile int *failed)
{
    const uint32_t a = smem_u32(bar);
    for (unsigned i = 0; i < ATT_SPIN_LIMIT; ++i) {
        unsigned ok;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(a), "r"(parity) : "memory");
        if (ok) return true;
        if ((i & 1023u) == 1023u && *failed) return false;
    }
    return false;
}
// D (+)= A B with the A operand in tensor memory (lane = row, 32-bit column c = elements 2c, 2c + 1 of the row)
// and B in shared memory
__device__ __forceinline__ void t5_mma_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t db, uint32_t idesc, uint32_t acc)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(tmem_d), "r"(tmem_a), "l"(db), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void t5_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 32 consecutive columns of this thread's tensor-memory lane
__device__ __forceinline__ void t5_ld32(uint32_t taddr, float *v)
{
    uint32_t r[32];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void t5_ld16(uint32_t taddr, float *v)
{
    uint32_t r[16];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ float t5_ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
template <int N>
__device__ __forceinline__ void t5_st_u32(uint32_t taddr, const uint32_t *v)   // N = 8, 16, 32 consecutive columns
{
    if constexpr (N == 8) {
        asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                     ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]) : "memory");
    } else if constexpr (N == 16) {
        asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
                     ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
                       "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]) : "memory");
    } else {
        static_assert(N == 32, "8, 16 or 32 columns");
        asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
                     "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
                     ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
                       "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
                       "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
                       "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31]) : "memory");
    }
}
__device__ __forceinline__ void t5_st32(uint32_t taddr, const float *v)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
                 "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
                 ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
                   "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
                   "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
                   "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
                   "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
                   "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
                   "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
                   "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
                 : "memory");
}

template <int DH, int G>
__global__ void __launch_bounds__(T5_THREADS, 1) attention_t5_kernel(const __grid_constant__ AttnParams p)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    // rings: slot s of K (V) is full when its copy has landed, empty when the MMAs that read it are complete
    __shared__ uint64_t kfull[MAX_ATT_STAGES], kempty[MAX_ATT_STAGES], vfull[MAX_ATT_STAGES], vempty[MAX_ATT_STAGES];
    // per buffer (tile parity): S complete / S read into registers / P written / O += P V complete
    __shared__ uint64_t bar_s[2], bar_sc[2], bar_p[2], bar_o[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int tile_row[T5_MAX_TILES];                        // pool row (within a layer's K or V) of each of this CTA's tiles
    __shared__ volatile int failed;                               // a bounded wait gave up: every later wait is skipped

    if (p.skip && *p.skip) return;
    if ((smem_u32(smem_raw) & 1023u) != 0u) {
        if (threadIdx.x == 0) atomicExch(p.err, 6);
        return;
    }
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (p.stamp && tid == 0 && blockIdx.x < STAMP_CTAS) p.stamp[blockIdx.x] = global_timer_ns();
    // tensor-memory columns: Q_hi [0, 64), Q_lo [64, 128) (dh / 2 each), S [128, 192) and [192, 256), O [256, 256 + dh),
    // P [384, 416) and [416, 448) (two keys per column)
    constexpr uint32_t TMEM_COLS = 512;
    // warps 0-3: softmax. One lane each of warp 4: S = Q K^T; warp 5: O += P V; warp 6: K copies; warp 7: V copies
    const bool softmax = warp < 4;
    const bool s_lane = warp == 4 && lane == 0, o_lane = warp == 5 && lane == 0;
    const bool k_lane = warp == 6 && lane == 0, v_lane = warp == 7 && lane == 0;
    const int NK = p.stages, NV = p.stages_v;
    if (tid == 0) {
        for (int s = 0; s < NK; ++s) { mbar_init(&kfull[s], 1); mbar_init(&kempty[s], 1); }
        for (int s = 0; s < NV; ++s) { mbar_init(&vfull[s], 1); mbar_init(&vempty[s], 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&bar_s[i], 1); mbar_init(&bar_sc[i], 128); mbar_init(&bar_p[i], 128); mbar_init(&bar_o[i], 1);
        }
        failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_s)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    // Only now may the kernel behind start: its CTAs allocate tensor memory too and then wait for this grid,
    // so every CTA here must hold its columns before any of them can arrive on its SM.
    pdl_trigger();
    const uint32_t tmem_q = tmem_base_s, tmem_s = tmem_base_s + 128u, tmem_o = tmem_base_s + 256u, tmem_p = tmem_base_s + 384u;

    const int C = p.C, rank = blockIdx.x % C, unit = blockIdx.x / C;
    const int q = unit / p.Hkv, kvh = unit % p.Hkv;
    const int b = q % p.B;
    const int Mq = p.Mq, rows = Mq * p.n_rep;
    constexpr int R = 128 / G;                                    // query rows a CTA can carry (rows <= R)
    constexpr int NC = TK / G;                                    // keys of a tile per thread
    constexpr int half = DH / 2;
    constexpr int CH = half / 8;
    constexpr uint32_t tile_bytes = TK * DH * 2;                  // one K (or V) tile: [DH/64][TK keys][128 B]

    uint8_t *kring = smem_raw;                                    // NK K tiles, then NV V tiles,
    uint8_t *vring = kring + (size_t)NK * tile_bytes;
    constexpr int QROW = DH * 2 + 16;                             // then the rotated queries on their way to tensor memory:
    uint8_t *q_st = vring + (size_t)NV * tile_bytes;              // two planes of [R][DH] bf16, rows 16 bytes apart in the banks;
    uint8_t *w_st = q_st;                                         // after that the window's K tiles, then its V tiles

    const int base = p.pos_override >= 0 ? p.pos_override : p.n_known[b] - 1;
    const int ctx = min(max(base, 0), p.max_seq);
    const int n_tiles = (ctx + TK - 1) / TK;
    const bool has_window = rank == C - 1;
    const int per = (n_tiles + 3 + C - 1) / C;
    const int t0 = min(n_tiles, rank * per);
    const int t1 = has_window ? n_tiles : min(n_tiles, (rank + 1) * per);
    const int my_tiles = t1 - t0;
    const int *pt = p.page_table + (size_t)q * p.pages_per_seq;

    bool dead = false;                                            // this thread has given up on a wait: it skips the others
    auto wait_on = [&](uint64_t *bar, unsigned parity, int code) {
        if (dead) return;
        if (!t5_wait(bar, parity, &failed)) {
            if (!failed) atomicExch(p.err, code);
            failed = 1;
            dead = true;
        }
    };
    // where each tile lies in the pool (one page-table read per tile, off the copy lanes' path)
    for (int t = tid; t < my_tiles; t += T5_THREADS) {
        const int pos = (t0 + t) * TK;
        tile_row[t] = (pt[pos >> p.page_shift] * p.Hkv + kvh) * p.page_tokens + (pos & (p.page_tokens - 1));
    }
    __syncthreads();
    // copy lanes: request the K (V) rows of context tile t0 + t into slot s of their ring
    auto issue = [&](int t, uint8_t *dst, uint64_t *bar, int row0) {
        mbar_expect_tx(bar, tile_bytes);
#pragma unroll
        for (int h = 0; h < DH / 64; ++h) tma_load_2d(&p.kv_map, bar, dst + h * (TK * 128), h * 64, row0 + tile_row[t]);
    };
    const int row0_k = (int)p.row0_k, row0_v = (int)p.row0_v;     // (the pool has fewer than 2^31 rows)
    // the first tiles do not depend on the kernel in front: on their way while it drains
    if (k_lane)
        for (int t = 0; t < min(NK, my_tiles); ++t) issue(t, kring + (size_t)t * tile_bytes, &kfull[t], row0_k);
    if (v_lane)
        for (int t = 0; t < min(NV, my_tiles); ++t) issue(t, vring + (size_t)t * tile_bytes, &vfull[t], row0_v);

    // softmax threads: lane = column group * R + query row
    const int grp = tid / R, row = tid % R;                       // (warps 0-3; R is a multiple of 32)
    const bool live = softmax && row < rows;
    const int qi = live ? row % Mq : 0;                           // query index inside the window
    const int c_lo = grp * NC;                                    // first key of a tile this thread takes
    const uint32_t lane_base = ((uint32_t)(warp & 3) * 32u) << 16; // this warp's quarter of the tensor-memory lanes

    // ---- Q, and in the cluster's last CTA the window's K and V: rotated, scaled, rounded by all threads (coalesced:
    // one item = 8 dims of both halves of a row). The rotation table does not depend on the kernel in front: its
    // values are in registers before that kernel is waited for.
    const size_t qstride = (size_t)(p.H + 2 * p.Hkv) * DH;
    constexpr int QI = (R * CH + T5_THREADS - 1) / T5_THREADS;    // query items per thread
    constexpr int WI = (TK * CH + T5_THREADS - 1) / T5_THREADS;   // K/V items per thread and window tile
    const int n_wt = has_window ? (Mq + TK - 1) / TK : 0;         // window tiles (at most 2: the host sizes the staging)
    Rope8 q_rope[QI], w_rope[2][WI];
#pragma unroll
    for (int k = 0; k < QI; ++k) {
        const int e = tid + k * T5_THREADS, rr = e / CH, j0 = (e % CH) * 8;
        const int pos = min(max(base + rr % Mq, 0), p.max_seq - 1);
        q_rope[k] = load_rope8(p.rope + (size_t)pos * half + j0);
    }
#pragma unroll
    for (int wt = 0; wt < 2; ++wt)
#pragma unroll
        for (int k = 0; k < WI; ++k) {
            const int e = tid + k * T5_THREADS, jr = e / CH, j0 = (e % CH) * 8;
            const int pos = min(max(base + wt * TK + jr, 0), p.max_seq - 1);
            if (wt < n_wt) w_rope[wt][k] = load_rope8(p.rope + (size_t)pos * half + j0);
        }

    pdl_wait();                                                   // the projections come from the GEMM in front

#pragma unroll
    for (int k = 0; k < QI; ++k) {
        const int e = tid + k * T5_THREADS, rr = e / CH, j0 = (e % CH) * 8;
        if (e < R * CH) {
            uint4 lo = make_uint4(0u, 0u, 0u, 0u), hi = lo, rlo = lo, rhi = lo;
            if (rr < rows) {
                const int i = rr % Mq, g = rr / Mq;
                const float *src = p.qkv + ((size_t)q * Mq + i) * qstride + (size_t)(kvh * p.n_rep + g) * DH;
                rotate8(src + j0, src + j0 + half, q_rope[k], p.qscale, lo, hi, &rlo, &rhi);
            }
            uint8_t *d0 = q_st + (size_t)rr * QROW, *d1 = d0 + (size_t)R * QROW;
            *(uint4 *)(d0 + j0 * 2) = lo;
            *(uint4 *)(d0 + (j0 + half) * 2) = hi;
            *(uint4 *)(d1 + j0 * 2) = rlo;
            *(uint4 *)(d1 + (j0 + half) * 2) = rhi;
        }
    }
    // the window's keys and values: into the cache now, into shared memory once the queries have left it
    uint4 w_k[2][WI][2], w_v[2][WI][2];
#pragma unroll
    for (int wt = 0; wt < 2; ++wt)
#pragma unroll
        for (int k = 0; k < WI; ++k) {
            const int e = tid + k * T5_THREADS, jr = e / CH, j0 = (e % CH) * 8;
            const int i = wt * TK + jr, pos = base + i;
            w_k[wt][k][0] = w_k[wt][k][1] = w_v[wt][k][0] = w_v[wt][k][1] = make_uint4(0u, 0u, 0u, 0u);
            if (wt < n_wt && e < TK * CH && i < Mq && pos >= 0 && pos < p.max_seq) {
                const float *src = p.qkv + ((size_t)q * Mq + i) * qstride + (size_t)(p.H + kvh) * DH;
                const float *vs = src + (size_t)p.Hkv * DH;
                w_v[wt][k][0] = round8(vs + j0);
                w_v[wt][k][1] = round8(vs + j0 + half);
                rotate8(src + j0, src + j0 + half, w_rope[wt][k], 1.0f, w_k[wt][k][0], w_k[wt][k][1]);
                const int page = pt[pos >> p.page_shift];
                const long long r = ((long long)page * p.Hkv + kvh) * p.page_tokens + (pos & (p.page_tokens - 1));
                __nv_bfloat16 *kd = p.pool + (size_t)(p.row0_k + r) * DH, *vd = p.pool + (size_t)(p.row0_v + r) * DH;
                *(uint4 *)(kd + j0) = w_k[wt][k][0]; *(uint4 *)(kd + j0 + half) = w_k[wt][k][1];
                *(uint4 *)(vd + j0) = w_v[wt][k][0]; *(uint4 *)(vd + j0 + half) = w_v[wt][k][1];
            }
        }
    __syncthreads();
    if (softmax) {
#pragma unroll
        for (int pl = 0; pl < 2; ++pl) {
            const uint8_t *srow = q_st + ((size_t)pl * R + row) * QROW;
#pragma unroll
            for (int c0 = 0; c0 < DH / 2; c0 += 16) {             // 16 columns = 32 dims = 64 bytes
                uint32_t w[16];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint4 x = *(const uint4 *)(srow + c0 * 4 + k * 16);
                    w[4 * k] = x.x; w[4 * k + 1] = x.y; w[4 * k + 2] = x.z; w[4 * k + 3] = x.w;
                }
                t5_st_u32<16>(tmem_q + lane_base + (uint32_t)pl * 64u + (uint32_t)c0, w);
            }
        }
        if (G > 1) {                                              // the columns of P this thread never writes stay zero
            uint32_t z[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) z[j] = 0u;
            t5_st_u32<32>(tmem_p + lane_base, z);
            t5_st_u32<32>(tmem_p + lane_base + 32u, z);
        }
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (n_wt > 0) {                                               // (the whole CTA or none of it)
#pragma unroll
        for (int wt = 0; wt < 2; ++wt)
#pragma unroll
            for (int k = 0; k < WI; ++k) {
                const int e = tid + k * T5_THREADS, jr = e / CH, j0 = (e % CH) * 8;
                if (wt < n_wt && e < TK * CH) {
                    uint8_t *kt = w_st + (size_t)wt * tile_bytes, *vt = w_st + (size_t)(n_wt + wt) * tile_bytes;
                    *(uint4 *)(kt + sw_off(TK, jr, j0)) = w_k[wt][k][0];
                    *(uint4 *)(kt + sw_off(TK, jr, j0 + half)) = w_k[wt][k][1];
                    *(uint4 *)(vt + sw_off(TK, jr, j0)) = w_v[wt][k][0];
                    *(uint4 *)(vt + sw_off(TK, jr, j0 + half)) = w_v[wt][k][1];
                }
            }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the MMAs read these tiles through the async proxy
        __syncthreads();
    }

    // instruction descriptors: fp32 accumulate, bf16 operands; S: N = 64, both K-major; PV: N = DH, B MN-major
    constexpr uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(TK >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
    constexpr uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(DH >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

    // S lane: S(t) = Q K(t)^T into S[t & 1], once the threads have read S(t - 2) out of it. The descriptors of
    // the k steps of one tile differ only in the start address field (bits 0-13, in 16-byte units; shared memory
    // ends far below 2^18 bytes, so adding there never carries out).
    auto mma_s = [&](int t, uint32_t kaddr) {
        if (t >= 2) wait_on(&bar_sc[t & 1], (unsigned)((t - 2) >> 1) & 1u, 10);
        const uint32_t d = tmem_s + (uint32_t)(t & 1) * 64u;
        const uint64_t dk = t5_desc_k(kaddr);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks) {
            const uint32_t koff = (uint32_t)(ks >> 2) * (uint32_t)(TK * 128) + (uint32_t)(ks & 3) * 32u;
            t5_mma_ts(d, tmem_q + (uint32_t)ks * 8u, dk + (koff >> 4), idesc_s, ks > 0 ? 1u : 0u);   // 16 dims = 8 columns
        }
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks) {
            const uint32_t koff = (uint32_t)(ks >> 2) * (uint32_t)(TK * 128) + (uint32_t)(ks & 3) * 32u;
            t5_mma_ts(d, tmem_q + 64u + (uint32_t)ks * 8u, dk + (koff >> 4), idesc_s, 1u);
        }
        t5_commit(&bar_s[t & 1]);
    };
    // O lane: O += P[t & 1] V(t) once the threads have written P(t)
    auto mma_o = [&](int t, uint32_t vaddr) {
        wait_on(&bar_p[t & 1], (unsigned)(t >> 1) & 1u, 8);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t pa = tmem_p + (uint32_t)(t & 1) * 32u;
        const uint64_t dv = t5_desc_mn(vaddr, (uint32_t)(TK * 128));
#pragma unroll
        for (int kk = 0; kk < TK / 16; ++kk)                      // 16 keys = 8 columns of P, 16 rows of V
            t5_mma_ts(tmem_o, pa + (uint32_t)kk * 8u, dv + (uint32_t)(kk * 2048 >> 4), idesc_o, (t > 0 || kk > 0) ? 1u : 0u);
        t5_commit(&bar_o[t & 1]);
    };

    float m_used = -INFINITY, l_run = 0.f;                        // softmax threads: the state of the lane's row

    // softmax threads: tile t, of which this row may attend to the first `lim` keys (0 .. TK)
    auto softmax_tile = [&](int t, int lim) {
        const int lim_l = min(max(lim - c_lo, 0), NC);            // ... of this thread's keys
        wait_on(&bar_s[t & 1], (unsigned)(t >> 1) & 1u, 7);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        float v[NC];
        const uint32_t s_addr = tmem_s + lane_base + (uint32_t)(t & 1) * 64u + (uint32_t)c_lo;
        if (NC == 16) t5_ld16(s_addr, v);
        else {
#pragma unroll
            for (int c0 = 0; c0 < NC; c0 += 32) t5_ld32(s_addr + (uint32_t)c0, v + c0);
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        mbar_arrive(&bar_sc[t & 1]);                              // S[t & 1] may be overwritten
        if (!__all_sync(0xffffffffu, lim_l == NC)) {
#pragma unroll
            for (int j = 0; j < NC; ++j) v[j] = j < lim_l ? v[j] : -INFINITY;
        }
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int j = 0; j < NC; ++j) mx4[j & 3] = fmaxf(mx4[j & 3], v[j]);
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        const bool raise = mx > m_used + T5_RAISE;                // (also the first keys this row meets: m_used = -inf)
        if (t == 0) {
            if (raise) m_used = mx;                               // nothing accumulated yet
        } else if (__any_sync(0xffffffffu, raise)) {
            // O holds the products up to tile t - 1: wait for them, rescale this row in tensor memory
            wait_on(&bar_o[(t - 1) & 1], (unsigned)((t - 1) >> 1) & 1u, 9);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const float alpha = raise ? exp2f(m_used - mx) : 1.0f;   // (m_used = -inf: the row of O is still zero)
#pragma unroll 1
            for (int c0 = 0; c0 < DH; c0 += 32) {
                float ov[32];
                t5_ld32(tmem_o + lane_base + (uint32_t)c0, ov);
#pragma unroll
                for (int j = 0; j < 32; ++j) ov[j] *= alpha;
                t5_st32(tmem_o + lane_base + (uint32_t)c0, ov);
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            l_run *= alpha;
            if (raise) m_used = mx;
        }
        const float msafe = m_used == -INFINITY ? 0.f : m_used;   // (a row without keys so far: every v is -inf)
        float sum4[4] = {0.f, 0.f, 0.f, 0.f};
        uint32_t pk[NC / 2];
#pragma unroll
        for (int j = 0; j < NC; j += 2) {
            const float p0 = t5_ex2(v[j] - msafe), p1 = t5_ex2(v[j + 1] - msafe);
            sum4[(j >> 1) & 3] += p0 + p1;
            pk[j >> 1] = pack_bf16(p0, p1);
        }
        l_run += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
        if (t >= 2) wait_on(&bar_o[t & 1], (unsigned)((t - 2) >> 1) & 1u, 9);   // P[t & 1] was read by the product of tile t - 2
        t5_st_u32<NC / 2>(tmem_p + lane_base + (uint32_t)(t & 1) * 32u + (uint32_t)(c_lo >> 1), pk);
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        mbar_arrive(&bar_p[t & 1]);
    };

    // ---- every role runs through the tiles on its own: the window's tiles first (they are in shared memory
    // already; the causal mask applies), then the committed context out of the rings -------------------------------
    const int t_done = n_wt + my_tiles;                           // tiles of this CTA
    if (s_lane) {
        for (int wt = 0; wt < n_wt; ++wt) mma_s(wt, smem_u32(w_st + (size_t)wt * tile_bytes));
        int s = 0;
        unsigned ph = 0;
        for (int t = 0; t < my_tiles; ++t) {
            wait_on(&kfull[s], ph, 5);
            mma_s(n_wt + t, smem_u32(kring + (size_t)s * tile_bytes));
            t5_commit(&kempty[s]);
            if (++s == NK) { s = 0; ph ^= 1u; }
        }
    } else if (o_lane) {
        for (int wt = 0; wt < n_wt; ++wt) mma_o(wt, smem_u32(w_st + (size_t)(n_wt + wt) * tile_bytes));
        int s = 0;
        unsigned ph = 0;
        for (int t = 0; t < my_tiles; ++t) {
            wait_on(&vfull[s], ph, 5);
            mma_o(n_wt + t, smem_u32(vring + (size_t)s * tile_bytes));
            t5_commit(&vempty[s]);
            if (++s == NV) { s = 0; ph ^= 1u; }
        }
    } else if (k_lane) {
        int s = 0;
        unsigned ph = 0;
        for (int t = NK; t < my_tiles; ++t) {                     // tile t goes where tile t - NK was
            wait_on(&kempty[s], ph, 4);
            if (!dead) issue(t, kring + (size_t)s * tile_bytes, &kfull[s], row0_k);
            if (++s == NK) { s = 0; ph ^= 1u; }
        }
    } else if (v_lane) {
        int s = 0;
        unsigned ph = 0;
        for (int t = NV; t < my_tiles; ++t) {
            wait_on(&vempty[s], ph, 4);
            if (!dead) issue(t, vring + (size_t)s * tile_bytes, &vfull[s], row0_v);
            if (++s == NV) { s = 0; ph ^= 1u; }
        }
    } else if (softmax) {
        for (int wt = 0; wt < n_wt; ++wt) {
            const int klim = min(Mq, p.max_seq - base) - wt * TK; // window keys that exist
            softmax_tile(wt, live ? max(0, min(min(TK, klim), qi - wt * TK + 1)) : 0);
        }
        for (int t = 0; t < my_tiles; ++t)
            softmax_tile(n_wt + t, live ? min(TK, ctx - (t0 + t) * TK) : 0);
    }
    if (t_done > 0) wait_on(&bar_o[(t_done - 1) & 1], (unsigned)((t_done - 1) >> 1) & 1u, 9);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    __syncthreads();                                              // every copy has landed, every MMA is complete

    // ---- finish: the parts of every row - G column groups here, C CTAs in the cluster - are merged ---------------
    const size_t ostride = (size_t)p.H * DH;
    constexpr int OROW = DH + 4;                                  // (rows 16 bytes apart in the banks)
    float *o_st = (float *)kring;                                 // parts: [128 lanes][OROW] fp32, then maxima and sums
    float *m_st = o_st + (size_t)128 * OROW;                      // per lane
    float *l_st = m_st + 128;
    float *m2_st = l_st + 128;                                    // per row, after the column groups were merged
    float *l2_st = m2_st + 128;
    if (softmax) {
#pragma unroll 1
        for (int c0 = 0; c0 < DH; c0 += 32) {
            float ov[32];
            t5_ld32(tmem_o + lane_base + (uint32_t)c0, ov);       // (warp-wide: dead rows read along)
            const bool keep = live && t_done > 0;
#pragma unroll
            for (int j = 0; j < 32; j += 4)
                *(float4 *)(o_st + (size_t)tid * OROW + c0 + j) = keep ? make_float4(ov[j], ov[j + 1], ov[j + 2], ov[j + 3])
                                                                     : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        m_st[tid] = live ? m_used : -INFINITY;
        l_st[tid] = live ? l_run : 0.f;
    }
    __syncthreads();
    // the column groups of each row: row r <- parts r, R + r, ..; one CTA: normalised and written out
    for (int e = tid; e < rows * (DH / 4); e += T5_THREADS) {
        const int rr = e / (DH / 4), col = (e % (DH / 4)) * 4;
        float mg[G], M = -INFINITY, L = 0.f;
#pragma unroll
        for (int g = 0; g < G; ++g) { mg[g] = m_st[g * R + rr]; M = fmaxf(M, mg[g]); }
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float wg = mg[g] == -INFINITY ? 0.f : exp2f(mg[g] - M);
            L += wg * l_st[g * R + rr];
            const float4 part = *(const float4 *)(o_st + (size_t)(g * R + rr) * OROW + col);
            acc.x += wg * part.x; acc.y += wg * part.y; acc.z += wg * part.z; acc.w += wg * part.w;
        }
        if (C == 1) {
            const float inv = L > 0.f ? 1.0f / L : 0.f;
            acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
            const int i = rr % Mq, gq = rr / Mq;
            __nv_bfloat16 *dst = p.out + ((size_t)q * Mq + i) * ostride + (size_t)(kvh * p.n_rep + gq) * DH + col;
            uint2 packed;
            packed.x = pack_bf16(acc.x, acc.y);
            packed.y = pack_bf16(acc.z, acc.w);
            *(uint2 *)dst = packed;
            packed.x = pack_bf16_rest(acc.x, acc.y);
            packed.y = pack_bf16_rest(acc.z, acc.w);
            *(uint2 *)(dst + p.out_plane) = packed;
        } else {
            if (G > 1) *(float4 *)(o_st + (size_t)rr * OROW + col) = acc;   // (part 0 of the row: only this item reads it)
            if (col == 0) { m2_st[rr] = M; l2_st[rr] = L; }
        }
    }
    if (C > 1) {
        __syncwarp();
        cluster_sync_all();
        {
            const int r_lo = (int)(((long long)rank * rows) / C), r_hi = (int)(((long long)(rank + 1) * rows) / C);
            const int nr = r_hi - r_lo;
            const uint32_t o_addr = smem_u32(o_st), m_addr = smem_u32(m2_st), l_addr = smem_u32(l2_st);
            for (int e = tid; e < nr * (DH / 4); e += T5_THREADS) {
                const int rl = e / (DH / 4), rr = r_lo + rl, col = (e % (DH / 4)) * 4;
                float4 part[8];
                float mp[8], lp[8];
#pragma unroll
                for (int peer = 0; peer < 8; ++peer) {
                    part[peer] = make_float4(0.f, 0.f, 0.f, 0.f);
                    mp[peer] = -INFINITY;
                    lp[peer] = 0.f;
                    if (peer < C) {
                        part[peer] = ld_cluster_f32x4(map_peer(o_addr + (uint32_t)(rr * OROW + col) * 4u, (uint32_t)peer));
                        mp[peer] = ld_cluster_f32(map_peer(m_addr + rr * 4u, (uint32_t)peer));
                        lp[peer] = ld_cluster_f32(map_peer(l_addr + rr * 4u, (uint32_t)peer));
                    }
                }
                float M = -INFINITY;
#pragma unroll
                for (int peer = 0; peer < 8; ++peer) M = fmaxf(M, mp[peer]);
                float L = 0.f;
#pragma unroll
                for (int peer = 0; peer < 8; ++peer) {
                    mp[peer] = mp[peer] == -INFINITY ? 0.f : exp2f(mp[peer] - M);
                    L += mp[peer] * lp[peer];
                }
                const float inv = L > 0.f ? 1.0f / L : 0.f;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int peer = 0; peer < 8; ++peer) {
                    const float wp = mp[peer] * inv;
                    acc.x += wp * part[peer].x; acc.y += wp * part[peer].y;
                    acc.z += wp * part[peer].z; acc.w += wp * part[peer].w;
                }
                const int i = rr % Mq, gq = rr / Mq;
                __nv_bfloat16 *dst = p.out + ((size_t)q * Mq + i) * ostride + (size_t)(kvh * p.n_rep + gq) * DH + col;
                uint2 packed;
                packed.x = pack_bf16(acc.x, acc.y);
                packed.y = pack_bf16(acc.z, acc.w);
                *(uint2 *)dst = packed;
                packed.x = pack_bf16_rest(acc.x, acc.y);
                packed.y = pack_bf16_rest(acc.z, acc.w);
                *(uint2 *)(dst + p.out_plane) = packed;
            }
        }
        __syncwarp();
        cluster_sync_all();
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 4) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base_s), "r"(TMEM_COLS) : "memory");
    }
    if (p.stamp && tid == 0 && blockIdx.x < STAMP_CTAS) p.stamp[STAMP_CTAS + blockIdx.x] = global_timer_ns();
}

struct AttnPlan {
    CUtensorMap kv_map;
    int sm_count;
    int t5_rows, t5_C;        // tcgen05 kernel: cluster size found for windows of t5_rows query rows (0: not looked for yet)
};

}  // namespace

bool attention_tc_supported(const scd_session *s, int Mq)
{
    const scd_model_config_t &c = s->model->cfg;
    const int n_rep = c.n_heads / c.n_kv_heads;
    return c.dtype == SCD_BF16 && s->attn_plan != nullptr && (c.head_dim == 64 || c.head_dim == 128) &&
           c.kv_page_tokens % TK == 0 && Mq * n_rep <= 128;
}

int attention_session_prepare(scd_session *s)
{
    const scd_model_config_t &c = s->model->cfg;
    s->attn_plan = nullptr;
    if (c.dtype != SCD_BF16 || !(c.head_dim == 64 || c.head_dim == 128) || c.kv_page_tokens % TK != 0) return SCD_OK;
    AttnPlan *plan = new AttnPlan();
    const unsigned long long total_rows = (unsigned long long)c.n_layers * 2ull * s->Q * s->pages_per_seq *
                                          c.n_kv_heads * c.kv_page_tokens;
    if (total_rows >= (1ull << 31)) { delete plan; return SCD_OK; }      // row coordinates are int32: keep the SIMT path
    int rc = make_tensor_map_bf16_2d(&plan->kv_map, s->kv_pool, total_rows, (unsigned long long)c.head_dim, TK, 64);
    if (rc != SCD_OK) { delete plan; return rc; }
    int dev = 0;
    cudaGetDevice(&dev);
    plan->sm_count = 148;
    cudaDeviceGetAttribute(&plan->sm_count, cudaDevAttrMultiProcessorCount, dev);
    s->attn_plan = plan;
    return SCD_OK;
}

void attention_session_release(scd_session *s)
{
    delete (AttnPlan *)s->attn_plan;
    s->attn_plan = nullptr;
}

// The kernel variant with two warps per query tile pays from about four key tiles per CTA on. The
// context length is device-side state; the host knows a floor of it (every iteration commits at
// least one token): s->ctx_floor. At most two query tiles (the CTA has four warps anyway).
static int attention_clusters(const scd_session *s, const AttnPlan *plan)
{
    const scd_model_config_t &c = s->model->cfg;
    const int units = s->Q * c.n_kv_heads;
    const int max_tiles = (c.max_seq + TK - 1) / TK;
    const int c_cap = std::max(1, std::min(std::min(8, max_tiles), (2 * plan->sm_count) / std::max(1, units)));
    int C = 1;
    while (C * 2 <= c_cap) C *= 2;
    return C;
}


using T5Kernel = void (*)(const AttnParams);
constexpr size_t T5_SMEM = 227 * 1024 - 8192;   // all of an SM's shared memory but the kernel's static part (some 5 KB)

static T5Kernel t5_kernel(int dh, int rows, int *G_out)
{
    const int G = rows > 64 ? 1 : rows > 32 ? 2 : 4;              // column groups: 128 / G query rows per CTA
    *G_out = G;
    return dh == 128 ? (G == 1 ? attention_t5_kernel<128, 1> : G == 2 ? attention_t5_kernel<128, 2> : attention_t5_kernel<128, 4>)
                     : (G == 1 ? attention_t5_kernel<64, 1> : G == 2 ? attention_t5_kernel<64, 2> : attention_t5_kernel<64, 4>);
}

// The largest cluster the tcgen05 kernel may use for windows of `rows` query rows: one CTA per SM and one wave,
// i.e. the device must hold one cluster per (sequence, KV head) at the same time. Any size up to 8 (the kernel
// splits tiles and rows evenly). The answer depends on how the SMs are grouped, so the runtime is asked - once.
static int t5_max_cluster(const scd_session *s, AttnPlan *plan, int rows)
{
    if (plan->t5_rows == rows) return plan->t5_C;
    const scd_model_config_t &c = s->model->cfg;
    const int units = s->Q * c.n_kv_heads;
    static DeviceOnce once;
    int dev = 0;
    if (current_device(&dev) != SCD_OK) return 0;
    const int rc = once.run(dev, [&]() -> int {
        SCD_CUDA_TRY(cudaFuncSetAttribute(attention_t5_kernel<128, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)T5_SMEM));
        SCD_CUDA_TRY(cudaFuncSetAttribute(attention_t5_kernel<128, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)T5_SMEM));
        SCD_CUDA_TRY(cudaFuncSetAttribute(attention_t5_kernel<128, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)T5_SMEM));
        SCD_CUDA_TRY(cudaFuncSetAttribute(attention_t5_kernel<64, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)T5_SMEM));
        SCD_CUDA_TRY(cudaFuncSetAttribute(attention_t5_kernel<64, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)T5_SMEM));
        SCD_CUDA_TRY(cudaFuncSetAttribute(attention_t5_kernel<64, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)T5_SMEM));
        return SCD_OK;
    });
    if (rc != SCD_OK) return 0;
    int G = 1;
    const T5Kernel fn = t5_kernel(c.head_dim, rows, &G);
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof(cfg));
    cfg.blockDim = dim3(T5_THREADS, 1, 1);
    cfg.dynamicSmemBytes = T5_SMEM;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 1;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int best = 1;
    for (int C = std::min(8, plan->sm_count / std::max(1, units)); C >= 2; --C) {
        cfg.gridDim = dim3((unsigned)(units * C), 1, 1);
        attr.val.clusterDim.x = (unsigned)C;
        int fit = 0;
        if (cudaOccupancyMaxActiveClusters(&fit, fn, &cfg) == cudaSuccess && fit >= units) { best = C; break; }
        cudaGetLastError();
    }
    plan->t5_rows = rows;
    plan->t5_C = best;
    return best;
}

// Low 4 bits: 0 = one warp per query tile; 1 = two warps per query tile; 2 = the tcgen05 kernel (at most 128 query
// rows per KV head, the units fit one wave), with its cluster size in the bits above. The choice
// follows `ctx`, the committed positions every live sequence is known to hold: the host's floor of it for a decoding
// step (a captured iteration is built for one value of the choice), the chunk's first position for a prefill chunk.
int attention_tc_variant(const scd_session *s, int Mq, long long ctx)
{
    const scd_model_config_t &c = s->model->cfg;
    AttnPlan *plan = (AttnPlan *)s->attn_plan;
    if (!plan) return 0;
    const int rows = Mq * (c.n_heads / c.n_kv_heads);
    const long long tiles = (std::max(0ll, ctx) + TK - 1) / TK;
    if (rows <= 128 && s->Q * c.n_kv_heads <= plan->sm_count && (c.max_seq + TK - 1) / TK <= T5_MAX_TILES && s->att_t5_min_ctx >= 0 &&
        ctx >= s->att_t5_min_ctx) {
        const int c_max = t5_max_cluster(s, plan, rows);
        // (the largest cluster at every context length: with fewer CTAs the kernel itself is faster on a short
        // context - no merge - but the GEMM behind, launched early onto the SMs this grid leaves free, crowds there:
        // measured, the iteration takes as long)
        if (c_max >= 1) return 2 | (c_max << 4);
    }
    const int n_mtiles = (rows + 15) / 16;
    if (n_mtiles > 2) return 0;
    const int C = attention_clusters(s, plan);
    return (tiles + 3 + C - 1) / C >= 4 ? 1 : 0;
}

static int attention_t5(scd_session *s, AttnParams &p, int C, cudaStream_t st)
{
    const scd_model_config_t &c = s->model->cfg;
    const int dh = c.head_dim, units = s->Q * c.n_kv_heads;
    const int rows = p.Mq * p.n_rep;
    int G = 1;
    const T5Kernel fn = t5_kernel(dh, rows, &G);
    const size_t tile_bytes = (size_t)TK * dh * 2;                // one K or V slot
    const size_t merge_bytes = (size_t)128 * (dh + 4 + 4) * sizeof(float);
    // All the shared memory a CTA can have: no CTA of another kernel fits beside this one, so the tensor
    // memory - all 512 columns - is never contended for (see the kernel's header).
    // Behind the rings: the rotated queries on their way to tensor memory, then the window's K and V tiles.
    const size_t q_stage = std::max((size_t)2 * (128 / G) * (dh * 2 + 16), (size_t)2 * ((p.Mq + TK - 1) / TK) * tile_bytes);
    const int slots = (int)std::min<size_t>(2 * MAX_ATT_STAGES, (T5_SMEM - q_stage) / tile_bytes);
    SCD_REQUIRE(slots >= 4 && (size_t)slots * tile_bytes >= merge_bytes, SCD_ERR_SHAPE, "attention: shared memory does not fit");
    p.stages = slots / 2;                                         // K ring
    p.stages_v = slots - slots / 2;                               // V ring: a V slot is held longer
    p.C = C;
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)(units * C), 1, 1);
    cfg.blockDim = dim3(T5_THREADS, 1, 1);
    cfg.dynamicSmemBytes = T5_SMEM;
    cfg.stream = st;
    cudaLaunchAttribute attrs[2];
    attrs[0].id = cudaLaunchAttributeClusterDimension;
    attrs[0].val.clusterDim.x = (unsigned)C;
    attrs[0].val.clusterDim.y = 1;
    attrs[0].val.clusterDim.z = 1;
    attrs[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attrs;
    cfg.numAttrs = 2;
    SCD_CUDA_TRY(cudaLaunchKernelEx(&cfg, fn, p));
    count_launches(1);
    return SCD_OK;
}

int attention_tc(scd_session *s, int layer, int Mq, int pos_override, cudaStream_t st)
{
    const scd_model_config_t &c = s->model->cfg;
    AttnPlan *plan = (AttnPlan *)s->attn_plan;
    AttnParams p;
    std::memset(&p, 0, sizeof(p));
    p.kv_map = plan->kv_map;
    p.qkv = (const float *)s->qkv;
    p.out = (__nv_bfloat16 *)s->att;
    p.out_plane = (long long)s->rows_cap * c.n_heads * c.head_dim;
    p.pool = (__nv_bfloat16 *)s->kv_pool;
    p.page_table = s->page_table;
    p.n_known = s->n_known;
    p.rope = s->model->rope_table;
    p.err = (int *)s->gemm_ws;
    p.skip = s->skip_now;
    p.stamp = take_stamp_slot();
    const long long rows_per_kind = (long long)s->Q * s->pages_per_seq * c.n_kv_heads * c.kv_page_tokens;
    p.row0_k = (long long)layer * 2 * rows_per_kind;
    p.row0_v = p.row0_k + rows_per_kind;
    p.B = s->B; p.Mq = Mq; p.H = c.n_heads; p.Hkv = c.n_kv_heads; p.n_rep = c.n_heads / c.n_kv_heads;
    p.pages_per_seq = s->pages_per_seq; p.page_tokens = c.kv_page_tokens;
    p.page_shift = __builtin_ctz((unsigned)c.kv_page_tokens);
    p.max_seq = c.max_seq; p.pos_override = pos_override;
    p.n_mtiles = (Mq * p.n_rep + 15) / 16;
    p.qscale = 1.4426950408889634f / sqrtf((float)c.head_dim);
    const int variant = attention_tc_variant(s, Mq, pos_override >= 0 ? (long long)pos_override : s->ctx_floor);
    if ((variant & 15) == 2) return attention_t5(s, p, variant >> 4, st);
    const int units = s->Q * c.n_kv_heads;
    // split-KV over a cluster: up to two CTAs per SM over the whole grid, a power of two (measured:
    // clusters of 7 take 1.8 times as long as clusters of 4 on the same problem)
    p.C = attention_clusters(s, plan);
    const int dh = c.head_dim;
    const size_t q_bytes = 2 * (((size_t)p.n_mtiles * 16 * dh * 2 + 1023) & ~(size_t)1023);   // two planes
    const size_t stage_bytes = (size_t)2 * TK * dh * 2;
    const size_t merge_bytes = (size_t)p.n_mtiles * 16 * (dh + 2) * sizeof(float);
    // a ring deep enough to keep ~64 KB in flight per CTA, and wide enough for the merge staging
    int stages = (int)std::max<size_t>(3, (96 * 1024) / stage_bytes);
    stages = std::min(stages, MAX_ATT_STAGES);
    {
        // One wave: all CTAs of the grid must be resident together (clusters start only when all
        // their CTAs find room, and a second wave doubles the kernel's time). If the grid needs r
        // CTAs per SM, shrink the ring - not below two slots - until r of them fit.
        const int ctas = units * p.C;
        const int r = (ctas + plan->sm_count - 1) / plan->sm_count;
        if (r >= 2) {
            // per CTA: 1 KB reserved by the system, the static part rounded up to the 1 KB alignment of
            // the dynamic part, and the dynamic part itself
            // (and 1 KB to spare: a grid that falls into a second wave takes twice as long)
            const size_t per_cta = (size_t)(228 * 1024) / (size_t)r - 1024 - 1024 - 1024;
            while (stages > 2 && q_bytes + (size_t)stages * stage_bytes > per_cta) --stages;
        }
    }
    while ((size_t)stages * stage_bytes < merge_bytes && stages < MAX_ATT_STAGES) ++stages;
    SCD_REQUIRE((size_t)stages * stage_bytes >= merge_bytes, SCD_ERR_SHAPE, "attention: merge staging does not fit");
    p.stages = stages;
    const size_t smem = q_bytes + (size_t)stages * stage_bytes;
    SCD_REQUIRE(smem <= 227 * 1024 - 4096, SCD_ERR_SHAPE, "attention needs %zu bytes of shared memory", smem);
    static DeviceOnce once;
    int dev = 0;
    int rc = current_device(&dev);
    if (rc != SCD_OK) return rc;
    rc = once.run(dev, [&]() -> int {
        const int lim = 227 * 1024 - 4096;
        SCD_CUDA_TRY(cudaFuncSetAttribute(attention_tc_kernel<128, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, lim));
        SCD_CUDA_TRY(cudaFuncSetAttribute(attention_tc_kernel<128, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, lim));
        SCD_CUDA_TRY(cudaFuncSetAttribute(attention_tc_kernel<64, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, lim));
        SCD_CUDA_TRY(cudaFuncSetAttribute(attention_tc_kernel<64, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, lim));
        return SCD_OK;
    });
    if (rc != SCD_OK) return rc;
    const bool wide = (variant & 15) == 1;                        // two warps per query tile
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)(units * p.C), 1, 1);
    cfg.blockDim = dim3((unsigned)(32 * std::max(4, p.n_mtiles)), 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attrs[2];
    attrs[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[0].val.programmaticStreamSerializationAllowed = 1;
    attrs[1].id = cudaLaunchAttributeClusterDimension;
    attrs[1].val.clusterDim.x = (unsigned)p.C;
    attrs[1].val.clusterDim.y = 1;
    attrs[1].val.clusterDim.z = 1;
    cfg.attrs = attrs;
    cfg.numAttrs = 2;
    if (dh == 128) {
        if (wide) SCD_CUDA_TRY(cudaLaunchKernelEx(&cfg, attention_tc_kernel<128, 2>, p));
        else SCD_CUDA_TRY(cudaLaunchKernelEx(&cfg, attention_tc_kernel<128, 1>, p));
    } else {
        if (wide) SCD_CUDA_TRY(cudaLaunchKernelEx(&cfg, attention_tc_kernel<64, 2>, p));
        else SCD_CUDA_TRY(cudaLaunchKernelEx(&cfg, attention_tc_kernel<64, 1>, p));
    }
    count_launches(1);
    return SCD_OK;
}

}  // namespace scd
