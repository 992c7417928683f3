// Weight-streaming bf16 GEMM for the window forward on sm_100a: tcgen05.mma with the fp32
// accumulator in tensor memory, operands staged by TMA through a shared-memory ring.
//
//   y[m, n] = sum_k x[m, k] * w[n, k]        x [M, K] bf16 (M <= 256 window rows, K-major)
//                                            w [N, K] bf16 (row-major weights, K-major)
//
// The window has few rows (M = S*B*L, 64 for the 7B workload), so the GEMM is bound by streaming
// the weights once from HBM. The operands are swapped with respect to the usual orientation: a
// tile of 128 WEIGHT rows sits on the UMMA M axis (A operand), the window rows sit on the N axis
// (B operand, N = M rounded up to 16). Both are K-major, 128-byte swizzled, 64 bf16 per K block.
// One CTA = one 128-row weight tile x one K slice:
//   warp 0 : TMA producer (one lane)      - ring of `stages` slots, full/empty mbarriers
//   warp 1 : tensor memory allocation; one lane issues tcgen05.mma and commits
//   warps 2-5 : epilogue - tcgen05.ld of the accumulator (lane = weight row) into shared memory,
//               then the reduction over the K slices and the fused output operation
// K is split across the CTAs of a thread-block cluster (at most 8). Each CTA leaves its partial
// tile in its own shared memory; after a cluster barrier CTA c adds the partials of window rows
// [c M / C, (c+1) M / C) over all C peers through distributed shared memory, always in peer order
// 0..C-1, and stores them: no scratch in global memory, no atomics, a result that does not
// depend on scheduling.
//
// CTAs are small (a ring of ~72 KB, so that three fit on an SM) and the grid is ONE wave of them:
// the shape rule picks the number of K slices so that every SM has two or three CTAs streaming
// (grids of at most two CTAs per SM get a deeper ring). The kernel is launched with programmatic
// stream serialisation: the weight tiles of the ring are requested before griddepcontrol.wait, so the
// weight stream of this GEMM starts while the kernel in front of it drains; everything that
// depends on that kernel (the x operand, the residual stream, the norm statistics) is touched
// only after the wait.
//
// Activations in two bf16 planes: a session keeps every GEMM input x as x_hi = bf16(x) and
// x_lo = bf16(x - x_hi) (16 significant bits together) and the kernel accumulates W x_hi + W x_lo into the
// same tensor-memory accumulator - twice the tensor-core work, which the weight stream hides, no extra HBM
// traffic, and the rounding of the activations drops out of the result (at 32 layers of the 7B shape it
// was the larger part of the distance to an fp32 evaluation). Weights stay single bf16 values.
//
// Fused operations
//   RMSNorm of the x rows: x holds bf16(h * gain) (not yet divided by the RMS); the sums of
//     squares of h arrive as `ss_parts` partial sums per row, and the accumulator column of row m
//     is scaled by 1 / sqrt(sum / K + eps) before the output operation.
//   output: bf16 store | fp32 store | residual add into the fp32 stream h (+ bf16(h * gain_next)
//     and this tile's partial sum of squares for the next norm) | SwiGLU, where the 128 tile rows
//     are 64 gate rows followed by the 64 up rows of the same features.
// Every mbarrier wait is bounded; on expiry the kernel raises an error word, drains, frees its
// tensor memory and returns (all CTAs still meet at the cluster barriers).
#include <cuda.h>
#include <cstring>
#include <algorithm>
#include <map>
#include <tuple>

#include "gemm.cuh"

namespace scd {

namespace {

constexpr int TILE_N = 128;          // accumulator rows per tile (UMMA M)
constexpr int BLOCK_K = 64;          // bf16 per K block = one 128-byte swizzle span
constexpr int UMMA_K = 16;
constexpr int MAX_SEG = 3;
constexpr int MAX_STAGES = 12;
constexpr int MAX_CLUSTER = 8;
constexpr int MAX_ROWS = 256;        // window rows one GEMM may carry
constexpr int GEMM_THREADS = 192;
constexpr unsigned SPIN_LIMIT = 1u << 22;

enum { EPI_BF16 = 0, EPI_F32 = 1, EPI_RESID = 2, EPI_SWIGLU = 3 };

struct GemmParams {
    CUtensorMap tmap_w[MAX_SEG];     // weight segments; SwiGLU: [0] gate, [1] up, boxes of 64 rows
    CUtensorMap tmap_x;
    int seg_tile0[MAX_SEG + 1];      // first tile of each segment
    int seg_row0[MAX_SEG];           // weight row of the segment's first tile
    int seg_nout[MAX_SEG];           // end (exclusive) of the segment's rows in its weight matrix
    int seg_col0[MAX_SEG];           // output column of row 0 of the segment's weight matrix
    int n_seg;
    int M;                           // live window rows
    int nbox;                        // rows of the x box = UMMA N (multiple of 16)
    int x_planes;                    // 1: x is one bf16 matrix (2-D map); 2: hi and lo plane [2][rows][K] (3-D map)
    long long out_plane;             // EPI_SWIGLU / xg_out: elements from the hi plane to the lo plane of the output (0: hi only)
    int k_blocks;                    // K / 64
    int k_splits;                    // = cluster size
    int tile_rows;                   // weight rows per tile (<= 128; SwiGLU: features per tile, <= 64)
    int stages;
    int aux_offset;                  // byte offset (from the aligned ring base) of the small per-row scratch
    int epi;
    void *out;                       // bf16 or fp32 [M][ldo]
    int ldo;
    // RMSNorm of the x rows (optional): ss_in [ss_parts][ss_stride] partial sums of squares
    const float *ss_in;
    int ss_parts, ss_stride;
    float inv_k, eps;
    // EPI_RESID extras (optional): the normalisation input of the next GEMM
    const __nv_bfloat16 *gain_next;  // [ldo]
    __nv_bfloat16 *xg_out;           // [M][ldo] bf16(h * gain_next)
    float *ss_out;                   // [tiles][ss_stride] this tile's sum of h^2 per row
    int *err;                        // device error word
    const int *skip;                 // optional device flag: set = nothing to do, return at once
    unsigned long long *stamp;       // optional [2][STAMP_CTAS]: %globaltimer at CTA entry and exit
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
// Bounded wait: false when the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, unsigned parity)
{
    const uint32_t a = smem_u32(bar);
    for (unsigned i = 0; i < SPIN_LIMIT; ++i) {
        unsigned ok;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(a), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}

__device__ __forceinline__ void tma_load_2d(const CUtensorMap *map, uint64_t *bar, void *dst, int x, int y,
                                            uint64_t policy)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
                 " [%0], [%1, {%3, %4}], [%2], %5;"
                 ::"r"(smem_u32(dst)), "l"((uint64_t)map), "r"(smem_u32(bar)), "r"(x), "r"(y), "l"(policy)
                 : "memory");
}
__device__ __forceinline__ void tma_load_3d(const CUtensorMap *map, uint64_t *bar, void *dst, int x, int y, int z,
                                            uint64_t policy)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
                 " [%0], [%1, {%3, %4, %5}], [%2], %6;"
                 ::"r"(smem_u32(dst)), "l"((uint64_t)map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z), "l"(policy)
                 : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap *map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)map) : "memory");
}

__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void epilogue_bar_sync()          // the four epilogue warps only
{
    asm volatile("bar.sync 1, 128;" ::: "memory");
}
__device__ __forceinline__ float ld_peer_f32(uint32_t local_smem_addr, uint32_t peer)
{
    uint32_t remote;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_smem_addr), "r"(peer));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}

// K-major, 128-byte-swizzled operand tile: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr)
{
    return (uint64_t)((smem_addr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float *v)
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
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float *v)
{
    uint32_t r[16];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ float4 ld_peer_f32x4(uint32_t local_smem_addr, uint32_t peer)
{
    uint32_t remote;
    float4 v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_smem_addr), "r"(peer));
    asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(remote) : "memory");
    return v;
}

// ---- the reduction over the K slices and the output operation ------------------------------------
// One epilogue warp owns a window row at a time; lane l owns the four consecutive output features
// 4l .. 4l+3 of the tile, so partials travel as 16-byte loads and results leave as 8/16-byte stores.
constexpr int RESID_PREFETCH = 2;    // residual rows per warp fetched before the accumulator is ready

struct OutCols {
    int col;        // first output column of this lane's four
    int n_ok;       // how many of the four exist (a prefix)
    bool vec;       // all four exist and 16-byte (fp32) / 8-byte (bf16) accesses are aligned
    float4 gain;    // gain of the next norm for the four columns
};

__device__ __forceinline__ OutCols out_cols(const GemmParams &p, int seg, int row0, int lane)
{
    OutCols oc;
    const int limit = min(p.tile_rows, p.seg_nout[seg] - row0);
    oc.col = p.seg_col0[seg] + row0 + 4 * lane;
    oc.n_ok = max(0, min(4, limit - 4 * lane));
    oc.vec = oc.n_ok == 4 && (p.ldo & 3) == 0 && (oc.col & 3) == 0 && ((uintptr_t)p.out & 15) == 0 &&
             ((uintptr_t)p.xg_out & 7) == 0;
    oc.gain = make_float4(0.f, 0.f, 0.f, 0.f);
    return oc;
}
__device__ __forceinline__ float4 load_f32x4(const float *src, const OutCols &oc)
{
    if (oc.vec) return __ldcg((const float4 *)src);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (oc.n_ok > 0) v.x = __ldcg(src);
    if (oc.n_ok > 1) v.y = __ldcg(src + 1);
    if (oc.n_ok > 2) v.z = __ldcg(src + 2);
    if (oc.n_ok > 3) v.w = __ldcg(src + 3);
    return v;
}
__device__ __forceinline__ float4 load_gain4(const __nv_bfloat16 *g, const OutCols &oc)
{
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (oc.n_ok > 0) v.x = __bfloat162float(g[oc.col]);
    if (oc.n_ok > 1) v.y = __bfloat162float(g[oc.col + 1]);
    if (oc.n_ok > 2) v.z = __bfloat162float(g[oc.col + 2]);
    if (oc.n_ok > 3) v.w = __bfloat162float(g[oc.col + 3]);
    return v;
}
__device__ __forceinline__ void store_f32x4(float *dst, float4 v, const OutCols &oc)
{
    if (oc.vec) { *(float4 *)dst = v; return; }
    if (oc.n_ok > 0) dst[0] = v.x;
    if (oc.n_ok > 1) dst[1] = v.y;
    if (oc.n_ok > 2) dst[2] = v.z;
    if (oc.n_ok > 3) dst[3] = v.w;
}
__device__ __forceinline__ void store_bf16x4(__nv_bfloat16 *dst, float4 v, int n_ok, bool vec)
{
    if (vec) {
        const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
        uint2 u;
        u.x = *(const uint32_t *)&lo;
        u.y = *(const uint32_t *)&hi;
        *(uint2 *)dst = u;
        return;
    }
    if (n_ok > 0) dst[0] = __float2bfloat16_rn(v.x);
    if (n_ok > 1) dst[1] = __float2bfloat16_rn(v.y);
    if (n_ok > 2) dst[2] = __float2bfloat16_rn(v.z);
    if (n_ok > 3) dst[3] = __float2bfloat16_rn(v.w);
}

// v as two bf16 planes: hi = bf16(v), lo = bf16(v - hi)
__device__ __forceinline__ void store_bf16x4_split(__nv_bfloat16 *hi, long long plane, float4 v, int n_ok, bool vec)
{
    store_bf16x4(hi, v, n_ok, vec);
    if (plane == 0) return;
    const float4 r = make_float4(v.x - __bfloat162float(__float2bfloat16_rn(v.x)), v.y - __bfloat162float(__float2bfloat16_rn(v.y)),
                                 v.z - __bfloat162float(__float2bfloat16_rn(v.z)), v.w - __bfloat162float(__float2bfloat16_rn(v.w)));
    store_bf16x4(hi + plane, r, n_ok, vec);
}

// Plain outputs (bf16 | fp32 | residual). Epilogue warp `ew` takes window rows m_lo + ew, + 4, ...;
// R of them per round, the loads from all peers for all R in flight before the first sum. The sum
// over the peers runs in peer order 0..C-1 for every element.
template <int CM, int R>
__device__ __forceinline__ void reduce_rows(const GemmParams &p, uint32_t base, int C, int ew, int lane, int m_lo,
                                            int m_hi, int tile, const float *inv_s, const OutCols &oc,
                                            const float4 (&hpre)[RESID_PREFETCH])
{
    const bool scale = p.ss_in != nullptr;
    const bool resid = p.epi == EPI_RESID;
    const bool norm_out = resid && p.xg_out != nullptr;
    bool first = true;
    for (int mb = m_lo + ew; mb < m_hi; mb += 4 * R, first = false) {
        float4 part[R][CM];
        float4 h[R];
#pragma unroll
        for (int j = 0; j < R; ++j) {
            const int m = mb + 4 * j;
            const bool on = m < m_hi;
#pragma unroll
            for (int peer = 0; peer < CM; ++peer)
                part[j][peer] = (on && peer < C) ? ld_peer_f32x4(base + (uint32_t)(m * TILE_N + 4 * lane) * 4u, (uint32_t)peer)
                                                 : make_float4(0.f, 0.f, 0.f, 0.f);
            h[j] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (resid) {
                if (first && j < RESID_PREFETCH) h[j] = hpre[j < RESID_PREFETCH ? j : 0];
                else if (on) h[j] = load_f32x4((const float *)p.out + (size_t)m * p.ldo + oc.col, oc);
            }
        }
#pragma unroll
        for (int j = 0; j < R; ++j) {
            const int m = mb + 4 * j;
            if (m >= m_hi) break;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int peer = 0; peer < CM; ++peer) {
                v.x += part[j][peer].x; v.y += part[j][peer].y; v.z += part[j][peer].z; v.w += part[j][peer].w;
            }
            if (scale) { const float is = inv_s[m - m_lo]; v.x *= is; v.y *= is; v.z *= is; v.w *= is; }
            const size_t o = (size_t)m * p.ldo + oc.col;
            if (p.epi == EPI_BF16) store_bf16x4((__nv_bfloat16 *)p.out + o, v, oc.n_ok, oc.vec);
            else if (p.epi == EPI_F32) store_f32x4((float *)p.out + o, v, oc);
            else {
                float4 hn = h[j];
                hn.x += v.x; hn.y += v.y; hn.z += v.z; hn.w += v.w;
                store_f32x4((float *)p.out + o, hn, oc);
                if (norm_out) {
                    store_bf16x4_split(p.xg_out + o, p.out_plane,
                                       make_float4(hn.x * oc.gain.x, hn.y * oc.gain.y, hn.z * oc.gain.z, hn.w * oc.gain.w),
                                       oc.n_ok, oc.vec);
                    // columns that do not exist hold h = 0; fixed-shape tree over the tile's 128 columns
                    float sq = (hn.x * hn.x + hn.y * hn.y) + (hn.z * hn.z + hn.w * hn.w);
#pragma unroll
                    for (int o2 = 16; o2 > 0; o2 >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o2);
                    if (lane == 0) p.ss_out[(size_t)tile * p.ss_stride + m] = sq;
                }
            }
        }
    }
}

// SwiGLU: accumulator rows f (gate) and 64 + f (up) belong to feature row0 + f. Half a warp owns a
// window row: lane l takes the features 4 (l & 15) .. + 3 of row m_lo + 2 ew + (l >> 4), + 8, ...
template <int CM, int R>
__device__ __forceinline__ void reduce_swiglu(const GemmParams &p, uint32_t base, int C, int ew, int lane, int m_lo,
                                              int m_hi, int row0, const float *inv_s)
{
    const bool scale = p.ss_in != nullptr;
    const int hl = lane & 15, sub = lane >> 4;
    const int col = row0 + 4 * hl;
    const int n_ok = max(0, min(4, min(p.tile_rows, p.seg_nout[0] - row0) - 4 * hl));
    const bool vec = n_ok == 4 && (p.ldo & 3) == 0 && (col & 3) == 0 && ((uintptr_t)p.out & 7) == 0;
    for (int mb = m_lo + 2 * ew + sub; mb < m_hi; mb += 8 * R) {
        float4 pg[R][CM], pu[R][CM];
#pragma unroll
        for (int j = 0; j < R; ++j) {
            const int m = mb + 8 * j;
#pragma unroll
            for (int peer = 0; peer < CM; ++peer) {
                const bool on = m < m_hi && peer < C;
                const uint32_t a = base + (uint32_t)(m * TILE_N + 4 * hl) * 4u;
                pg[j][peer] = on ? ld_peer_f32x4(a, (uint32_t)peer) : make_float4(0.f, 0.f, 0.f, 0.f);
                pu[j][peer] = on ? ld_peer_f32x4(a + 64u * 4u, (uint32_t)peer) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
#pragma unroll
        for (int j = 0; j < R; ++j) {
            const int m = mb + 8 * j;
            if (m >= m_hi) break;
            float4 g = make_float4(0.f, 0.f, 0.f, 0.f), u = g;
#pragma unroll
            for (int peer = 0; peer < CM; ++peer) {
                g.x += pg[j][peer].x; g.y += pg[j][peer].y; g.z += pg[j][peer].z; g.w += pg[j][peer].w;
                u.x += pu[j][peer].x; u.y += pu[j][peer].y; u.z += pu[j][peer].z; u.w += pu[j][peer].w;
            }
            if (scale) {
                const float is = inv_s[m - m_lo];
                g.x *= is; g.y *= is; g.z *= is; g.w *= is;
                u.x *= is; u.y *= is; u.z *= is; u.w *= is;
            }
            const float4 y = make_float4(g.x / (1.0f + expf(-g.x)) * u.x, g.y / (1.0f + expf(-g.y)) * u.y,
                                         g.z / (1.0f + expf(-g.z)) * u.z, g.w / (1.0f + expf(-g.w)) * u.w);
            store_bf16x4_split((__nv_bfloat16 *)p.out + (size_t)m * p.ldo + col, p.out_plane, y, n_ok, vec);
        }
    }
}

__global__ void __launch_bounds__(GEMM_THREADS, 3) gemm_ws_kernel(const __grid_constant__ GemmParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[MAX_STAGES], empty_bar[MAX_STAGES], acc_bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;
    __shared__ int healthy_s[4];               // per epilogue warp: accumulator complete, no error raised

    pdl_trigger();                     // the next kernel may take the SM slots this grid leaves free
    if (p.skip && *p.skip) return;     // (the flag is older than this iteration: the same answer in every CTA)
    if (p.stamp && threadIdx.x == 0 && blockIdx.x < STAMP_CTAS) p.stamp[blockIdx.x] = global_timer_ns();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int C = p.k_splits;
    const int tile = blockIdx.x / C, split = blockIdx.x % C;      // split == rank in the cluster
    const int kb0 = (int)(((long long)split * p.k_blocks) / C);
    const int kb1 = (int)(((long long)(split + 1) * p.k_blocks) / C);
    const int nk = kb1 - kb0;
    const int nbox = p.nbox;
    const bool pair = p.epi == EPI_SWIGLU;

    // segment of this tile
    int seg = 0;
    if (!pair) { while (seg + 1 < p.n_seg && tile >= p.seg_tile0[seg + 1]) ++seg; }
    // first weight row of the tile (SwiGLU: 64 gate rows + 64 up rows of features row0 .. row0 + 63)
    const int row0 = p.seg_row0[seg] + (tile - p.seg_tile0[seg]) * p.tile_rows;

    uint8_t *stage_base = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t a_bytes = TILE_N * BLOCK_K * 2, b_plane = (uint32_t)nbox * BLOCK_K * 2;
    const uint32_t b_bytes = b_plane * (uint32_t)p.x_planes;      // hi tile, then lo tile
    const uint32_t stage_bytes = a_bytes + b_bytes;
    // bytes one K block brings: the tile's weight rows (the TMA box is tile_rows high) and the x rows
    const uint32_t load_bytes = (uint32_t)p.tile_rows * 128u * (pair ? 2u : 1u) + b_bytes;

    // The producer lane sets the barriers up and, before anything else happens in the CTA, requests
    // the first ring slots of weights: they depend on no kernel in front, so this stream starts while
    // tensor memory is still being allocated and while the kernel in front drains.
    uint64_t pol_w = 0, pol_x = 0;
    auto load_w = [&](int i, int s) {
        uint8_t *sa = stage_base + (size_t)s * stage_bytes;
        const int kx = (kb0 + i) * BLOCK_K;
        if (pair) {
            tma_load_2d(&p.tmap_w[0], &full_bar[s], sa, kx, row0, pol_w);
            tma_load_2d(&p.tmap_w[1], &full_bar[s], sa + a_bytes / 2, kx, row0, pol_w);
        } else {
            tma_load_2d(&p.tmap_w[seg], &full_bar[s], sa, kx, row0, pol_w);
        }
    };
    const int pre = min(p.stages, nk);
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        mbar_init(&acc_bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_w));
        asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_x));
        for (int i = 0; i < pre; ++i) {
            mbar_expect_tx(&full_bar[i], load_bytes);
            load_w(i, i);
        }
        tma_prefetch_desc(&p.tmap_x);
    }
    // Two planes of up to 128 rows: ONE instruction per K step multiplies the weight tile with the hi and
    // the lo tile together (they lie back to back in the slot: a B operand of 2 nbox rows); accumulator
    // columns [0, nbox) receive W x_hi, [nbox, 2 nbox) W x_lo, and the epilogue adds the halves. The
    // weight tile is then read from shared memory once per K step, not twice.
    const bool fused2 = p.x_planes == 2 && 2 * nbox <= 256;
    const int acc_cols = fused2 ? 2 * nbox : nbox;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < acc_cols) tmem_cols <<= 1;
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_s)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_s;

    // this CTA's partial tile for the cluster reduction: [window row][accumulator row] fp32; it
    // reuses the ring once every copy has landed and every MMA has read its operands
    float *stage_part = (float *)stage_base;
    // behind the ring: 1 / rms of the x rows this CTA reduces
    float *inv_s = (float *)(stage_base + p.aux_offset);
    // window rows this CTA reduces and stores
    const int m_lo = (int)(((long long)split * p.M) / C), m_hi = (int)(((long long)(split + 1) * p.M) / C);

    if (warp == 0 && lane == 0) {
        // ---------------- TMA producer ----------------
        pdl_wait();                                    // x is written by the kernel in front
        auto load_x = [&](int i, int s) {
            uint8_t *sb = stage_base + (size_t)s * stage_bytes + a_bytes;
            // (two planes: one copy of the box [2][nbox][64] - the hi tile, then the lo tile)
            if (p.x_planes == 2) tma_load_3d(&p.tmap_x, &full_bar[s], sb, (kb0 + i) * BLOCK_K, 0, 0, pol_x);
            else tma_load_2d(&p.tmap_x, &full_bar[s], sb, (kb0 + i) * BLOCK_K, 0, pol_x);
        };
        for (int i = 0; i < pre; ++i) load_x(i, i);
        int issued = pre;
        // (slot and round as running counters: a division per K block is a long way for one lane)
        for (int i = pre, s = pre == p.stages ? 0 : pre, round = pre == p.stages ? 1 : 0; i < nk; ++i) {
            if (!mbar_wait(&empty_bar[s], (round & 1) ^ 1)) { atomicExch(p.err, 1); abort_flag = 1; break; }
            mbar_expect_tx(&full_bar[s], load_bytes);
            load_w(i, s);
            load_x(i, s);
            issued = i + 1;
            if (++s == p.stages) { s = 0; ++round; }
        }
        if (abort_flag) {
            // drain: give the copies already issued a bounded time to land before the CTA exits
            for (int i = max(0, issued - p.stages); i < issued; ++i)
                mbar_wait(&full_bar[i % p.stages], (i / p.stages) & 1);
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------- MMA issuer ----------------
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(acc_cols >> 3) << 17) |
                               ((uint32_t)(TILE_N >> 4) << 24);
        bool ok = true;
        const bool second = p.x_planes == 2 && !fused2;
        for (int i = 0, s = 0, round = 0; i < nk && ok; ++i) {
            ok = mbar_wait(&full_bar[s], round & 1);
            if (!ok) { atomicExch(p.err, 2); break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t sa = smem_u32(stage_base + (size_t)s * stage_bytes);
            // (the descriptors of the K steps differ in the start address field only: 16-byte units, no carry out of it)
            const uint64_t da = umma_desc(sa), db = umma_desc(sa + a_bytes), db2 = umma_desc(sa + a_bytes + b_plane);
#pragma unroll
            for (int k = 0; k < BLOCK_K / UMMA_K; ++k) {
                const uint32_t koff = (uint32_t)(k * UMMA_K * 2) >> 4;
                umma_bf16(tmem_base, da + koff, db + koff, idesc, (i > 0 || k > 0) ? 1u : 0u);
                if (second) umma_bf16(tmem_base, da + koff, db2 + koff, idesc, 1u);
            }
            umma_commit(&empty_bar[s]);        // frees the slot once these MMAs have read it
            if (++s == p.stages) { s = 0; ++round; }
        }
        umma_commit(&acc_bar);                 // accumulator complete (or abandoned)
    }

    // ---------------- epilogue (warps 2-5) ----------------
    const int et = threadIdx.x - 64;           // 0..127 among the epilogue threads
    const int ew = warp - 2;                   // epilogue warp 0..3
    bool healthy = true;
    OutCols oc = {};
    float4 hpre[RESID_PREFETCH] = {};
    if (warp >= 2) {
        const int quarter = warp & 3;          // the TMEM lane quarter this warp may read
        const int r = quarter * 32 + lane;     // accumulator row
        pdl_wait();                            // norm statistics / outputs belong to kernels in front
        // 1 / rms of the rows this CTA will reduce, while the main loop streams
        if (p.ss_in) {
            for (int m = m_lo + et; m < m_hi; m += 128) {
                float ss = 0.f;
                for (int part = 0; part < p.ss_parts; ++part) ss += __ldcg(p.ss_in + (size_t)part * p.ss_stride + m);
                inv_s[m - m_lo] = rsqrtf(ss * p.inv_k + p.eps);
            }
        }
        // the residual rows this thread will add to, and the next norm's gain: fetched while the
        // main loop streams
        if (!pair) {
            oc = out_cols(p, seg, row0, lane);
            if (p.epi == EPI_RESID) {
                if (p.xg_out) oc.gain = load_gain4(p.gain_next, oc);
#pragma unroll
                for (int j = 0; j < RESID_PREFETCH; ++j) {
                    const int m = m_lo + ew + 4 * j;
                    hpre[j] = m < m_hi ? load_f32x4((const float *)p.out + (size_t)m * p.ldo + oc.col, oc)
                                       : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
        }
        const bool ok = mbar_wait(&acc_bar, 0);
        if (!ok) atomicExch(p.err, 3);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16);
        int errw = 0;
        if (lane == 0) errw = *(volatile int *)p.err;
        errw = __shfl_sync(0xffffffffu, errw, 0);
        healthy = __all_sync(0xffffffffu, ok) && errw == 0;   // warp-uniform
        if (lane == 0) healthy_s[warp - 2] = healthy ? 1 : 0;
        if (healthy) {
            // all copies into the ring have landed and all MMAs have read them (acc_bar)
            int c = 0;
            for (; c + 32 <= nbox; c += 32) {            // 32 accumulator columns per tensor-memory load
                float v[32];
                tmem_ld32(taddr + c, v);
                if (fused2) {
                    float v2[32];
                    tmem_ld32(taddr + nbox + c, v2);
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] += v2[j];
                }
#pragma unroll
                for (int j = 0; j < 32; ++j) stage_part[(size_t)(c + j) * TILE_N + r] = v[j];
            }
            for (; c < nbox; c += 16) {
                float v[16];
                tmem_ld16(taddr + c, v);
                if (fused2) {
                    float v2[16];
                    tmem_ld16(taddr + nbox + c, v2);
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] += v2[j];
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) stage_part[(size_t)(c + j) * TILE_N + r] = v[j];
            }
        }
    }
    if (C > 1) { __syncwarp(); cluster_sync_all(); }      // every CTA of the cluster has staged its partial
    else if (warp >= 2) epilogue_bar_sync();
    // the same decision in all four epilogue warps (they meet again at a named barrier below)
    if (warp >= 2) healthy = (healthy_s[0] & healthy_s[1] & healthy_s[2] & healthy_s[3]) != 0;

    if (warp >= 2 && healthy) {
        const uint32_t base = smem_u32(stage_part);
        if (!pair) {
            if (C <= 2) reduce_rows<2, 4>(p, base, C, ew, lane, m_lo, m_hi, tile, inv_s, oc, hpre);
            else if (C <= 4) reduce_rows<4, 2>(p, base, C, ew, lane, m_lo, m_hi, tile, inv_s, oc, hpre);
            else reduce_rows<8, 1>(p, base, C, ew, lane, m_lo, m_hi, tile, inv_s, oc, hpre);
        } else {
            if (C <= 2) reduce_swiglu<2, 2>(p, base, C, ew, lane, m_lo, m_hi, row0, inv_s);
            else if (C <= 4) reduce_swiglu<4, 1>(p, base, C, ew, lane, m_lo, m_hi, row0, inv_s);
            else reduce_swiglu<8, 1>(p, base, C, ew, lane, m_lo, m_hi, row0, inv_s);
        }
    }
    if (C > 1) { __syncwarp(); cluster_sync_all(); }      // nobody leaves while a peer still reads its partial
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
    if (p.stamp && threadIdx.x == 0 && blockIdx.x < STAMP_CTAS) p.stamp[STAMP_CTAS + blockIdx.x] = global_timer_ns();
}

// ------------------------------------------------------------------------------------------ host
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)sym;
    }
    return fn;
}

}  // namespace

int make_tensor_map_bf16_2d(void *map, const void *ptr, unsigned long long rows, unsigned long long cols,
                            unsigned box_rows, unsigned box_cols)
{
    EncodeTiledFn fn = encode_fn();
    SCD_REQUIRE(fn, SCD_ERR_CUDA, "cuTensorMapEncodeTiled entry point not found");
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn((CUtensorMap *)map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides,
                    box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    SCD_REQUIRE(r == CUDA_SUCCESS, SCD_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d) rows %llu cols %llu box %u x %u",
                (int)r, rows, cols, box_rows, box_cols);
    return SCD_OK;
}

namespace {

// 2-D bf16 row-major matrix [rows][K], box = 64 (K) x box_rows, 128-byte swizzle.
int make_map(CUtensorMap *map, const void *ptr, uint64_t rows, uint64_t K, uint32_t box_rows)
{
    return make_tensor_map_bf16_2d(map, ptr, rows, K, box_rows, BLOCK_K);
}

// Two-plane activation buffer [2][rows][K] bf16: box = 64 (K) x box_rows x both planes, 128-byte swizzle.
// (rows: rows of a plane that the map covers from ptr on; plane_rows: rows from one plane to the other)
int make_map_planes(CUtensorMap *map, const void *ptr, uint64_t rows, uint64_t plane_rows, uint64_t K, uint32_t box_rows)
{
    EncodeTiledFn fn = encode_fn();
    SCD_REQUIRE(fn, SCD_ERR_CUDA, "cuTensorMapEncodeTiled entry point not found");
    cuuint64_t dims[3] = {K, rows, 2};
    cuuint64_t strides[2] = {K * 2, plane_rows * K * 2};
    cuuint32_t box[3] = {BLOCK_K, box_rows, 2};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    SCD_REQUIRE(r == CUDA_SUCCESS, SCD_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d) rows %llu K %llu box rows %u, two planes",
                (int)r, (unsigned long long)rows, (unsigned long long)K, box_rows);
    return SCD_OK;
}

struct GemmPlan {                    // per model: weight-side tensor maps, built on first use
    std::map<std::tuple<const void *, int, int, int>, CUtensorMap> wmaps;   // (matrix, rows, K, box rows)
    int sm_count;
    int kind_splits[GEMM_KINDS];     // K slices per GEMM kind chosen by gemm_set_kind_splits (0: the rule)
    int forced_splits, forced_stages; // scd_model_gemm_tune (0: the rule)
};

inline int round16(int m) { return std::max(16, (m + 15) & ~15); }

inline size_t stage_bytes_of(int nbox, int planes) { return (size_t)TILE_N * BLOCK_K * 2 + (size_t)planes * nbox * BLOCK_K * 2; }
inline size_t staging_bytes_of(int nbox) { return (size_t)nbox * TILE_N * sizeof(float); }
constexpr size_t SMEM_LIMIT = 227 * 1024 - 8192;   // dynamic shared memory one CTA may ask for

struct Segment { const void *w; int rows, K; int row0, row_end, col0; };   // weight rows [row0, row_end) -> columns col0 + row

int tiles_for(const Segment *segs, int n_seg, bool pair, int h)
{
    int t = 0;
    for (int i = 0; i < (pair ? 1 : n_seg); ++i) t += (segs[i].row_end - segs[i].row0 + h - 1) / h;
    return t;
}

// Launch shape of one GEMM: K slices C (= cluster size, at most 8, the portable limit) and tile
// height h. Measured on B200: one wave of CTAs streams best (three CTAs fit per SM, clusters
// leave some slots unused; a second wave costs 30-50 %), full-height tiles beat lower ones (the x
// tile is re-read per weight tile), and a CTA should stream at most ~32 K blocks. So: full-height
// tiles and the smallest C that gives every SM two CTAs.
void choose_shape(const Segment *segs, int n_seg, bool pair, int k_blocks, int sm_count, int *C_out, int *h_out,
                  int *tiles_out, int tuned = 0, int forced = 0)
{
    const int h = pair ? TILE_N / 2 : TILE_N;
    const int tiles = tiles_for(segs, n_seg, pair, h);
    int C;
    if (forced > 0) C = forced;
    else if (tuned > 0) C = tuned;
    else {
        C = (k_blocks + 31) / 32;
        while (C < MAX_CLUSTER && tiles * C < 2 * sm_count && k_blocks / (C + 1) >= 2) ++C;
    }
    *C_out = std::max(1, std::min(std::min(C, k_blocks), MAX_CLUSTER));
    *h_out = h;
    *tiles_out = tiles;
}

// Ring slots: about 72 KB per CTA so that three CTAs share an SM - or about 100 KB when the grid has
// at most two CTAs per SM anyway (measured: the deeper ring then wins a few percent) - and never
// less than the partial-tile staging.
int choose_stages(int nbox, int planes, int k_blocks_per_cta, bool two_per_sm, int forced = 0)
{
    const int stage_bytes = (int)stage_bytes_of(nbox, planes);
    int st = std::max(2, ((two_per_sm ? 100 : 73) * 1024) / stage_bytes);
    if (forced > 0) st = forced;
    st = std::min(st, (int)((SMEM_LIMIT - 1024) / stage_bytes));
    st = std::min(st, MAX_STAGES);
    st = std::min(st, std::max(2, k_blocks_per_cta));
    return std::max(st, 1);
}

int launch(GemmParams &p, int tiles, cudaStream_t st)
{
    const size_t ring = std::max((size_t)p.stages * stage_bytes_of(p.nbox, p.x_planes), staging_bytes_of(p.nbox));
    p.aux_offset = (int)ring;
    const size_t rows_per_cta = (size_t)(p.M + p.k_splits - 1) / p.k_splits;
    size_t smem = ring + 5 * rows_per_cta * sizeof(float) + 1024;
    SCD_REQUIRE(smem <= SMEM_LIMIT, SCD_ERR_SHAPE, "GEMM needs %zu bytes of shared memory", smem);
    SCD_REQUIRE(p.M <= MAX_ROWS, SCD_ERR_SHAPE, "GEMM carries at most %d window rows", MAX_ROWS);
    static DeviceOnce once;
    int dev = 0;
    int rc = current_device(&dev);
    if (rc != SCD_OK) return rc;
    rc = once.run(dev, [&]() -> int {
        SCD_CUDA_TRY(cudaFuncSetAttribute(gemm_ws_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_LIMIT));
        return SCD_OK;
    });
    if (rc != SCD_OK) return rc;
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)(tiles * p.k_splits), 1, 1);
    cfg.blockDim = dim3(GEMM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attrs[2];
    attrs[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[0].val.programmaticStreamSerializationAllowed = 1;
    attrs[1].id = cudaLaunchAttributeClusterDimension;
    attrs[1].val.clusterDim.x = (unsigned)p.k_splits;
    attrs[1].val.clusterDim.y = 1;
    attrs[1].val.clusterDim.z = 1;
    cfg.attrs = attrs;
    cfg.numAttrs = 2;
    SCD_CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_ws_kernel, p));
    count_launches(1);
    return SCD_OK;
}

struct SessionGemm {                 // activation-side tensor maps of a session, by (buffer, K, box rows)
    std::map<std::tuple<const void *, int, int>, CUtensorMap> xmaps;
};

// (planes = 2: both planes of an activation buffer in one map; 1: its hi plane alone; m0: first row the map covers)
int x_map(scd_session *s, const void *buf, int K, int nbox, int planes, int m0, CUtensorMap *out)
{
    SessionGemm *sg = (SessionGemm *)s->gemm_state;
    buf = (const __nv_bfloat16 *)buf + (size_t)m0 * K;
    auto key = std::make_tuple(buf, K, nbox * 4 + planes);
    auto it = sg->xmaps.find(key);
    if (it == sg->xmaps.end()) {
        CUtensorMap m;
        int rc = planes == 2 ? make_map_planes(&m, buf, (uint64_t)(s->rows_cap - m0), (uint64_t)s->rows_cap, (uint64_t)K, (uint32_t)nbox)
                             : make_map(&m, buf, (uint64_t)(s->rows_cap - m0), (uint64_t)K, (uint32_t)nbox);
        if (rc != SCD_OK) return rc;
        it = sg->xmaps.emplace(key, m).first;
    }
    *out = it->second;
    return SCD_OK;
}


struct NormIn { const float *ss; int parts; };                 // statistics of the x rows
struct NormOut { const void *gain; void *xg; float *ss; };     // what a residual GEMM leaves behind

int g_last_tiles = 0;                 // weight tiles of the most recent GEMM launch

int w_map(GemmPlan *plan, const Segment &sg, int box_rows, CUtensorMap *out)
{
    auto key = std::make_tuple(sg.w, sg.rows, sg.K, box_rows);
    auto it = plan->wmaps.find(key);
    if (it == plan->wmaps.end()) {
        CUtensorMap tm;
        int rc = make_map(&tm, sg.w, (uint64_t)sg.rows, (uint64_t)sg.K, (uint32_t)box_rows);
        if (rc != SCD_OK) return rc;
        it = plan->wmaps.emplace(key, tm).first;
    }
    *out = it->second;
    return SCD_OK;
}

// x_planes: 2 = multiply with both planes of x, 1 = with its hi plane alone (where the output is rounded to
// bf16 right away - Q, K, V - or is the last stage - the logits - the remainder plane buys nothing)
// (the window rows m0 .. m0 + rows - 1, at most 256: one accumulator holds all rows of a weight tile)
int run_gemm_rows(scd_session *s, int kind, const Segment *segs, int n_seg, int epi, const void *x, int K, int m0, int rows,
                  void *out, int ldo, const NormIn *nin, const NormOut *nout, int x_planes, cudaStream_t st)
{
    GemmPlan *plan = (GemmPlan *)s->model->gemm_plan;
    const bool pair = epi == EPI_SWIGLU;
    GemmParams p;
    std::memset(&p, 0, sizeof(p));
    p.k_blocks = K / BLOCK_K;
    int tiles = 0;
    choose_shape(segs, n_seg, pair, p.k_blocks, plan->sm_count, &p.k_splits, &p.tile_rows, &tiles,
                 plan->kind_splits[kind], plan->forced_splits);
    int t0 = 0;
    for (int i = 0; i < n_seg; ++i) {
        int rc = w_map(plan, segs[i], p.tile_rows, &p.tmap_w[i]);
        if (rc != SCD_OK) return rc;
        p.seg_row0[i] = segs[i].row0;
        p.seg_nout[i] = segs[i].row_end;
        p.seg_col0[i] = segs[i].col0;
        if (!pair) { p.seg_tile0[i] = t0; t0 += (segs[i].row_end - segs[i].row0 + p.tile_rows - 1) / p.tile_rows; }
    }
    p.seg_tile0[pair ? 1 : n_seg] = tiles;
    p.n_seg = pair ? 1 : n_seg;
    p.M = rows;
    p.nbox = round16(rows);
    p.x_planes = x_planes;
    p.out_plane = (long long)s->rows_cap * ldo;           // (used by the outputs that are GEMM inputs themselves)
    p.stages = choose_stages(p.nbox, p.x_planes, (p.k_blocks + p.k_splits - 1) / p.k_splits,
                             tiles * p.k_splits <= 2 * plan->sm_count, plan->forced_stages);
    p.epi = epi;
    // everything indexed by window row starts at row m0
    const size_t out_elem = (epi == EPI_BF16 || epi == EPI_SWIGLU) ? 2 : 4;
    p.out = (char *)out + (size_t)m0 * ldo * out_elem;
    p.ldo = ldo;
    p.ss_stride = s->rows_cap;
    if (nin && nin->ss) {
        p.ss_in = nin->ss + m0; p.ss_parts = nin->parts;
        p.inv_k = 1.0f / (float)K; p.eps = s->model->cfg.rms_eps;
    }
    if (nout && nout->xg) {
        SCD_REQUIRE(tiles <= s->ss_parts_cap, SCD_ERR_SHAPE, "norm statistics: %d tiles > %d", tiles, s->ss_parts_cap);
        p.gain_next = (const __nv_bfloat16 *)nout->gain;
        p.xg_out = (__nv_bfloat16 *)nout->xg + (size_t)m0 * ldo;
        p.ss_out = nout->ss + m0;
    }
    int rc = x_map(s, x, K, p.nbox, p.x_planes, m0, &p.tmap_x);
    if (rc != SCD_OK) return rc;
    p.err = (int *)s->gemm_ws;
    p.skip = s->skip_now;
    p.stamp = take_stamp_slot();
    g_last_tiles = tiles;
    return launch(p, tiles, st);
}

// More than 256 window rows: one pass over the weights per block of 256 rows.
int run_gemm(scd_session *s, int kind, const Segment *segs, int n_seg, int epi, const void *x, int K, int rows,
             void *out, int ldo, const NormIn *nin, const NormOut *nout, int x_planes, cudaStream_t st)
{
    for (int m0 = 0; m0 < rows; m0 += 256) {
        const int rc = run_gemm_rows(s, kind, segs, n_seg, epi, x, K, m0, std::min(256, rows - m0), out, ldo, nin, nout, x_planes, st);
        if (rc != SCD_OK) return rc;
    }
    return SCD_OK;
}

}  // namespace

int gemm_plan_create(scd_model *m)
{
    GemmPlan *plan = new GemmPlan();
    int dev = 0;
    cudaGetDevice(&dev);
    plan->sm_count = 148;
    for (int k = 0; k < GEMM_KINDS; ++k) plan->kind_splits[k] = 0;
    plan->forced_splits = plan->forced_stages = 0;
    if (cudaDeviceGetAttribute(&plan->sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        delete plan;
        return cuda_fail(cudaGetLastError(), "cudaDeviceGetAttribute");
    }
    m->gemm_plan = plan;
    return SCD_OK;
}

void gemm_plan_destroy(scd_model *m)
{
    delete (GemmPlan *)m->gemm_plan;
    m->gemm_plan = nullptr;
}

// The norm statistics of the rows in xn: the producer of xn left `ss_parts` partial sums of squares.
int gemm_tc_qkv(scd_session *s, int l, int rows, int ss_parts, cudaStream_t st)
{
    const scd_model *m = s->model;
    const scd_model_config_t &c = m->cfg;
    const int d = c.d_model, dq = c.n_heads * c.head_dim, dkv = c.n_kv_heads * c.head_dim;
    const Segment segs[3] = {{m->wq[l], dq, d, 0, dq, 0}, {m->wk[l], dkv, d, 0, dkv, dq}, {m->wv[l], dkv, d, 0, dkv, dq + dkv}};
    const NormIn nin = {s->ss, ss_parts};
    // fp32 out: the attention kernel rotates Q and K in fp32 and rounds each of Q, K, V to bf16 once
    return run_gemm(s, GEMM_QKV, segs, 3, EPI_F32, s->xn, d, rows, s->qkv, dq + 2 * dkv, &nin, nullptr, 1, st);
}

int gemm_tc_residual(scd_session *s, int l, int which, int rows, const void *gain_next, int *parts_out,
                     cudaStream_t st)
{
    const scd_model *m = s->model;
    const scd_model_config_t &c = m->cfg;
    const int dq = c.n_heads * c.head_dim;
    const int K = which == 0 ? dq : c.d_ffn;
    const Segment segs[1] = {{which == 0 ? m->wo[l] : m->w_down[l], c.d_model, K, 0, c.d_model, 0}};
    const NormOut nout = {gain_next, s->xn, s->ss};
    const int rc = run_gemm(s, which == 0 ? GEMM_O : GEMM_DOWN, segs, 1, EPI_RESID, which == 0 ? s->att : s->act, K, rows,
                            s->h, c.d_model, nullptr,
                            &nout, 2, st);
    *parts_out = g_last_tiles;                          // one partial sum of squares per output tile
    return rc;
}

int gemm_tc_gate_up(scd_session *s, int l, int rows, int ss_parts, cudaStream_t st)
{
    const scd_model *m = s->model;
    const scd_model_config_t &c = m->cfg;
    const Segment segs[2] = {{m->w_gate[l], c.d_ffn, c.d_model, 0, c.d_ffn, 0}, {m->w_up[l], c.d_ffn, c.d_model, 0, c.d_ffn, 0}};
    const NormIn nin = {s->ss, ss_parts};
    return run_gemm(s, GEMM_GATE_UP, segs, 2, EPI_SWIGLU, s->xn, c.d_model, rows, s->act, c.d_ffn, &nin, nullptr, 2, st);
}

// Logits of the ids [lo, hi) and, when eol >= 0, of id eol; other columns of `logits` are left
// untouched (the sampler reads no others). lo = 0, hi = V: the whole row.
int gemm_tc_lm_head(scd_session *s, int rows, float *logits, int lo, int hi, int eol, int ss_parts, cudaStream_t st)
{
    const scd_model_config_t &c = s->model->cfg;
    Segment segs[2];
    int n = 0;
    const int lo8 = lo & ~7;
    segs[n++] = {s->model->lm_head, c.vocab_out, c.d_model, lo8, hi, 0};
    if (eol >= 0 && !(eol >= lo8 && eol < hi))
        segs[n++] = {s->model->lm_head, c.vocab_out, c.d_model, eol & ~7, std::min(c.vocab_out, (eol & ~7) + 8), 0};
    const NormIn nin = {s->ss, ss_parts};
    return run_gemm(s, GEMM_LM_HEAD, segs, n, EPI_F32, s->xn, c.d_model, rows, logits, c.vocab_out, &nin, nullptr, 1, st);
}

void gemm_set_kind_splits(scd_model *m, int kind, int k_splits)
{
    GemmPlan *plan = (GemmPlan *)m->gemm_plan;
    if (plan && kind >= 0 && kind < GEMM_KINDS) plan->kind_splits[kind] = std::max(0, std::min(k_splits, MAX_CLUSTER));
}

// Upper bound of the partial sums of squares a residual GEMM leaves per row (= its output tiles).
int gemm_norm_parts_cap(const scd_session *s) { return std::max(1024, (s->model->cfg.d_model + 7) / 8); }

// Per-session state: the activation-side tensor maps and the device error word.
int gemm_session_prepare(scd_session *s)
{
    s->gemm_state = new SessionGemm();
    SCD_CUDA_TRY(cudaMalloc(&s->gemm_ws, 256));
    SCD_CUDA_TRY(cudaMemset(s->gemm_ws, 0, 256));
    s->gemm_ws_bytes = 256;
    return SCD_OK;
}

void gemm_session_release(scd_session *s)
{
    delete (SessionGemm *)s->gemm_state;
    s->gemm_state = nullptr;
}

int gemm_error_word(scd_session *s, int *host_value, cudaStream_t st)
{
    *host_value = 0;
    if (!s->gemm_ws) return SCD_OK;
    SCD_CUDA_TRY(cudaMemcpyAsync(host_value, s->gemm_ws, sizeof(int), cudaMemcpyDeviceToHost, st));
    SCD_CUDA_TRY(cudaStreamSynchronize(st));
    return SCD_OK;
}

}  // namespace scd

// ------------------------------------------------------------------------------------------ hook
using namespace scd;

extern "C" {

int64_t scd_gemm_workspace_bytes(int32_t M, int32_t N, int32_t K)
{
    if (M < 1 || M > 256 || N < 1 || K < BLOCK_K || K % BLOCK_K) return SCD_ERR_SHAPE;
    return 256;                                           // the device error word
}

int scd_model_gemm_tune(scd_model_t *m, int32_t k_splits, int32_t stages)
{
    SCD_REQUIRE(m, SCD_ERR_ARG, "scd_model_gemm_tune: NULL model");
    SCD_REQUIRE(k_splits >= 0 && k_splits <= MAX_CLUSTER && stages >= 0 && stages <= MAX_STAGES, SCD_ERR_ARG,
                "scd_model_gemm_tune: k_splits %d (0..%d), stages %d (0..%d)", k_splits, MAX_CLUSTER, stages, MAX_STAGES);
    GemmPlan *plan = (GemmPlan *)m->gemm_plan;
    if (!plan) return SCD_OK;                             // fp32 model: no tcgen05 GEMMs to shape
    plan->forced_splits = k_splits;
    plan->forced_stages = stages;
    return SCD_OK;
}

int scd_gemm_bf16_shaped(const void *x, const void *w, float *y, int32_t M, int32_t N, int32_t K, int32_t k_splits,
                         int32_t stages, void *workspace, void *stream)
{
    SCD_REQUIRE(x && w && y && workspace, SCD_ERR_ARG, "scd_gemm_bf16: NULL argument");
    SCD_REQUIRE(M >= 1 && M <= 256 && N >= 1 && N % 8 == 0 && K >= BLOCK_K && K % BLOCK_K == 0, SCD_ERR_SHAPE,
                "scd_gemm_bf16: M %d (1..256), N %d (multiple of 8), K %d (multiple of 64)", M, N, K);
    SCD_REQUIRE(k_splits >= 0 && k_splits <= MAX_CLUSTER && stages >= 0 && stages <= MAX_STAGES, SCD_ERR_ARG,
                "scd_gemm_bf16: k_splits %d (0..%d), stages %d (0..%d)", k_splits, MAX_CLUSTER, stages, MAX_STAGES);
    SCD_REQUIRE((((uintptr_t)x | (uintptr_t)w | (uintptr_t)workspace) & 15) == 0, SCD_ERR_ARG,
                "scd_gemm_bf16: pointers must be 16-byte aligned");
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    GemmParams p;
    std::memset(&p, 0, sizeof(p));
    p.k_blocks = K / BLOCK_K;
    const Segment seg = {w, N, K, 0, N, 0};
    int tiles = 0;
    choose_shape(&seg, 1, false, p.k_blocks, sms, &p.k_splits, &p.tile_rows, &tiles, 0, k_splits);
    int rc = make_map(&p.tmap_w[0], w, (uint64_t)N, (uint64_t)K, (uint32_t)p.tile_rows);
    if (rc != SCD_OK) return rc;
    p.nbox = round16(M);
    // the x box may reach past row M: rows beyond the matrix are zero-filled by TMA
    rc = make_map(&p.tmap_x, x, (uint64_t)M, (uint64_t)K, (uint32_t)p.nbox);
    if (rc != SCD_OK) return rc;
    p.seg_tile0[0] = 0; p.seg_tile0[1] = tiles; p.seg_row0[0] = 0; p.seg_nout[0] = N; p.seg_col0[0] = 0; p.n_seg = 1;
    p.M = M;
    p.x_planes = 1;                                       // the hook multiplies one bf16 matrix
    p.stages = choose_stages(p.nbox, 1, (p.k_blocks + p.k_splits - 1) / p.k_splits, tiles * p.k_splits <= 2 * sms, stages);
    p.epi = EPI_F32;
    p.out = y;
    p.ldo = N;
    p.err = (int *)workspace;                             // must be zero on entry; stays zero unless a wait gave up
    return launch(p, tiles, (cudaStream_t)stream);
}

int scd_gemm_bf16(const void *x, const void *w, float *y, int32_t M, int32_t N, int32_t K, void *workspace,
                  void *stream)
{
    return scd_gemm_bf16_shaped(x, w, y, M, N, K, 0, 0, workspace, stream);
}

}  // extern "C"
