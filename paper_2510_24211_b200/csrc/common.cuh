// Shared device helpers of the SCD CUDA library: status handling, counter-based noise,
// the specified exponential, integer-weight arithmetic and block reductions.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <mutex>

#include "../../include/scd_hooks.h"

namespace scd {

typedef unsigned __int128 u128;

// ---------------------------------------------------------------------------- host-side errors
void set_last_error(const char *fmt, ...);
int cuda_fail(cudaError_t e, const char *what);
// Kernels enqueued by this process so far: every launch site counts itself.
void count_launches(long long n);

// Set-up that a CUDA device needs once (a kernel's shared-memory opt-in is a per-device attribute, the
// address of a __device__ array differs per device): `done` remembers the ordinals it has run on, the
// lock keeps a second host thread from launching before the first has finished the set-up.
struct DeviceOnce {
    static constexpr int kSlots = 64;
    std::mutex lock;
    bool done[kSlots] = {};
    // Runs setup() unless it already succeeded on `device`; ordinals beyond the table run it every time.
    template <class F>
    int run(int device, F setup)
    {
        std::lock_guard<std::mutex> g(lock);
        if (device >= 0 && device < kSlots && done[device]) return SCD_OK;
        const int rc = setup();
        if (rc == SCD_OK && device >= 0 && device < kSlots) done[device] = true;
        return rc;
    }
};
int current_device(int *device);    // cudaGetDevice as a status code

#define SCD_CUDA_TRY(expr)                                                     \
    do {                                                                       \
        cudaError_t e__ = (expr);                                              \
        if (e__ != cudaSuccess) return ::scd::cuda_fail(e__, #expr);           \
    } while (0)

#define SCD_REQUIRE(cond, code, ...)                                           \
    do {                                                                       \
        if (!(cond)) { ::scd::set_last_error(__VA_ARGS__); return (code); }    \
    } while (0)

// nanoseconds of the GPU-wide timer (time stamps of scd_step_timeline)
__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// ---------------------------------------------------------------------------- dependent launch
// Programmatic dependent launch. A kernel launched with programmatic stream serialisation may
// start while the kernel in front of it still runs; it must call pdl_wait() before it touches
// anything that kernel writes. pdl_trigger() lets the kernel behind this one start early.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---------------------------------------------------------------------------- noise
// Philox4x32-10 (Salmon et al., SC'11). key = 64-bit seed; counter = (sub, position, iteration,
// stream | batch << 8); the uniform variate is the top 24 bits of output word 0.
enum { NOISE_ACCEPT = 1, NOISE_RESIDUAL = 2, NOISE_INIT = 3, NOISE_INDEP = 4, NOISE_ALPHA = 5, NOISE_GUMBEL = 6 };

__device__ __forceinline__ uint32_t philox_word0(uint32_t k0, uint32_t k1, uint32_t c0, uint32_t c1,
                                                 uint32_t c2, uint32_t c3)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = hi1 ^ c1 ^ k0;
        const uint32_t n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return c0;
}

__device__ __forceinline__ uint32_t noise_u24(uint64_t seed, uint32_t stream, uint32_t batch,
                                              int64_t position, uint32_t iteration, uint32_t sub)
{
    return philox_word0((uint32_t)seed, (uint32_t)(seed >> 32), sub, (uint32_t)position, iteration,
                        stream | (batch << 8)) >> 8;
}

// ---------------------------------------------------------------------------- race times
// Gumbel-max (Algorithm 4) as an exponential race: argmax(log P_v + g_v) = argmin(E_v / P_v) with
// E_v = -log u_v. This is -log2 u for u = (U + 1/2) / 2^24 = n / 2^25, n = 2U + 1, as an integer
// with 40 fraction bits: 25 - log2 n. The mantissa m = n / 2^e in [1, 2) is held as m * 2^63;
// squaring it yields one binary digit of log2 m per step (digit 1 and m <- m^2 / 2 when m^2 >= 2),
// every square truncated to its upper 64 bits. The factor ln 2 does not change an argmin.
__device__ __forceinline__ unsigned long long neglog2_q40(unsigned U)
{
    const unsigned n = 2u * (U & 0xFFFFFFu) + 1u;      // odd, 1 .. 2^25 - 1
    const int e = 31 - __clz(n);
    unsigned long long x = (unsigned long long)n << (63 - e);
    unsigned long long frac = 0;
#pragma unroll 8
    for (int i = 0; i < 40; ++i) {
        const unsigned long long y = __umul64hi(x, x);  // m^2 * 2^62
        frac <<= 1;
        if (y >> 63) { frac |= 1ull; x = y; }
        else x = y << 1;
    }
    return (25ull << 40) - (((unsigned long long)e << 40) | frac);
}

// ---------------------------------------------------------------------------- scd_exp
// e^x for x <= 0 as a fixed sequence of round-to-nearest fp32 operations:
//   x < -22 -> 0;  n = rint(x * log2 e);  r = x - n ln2 (hi/lo split, fused);
//   degree-6 Taylor polynomial of e^r in Horner form (fused);  result = poly * 2^n.
// Every operation is an explicit intrinsic so that the compiler neither contracts nor
// reassociates: the integer weights derived from the result decide accept / reject.
__device__ __forceinline__ float scd_exp(float x)
{
    if (!(x >= -22.0f)) return 0.0f;
    if (x > 0.0f) x = 0.0f;
    const float t = __fmul_rn(x, 0x1.715476p+0f);
    const float n = rintf(t);
    float r = __fmaf_rn(n, -0x1.62e400p-1f, x);
    r = __fmaf_rn(n, -0x1.7f7d1cp-20f, r);
    float p = 0x1.6c16c2p-10f;
    p = __fmaf_rn(p, r, 0x1.111112p-7f);
    p = __fmaf_rn(p, r, 0x1.555556p-5f);
    p = __fmaf_rn(p, r, 0x1.555556p-3f);
    p = __fmaf_rn(p, r, 0.5f);
    p = __fmaf_rn(p, r, 1.0f);
    p = __fmaf_rn(p, r, 1.0f);
    const float scale = __int_as_float(((int)n + 127) << 23);
    return __fmul_rn(p, scale);
}

// Integer weight of a post-processed logit: W = trunc(scd_exp(x - m) * 2^30), 0 below the
// top-k threshold.
__device__ __forceinline__ uint32_t weight_of(float x, float m, float tau)
{
    if (!(x >= tau)) return 0u;
    const float e = scd_exp(__fsub_rn(x, m));
    return (uint32_t)__fmul_rn(e, 1073741824.0f);
}
// ... and 0 below the nucleus threshold theta (theta = 0: no top-p)
__device__ __forceinline__ uint32_t weight_of(float x, float m, float tau, uint32_t theta)
{
    const uint32_t w = weight_of(x, m, tau);
    return w >= theta ? w : 0u;
}

// Order-preserving map float -> uint32 (for radix selection of the k-th largest logit).
__device__ __forceinline__ uint32_t float_key(float f)
{
    const uint32_t b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key_float(uint32_t k)
{
    const uint32_t b = (k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k;
    return __uint_as_float(b);
}

// ---------------------------------------------------------------------------- wide sums
// A sum of up to 2^16 terms of at most 2^77 each, kept as two independent 64-bit limbs
// (low 40 bits / the rest) so that partial sums combine with plain, associative 64-bit adds.
struct Limbs {
    unsigned long long lo, hi;
    __device__ __forceinline__ void add(u128 v)
    {
        lo += (unsigned long long)(v & (((u128)1 << 40) - 1));
        hi += (unsigned long long)(v >> 40);
    }
    __device__ __forceinline__ u128 value() const { return ((u128)hi << 40) + lo; }
};

__device__ __forceinline__ Limbs warp_sum(Limbs v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        v.lo += __shfl_xor_sync(0xffffffffu, v.lo, o);
        v.hi += __shfl_xor_sync(0xffffffffu, v.hi, o);
    }
    return v;
}

__device__ __forceinline__ Limbs warp_scan_inclusive(Limbs v, int lane)
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long l = __shfl_up_sync(0xffffffffu, v.lo, o);
        const unsigned long long h = __shfl_up_sync(0xffffffffu, v.hi, o);
        if (lane >= o) { v.lo += l; v.hi += h; }
    }
    return v;
}

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

__device__ __forceinline__ float warp_sum_f(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

}  // namespace scd
