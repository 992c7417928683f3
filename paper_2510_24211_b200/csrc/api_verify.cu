// C-ABI entry points that do not need a session: error strings, the stand-alone verify hook
// and the noise hook.
#include <cstdarg>
#include <cstdio>

#include "verify.cuh"

namespace scd {

static thread_local char g_last_error[512] = "";

void set_last_error(const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_last_error, sizeof(g_last_error), fmt, ap);
    va_end(ap);
}

int cuda_fail(cudaError_t e, const char *what)
{
    set_last_error("CUDA error %d (%s) in %s", (int)e, cudaGetErrorString(e), what);
    return SCD_ERR_CUDA;
}

int current_device(int *device)
{
    SCD_CUDA_TRY(cudaGetDevice(device));
    return SCD_OK;
}

int validate_decode_config(const scd_decode_config_t *cfg, int V)
{
    SCD_REQUIRE(cfg != nullptr, SCD_ERR_ARG, "decode config is NULL");
    SCD_REQUIRE(cfg->mode == SCD_MODE_AR || cfg->mode == SCD_MODE_SJD || cfg->mode == SCD_MODE_SCD_MC ||
                cfg->mode == SCD_MODE_SCD_GS || cfg->mode == SCD_MODE_ALPHA, SCD_ERR_ARG, "unknown decode mode %d", cfg->mode);
    if (cfg->mode == SCD_MODE_ALPHA)
        SCD_REQUIRE(cfg->alpha >= 0.0f && cfg->alpha <= 1.0f, SCD_ERR_ARG, "alpha %g outside [0, 1]",
                    (double)cfg->alpha);
    SCD_REQUIRE(cfg->batch >= 1 && cfg->batch <= 255, SCD_ERR_ARG, "batch %d outside 1..255", cfg->batch);
    SCD_REQUIRE(cfg->window_L >= 1 && cfg->window_L <= 256, SCD_ERR_ARG,
                "window_L %d outside 1..256", cfg->window_L);
    SCD_REQUIRE(cfg->temperature > 0.0f, SCD_ERR_ARG, "temperature must be positive");
    SCD_REQUIRE(V >= 1, SCD_ERR_ARG, "vocabulary size %d", V);
    SCD_REQUIRE(cfg->allowed_lo >= 0 && cfg->allowed_hi <= V && cfg->allowed_lo < cfg->allowed_hi,
                SCD_ERR_ARG, "allowed id range [%d, %d) not inside [0, %d)", cfg->allowed_lo,
                cfg->allowed_hi, V);
    SCD_REQUIRE(cfg->row_period >= 0, SCD_ERR_ARG, "row_period %d", cfg->row_period);
    if (cfg->row_period > 0)
        SCD_REQUIRE(cfg->eol_id >= 0 && cfg->eol_id < V, SCD_ERR_ARG, "eol_id %d outside [0, %d)",
                    cfg->eol_id, V);
    return SCD_OK;
}

void fill_verify_params(VerifyParams &p, const scd_decode_config_t *cfg, int V)
{
    p = VerifyParams{};
    p.mode = cfg->mode;
    p.B = cfg->batch;
    p.L = cfg->mode == SCD_MODE_AR ? 1 : cfg->window_L;
    p.V = V;
    p.S = cfg->cfg_lambda != 0.0f ? 2 : 1;
    p.temperature = cfg->temperature;
    p.lam = cfg->cfg_lambda;
    p.one_plus_lam = 1.0f + cfg->cfg_lambda;
    p.top_k = cfg->top_k;
    p.top_p24 = (cfg->top_p > 0.0f && cfg->top_p < 1.0f) ? (unsigned)((double)cfg->top_p * 16777216.0 + 0.5) : 0u;
    if (p.top_p24 == 0u && cfg->top_p > 0.0f && cfg->top_p < 1.0f) p.top_p24 = 1u;   // (tiny top_p: still on)
    p.seed = cfg->seed;
    p.alpha = cfg->mode == SCD_MODE_ALPHA ? cfg->alpha : 1.0f;
    p.allowed_lo = cfg->allowed_lo;
    p.allowed_hi = cfg->allowed_hi;
    p.row_period = cfg->row_period;
    p.eol_id = cfg->eol_id;
}

static inline int64_t align256(int64_t x) { return (x + 255) & ~(int64_t)255; }

struct VerifyWorkspace {
    int64_t xbuf, stats0, stats1, row_y, row_y_indep, done, total;
};

static VerifyWorkspace verify_layout(int B, int L, int V)
{
    VerifyWorkspace w;
    int64_t off = 0;
    const int64_t rows = (int64_t)B * L;
    w.xbuf = off;        off = align256(off + rows * V * (int64_t)sizeof(float));
    w.stats0 = off;      off = align256(off + rows * (int64_t)sizeof(RowStats));
    w.stats1 = off;      off = align256(off + rows * (int64_t)sizeof(RowStats));
    w.row_y = off;       off = align256(off + rows * 4);
    w.row_y_indep = off; off = align256(off + rows * 8);
    w.done = off;        off = align256(off + (int64_t)B * 4);
    w.total = off;
    return w;
}

__global__ void noise_kernel(unsigned long long seed, unsigned stream, unsigned batch,
                             const long long *positions, unsigned iteration, unsigned sub,
                             long long n, unsigned *out)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = noise_u24(seed, stream, batch, positions[i], iteration, sub);
}

// ---- scratch of scd_verify_noalloc -----------------------------------------------------------
// The array lives in every GPU context that loads the library, until the process exits. Its
// name is only a host-side stand-in: the device address is looked up once per device.
#define SCD_NOALLOC_SCRATCH_BYTES (16u << 20)
static __device__ __align__(256) unsigned char g_noalloc_scratch[SCD_NOALLOC_SCRATCH_BYTES];
static void *g_noalloc_scratch_addr[DeviceOnce::kSlots];      // per device ordinal, filled under g_noalloc_once
static DeviceOnce g_noalloc_once;

}  // namespace scd

using namespace scd;

extern "C" {

const char *scd_strerror(int code)
{
    switch (code) {
        case SCD_OK: return "ok";
        case SCD_ERR_ARG: return "bad argument";
        case SCD_ERR_SHAPE: return "unsupported shape";
        case SCD_ERR_CAPACITY: return "capacity exceeded";
        case SCD_ERR_STATE: return "call out of order";
        case SCD_ERR_CUDA: return "CUDA error";
        case SCD_ERR_TIMEOUT: return "device-side wait timed out";
        case SCD_ERR_UNSUPPORTED: return "not implemented";
        default: return "unknown status";
    }
}

const char *scd_last_error(void) { return g_last_error; }

int64_t scd_verify_workspace_bytes(const scd_decode_config_t *cfg, int32_t V)
{
    if (validate_decode_config(cfg, V) != SCD_OK) return SCD_ERR_ARG;
    const int L = cfg->mode == SCD_MODE_AR ? 1 : cfg->window_L;
    return verify_layout(cfg->batch, L, V).total;
}

int scd_verify(const scd_decode_config_t *cfg, int32_t V, const float *p_logits,
               const float *q_logits, const int32_t *draft_ids, const int64_t *positions,
               int64_t iteration, int32_t *n_commit, int32_t *committed_ids,
               int32_t *next_draft_ids, uint8_t *accept_flags, void *workspace, void *stream)
{
    int rc = validate_decode_config(cfg, V);
    if (rc != SCD_OK) return rc;
    SCD_REQUIRE(p_logits && draft_ids && positions && n_commit && committed_ids && next_draft_ids &&
                accept_flags && workspace, SCD_ERR_ARG, "scd_verify: NULL argument");
    SCD_REQUIRE(((uintptr_t)workspace & 255) == 0, SCD_ERR_ARG, "workspace must be 256-byte aligned");
    SCD_REQUIRE(iteration >= 0 && iteration <= 0xFFFFFFFFll, SCD_ERR_ARG, "iteration out of range");
    VerifyParams p;
    fill_verify_params(p, cfg, V);
    const VerifyWorkspace w = verify_layout(p.B, p.L, V);
    char *ws = (char *)workspace;
    cudaStream_t st = (cudaStream_t)stream;
    p.p_logits = p_logits;
    p.xbuf[0] = (float *)(ws + w.xbuf);
    p.xbuf[1] = const_cast<float *>(q_logits);
    p.stats[0] = (RowStats *)(ws + w.stats0);
    p.stats[1] = (RowStats *)(ws + w.stats1);
    p.q_is_raw = 1;
    p.keep_x = 0;                                       // stand-alone: nothing reads the post-processed row later
    p.q_present = q_logits != nullptr;
    p.positions = (const long long *)positions;
    p.iteration = iteration;
    p.prompt_len = 0;
    p.draft_in = draft_ids;
    p.draft_out = next_draft_ids;
    p.n_commit = n_commit;
    p.committed_ids = committed_ids;
    p.accept_flags = accept_flags;
    p.row_y = (int *)(ws + w.row_y);
    p.row_y_indep = (int *)(ws + w.row_y_indep);
    p.done_count = (unsigned *)(ws + w.done);
    SCD_CUDA_TRY(cudaMemsetAsync(p.done_count, 0, (size_t)p.B * 4, st));
    count_launches(1);
    return launch_verify(p, st);
}

int scd_noise_u24(uint64_t seed, uint32_t noise_stream, uint32_t batch, const int64_t *positions,
                  uint32_t iteration, uint32_t sub, int64_t n, uint32_t *out, void *stream)
{
    SCD_REQUIRE(positions && out && n >= 0, SCD_ERR_ARG, "scd_noise_u24: bad argument");
    if (n == 0) return SCD_OK;
    const unsigned blocks = (unsigned)((n + 255) / 256);
    noise_kernel<<<blocks, 256, 0, (cudaStream_t)stream>>>(seed, noise_stream, batch,
                                                           (const long long *)positions, iteration,
                                                           sub, n, out);
    SCD_CUDA_TRY(cudaGetLastError());
    return SCD_OK;
}

int scd_selftest_device_once(void)
{
    // host-only: the per-device bookkeeping behind the kernels' one-time set-up
    DeviceOnce once;
    int runs = 0;
    auto ok = [&]() -> int { ++runs; return SCD_OK; };
    auto bad = [&]() -> int { ++runs; return SCD_ERR_CUDA; };
    if (once.run(0, ok) != SCD_OK || runs != 1) return 1;
    if (once.run(0, ok) != SCD_OK || runs != 1) return 2;          // second use of device 0: skipped
    if (once.run(1, ok) != SCD_OK || runs != 2) return 3;          // another device: runs again
    if (once.run(2, bad) != SCD_ERR_CUDA || runs != 3) return 4;   // a failed set-up ...
    if (once.run(2, ok) != SCD_OK || runs != 4) return 5;          // ... is tried again
    if (once.run(2, ok) != SCD_OK || runs != 4) return 6;
    if (once.run(DeviceOnce::kSlots + 3, ok) != SCD_OK || once.run(DeviceOnce::kSlots + 3, ok) != SCD_OK || runs != 6)
        return 7;                                                  // beyond the table: every time
    return 0;
}

int64_t scd_verify_noalloc_max_bytes(void) { return (int64_t)SCD_NOALLOC_SCRATCH_BYTES; }

int scd_verify_noalloc(const scd_decode_config_t *cfg, int32_t V, const float *p_logits,
                       const float *q_logits, const int32_t *draft_ids, const int64_t *positions,
                       int64_t iteration, int32_t *n_commit, int32_t *committed_ids,
                       int32_t *next_draft_ids, uint8_t *accept_flags, void *stream)
{
    int rc = validate_decode_config(cfg, V);
    if (rc != SCD_OK) return rc;
    const int64_t need = scd_verify_workspace_bytes(cfg, V);
    SCD_REQUIRE(need >= 0 && need <= (int64_t)SCD_NOALLOC_SCRATCH_BYTES, SCD_ERR_CAPACITY,
                "scd_verify_noalloc: batch %d x window %d x V %d needs %lld bytes of scratch, the built-in "
                "buffer holds %u; use scd_verify with a caller-allocated workspace", cfg->batch,
                cfg->window_L, V, (long long)need, SCD_NOALLOC_SCRATCH_BYTES);
    int dev = 0;
    rc = current_device(&dev);
    if (rc != SCD_OK) return rc;
    SCD_REQUIRE(dev >= 0 && dev < DeviceOnce::kSlots, SCD_ERR_UNSUPPORTED, "scd_verify_noalloc: device ordinal %d", dev);
    // first call on this device: resolve the device address of the built-in buffer (this is also the
    // moment the CUDA runtime loads this module on the device and gives the array its memory)
    rc = g_noalloc_once.run(dev, [&]() -> int {
        void *ptr = nullptr;
        SCD_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
        SCD_REQUIRE(ptr != nullptr, SCD_ERR_CUDA, "scd_verify_noalloc: no device address for the scratch buffer");
        g_noalloc_scratch_addr[dev] = ptr;
        return SCD_OK;
    });
    if (rc != SCD_OK) return rc;
    // scd_verify zeroes the part of the workspace that must start at zero (the per-sequence
    // tickets) on `stream` before the kernel; everything else is written before it is read
    return scd_verify(cfg, V, p_logits, q_logits, draft_ids, positions, iteration, n_commit, committed_ids,
                      next_draft_ids, accept_flags, g_noalloc_scratch_addr[dev], stream);
}

}  // extern "C"
