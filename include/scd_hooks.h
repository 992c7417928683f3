/*
 * scd_hooks.h - test, timing and tuning hooks of the SCD library. Nothing here is needed to decode;
 * the product calls are in scd.h, whose conventions (status codes, [dev] / [host] pointers, streams)
 * apply unchanged.
 */
#ifndef SCD_HOOKS_H_
#define SCD_HOOKS_H_

#include "scd.h"

#ifdef __cplusplus
extern "C" {
#endif

/* scd_step_profile: one iteration exactly like scd_step, with a CUDA event recorded on `stream`
 * in front of every kernel; the device time between consecutive events is ADDED to
 * ms_by_class[c] and the kernel count to launches_by_class[c] ([host] arrays of
 * SCD_PROF_CLASSES entries, which the caller zeroes), c being the class of the kernel launched
 * between them. Blocking. Used to attribute the time of an iteration (Sec. 4.3, latency
 * breakdown per NFE step) to its kernels. */
enum { SCD_PROF_EMBED = 0, SCD_PROF_RMSNORM, SCD_PROF_GEMM_QKV, SCD_PROF_ROPE_KV, SCD_PROF_ATTENTION,
       SCD_PROF_GEMM_O, SCD_PROF_GEMM_GATE_UP, SCD_PROF_GEMM_DOWN, SCD_PROF_GEMM_LM_HEAD,
       SCD_PROF_VERIFY, SCD_PROF_OTHER, SCD_PROF_CLASSES };
int scd_step_profile(scd_session_t *session, float *ms_by_class, int32_t *launches_by_class,
                     void *stream);

/* scd_session_attention_min_ctx: the forwards of a bf16 session (decoding steps, prefill chunks, explicit
 * windows) use the tcgen05 attention kernel (Sec. 4.3: the window's attention over the committed
 * context) once every live sequence is known to hold at least min_ctx committed positions, and the
 * mma.sync kernel below that; the default is 512. min_ctx = 0 selects the tcgen05 kernel for every
 * forward, a negative value never. Both kernels compute the same attention; their fp32 additions
 * differ in order. Takes effect at the next forward. Errors: SCD_ERR_ARG for a null session. */
int scd_session_attention_min_ctx(scd_session_t *session, int64_t min_ctx);

/* scd_kernel_launches: number of CUDA kernels this process has enqueued through the library. */
int64_t scd_kernel_launches(void);
/* scd_autotune: measures, for this model and this session's window shape, how many K slices
 * (1..8, = cluster size) make each kind of weight GEMM of the layer - QKV, output projection,
 * gate/up, down - fastest inside a whole window forward, and keeps the winners for every later
 * launch on this model (all its sessions). It runs a few dozen window forwards without verify and
 * without commit: tokens, counters and the committed KV cache do not change. k_splits_out (host,
 * 4 entries, optional) receives the choices (0: the built-in rule stays). The slicing changes the
 * order of the fp32 additions of a GEMM, so logits may differ in their last bits from an untuned
 * run, and with them the sampled tokens: call it (or not) consistently where runs must be
 * comparable token by token. fp32 models: no-op. Blocking. Errors: SCD_ERR_STATE before
 * scd_prefill, SCD_ERR_CUDA. */
int scd_autotune(scd_session_t *session, int32_t *k_splits_out, void *stream);
/* Like scd_step_profile (one iteration, same arrays, same classes, blocking), but without events
 * between the kernels: the GEMM and attention kernels write the GPU timer at CTA entry and exit
 * into a device buffer, so neighbouring kernels overlap exactly as in scd_step. The time from the
 * end of the previous stamped kernel to the end of a kernel is charged to that kernel's class; the
 * embedding gather and the verify kernel leave no stamps and are not counted (their classes stay 0).
 * The first call allocates the stamp buffer (a few MiB, freed with the session). */
int scd_step_timeline(scd_session_t *session, float *ms_by_class, int32_t *launches_by_class, void *stream);

/* scd_debug_read: copies a piece of session state to host memory, for step-level parity tests.
 * what = 0: the logits of the last step, f32 [S*B, L, V]; what = 1: the current drafts,
 * i32 [B, L]. `bytes` must equal the size of that piece. Blocking. */
int scd_debug_read(scd_session_t *session, int32_t what, void *out, int64_t bytes, void *stream);

/* scd_noise_u24: the counter-based noise of the sampler, for bit-exactness tests.
 * out[i] = top 24 bits of word 0 of Philox4x32-10(key = seed,
 *          counter = (sub, positions[i], iteration, noise_stream | batch << 8)). [dev] arrays. */
int scd_noise_u24(uint64_t seed, uint32_t noise_stream, uint32_t batch, const int64_t *positions,
                  uint32_t iteration, uint32_t sub, int64_t n, uint32_t *out, void *stream);

/* scd_gemm_bf16: the tcgen05 weight-streaming GEMM alone, y[M,N] = x[M,K] * w[N,K]^T with fp32
 * accumulation in tensor memory. x, w [dev] bf16 row-major, y [dev] f32. M <= 256;
 * K % 64 == 0; N % 8 == 0. workspace: [dev] scratch of scd_gemm_workspace_bytes(M, N, K)
 * bytes. */
/* The workspace must be zero-filled before its first use (it holds an error word that every call leaves
 * at zero unless a bounded wait gave up). scd_gemm_bf16_shaped is the same GEMM with the number of K
 * slices (= cluster size, 1..8) and ring slots given by the caller (0 = the built-in rule), for tests
 * that walk through the launch shapes. scd_model_gemm_tune does that for every later GEMM launch of one
 * model (all its sessions), for benchmarking; 0, 0 restores the rule. */
int64_t scd_gemm_workspace_bytes(int32_t M, int32_t N, int32_t K);
int scd_model_gemm_tune(scd_model_t *model, int32_t k_splits, int32_t stages);
int scd_gemm_bf16_shaped(const void *x, const void *w, float *y, int32_t M, int32_t N, int32_t K,
                         int32_t k_splits, int32_t stages, void *workspace, void *stream);
int scd_gemm_bf16(const void *x, const void *w, float *y, int32_t M, int32_t N, int32_t K,
                  void *workspace, void *stream);


/* scd_selftest_device_once: host-only check of the bookkeeping behind the kernels' per-device set-up
 * (shared-memory opt-in, address of the built-in scratch): a set-up runs once per device ordinal, again
 * after a failure, and every time for ordinals beyond the table. Returns 0 when it behaves. Needs no GPU. */
int scd_selftest_device_once(void);

#ifdef __cplusplus
}
#endif
#endif /* SCD_HOOKS_H_ */
