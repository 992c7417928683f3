// Launch interface of the tcgen05 weight-streaming GEMMs used by the bf16 window forward.
#pragma once
#include "model.cuh"

namespace scd {

// In bf16 sessions the RMSNorm is folded into the GEMMs: s->xn holds h * gain and s->ss the
// partial sums of squares of h ([parts][rows_cap]); a GEMM that reads xn scales its output rows by
// 1 / rms, a residual GEMM refreshes h, xn (with the gain of the NEXT norm) and ss.
// Every GEMM input of a session (xn, att, act) is kept as two bf16 planes [2][rows_cap][K]: hi = bf16(x),
// lo = bf16(x - hi); the GEMMs multiply the weights with both.
// qkv[rows][(H+2Hkv)*dh] = norm(h) * [Wq; Wk; Wv]^T                          (fp32 out)
int gemm_tc_qkv(scd_session *s, int layer, int rows, int ss_parts, cudaStream_t st);
// which = 0: h += att * Wo^T;  which = 1: h += act * Wdown^T                   (fp32 residual)
// then xn = bf16(h * gain_next), ss = per-tile sums of h^2
// *parts_out = partial sums of squares it left per row (to be passed to the GEMM that reads xn)
int gemm_tc_residual(scd_session *s, int layer, int which, int rows, const void *gain_next, int *parts_out,
                     cudaStream_t st);
// act[rows][F] = silu(norm(h) * Wgate^T) * (norm(h) * Wup^T)                    (two bf16 planes out)
int gemm_tc_gate_up(scd_session *s, int layer, int rows, int ss_parts, cudaStream_t st);
// logits[rows][v] = norm(h) * Wlm[v]^T for lo <= v < hi and, if eol >= 0, for v = eol    (fp32 out)
int gemm_tc_lm_head(scd_session *s, int rows, float *logits, int lo, int hi, int eol, int ss_parts, cudaStream_t st);
// The number of K slices (= cluster size) of every launch of one kind of GEMM follows a rule (see
// choose_shape); gemm_set_kind_splits replaces it for a model (0: back to the rule). The result of a
// GEMM depends on the slicing only through the order of its fp32 additions.
enum { GEMM_QKV = 0, GEMM_O, GEMM_GATE_UP, GEMM_DOWN, GEMM_LM_HEAD, GEMM_KINDS };
void gemm_set_kind_splits(scd_model *m, int kind, int k_splits);
// upper bound of the partial sums a residual GEMM leaves per row (sizes the session's ss buffer)
int gemm_norm_parts_cap(const scd_session *s);

// 2-D bf16 row-major matrix [rows][cols] as a TMA tensor map with box [box_rows][box_cols] and
// the 128-byte swizzle (box_cols * 2 bytes <= 128).
int make_tensor_map_bf16_2d(void *map, const void *ptr, unsigned long long rows, unsigned long long cols,
                            unsigned box_rows, unsigned box_cols);

// tensor-core window attention for bf16 sessions (attention_tc.cu)
bool attention_tc_supported(const scd_session *s, int Mq);
int attention_session_prepare(scd_session *s);
void attention_session_release(scd_session *s);
// RoPE + KV write of the window rows + attention of all Mq rows per stream-sequence
int attention_tc(scd_session *s, int layer, int Mq, int pos_override, cudaStream_t st);
// whether the next window forward of the session (Mq rows per stream-sequence) takes the kernel
// variant for long contexts; a captured iteration is valid only while this does not change
int attention_tc_variant(const scd_session *s, int Mq, long long ctx);

// per-session state (activation tensor maps, device error word); bf16 sessions only
int gemm_session_prepare(scd_session *s);
void gemm_session_release(scd_session *s);
// reads the device error word that a bounded wait sets when it gives up (0 = healthy). Blocking.
int gemm_error_word(scd_session *s, int *host_value, cudaStream_t st);

}  // namespace scd
