"""Thin ctypes binding of libscd.so: same names as the C ABI, argument marshalling only.

PyTorch supplies device memory (tensor.data_ptr()) and streams; every step of the decode path
runs in the library's CUDA kernels. Loading fails loudly when the library has not been built."""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libscd.so")

SCD_OK = 0
SCD_ERR_ARG, SCD_ERR_SHAPE, SCD_ERR_CAPACITY, SCD_ERR_STATE = -1, -2, -3, -4
SCD_ERR_CUDA, SCD_ERR_TIMEOUT, SCD_ERR_UNSUPPORTED = -5, -6, -7
SCD_F32, SCD_BF16 = 0, 1
SCD_MODE_AR, SCD_MODE_SJD, SCD_MODE_SCD_MC, SCD_MODE_SCD_GS, SCD_MODE_ALPHA = 0, 1, 2, 3, 4

EXPORTS = (
    "scd_strerror", "scd_last_error", "scd_init_model", "scd_free_model", "scd_session_create",
    "scd_session_free", "scd_prefill", "scd_step", "scd_step_result", "scd_generate",
    "scd_read_tokens", "scd_verify_workspace_bytes", "scd_verify", "scd_forward_window",
    "scd_noise_u24", "scd_gemm_workspace_bytes", "scd_gemm_bf16", "scd_debug_read", "scd_model_gemm_tune", "scd_gemm_bf16_shaped", "scd_selftest_device_once",
    "scd_step_profile", "scd_step_timeline", "scd_session_attention_min_ctx", "scd_autotune", "scd_kernel_launches", "scd_verify_noalloc", "scd_verify_noalloc_max_bytes",
)

PROF_CLASSES = ("embed", "rmsnorm", "gemm_qkv", "rope_kv", "attention", "gemm_o", "gemm_gate_up",
                "gemm_down", "gemm_lm_head", "verify", "other")


class ScdError(RuntimeError):
    def __init__(self, code, detail):
        super().__init__(f"scd error {code}: {detail}")
        self.code = code


class ModelConfig(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("d_ffn", C.c_int32),
                ("vocab_out", C.c_int32), ("vocab_in", C.c_int32), ("rope_base", C.c_float),
                ("rms_eps", C.c_float), ("dtype", C.c_int32), ("max_seq", C.c_int32),
                ("kv_page_tokens", C.c_int32)]


class Weights(C.Structure):
    _fields_ = [("tok_emb", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p)] + \
               [(k, C.POINTER(C.c_void_p)) for k in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm",
                                                     "w_gate", "w_up", "w_down")]


class DecodeConfig(C.Structure):
    _fields_ = [("mode", C.c_int32), ("batch", C.c_int32), ("window_L", C.c_int32),
                ("temperature", C.c_float), ("top_k", C.c_int32), ("cfg_lambda", C.c_float),
                ("seed", C.c_uint64), ("allowed_lo", C.c_int32), ("allowed_hi", C.c_int32),
                ("row_period", C.c_int32), ("eol_id", C.c_int32), ("alpha", C.c_float),
                ("top_p", C.c_float)]


class Stats(C.Structure):
    _fields_ = [("forwards", C.c_int64), ("committed", C.c_int64), ("accept_hist", C.c_int64 * 257),
                ("elapsed_ms", C.c_float)]


_lib = None


def lib():
    """The loaded library. Raises if libscd.so is missing: there is no fallback path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} not found: build it with `python -m paper_2510_24211_b200.build` "
                "(the CUDA library is the only implementation; there is no CPU fallback)")
        l = C.CDLL(LIB_PATH)
        _declare(l)
        _lib = l
    return _lib


def _declare(l):
    vp, i32p, i64p = C.c_void_p, C.c_void_p, C.c_void_p
    l.scd_strerror.argtypes = [C.c_int]
    l.scd_strerror.restype = C.c_char_p
    l.scd_last_error.argtypes = []
    l.scd_last_error.restype = C.c_char_p
    l.scd_verify_workspace_bytes.argtypes = [C.POINTER(DecodeConfig), C.c_int32]
    l.scd_verify_workspace_bytes.restype = C.c_int64
    l.scd_verify.argtypes = [C.POINTER(DecodeConfig), C.c_int32, vp, vp, i32p, i64p, C.c_int64,
                             i32p, i32p, i32p, vp, vp, vp]
    l.scd_verify.restype = C.c_int
    l.scd_verify_noalloc.argtypes = [C.POINTER(DecodeConfig), C.c_int32, vp, vp, i32p, i64p, C.c_int64,
                                     i32p, i32p, i32p, vp, vp]
    l.scd_verify_noalloc.restype = C.c_int
    l.scd_verify_noalloc_max_bytes.argtypes = []
    l.scd_verify_noalloc_max_bytes.restype = C.c_int64
    l.scd_noise_u24.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, vp, C.c_uint32, C.c_uint32,
                                C.c_int64, vp, vp]
    l.scd_noise_u24.restype = C.c_int
    l.scd_init_model.argtypes = [C.POINTER(ModelConfig), C.POINTER(Weights), C.POINTER(C.c_void_p)]
    l.scd_init_model.restype = C.c_int
    l.scd_free_model.argtypes = [vp]
    l.scd_free_model.restype = C.c_int
    l.scd_session_create.argtypes = [vp, C.POINTER(DecodeConfig), C.POINTER(C.c_void_p)]
    l.scd_session_create.restype = C.c_int
    l.scd_session_free.argtypes = [vp]
    l.scd_session_free.restype = C.c_int
    l.scd_prefill.argtypes = [vp, vp, C.c_int32, C.c_int32, vp]
    l.scd_prefill.restype = C.c_int
    l.scd_step.argtypes = [vp, vp]
    l.scd_step.restype = C.c_int
    l.scd_step_result.argtypes = [vp, vp, vp, vp, vp]
    l.scd_step_result.restype = C.c_int
    l.scd_generate.argtypes = [vp, vp, C.POINTER(Stats), vp]
    l.scd_generate.restype = C.c_int
    l.scd_read_tokens.argtypes = [vp, C.c_int32, C.c_int32, vp, vp]
    l.scd_read_tokens.restype = C.c_int
    l.scd_forward_window.argtypes = [vp, vp, C.c_int32, vp, vp, C.c_int32, vp]
    l.scd_forward_window.restype = C.c_int
    l.scd_debug_read.argtypes = [vp, C.c_int32, vp, C.c_int64, vp]
    l.scd_debug_read.restype = C.c_int
    l.scd_step_profile.argtypes = [vp, vp, vp, vp]
    l.scd_step_profile.restype = C.c_int
    l.scd_autotune.argtypes = [vp, vp, vp]
    l.scd_autotune.restype = C.c_int
    l.scd_step_timeline.argtypes = [vp, vp, vp, vp]
    l.scd_step_timeline.restype = C.c_int
    l.scd_session_attention_min_ctx.argtypes = [vp, C.c_int64]
    l.scd_session_attention_min_ctx.restype = C.c_int
    l.scd_kernel_launches.argtypes = []
    l.scd_kernel_launches.restype = C.c_int64
    l.scd_gemm_workspace_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32]
    l.scd_gemm_workspace_bytes.restype = C.c_int64
    l.scd_gemm_bf16.argtypes = [vp, vp, vp, C.c_int32, C.c_int32, C.c_int32, vp, vp]
    l.scd_gemm_bf16.restype = C.c_int
    l.scd_gemm_bf16_shaped.argtypes = [vp, vp, vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, vp, vp]
    l.scd_gemm_bf16_shaped.restype = C.c_int
    l.scd_model_gemm_tune.argtypes = [vp, C.c_int32, C.c_int32]
    l.scd_model_gemm_tune.restype = C.c_int
    l.scd_selftest_device_once.argtypes = []
    l.scd_selftest_device_once.restype = C.c_int


def _check(rc):
    if rc != SCD_OK:
        raise ScdError(rc, f"{lib().scd_strerror(rc).decode()}: {lib().scd_last_error().decode()}")


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _ptr(t):
    return C.c_void_p(0) if t is None else C.c_void_p(t.data_ptr())


def scd_strerror(code: int) -> str:
    return lib().scd_strerror(code).decode()


def decode_config(mode=SCD_MODE_SCD_MC, batch=1, window_L=16, temperature=1.0, top_k=0,
                  cfg_lambda=0.0, seed=0, allowed_lo=0, allowed_hi=0, row_period=0, eol_id=0, alpha=1.0,
                  top_p=0.0):
    return DecodeConfig(mode, batch, window_L, temperature, top_k, cfg_lambda, seed, allowed_lo,
                        allowed_hi, row_period, eol_id, alpha, top_p)


# ------------------------------------------------------------------------------------ hooks
def scd_noise_u24(seed, noise_stream, batch, positions: torch.Tensor, iteration, sub=0, stream=None):
    assert positions.dtype == torch.int64 and positions.is_cuda
    out = torch.empty(positions.numel(), dtype=torch.int32, device=positions.device)
    _check(lib().scd_noise_u24(seed, noise_stream, batch, _ptr(positions), iteration, sub,
                               positions.numel(), _ptr(out), _stream(stream)))
    return out


def scd_verify_workspace_bytes(cfg: DecodeConfig, V: int) -> int:
    n = lib().scd_verify_workspace_bytes(C.byref(cfg), V)
    if n < 0:
        _check(int(n))
    return int(n)


def scd_verify(cfg: DecodeConfig, p_logits, q_logits, draft_ids, positions, iteration,
               workspace=None, stream=None):
    """Fused verify-and-redraft on caller-supplied logits. Returns
    (n_commit [B], committed_ids [B,L], next_draft_ids [B,L], accept_flags [B,L])."""
    V = p_logits.shape[-1]
    B = cfg.batch
    L = 1 if cfg.mode == SCD_MODE_AR else cfg.window_L
    dev = p_logits.device
    assert p_logits.dtype == torch.float32 and p_logits.is_contiguous()
    assert q_logits is None or (q_logits.dtype == torch.float32 and q_logits.is_contiguous())
    assert draft_ids.dtype == torch.int32 and positions.dtype == torch.int64
    if workspace is None:
        workspace = torch.empty(scd_verify_workspace_bytes(cfg, V), dtype=torch.uint8, device=dev)
    n_commit = torch.empty(B, dtype=torch.int32, device=dev)
    committed = torch.zeros(B, L, dtype=torch.int32, device=dev)
    next_drafts = torch.empty(B, L, dtype=torch.int32, device=dev)
    flags = torch.zeros(B, L, dtype=torch.uint8, device=dev)
    _check(lib().scd_verify(C.byref(cfg), V, _ptr(p_logits), _ptr(q_logits), _ptr(draft_ids),
                            _ptr(positions), iteration, _ptr(n_commit), _ptr(committed),
                            _ptr(next_drafts), _ptr(flags), _ptr(workspace), _stream(stream)))
    return n_commit, committed, next_drafts, flags


def scd_verify_noalloc_max_bytes() -> int:
    return int(lib().scd_verify_noalloc_max_bytes())


def scd_verify_noalloc(cfg: DecodeConfig, p_logits, q_logits, draft_ids, positions, iteration, out,
                       stream=None):
    """scd_verify on the library's built-in scratch buffer: the call allocates nothing, so the
    caller passes the four output tensors in ``out`` = (n_commit [B] i32, committed_ids [B,L] i32,
    next_draft_ids [B,L] i32, accept_flags [B,L] u8), already allocated on the device."""
    V = p_logits.shape[-1]
    n_commit, committed, next_drafts, flags = out
    _check(lib().scd_verify_noalloc(C.byref(cfg), V, _ptr(p_logits), _ptr(q_logits), _ptr(draft_ids),
                                    _ptr(positions), iteration, _ptr(n_commit), _ptr(committed),
                                    _ptr(next_drafts), _ptr(flags), _stream(stream)))
    return out


def scd_gemm_workspace_bytes(M, N, K) -> int:
    n = lib().scd_gemm_workspace_bytes(M, N, K)
    if n < 0:
        _check(int(n))
    return int(n)


def scd_gemm_bf16(x, w, y=None, workspace=None, stream=None, k_splits=0, stages=0):
    """y[M,N] = x[M,K] @ w[N,K]^T (bf16 in, fp32 out) on the tcgen05 weight-streaming kernel
    (scd_gemm_bf16_shaped when a launch shape is given)."""
    M, K = x.shape
    N = w.shape[0]
    assert x.dtype == torch.bfloat16 and w.dtype == torch.bfloat16 and w.shape[1] == K
    assert x.is_contiguous() and w.is_contiguous()
    if y is None:
        y = torch.empty(M, N, dtype=torch.float32, device=x.device)
    if workspace is None:
        workspace = torch.zeros(max(scd_gemm_workspace_bytes(M, N, K), 256), dtype=torch.uint8,
                                device=x.device)
    if k_splits or stages:
        _check(lib().scd_gemm_bf16_shaped(_ptr(x), _ptr(w), _ptr(y), M, N, K, k_splits, stages, _ptr(workspace),
                                          _stream(stream)))
    else:
        _check(lib().scd_gemm_bf16(_ptr(x), _ptr(w), _ptr(y), M, N, K, _ptr(workspace), _stream(stream)))
    return y


def scd_kernel_launches() -> int:
    return int(lib().scd_kernel_launches())


def scd_selftest_device_once() -> int:
    return int(lib().scd_selftest_device_once())


# ------------------------------------------------------------------------------------ model / session
LAYER_KEYS = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


class Model:
    """scd_init_model / scd_free_model. ``weights``: dict of CUDA tensors (per-layer lists)."""

    def __init__(self, shape: dict, weights: dict, max_seq: int, kv_page_tokens: int = 128):
        dt = SCD_F32 if shape["dtype"] == "f32" else SCD_BF16
        want = torch.float32 if dt == SCD_F32 else torch.bfloat16
        self.shape = dict(shape)
        self.max_seq = max_seq
        self._keep = weights
        nl = shape["n_layers"]
        w = Weights()
        for k in ("tok_emb", "final_norm", "lm_head"):
            t = weights[k]
            assert t.is_cuda and t.dtype == want and t.is_contiguous(), k
            setattr(w, k, t.data_ptr())
        self._arrs = {}
        for k in LAYER_KEYS:
            for t in weights[k]:
                assert t.is_cuda and t.dtype == want and t.is_contiguous(), k
            arr = (C.c_void_p * nl)(*[t.data_ptr() for t in weights[k]])
            self._arrs[k] = arr
            setattr(w, k, C.cast(arr, C.POINTER(C.c_void_p)))
        cfg = ModelConfig(nl, shape["d_model"], shape["n_heads"], shape["n_kv_heads"], shape["head_dim"],
                          shape["d_ffn"], shape["vocab_out"], shape["vocab_in"],
                          shape.get("rope_base", 10000.0), shape.get("rms_eps", 1e-5), dt, max_seq,
                          kv_page_tokens)
        h = C.c_void_p()
        _check(lib().scd_init_model(C.byref(cfg), C.byref(w), C.byref(h)))
        self.handle = h

    def scd_model_gemm_tune(self, k_splits: int = 0, stages: int = 0):
        _check(lib().scd_model_gemm_tune(self.handle, k_splits, stages))

    def close(self):
        if getattr(self, "handle", None):
            lib().scd_free_model(self.handle)
            self.handle = None

    def __del__(self):
        self.close()


class Session:
    """scd_session_create and the calls that take a session."""

    def __init__(self, model: Model, cfg: DecodeConfig):
        self.model = model
        self.cfg = cfg
        self.B = cfg.batch
        self.S = 2 if cfg.cfg_lambda != 0.0 else 1
        self.L = 1 if cfg.mode == SCD_MODE_AR else cfg.window_L
        h = C.c_void_p()
        _check(lib().scd_session_create(model.handle, C.byref(cfg), C.byref(h)))
        self.handle = h
        self.n_new = 0

    def close(self):
        if getattr(self, "handle", None):
            lib().scd_session_free(self.handle)
            self.handle = None

    def __del__(self):
        self.close()

    def scd_prefill(self, prompt_ids, n_new: int, stream=None):
        """prompt_ids: host int32 array-like [S*B, P]."""
        import numpy as np
        ids = np.ascontiguousarray(prompt_ids, dtype=np.int32)
        assert ids.ndim == 2 and ids.shape[0] == self.S * self.B, ids.shape
        self.P = ids.shape[1]
        self.n_new = n_new
        _check(lib().scd_prefill(self.handle, ids.ctypes.data_as(C.c_void_p), ids.shape[1], n_new,
                                 _stream(stream)))

    def scd_step(self, stream=None):
        _check(lib().scd_step(self.handle, _stream(stream)))

    def scd_step_profile(self, ms=None, launches=None, stream=None):
        """One iteration with per-kernel-class device timing; accumulates into (ms, launches)."""
        import numpy as np
        n = len(PROF_CLASSES)
        ms = np.zeros(n, dtype=np.float32) if ms is None else ms
        launches = np.zeros(n, dtype=np.int32) if launches is None else launches
        _check(lib().scd_step_profile(self.handle, ms.ctypes.data_as(C.c_void_p),
                                      launches.ctypes.data_as(C.c_void_p), _stream(stream)))
        return ms, launches

    def scd_autotune(self, stream=None):
        """Pick the K slicing of the four layer GEMMs by timing window forwards; returns the choices."""
        import numpy as np
        out = np.zeros(4, dtype=np.int32)
        _check(lib().scd_autotune(self.handle, out.ctypes.data_as(C.c_void_p), _stream(stream)))
        return out

    def scd_session_attention_min_ctx(self, min_ctx):
        _check(lib().scd_session_attention_min_ctx(self.handle, int(min_ctx)))

    def scd_step_timeline(self, ms=None, launches=None, stream=None):
        """One iteration timed by device time stamps inside the kernels (no events between them)."""
        import numpy as np
        n = len(PROF_CLASSES)
        ms = np.zeros(n, dtype=np.float32) if ms is None else ms
        launches = np.zeros(n, dtype=np.int32) if launches is None else launches
        _check(lib().scd_step_timeline(self.handle, ms.ctypes.data_as(C.c_void_p),
                                       launches.ctypes.data_as(C.c_void_p), _stream(stream)))
        return ms, launches

    def scd_step_result(self, stream=None):
        import numpy as np
        a = np.zeros(self.B, dtype=np.int32)
        n = np.zeros(self.B, dtype=np.int32)
        kv = np.zeros(self.B, dtype=np.int32)
        _check(lib().scd_step_result(self.handle, a.ctypes.data_as(C.c_void_p),
                                     n.ctypes.data_as(C.c_void_p), kv.ctypes.data_as(C.c_void_p),
                                     _stream(stream)))
        return a, n, kv

    def scd_generate(self, stream=None):
        """Runs to completion. Returns (tokens [B, n_new] int32 numpy, Stats)."""
        import numpy as np
        out = np.zeros((self.B, self.n_new), dtype=np.int32)
        st = Stats()
        _check(lib().scd_generate(self.handle, out.ctypes.data_as(C.c_void_p), C.byref(st),
                                  _stream(stream)))
        return out, st

    def scd_read_tokens(self, first: int, count: int, stream=None):
        import numpy as np
        out = np.zeros((self.B, count), dtype=np.int32)
        _check(lib().scd_read_tokens(self.handle, first, count, out.ctypes.data_as(C.c_void_p),
                                     _stream(stream)))
        return out

    def scd_debug_read(self, what: str, stream=None):
        """'logits' -> float32 [S*B, L, V] of the last step; 'drafts' -> int32 [B, L]."""
        import numpy as np
        if what == "logits":
            out = np.zeros((self.S * self.B, self.L, self.model.shape["vocab_out"]), dtype=np.float32)
            code = 0
        else:
            out = np.zeros((self.B, self.L), dtype=np.int32)
            code = 1
        _check(lib().scd_debug_read(self.handle, code, out.ctypes.data_as(C.c_void_p), out.nbytes,
                                    _stream(stream)))
        return out

    def scd_forward_window(self, ids: torch.Tensor, commit: bool = False, want_hidden: bool = False,
                           stream=None):
        """ids: CUDA int32 [S*B, M]. Returns logits [S*B, M, V] (and hidden [S*B, M, d])."""
        assert ids.is_cuda and ids.dtype == torch.int32 and ids.is_contiguous()
        rows, M = ids.shape
        V, d = self.model.shape["vocab_out"], self.model.shape["d_model"]
        logits = torch.empty(rows, M, V, dtype=torch.float32, device=ids.device)
        hidden = torch.empty(rows, M, d, dtype=torch.float32, device=ids.device) if want_hidden else None
        _check(lib().scd_forward_window(self.handle, _ptr(ids), M, _ptr(logits), _ptr(hidden),
                                        1 if commit else 0, _stream(stream)))
        return (logits, hidden) if want_hidden else logits
