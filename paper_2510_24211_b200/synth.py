"""Seeded synthetic inputs: model shapes, random-init weights, prompts and verify-only logits.

This module serves the CUDA library's tests and benchmark AND the CPU oracle's tests. It holds
none of the method's arithmetic (no sampling rule, no post-processing, no noise keyed by
position): it only produces the arrays both sides are given.

The paper evaluates trained models (Lumina-mGPT 7B, LlamaGen-XL, Cosmos-1-AR) on MS-COCO,
Parti-prompt and RealEstate-10k inputs. Neither weights nor datasets exist here, so random-init
decoders with the same shapes and random token prefixes stand in for them.
"""
from __future__ import annotations

import numpy as np
import torch

# name -> shape / decode recipe. "tiny" runs on the CPU oracle in seconds; the others follow the
# shapes of the paper's image and video models.
WORKLOADS = {
    "tiny": dict(
        n_layers=4, d_model=256, n_heads=4, n_kv_heads=4, head_dim=64, d_ffn=688,
        vocab_out=1024, vocab_in=1024 + 8, dtype="f32", rope_base=10000.0, rms_eps=1e-5,
        prompt_len=1, n_gen=256, window_L=16, temperature=1.0, top_k=64, cfg_lambda=0.0,
        allowed_lo=0, allowed_hi=1024, row_period=0, eol_id=0, seed=0),
    "llamagen_xl": dict(
        n_layers=36, d_model=1280, n_heads=20, n_kv_heads=20, head_dim=64, d_ffn=3456,
        vocab_out=16384, vocab_in=16384 + 1024, dtype="bf16", rope_base=10000.0, rms_eps=1e-5,
        prompt_len=1, n_gen=576, window_L=32, temperature=1.0, top_k=2000, cfg_lambda=2.0,
        allowed_lo=0, allowed_hi=16384, row_period=0, eol_id=0, seed=0),
    "lumina_7b": dict(
        n_layers=32, d_model=4096, n_heads=32, n_kv_heads=32, head_dim=128, d_ffn=11008,
        vocab_out=65536, vocab_in=65536, dtype="bf16", rope_base=10000.0, rms_eps=1e-5,
        prompt_len=120, n_gen=2352, window_L=32, temperature=1.0, top_k=2000, cfg_lambda=3.0,
        allowed_lo=4096, allowed_hi=4096 + 8192, row_period=49, eol_id=12288 + 5, seed=0),
    "video_4b": dict(
        n_layers=28, d_model=3072, n_heads=24, n_kv_heads=24, head_dim=128, d_ffn=8192,
        vocab_out=64000, vocab_in=64000, dtype="bf16", rope_base=10000.0, rms_eps=1e-5,
        prompt_len=2560, n_gen=10240, window_L=64, temperature=1.0, top_k=1000, cfg_lambda=0.0,
        allowed_lo=0, allowed_hi=64000, row_period=0, eol_id=0, seed=0),
    # the paper's Janus-Pro setting on a 7B-shaped decoder: 24 x 24 image tokens, guidance 5, top-k 1000
    "janus_like": dict(
        n_layers=30, d_model=4096, n_heads=32, n_kv_heads=32, head_dim=128, d_ffn=11008,
        vocab_out=16384, vocab_in=16384 + 1024, dtype="bf16", rope_base=10000.0, rms_eps=1e-5,
        prompt_len=64, n_gen=576, window_L=32, temperature=1.0, top_k=1000, cfg_lambda=5.0,
        allowed_lo=0, allowed_hi=16384, row_period=0, eol_id=0, seed=0),
    # the paper's video setting on the video-shaped decoder: nucleus 0.8, no top-k
    "video_4b_top_p": dict(
        n_layers=28, d_model=3072, n_heads=24, n_kv_heads=24, head_dim=128, d_ffn=8192,
        vocab_out=64000, vocab_in=64000, dtype="bf16", rope_base=10000.0, rms_eps=1e-5,
        prompt_len=2560, n_gen=10240, window_L=64, temperature=1.0, top_k=0, top_p=0.8, cfg_lambda=0.0,
        allowed_lo=0, allowed_hi=64000, row_period=0, eol_id=0, seed=0),
}

LAYER_KEYS = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


def layer_shapes(s: dict) -> dict:
    d, dq, dkv, f = s["d_model"], s["n_heads"] * s["head_dim"], s["n_kv_heads"] * s["head_dim"], s["d_ffn"]
    return dict(attn_norm=(d,), wq=(dq, d), wk=(dkv, d), wv=(dkv, d), wo=(d, dq), ffn_norm=(d,),
                w_gate=(f, d), w_up=(f, d), w_down=(d, f))


def make_weights(shape: dict, seed: int = 1234, device: str = "cpu", std: float = 0.02) -> dict:
    """Random-init weights: matrices N(0, std), norm gains 1, in the workload's dtype.

    Returns torch tensors on ``device`` (row-major [out, in]); per-layer entries are lists."""
    dt = torch.float32 if shape["dtype"] == "f32" else torch.bfloat16
    g = torch.Generator(device=device)
    g.manual_seed(seed)

    def mat(*dims):
        return (torch.randn(*dims, generator=g, device=device, dtype=torch.float32) * std).to(dt)

    w = {"tok_emb": mat(shape["vocab_in"], shape["d_model"]),
         "final_norm": torch.ones(shape["d_model"], device=device, dtype=dt),
         "lm_head": None}
    ls = layer_shapes(shape)
    for k in LAYER_KEYS:
        w[k] = []
    for _ in range(shape["n_layers"]):
        for k in LAYER_KEYS:
            if k.endswith("norm"):
                w[k].append(torch.ones(ls[k], device=device, dtype=dt))
            else:
                w[k].append(mat(*ls[k]))
    w["lm_head"] = mat(shape["vocab_out"], shape["d_model"])
    return w


def perturb_norm_gains(w: dict, seed: int = 7, spread: float = 0.2) -> dict:
    """Replace the all-ones norm gains by 1 + U(-spread, spread), so that a test can tell a
    missing or misplaced gain from a correct one."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)

    def jitter(t):
        r = (torch.rand(t.shape, generator=g) * 2 - 1) * spread + 1.0
        return r.to(device=t.device, dtype=t.dtype)

    w["final_norm"] = jitter(w["final_norm"])
    for k in ("attn_norm", "ffn_norm"):
        w[k] = [jitter(t) for t in w[k]]
    return w


def to_numpy(t: torch.Tensor) -> np.ndarray:
    """float32 -> float32 array; bfloat16 -> uint16 array of the bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.uint16).numpy()
    return t.numpy()


def weights_to_numpy(w: dict) -> dict:
    out = {}
    for k, v in w.items():
        out[k] = [to_numpy(t) for t in v] if isinstance(v, list) else to_numpy(v)
    return out


def make_prompt(shape: dict, batch: int = 1, seed: int = 99):
    """Conditional and unconditional prompt ids, [batch, prompt_len] int32 each.

    Prompt ids are drawn outside the generated-code range where the vocabulary has room
    (class / text ids); the unconditional stream replaces every prompt id by one null id."""
    rng = np.random.default_rng(seed)
    P = shape["prompt_len"]
    lo, hi = shape["allowed_lo"], shape["allowed_hi"]
    vin = shape["vocab_in"]
    if vin > hi:
        ids = rng.integers(hi, vin - 1, size=(batch, P))
        null_id = vin - 1
    elif lo > 0:
        ids = rng.integers(0, lo - 1, size=(batch, P))
        null_id = lo - 1
    else:
        ids = rng.integers(0, vin, size=(batch, P))
        null_id = 0
    cond = ids.astype(np.int32)
    uncond = np.full_like(cond, null_id)
    return cond, uncond


def verify_logits(seed: int, iteration: int, B: int, L: int, V: int, device: str = "cpu",
                  streams: int = 1):
    """Verify-only workload: target logits N(0,1) scaled per row by s ~ U(2,6); draft logits are
    the target logits plus N(0, 0.3) noise (a stand-in for the previous Jacobi iteration's
    logits, which differ from the current ones by a small context change).

    Returns (p_logits [streams,B,L,V], q_logits [B,L,V]) float32."""
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1000003 + iteration) * 2 + 1)
    z = torch.randn(streams, B, L, V, generator=g, device=device, dtype=torch.float32)
    s = torch.rand(1, B, L, 1, generator=g, device=device, dtype=torch.float32) * 4.0 + 2.0
    p = z * s
    q = p[0] + 0.3 * torch.randn(B, L, V, generator=g, device=device, dtype=torch.float32)
    return p.contiguous(), q.contiguous()


def draft_ids_from_logits(q_logits: torch.Tensor, top_k: int, seed: int) -> torch.Tensor:
    """Draft tokens drawn from softmax of the top-k draft logits (so that X ~ q up to rounding),
    with torch's own sampler. [B,L,V] -> [B,L] int32."""
    g = torch.Generator(device=q_logits.device)
    g.manual_seed(seed * 7919 + 13)
    B, L, V = q_logits.shape
    x = q_logits.reshape(B * L, V)
    if 0 < top_k < V:
        kth = torch.topk(x, top_k, dim=-1).values[:, -1:]
        x = torch.where(x >= kth, x, torch.full_like(x, float("-inf")))
    pr = torch.softmax(x, dim=-1)
    ids = torch.multinomial(pr, 1, generator=g).reshape(B, L)
    return ids.to(torch.int32)
