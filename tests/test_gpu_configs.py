"""GPU parity at the shapes of every benchmark workload, at full depth, on long vocabulary rows, and
of the sampler's output distribution itself.

  - layer shapes of the LlamaGen-XL-like and the video-like decoders (two-layer truncations, every
    logit and hidden state against the oracle's forward);
  - full-depth window forwards (36 and 32 layers): the bf16 error at the depth the benchmark runs;
  - sessions whose vocabulary rows do not fit in shared memory (the integer draft weights of the
    previous iteration are read back from global memory), replayed decision by decision;
  - the KV cache after partial accepts: logits of later iterations against the oracle's own forward,
    teacher-forced on the tokens the GPU committed;
  - chi-square of the GPU path's generated sequences against the exact autoregressive joint
    prod_i p_i(x_i | x_<i) (Sec. 2.1; correctness theorem of Sec. 4: any coupling is lossless)."""
import itertools
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2510_24211_b200 import binding as scd
from paper_2510_24211_b200 import synth
from test_gpu_session import MID_BF16_D64, MODES, _models, _rel, _replay_case

pytestmark = pytest.mark.gpu


# ---- layer shapes of the other two benchmark workloads ----------------------------------------------
@pytest.mark.parametrize("name", ["llamagen_xl", "video_4b"])
def test_workload_layer_shape_forward_matches_oracle(name):
    shape = dict(synth.WORKLOADS[name], n_layers=2)
    P, L = 70, shape["window_L"]
    gm, om = _models(shape, max_seq=P + 2 * L + 8, seed=23, std=0.02, page=64)
    rng = np.random.default_rng(23)
    prompt = rng.integers(0, shape["vocab_in"], size=(1, P)).astype(np.int32)
    sess = scd.Session(gm, scd.decode_config(batch=1, window_L=L, allowed_hi=shape["vocab_out"]))
    sess.scd_prefill(prompt, n_new=L + 8)
    om.forward(prompt[0, :-1], 0)
    ids = np.concatenate([prompt[0, -1:], rng.integers(0, shape["vocab_in"], size=L - 1)]).astype(np.int32)
    logits, hidden = sess.scd_forward_window(torch.from_numpy(ids[None]).cuda(), want_hidden=True)
    ref_logits, ref_hidden = om.forward(ids, P - 1, want_hidden=True)
    assert _rel(hidden[0].cpu().numpy(), ref_hidden) <= 3e-2
    assert _rel(logits[0].cpu().numpy(), ref_logits) <= 3e-2


# ---- full depth -------------------------------------------------------------------------------------
@pytest.mark.parametrize("name,rows,att_min_ctx", [("llamagen_xl", 32, -1), ("lumina_7b", 32, -1), ("lumina_7b", 32, 0)])
def test_full_depth_window_logits_match_oracle(name, rows, att_min_ctx):
    """All layers of the workload's decoder, one window on top of a short prompt: the error of the bf16
    path (activations rounded to bf16 between kernels, fp32 accumulation) has the whole depth to grow."""
    shape = synth.WORKLOADS[name]
    P = 9
    w = synth.make_weights(shape, seed=1234, device="cuda")
    gm = scd.Model(shape, w, max_seq=P + rows + 8, kv_page_tokens=64)
    wn = synth.weights_to_numpy(w)
    om = oracle.Model(dict(shape, max_seq=P + rows + 8), wn)
    rng = np.random.default_rng(31)
    prompt = rng.integers(0, shape["vocab_in"], size=(1, P)).astype(np.int32)
    sess = scd.Session(gm, scd.decode_config(batch=1, window_L=rows, allowed_hi=shape["vocab_out"]))
    sess.scd_session_attention_min_ctx(att_min_ctx)        # -1: the mma.sync attention kernel, 0: the tcgen05 one
    sess.scd_prefill(prompt, n_new=rows + 4)
    om.forward(prompt[0, :-1], 0)
    ids = np.concatenate([prompt[0, -1:], rng.integers(0, shape["vocab_in"], size=rows - 1)]).astype(np.int32)
    logits, hidden = sess.scd_forward_window(torch.from_numpy(ids[None]).cuda(), want_hidden=True)
    ref_logits, ref_hidden = om.forward(ids, P - 1, want_hidden=True)
    e_h, e_l = _rel(hidden[0].cpu().numpy(), ref_hidden), _rel(logits[0].cpu().numpy(), ref_logits)
    print(f"\n{name}: {shape['n_layers']} layers, attention min_ctx {att_min_ctx}, max-relative error hidden {e_h:.3e}, logits {e_l:.3e}")
    assert e_h <= 3e-2 and e_l <= 3e-2


# ---- long vocabulary rows in a session ------------------------------------------------------------------
WIDE_VOCAB = dict(n_layers=2, d_model=128, n_heads=2, n_kv_heads=2, head_dim=64, d_ffn=192,
                  vocab_out=64000, vocab_in=64000, dtype="bf16", rope_base=10000.0, rms_eps=1e-5)


@pytest.mark.parametrize("mode,V,top_k,top_p", [
    (oracle.MODE_SCD_MC, 64000, 1000, 0.0),      # the video workload's row: no row fits in shared memory
    (oracle.MODE_SCD_GS, 64000, 1000, 0.0),
    (oracle.MODE_SCD_MC, 40000, 500, 0.0),       # the target row fits, the draft row does not
    (oracle.MODE_SCD_MC, 64000, 0, 0.8),         # the paper's video setting: nucleus 0.8, no top-k
])
def test_step_replay_long_vocabulary_rows(mode, V, top_k, top_p):
    shape = dict(WIDE_VOCAB, vocab_out=V, vocab_in=V)
    _replay_case(shape, mode, B=1, L=8, P=5, n_new=48, top_k=top_k, seed=41, std=0.35, page=64, top_p=top_p)


# ---- KV cache after partial accepts --------------------------------------------------------------------
@pytest.mark.parametrize("att_min_ctx", [-1, 0])        # the mma.sync attention kernel, the tcgen05 one
def test_bf16_logits_after_partial_accepts_match_oracle_forward(att_min_ctx):
    """A stale or misplaced K/V row left behind by an accept or a reject would change the logits of
    every later iteration. Here the GPU session runs on its own (CUDA-graph iterations, CFG pair,
    two sequences, pages of 64 tokens crossed during generation); afterwards the oracle's forward is
    teacher-forced, iteration by iteration, on the tokens the GPU committed and the drafts it fed, and
    its logits are compared with those the GPU produced at that iteration."""
    shape, B, L, P, n_new = MID_BF16_D64, 2, 16, 58, 96
    # small weights keep the bf16 path accurate; a scaled-up LM head makes the next token nearly
    # certain, so that drafts are accepted in runs and the window slides by more than one position
    w = synth.perturb_norm_gains(synth.make_weights(shape, seed=13, std=0.06))
    w["lm_head"] = (w["lm_head"].float() * 10.0).to(w["lm_head"].dtype)
    wg = {k: ([t.cuda() for t in v] if isinstance(v, list) else v.cuda()) for k, v in w.items()}
    max_seq = P + n_new + L + 4
    gm = scd.Model(shape, wg, max_seq=max_seq, kv_page_tokens=64)
    om = oracle.Model(dict(shape, max_seq=max_seq), synth.weights_to_numpy(w), n_streams=2 * B)
    rng = np.random.default_rng(77)
    cond = rng.integers(0, shape["vocab_in"], size=(B, P)).astype(np.int32)
    uncond = np.full_like(cond, shape["vocab_in"] - 1)
    cfg = scd.decode_config(mode=scd.SCD_MODE_SCD_MC, batch=B, window_L=L, top_k=4, cfg_lambda=1.5, seed=3,
                            allowed_hi=shape["vocab_out"])
    sess = scd.Session(gm, cfg)
    sess.scd_session_attention_min_ctx(att_min_ctx)
    sess.scd_prefill(np.concatenate([cond, uncond]), n_new=n_new)
    rec = []
    n_total = P + n_new
    for _ in range(n_new + 2):
        _, n_now, kv = sess.scd_step_result()
        if (n_now >= n_total).all():
            break
        drafts = sess.scd_debug_read("drafts").copy()
        sess.scd_step()
        rec.append((n_now.copy(), drafts, sess.scd_debug_read("logits").copy(), sess.scd_step_result()[0].copy()))
    tokens = sess.scd_read_tokens(0, n_total)
    accepts = np.array([r[3] for r in rec])
    assert (accepts > 1).any() and (accepts == 1).any()          # mixed accept counts: the window really slides
    worst = 0.0
    for b in range(B):
        for s in range(2):
            q = s * B + b                                         # stream-sequence index on both sides
            prompt = cond[b] if s == 0 else uncond[b]
            om.forward(prompt[:-1], 0, stream=q)
            for n_now, drafts, logits, _ in rec:
                n = int(n_now[b])
                Lw = min(L, n_total - n)
                if Lw <= 0:
                    continue
                last = prompt[-1] if n == P else tokens[b, n - 1]
                ids = np.concatenate([[last], drafts[b, :Lw - 1]]).astype(np.int32)
                ref = om.forward(ids, n - 1, stream=q)
                worst = max(worst, _rel(logits[q, :Lw], ref))
    assert worst <= 3e-2, worst


# ---- losslessness of the CUDA path itself -------------------------------------------------------------------
CHI_SHAPE = dict(n_layers=1, d_model=64, n_heads=2, n_kv_heads=2, head_dim=32, d_ffn=96,
                 vocab_out=8, vocab_in=12, dtype="f32", rope_base=10000.0, rms_eps=1e-5)


@pytest.mark.parametrize("mode,L", [(oracle.MODE_SCD_MC, 2), (oracle.MODE_SCD_GS, 3), (oracle.MODE_SCD_MC, 4)])
def test_generated_sequences_follow_the_exact_ar_joint(mode, L):
    """3 generated tokens over a vocabulary of 8, more than 2 * 10^4 generations through scd_prefill +
    scd_generate (200 sequences per session share a prompt and differ in their batch index, which keys
    the noise; every session has its own seed). The histogram of the 512 possible sequences is compared
    with prod_i p_i(x_i | x_<i), p_i from the oracle's forward and post-processing."""
    shape, P, n_gen, top_k, B, n_sessions = CHI_SHAPE, 2, 3, 6, 200, 110
    V = shape["vocab_out"]
    gm, om = _models(shape, max_seq=16, seed=5, std=0.6)
    prompt = np.array([9, 10], dtype=np.int32)
    joint = {}
    for seq in itertools.product(range(V), repeat=n_gen):
        pr = 1.0
        for i in range(n_gen):
            ids = np.concatenate([prompt, np.array(seq[:i], dtype=np.int32)]).astype(np.int32)
            W, Z = oracle.postprocess(om.forward(ids, 0)[-1], None, temperature=1.0, top_k=top_k)
            pr *= float(W[seq[i]]) / float(Z)
            if pr == 0.0:
                break
        joint[seq] = pr
    assert abs(sum(joint.values()) - 1.0) < 1e-9
    hist, committed = {}, 0
    prompts = np.repeat(prompt[None], B, axis=0)
    for s in range(n_sessions):
        cfg = scd.decode_config(mode=MODES[mode], batch=B, window_L=L, top_k=top_k, seed=1000 + s, allowed_hi=V)
        sess = scd.Session(gm, cfg)
        sess.scd_prefill(prompts, n_new=n_gen)
        toks, st = sess.scd_generate()
        committed += st.committed
        for row in toks:
            key = tuple(int(t) for t in row)
            hist[key] = hist.get(key, 0) + 1
        sess.close()
    n = B * n_sessions
    assert n >= 20_000 and sum(hist.values()) == n and committed == n * n_gen
    # cells with fewer than 8 expected draws are pooled into one (the chi-square approximation needs it)
    chi2, dof, pool_e, pool_o = 0.0, -1, 0.0, 0
    for seq, pr in joint.items():
        got = hist.get(seq, 0)
        if pr < 1e-12:
            assert got == 0, f"sequence {seq} has probability 0 but was generated"
        elif n * pr < 8.0:
            pool_e += n * pr
            pool_o += got
        else:
            chi2 += (got - n * pr) ** 2 / (n * pr)
            dof += 1
    if pool_e > 0.0:
        chi2 += (pool_o - pool_e) ** 2 / pool_e
        dof += 1
    assert dof >= 20
    assert chi2 < dof + 4.5 * math.sqrt(2 * dof), (chi2, dof)


# ---- the paper's other two settings as workloads (reduced depth) -------------------------------------------
@pytest.mark.parametrize("name", ["janus_like", "video_4b_top_p"])
def test_step_replay_paper_settings_reduced_depth(name):
    """Janus-Pro-like (guidance 5, top-k 1000, 24 x 24 tokens) and the video setting with nucleus 0.8 and no
    top-k (App. "Experimental Details"), on two layers of the workload's shape: every decision of a short
    generation replayed through the oracle's loop."""
    w = synth.WORKLOADS[name]
    shape = dict(w, n_layers=2)
    _replay_case(shape, oracle.MODE_SCD_MC, B=1, L=w["window_L"], P=6, n_new=70, top_k=w["top_k"], lam=w["cfg_lambda"],
                 seed=19, lo=w["allowed_lo"], hi=w["allowed_hi"], std=0.02, page=64, top_p=w.get("top_p", 0.0))
