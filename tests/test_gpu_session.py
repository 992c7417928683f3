"""GPU parity of the window forward and of the whole SCD iteration against the CPU oracle.

  - logits / hidden states: max |a-b| / max |b| <= 2e-3 (fp32 models), <= 3e-2 (bf16 models);
  - step-level decisions: the logits the GPU produced at every iteration are replayed through the
    oracle's own decode loop, and accept counts, committed tokens, drafts and KV length must be
    identical (bit-exact given the same fp32 logits and Philox key);
  - end to end on the tiny workload: same tokens as the oracle running its own forward."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_24211_b200 import binding as scd
from paper_2510_24211_b200 import synth

pytestmark = pytest.mark.gpu

SMALL = dict(n_layers=2, d_model=128, n_heads=4, n_kv_heads=2, head_dim=32, d_ffn=208,
             vocab_out=300, vocab_in=310, dtype="f32", rope_base=10000.0, rms_eps=1e-5)
SMALL_BF16 = dict(n_layers=3, d_model=128, n_heads=4, n_kv_heads=4, head_dim=32, d_ffn=192,
                  vocab_out=512, vocab_in=520, dtype="bf16", rope_base=10000.0, rms_eps=1e-5)
MODES = {oracle.MODE_AR: scd.SCD_MODE_AR, oracle.MODE_SJD: scd.SCD_MODE_SJD,
         oracle.MODE_SCD_MC: scd.SCD_MODE_SCD_MC, oracle.MODE_ALPHA: scd.SCD_MODE_ALPHA,
         oracle.MODE_SCD_GS: scd.SCD_MODE_SCD_GS}


def _rel(a, b):
    return float(np.abs(a - b).max() / np.abs(b).max())


def _models(shape, max_seq, seed=3, std=0.05, n_streams=1, page=16):
    w = synth.perturb_norm_gains(synth.make_weights(shape, seed=seed, std=std))
    wg = {k: ([t.cuda() for t in v] if isinstance(v, list) else v.cuda()) for k, v in w.items()}
    gm = scd.Model(shape, wg, max_seq=max_seq, kv_page_tokens=page)
    om = oracle.Model(dict(shape, max_seq=max_seq), synth.weights_to_numpy(w), n_streams=n_streams)
    return gm, om


@pytest.mark.parametrize("shape,tol", [(SMALL, 2e-3), (SMALL_BF16, 3e-2)])
def test_forward_window_logits_and_hidden(shape, tol):
    gm, om = _models(shape, max_seq=96)
    rng = np.random.default_rng(0)
    P, M = 21, 8
    prompt = rng.integers(0, shape["vocab_in"], size=(1, P)).astype(np.int32)
    sess = scd.Session(gm, scd.decode_config(batch=1, window_L=M, allowed_hi=shape["vocab_out"]))
    sess.scd_prefill(prompt, n_new=40)
    om.forward(prompt[0, :-1], 0)
    nxt = rng.integers(0, shape["vocab_in"], size=M - 1).astype(np.int32)
    ids = np.concatenate([prompt[0, -1:], nxt])
    logits, hidden = sess.scd_forward_window(torch.from_numpy(ids[None]).cuda(), commit=True, want_hidden=True)
    ref_logits, ref_hidden = om.forward(ids, P - 1, want_hidden=True)
    assert _rel(logits[0].cpu().numpy(), ref_logits) <= tol
    assert _rel(hidden[0].cpu().numpy(), ref_hidden) <= tol
    # a second window on top of the committed one: KV of the first must have been kept
    a, n, kv = sess.scd_step_result()
    assert n[0] == P + M - 1 and kv[0] == n[0] - 1
    ids2 = np.concatenate([ids[-1:], rng.integers(0, shape["vocab_in"], size=5).astype(np.int32)])
    logits2 = sess.scd_forward_window(torch.from_numpy(ids2[None]).cuda())
    ref2 = om.forward(ids2, P - 1 + M - 1)
    assert _rel(logits2[0].cpu().numpy(), ref2) <= tol
    # single-token window == row 0 of the wider one (causality)
    logits3 = sess.scd_forward_window(torch.from_numpy(ids2[None, :1].copy()).cuda())
    assert _rel(logits3[0, 0].cpu().numpy(), ref2[0]) <= tol


def test_forward_long_prompt_crosses_pages_and_chunks():
    gm, om = _models(SMALL, max_seq=400, seed=5)
    rng = np.random.default_rng(1)
    P = 300                                            # > prefill chunk (128) and many 16-token pages
    prompt = rng.integers(0, SMALL["vocab_in"], size=(1, P)).astype(np.int32)
    sess = scd.Session(gm, scd.decode_config(batch=1, window_L=4, allowed_hi=SMALL["vocab_out"]))
    sess.scd_prefill(prompt, n_new=10)
    om.forward(prompt[0, :-1], 0)
    ids = np.concatenate([prompt[0, -1:], [5, 6, 7]]).astype(np.int32)
    logits = sess.scd_forward_window(torch.from_numpy(ids[None]).cuda())
    assert _rel(logits[0].cpu().numpy(), om.forward(ids, P - 1)) <= 2e-3


# bf16 shapes that take the tensor-core attention path (head_dim 64 / 128, pages of 64 / 128 tokens)
MID_BF16_D64 = dict(n_layers=2, d_model=256, n_heads=4, n_kv_heads=4, head_dim=64, d_ffn=320,
                    vocab_out=384, vocab_in=400, dtype="bf16", rope_base=10000.0, rms_eps=1e-5)
MID_BF16_D128_GQA = dict(n_layers=2, d_model=256, n_heads=2, n_kv_heads=1, head_dim=128, d_ffn=320,
                         vocab_out=384, vocab_in=400, dtype="bf16", rope_base=10000.0, rms_eps=1e-5)


@pytest.mark.parametrize("shape,page,P,M", [
    (MID_BF16_D64, 64, 300, 32),       # 5 context tiles, ragged last tile, several pages
    (MID_BF16_D64, 128, 65, 16),       # one full tile + 1 key
    (MID_BF16_D128_GQA, 128, 300, 32), # two query heads share one KV head
    (MID_BF16_D128_GQA, 64, 2, 64),    # (almost) no context: only the window, L = 64
    (MID_BF16_D128_GQA, 64, 700, 1),   # single-row window (the AR shape), 11 tiles over the cluster
    (MID_BF16_D128_GQA, 128, 2000, 64),  # long context, L = 64 with two query heads per KV head (8 row tiles)
    (MID_BF16_D64, 64, 900, 128),      # the largest window of the video table: 128 rows, two window tiles
    (MID_BF16_D64, 64, 2000, 32),      # long context, 32 rows: five tiles per CTA, two warps per query tile
    (MID_BF16_D128_GQA, 128, 1500, 16),  # the same with head_dim 128 and a window CTA without context tiles
    (MID_BF16_D128_GQA, 64, 1100, 1),  # single row, long context
])
@pytest.mark.parametrize("kernel", ["mma_sync", "tcgen05"])
def test_forward_tensor_core_attention(shape, page, P, M, kernel):
    gm, om = _models(shape, max_seq=P + 2 * M + 70, seed=9, std=0.08, page=page)
    rng = np.random.default_rng(P)
    prompt = rng.integers(0, shape["vocab_in"], size=(1, P)).astype(np.int32)
    sess = scd.Session(gm, scd.decode_config(batch=1, window_L=M, allowed_hi=shape["vocab_out"]))
    sess.scd_session_attention_min_ctx(0 if kernel == "tcgen05" else -1)   # every context length through each kernel
    sess.scd_prefill(prompt, n_new=M + 40)
    om.forward(prompt[0, :-1], 0)
    ids = np.concatenate([prompt[0, -1:], rng.integers(0, shape["vocab_in"], size=M - 1)]).astype(np.int32)
    logits, hidden = sess.scd_forward_window(torch.from_numpy(ids[None]).cuda(), commit=True, want_hidden=True)
    ref_logits, ref_hidden = om.forward(ids, P - 1, want_hidden=True)
    assert _rel(hidden[0].cpu().numpy(), ref_hidden) <= 3e-2
    assert _rel(logits[0].cpu().numpy(), ref_logits) <= 3e-2
    # the window's K/V must have reached the cache: a second window on top of the first
    ids2 = np.concatenate([ids[-1:], rng.integers(0, shape["vocab_in"], size=min(M, 7))]).astype(np.int32)
    if len(ids2) <= sess.L or len(ids2) <= 128:
        logits2 = sess.scd_forward_window(torch.from_numpy(ids2[None]).cuda())
        ref2 = om.forward(ids2, P - 1 + M - 1)
        assert _rel(logits2[0].cpu().numpy(), ref2) <= 3e-2


@pytest.mark.parametrize("att_min_ctx", [-1, 0])
def test_step_replay_bf16_tensor_core_attention_cfg_batch(att_min_ctx):
    # CFG pair of streams x 2 sequences through the tensor-core attention (the mma.sync kernel, then the
    # tcgen05 kernel, inside the captured iteration) and the cluster GEMMs
    _replay_case(MID_BF16_D64, oracle.MODE_SCD_MC, B=2, L=16, P=70, n_new=60, top_k=40, lam=2.0, seed=8,
                 page=64, att_min_ctx=att_min_ctx)


def test_step_replay_attention_kernel_changes_inside_a_generation():
    # the committed context passes 512 positions while the sequence is generated: the captured iteration is built
    # again with the tcgen05 attention kernel in place of the mma.sync one, and the decisions still replay
    _replay_case(MID_BF16_D64, oracle.MODE_SCD_MC, B=1, L=16, P=490, n_new=80, top_k=40, seed=31, page=64)


def _replay_case(shape, mode, B, L, P, n_new, top_k, lam=0.0, temperature=1.0, seed=0, lo=0, hi=None,
                 row_period=0, eol_id=0, std=0.3, page=16, alpha=1.0, top_p=0.0, autotune=False, gm=None,
                 att_min_ctx=None):
    """Run the GPU session step by step, then replay its logits through the oracle's loop."""
    hi = shape["vocab_out"] if hi is None else hi
    S = 2 if lam != 0.0 else 1
    if gm is None:
        gm, _ = _models(shape, max_seq=P + n_new + 4, seed=11, std=std, page=page)
    rng = np.random.default_rng(seed + 100)
    cond = rng.integers(0, shape["vocab_in"], size=(B, P)).astype(np.int32)
    uncond = np.full_like(cond, shape["vocab_in"] - 1)
    prompts = np.concatenate([cond, uncond]) if S == 2 else cond
    cfg = scd.decode_config(mode=MODES[mode], batch=B, window_L=L, temperature=temperature, top_k=top_k,
                            cfg_lambda=lam, seed=seed, allowed_lo=lo, allowed_hi=hi,
                            row_period=row_period, eol_id=eol_id, alpha=alpha, top_p=top_p)
    sess = scd.Session(gm, cfg)
    if att_min_ctx is not None:
        sess.scd_session_attention_min_ctx(att_min_ctx)
    sess.scd_prefill(prompts, n_new=n_new)
    if autotune:
        before = [x.copy() for x in sess.scd_step_result()] + [sess.scd_debug_read("drafts").copy()]
        chosen = sess.scd_autotune()
        assert chosen.shape == (4,) and ((chosen >= 0) & (chosen <= 8)).all()
        after = [x.copy() for x in sess.scd_step_result()] + [sess.scd_debug_read("drafts").copy()]
        for x, y in zip(before, after):
            assert np.array_equal(x, y)                  # tuning runs forwards only: the state did not move
    Lw = sess.L
    rec_logits, rec_drafts, rec_a, rec_n = [], [], [], []
    n_total = P + n_new
    for _ in range(n_new + 2):
        a_prev, n_now, kv = sess.scd_step_result()
        assert (kv == n_now - 1).all()
        if (n_now >= n_total).all():
            break
        rec_drafts.append(sess.scd_debug_read("drafts"))
        sess.scd_step()
        rec_logits.append(sess.scd_debug_read("logits"))
        a, n_after, _ = sess.scd_step_result()
        rec_a.append(a.copy())
        rec_n.append(n_now.copy())
    gpu_tokens = sess.scd_read_tokens(0, n_total)
    V = shape["vocab_out"]
    for b in range(B):
        # the oracle's loop over the GPU's logits: call i of each stream is GPU iteration i
        # (sequences that finished early stop calling)
        calls = {0: 0, 1: 0}

        def fwd(stream, ids, pos0, b=b, calls=calls):
            idx = calls[stream]
            calls[stream] += 1
            if P > 1:                                   # the first call of a stream is the prefill
                if idx == 0:
                    assert pos0 == 0 and len(ids) == P - 1
                    return np.zeros((len(ids), V), dtype=np.float32)
                idx -= 1
            assert pos0 == rec_n[idx][b] - 1
            if mode != oracle.MODE_AR and len(ids) > 1:           # inputs = [last token, drafts]
                assert np.array_equal(ids[1:], rec_drafts[idx][b, :len(ids) - 1])
            return rec_logits[idx][stream * B + b, :len(ids)]

        dec = oracle.Decode(mode=mode, window_L=L, top_k=top_k, cfg_lambda=lam, temperature=temperature,
                            seed=seed, batch_index=b, allowed_lo=lo, allowed_hi=hi, row_period=row_period,
                            eol_id=eol_id, alpha=alpha, top_p=top_p)
        res = oracle.CallbackModel(V, fwd).generate(dec, cond[b], n_total, uncond[b] if S == 2 else None)
        assert np.array_equal(res.tokens, gpu_tokens[b]), (b, res.tokens, gpu_tokens[b])
        got_a = [int(x[b]) for x in rec_a if x[b] > 0][:res.forwards]
        assert got_a == res.trace_a.tolist()
    return rec_a


@pytest.mark.parametrize("mode", [oracle.MODE_SCD_MC, oracle.MODE_SJD, oracle.MODE_AR])
def test_step_decisions_replayed_through_oracle(mode):
    _replay_case(SMALL, mode, B=1, L=6, P=5, n_new=40, top_k=30)


@pytest.mark.parametrize("alpha", [0.25, 0.8])
def test_step_replay_alpha_coupling(alpha):
    # Algorithm 5 end to end: window slide, fresh rows and the coin per redrafted row
    _replay_case(SMALL, oracle.MODE_ALPHA, B=2, L=6, P=5, n_new=40, top_k=30, seed=9, alpha=alpha)


def test_step_replay_gumbel_sharing():
    # Algorithm 7 end to end: initial drafts, redrafts and fresh rows all come from the shared-noise race
    _replay_case(SMALL, oracle.MODE_SCD_GS, B=1, L=6, P=5, n_new=40, top_k=30, seed=12)
    _replay_case(SMALL, oracle.MODE_SCD_GS, B=2, L=5, P=3, n_new=33, top_k=20, lam=1.5, temperature=0.9,
                 seed=13, lo=10, hi=250, row_period=7, eol_id=260)


def test_step_replay_nucleus_truncation():
    # top-p end to end: the truncated p of one iteration is the draft distribution of the next
    _replay_case(SMALL, oracle.MODE_SCD_MC, B=2, L=6, P=5, n_new=40, top_k=0, seed=14, top_p=0.8)
    _replay_case(SMALL, oracle.MODE_SCD_GS, B=1, L=6, P=5, n_new=40, top_k=30, seed=15, top_p=0.6)


def test_step_replay_wide_window_ragged_batch_bf16():
    # L = 48 through the tensor-core path with three sequences that progress at different speeds
    _replay_case(MID_BF16_D64, oracle.MODE_SCD_MC, B=3, L=48, P=66, n_new=120, top_k=60, seed=17, page=64)


def test_step_replay_four_cfg_pairs_fill_one_row_block():
    # B = 4 with guidance at L = 32: 256 window rows, the most one GEMM launch carries
    _replay_case(MID_BF16_D64, oracle.MODE_SCD_MC, B=4, L=32, P=40, n_new=70, top_k=40, lam=1.5, seed=23, page=64)


def test_step_replay_more_rows_than_one_gemm_block():
    # B = 5 with guidance at L = 32: 320 window rows, two passes over the weights per GEMM (256 + 64 rows);
    # and a session beyond the 1024 rows that are accepted
    _replay_case(MID_BF16_D64, oracle.MODE_SCD_MC, B=5, L=32, P=40, n_new=50, top_k=40, lam=1.5, seed=29, page=64)
    gm, _ = _models(MID_BF16_D64, max_seq=128, seed=11, std=0.3, page=64)
    with pytest.raises(scd.ScdError) as e:
        scd.Session(gm, scd.decode_config(batch=17, window_L=32, cfg_lambda=1.5, allowed_hi=MID_BF16_D64["vocab_out"]))
    assert e.value.code == scd.SCD_ERR_CAPACITY


def test_autotune_keeps_state_and_parity():
    # the K slicing chosen by timing changes launch shapes only: decisions still replay through the oracle
    _replay_case(MID_BF16_D64, oracle.MODE_SCD_MC, B=2, L=16, P=70, n_new=60, top_k=40, lam=2.0, seed=19,
                 page=64, autotune=True)


def test_step_replay_batch_cfg_ragged_end_and_forced_tokens():
    # two sequences progress at different speeds; CFG pair of streams; generation length not a
    # multiple of L; every 7th generated token forced
    _replay_case(SMALL, oracle.MODE_SCD_MC, B=2, L=5, P=3, n_new=33, top_k=20, lam=1.5, temperature=0.9,
                 seed=3, lo=10, hi=250, row_period=7, eol_id=260)
    _replay_case(SMALL, oracle.MODE_SCD_MC, B=3, L=8, P=1, n_new=21, top_k=0, seed=4)


def test_step_replay_bf16_model():
    _replay_case(SMALL_BF16, oracle.MODE_SCD_MC, B=1, L=8, P=4, n_new=40, top_k=50, seed=6)


def test_generate_matches_stepwise_and_counts():
    gm, _ = _models(SMALL, max_seq=80, seed=11, std=0.3)
    prompt = np.array([[7, 8, 9]], dtype=np.int32)
    cfg = scd.decode_config(batch=1, window_L=6, top_k=30, seed=5, allowed_hi=SMALL["vocab_out"])
    s1 = scd.Session(gm, cfg)
    s1.scd_prefill(prompt, n_new=50)
    toks, st = s1.scd_generate()
    assert st.committed == 50 and sum(a * c for a, c in enumerate(st.accept_hist)) == 50
    assert st.forwards == sum(st.accept_hist) and st.elapsed_ms > 0
    s2 = scd.Session(gm, cfg)
    s2.scd_prefill(prompt, n_new=50)
    for _ in range(st.forwards):
        s2.scd_step()
    a, n, kv = s2.scd_step_result()
    assert n[0] == 53 and kv[0] == 52
    assert np.array_equal(s2.scd_read_tokens(3, 50), toks)
    # same seed -> same tokens; prefill resets the session
    s1.scd_prefill(prompt, n_new=50)
    toks2, _ = s1.scd_generate()
    assert np.array_equal(toks, toks2)


def test_tiny_workload_end_to_end_tokens_equal_oracle():
    shape = synth.WORKLOADS["tiny"]
    w = synth.make_weights(shape, seed=1234)
    wg = {k: ([t.cuda() for t in v] if isinstance(v, list) else v.cuda()) for k, v in w.items()}
    P, N = shape["prompt_len"], shape["n_gen"]
    gm = scd.Model(shape, wg, max_seq=P + N + 8)
    cond, _ = synth.make_prompt(shape)
    om = oracle.Model(dict(shape, max_seq=P + N + 8), synth.weights_to_numpy(w))
    results = {}
    for mode in (oracle.MODE_SCD_MC, oracle.MODE_AR):
        cfg = scd.decode_config(mode=MODES[mode], batch=1, window_L=shape["window_L"],
                                temperature=shape["temperature"], top_k=shape["top_k"], seed=shape["seed"],
                                allowed_lo=shape["allowed_lo"], allowed_hi=shape["allowed_hi"])
        sess = scd.Session(gm, cfg)
        sess.scd_prefill(cond, n_new=N)
        toks, st = sess.scd_generate()
        dec = oracle.Decode(mode=mode, window_L=shape["window_L"], top_k=shape["top_k"], seed=shape["seed"],
                            temperature=shape["temperature"], allowed_lo=shape["allowed_lo"],
                            allowed_hi=shape["allowed_hi"])
        ref = om.generate(dec, cond[0], P + N)
        assert np.array_equal(toks[0], ref.tokens[P:])
        assert st.forwards == ref.forwards and st.committed == N
        results[mode] = st.forwards
    assert results[oracle.MODE_AR] == N and results[oracle.MODE_SCD_MC] <= N


def test_session_error_paths_leave_context_usable():
    gm, _ = _models(SMALL, max_seq=64)
    with pytest.raises(scd.ScdError) as e:
        scd.Session(gm, scd.decode_config(batch=1, window_L=300, allowed_hi=300))
    assert e.value.code == scd.SCD_ERR_ARG
    sess = scd.Session(gm, scd.decode_config(batch=1, window_L=4, allowed_hi=300))
    with pytest.raises(scd.ScdError) as e:
        sess.scd_step()
    assert e.value.code == scd.SCD_ERR_STATE
    with pytest.raises(scd.ScdError) as e:
        sess.scd_prefill(np.zeros((1, 10), dtype=np.int32), n_new=60)      # 70 > max_seq
    assert e.value.code == scd.SCD_ERR_CAPACITY
    with pytest.raises(scd.ScdError) as e:
        sess.scd_prefill(np.full((1, 4), 999, dtype=np.int32), n_new=4)     # id outside vocab_in
    assert e.value.code == scd.SCD_ERR_ARG
    bad = dict(SMALL, head_dim=24)
    w = synth.make_weights(SMALL)
    wg = {k: ([t.cuda() for t in v] if isinstance(v, list) else v.cuda()) for k, v in w.items()}
    with pytest.raises(scd.ScdError) as e:
        scd.Model(bad, wg, max_seq=64)
    assert e.value.code == scd.SCD_ERR_SHAPE
    sess.scd_prefill(np.ones((1, 3), dtype=np.int32), n_new=8)
    toks, st = sess.scd_generate()
    assert toks.shape == (1, 8) and st.committed == 8


@pytest.mark.gpu
def test_step_timeline_advances_like_step_and_charges_every_class():
    """scd_step_timeline (time stamps inside the kernels, no events between them) advances the
    session exactly like scd_step and charges time to every GEMM / attention class."""
    shape, B, L, P, n_new = MID_BF16_D64, 1, 16, 70, 48
    gm, _ = _models(shape, max_seq=P + n_new + 4, seed=11, std=0.3, page=64)
    rng = np.random.default_rng(5)
    prompts = rng.integers(0, shape["vocab_in"], size=(B, P)).astype(np.int32)
    cfg = scd.decode_config(mode=scd.SCD_MODE_SCD_MC, batch=B, window_L=L, temperature=1.0, top_k=40,
                            cfg_lambda=0.0, seed=3, allowed_lo=0, allowed_hi=shape["vocab_out"])
    a, b = scd.Session(gm, cfg), scd.Session(gm, cfg)
    a.scd_prefill(prompts, n_new=n_new)
    b.scd_prefill(prompts, n_new=n_new)
    names = list(scd.PROF_CLASSES)
    for _ in range(3):
        a.scd_step()
        ms, n = b.scd_step_timeline()
        for x, y in zip(a.scd_step_result(), b.scd_step_result()):
            assert (x == y).all()
        for c in ("gemm_qkv", "attention", "gemm_o", "gemm_gate_up", "gemm_down"):
            assert n[names.index(c)] == shape["n_layers"] and ms[names.index(c)] > 0
        assert n[names.index("gemm_lm_head")] == 1 and ms[names.index("gemm_lm_head")] > 0
        assert 0 < float(ms.sum()) < 50.0
    known = int(a.scd_step_result()[1].min())                    # tokens committed so far
    assert known > P
    assert (a.scd_read_tokens(0, known) == b.scd_read_tokens(0, known)).all()


# ---- the benchmark's own configuration (7B-shaped decoder, L = 32, CFG pair, 8192 allowed ids) ----------
def test_benchmark_layer_shape_forward_matches_oracle():
    """Full layer sizes (d 4096, 32 heads of 128, FFN 11008, vocabulary 65536: the GEMM, attention and
    LM-head launches are the ones bench.py times) on a model of two layers, which the oracle still
    evaluates in seconds: every logit of the window against the oracle."""
    shape = dict(synth.WORKLOADS["lumina_7b"], n_layers=2)
    P, L = 70, shape["window_L"]
    gm, om = _models(shape, max_seq=P + 2 * L + 8, seed=21, std=0.02, page=64)
    rng = np.random.default_rng(21)
    prompt = rng.integers(0, shape["vocab_in"], size=(1, P)).astype(np.int32)
    sess = scd.Session(gm, scd.decode_config(batch=1, window_L=L, allowed_hi=shape["vocab_out"]))
    sess.scd_prefill(prompt, n_new=L + 8)
    om.forward(prompt[0, :-1], 0)
    ids = np.concatenate([prompt[0, -1:], rng.integers(0, shape["vocab_in"], size=L - 1)]).astype(np.int32)
    logits, hidden = sess.scd_forward_window(torch.from_numpy(ids[None]).cuda(), want_hidden=True)
    ref_logits, ref_hidden = om.forward(ids, P - 1, want_hidden=True)
    assert _rel(hidden[0].cpu().numpy(), ref_hidden) <= 3e-2
    assert _rel(logits[0].cpu().numpy(), ref_logits) <= 3e-2


def test_benchmark_configuration_decisions_replay_through_oracle():
    """The whole 32-layer model in the launch configuration of bench.py (one CUDA graph per iteration,
    CFG pair of streams, 8192 allowed ids out of 65536, a forced end-of-row token every 49 positions):
    every accept / reject decision, residual sample and redraft of a generation replayed by the oracle
    from the logits the GPU produced - bit-exact at any size."""
    shape = synth.WORKLOADS["lumina_7b"]
    P, n_new = 24, 60
    w = synth.make_weights(shape, seed=1234, device="cuda")
    gm = scd.Model(shape, w, max_seq=P + n_new + 4)
    _replay_case(shape, oracle.MODE_SCD_MC, B=1, L=shape["window_L"], P=P, n_new=n_new, top_k=shape["top_k"],
                 lam=shape["cfg_lambda"], seed=5, lo=shape["allowed_lo"], hi=shape["allowed_hi"],
                 row_period=shape["row_period"], eol_id=shape["eol_id"], gm=gm)
