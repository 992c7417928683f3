"""GPU parity of the fused verify-and-redraft kernel against the CPU oracle, through the C ABI.

Bit-exact comparison of accept counts, accept flags, committed ids and next drafts on the same
fp32 logits and the same Philox key."""
import os

import numpy as np
import pytest
import torch

import oracle
from helpers import oracle_verify
from paper_2510_24211_b200 import binding as scd
from paper_2510_24211_b200 import synth

pytestmark = pytest.mark.gpu
MODES = {"ar": scd.SCD_MODE_AR, "sjd": scd.SCD_MODE_SJD, "scd": scd.SCD_MODE_SCD_MC,
         "alpha": scd.SCD_MODE_ALPHA, "gs": scd.SCD_MODE_SCD_GS}


def _run_case(mode, B, L, V, iteration, seed, temperature=1.0, top_k=0, lam=0.0, lo=0, hi=None,
              row_period=0, eol_id=0, q_present=True, quantise=None, pos_base=1000, alpha=1.0, top_p=0.0):
    hi = V if hi is None else hi
    S = 2 if lam != 0.0 else 1
    p, q = synth.verify_logits(seed, iteration, B, L, V, device="cuda", streams=S)
    if quantise:
        p = torch.round(p / quantise) * quantise      # many exact ties
        q = torch.round(q / quantise) * quantise
    if mode == "ar":
        p = p[:, :, :1].contiguous()
        q = q[:, :1].contiguous()
    Lk = p.shape[2]
    qm = q.clone()
    qm[..., :lo] = float("-inf")
    qm[..., hi:] = float("-inf")
    drafts = synth.draft_ids_from_logits(qm / temperature, top_k, seed * 100 + iteration)
    positions = torch.tensor([pos_base + 37 * b + iteration for b in range(B)], dtype=torch.int64,
                             device="cuda")
    cfg = scd.decode_config(mode=MODES[mode], batch=B, window_L=L, temperature=temperature,
                            top_k=top_k, cfg_lambda=lam, seed=seed, allowed_lo=lo, allowed_hi=hi,
                            row_period=row_period, eol_id=eol_id, alpha=alpha, top_p=top_p)
    got = scd.scd_verify(cfg, p, q if q_present else None, drafts, positions, iteration)
    torch.cuda.synchronize()
    n_commit, committed, next_drafts, flags = [t.cpu().numpy() for t in got]
    want = oracle_verify(mode, p.cpu().numpy(), q.cpu().numpy() if q_present else None,
                         drafts.cpu().numpy(), positions.cpu().numpy(), iteration, seed, temperature,
                         top_k, lam, lo, hi, row_period, eol_id, alpha, top_p)
    assert np.array_equal(n_commit, want["n_commit"]), (n_commit, want["n_commit"])
    assert np.array_equal(flags[:, :Lk], want["flags"])
    for b in range(B):
        a = int(n_commit[b])
        assert np.array_equal(committed[b, :a], want["committed"][b, :a])
    if mode != "ar":
        assert np.array_equal(next_drafts, want["next_drafts"])
    return n_commit


def test_noise_matches_oracle_bitwise():
    pos = torch.arange(0, 1_000_000, dtype=torch.int64, device="cuda") * 7 + 3
    got = scd.scd_noise_u24(0xDEADBEEF12345678, oracle.NOISE_RESIDUAL, 5, pos, 77, 2).cpu().numpy()
    idx = np.concatenate([np.arange(0, 2000), np.random.default_rng(0).integers(0, 1_000_000, 3000)])
    for i in idx:
        assert int(got[i]) == oracle.noise_u24(0xDEADBEEF12345678, oracle.NOISE_RESIDUAL, 5,
                                               int(pos[i]), 77, 2)
    hist = np.bincount(got.astype(np.int64) >> 18, minlength=64)
    chi2 = ((hist - 1e6 / 64) ** 2 / (1e6 / 64)).sum()
    assert chi2 < 63 + 5 * np.sqrt(126)


@pytest.mark.parametrize("B", [1, 2, 8])
def test_verify_workload_shape(B):
    # the verify-only workload: L = 32, V = 16384, temperature 1, top-k 2000
    iters = int(os.environ.get("SCD_VERIFY_ITERS", "12" if B < 8 else "4"))
    accepted = []
    for seed in (0, 1, 2):
        for it in range(iters):
            accepted.append(_run_case("scd", B, 32, 16384, it, seed, top_k=2000))
    mean_a = float(np.concatenate(accepted).mean())
    assert 1.0 <= mean_a <= 32.0


@pytest.mark.parametrize("mode", ["scd", "sjd", "ar"])
def test_verify_modes_small_ragged(mode):
    # ragged vocabulary (not a multiple of the CTA width), short window
    for it in range(6):
        _run_case(mode, 3, 5, 1000, it, seed=4, top_k=50)
        _run_case(mode, 2, 7, 33, it, seed=5, top_k=0)


@pytest.mark.parametrize("alpha", [0.0, 0.3, 0.75, 1.0])
def test_verify_alpha_coupling(alpha):
    # Algorithm 5: rows beyond the committed prefix keep the coupled redraft with probability alpha
    for it in range(8):
        _run_case("alpha", 3, 12, 1000, it, seed=21, top_k=50, alpha=alpha)
        _run_case("alpha", 2, 9, 257, it, seed=22, top_k=0, lam=1.5, alpha=alpha)


def test_verify_gumbel_sharing_coupling():
    # Algorithm 7: verify as Algorithm 1, redraft and fresh rows by the shared-noise Gumbel race
    for it in range(6):
        _run_case("gs", 3, 12, 1000, it, seed=31, top_k=50)
        _run_case("gs", 2, 9, 257, it, seed=32, top_k=0, lam=1.5, temperature=0.8)
        _run_case("gs", 2, 12, 777, it, seed=33, top_k=40, lo=10, hi=700, row_period=5, eol_id=720,
                  pos_base=0)
    _run_case("gs", 2, 8, 300, 0, seed=34, top_k=20, q_present=False)
    _run_case("gs", 1, 32, 16384, 1, seed=35, top_k=2000)
    _run_case("gs", 2, 6, 1500, 2, seed=36, top_k=100, quantise=0.5)     # equal weights: ties in the race


@pytest.mark.parametrize("top_p", [0.8, 0.3, 0.999, 1e-4])
def test_verify_nucleus_truncation(top_p):
    # top-p after top-k (and alone), on p and on the raw draft rows; ties from quantised logits
    for it in range(4):
        _run_case("scd", 2, 8, 4099, it, seed=41, top_k=300, top_p=top_p)
        _run_case("scd", 2, 8, 1000, it, seed=42, top_k=0, lam=1.5, temperature=0.8, top_p=top_p)
        _run_case("scd", 1, 6, 1500, it, seed=43, top_k=0, quantise=0.5, top_p=top_p)
    _run_case("gs", 2, 8, 777, 0, seed=44, top_k=0, top_p=top_p)
    _run_case("sjd", 2, 8, 777, 1, seed=45, top_k=50, top_p=top_p)
    _run_case("ar", 3, 1, 2048, 2, seed=46, top_k=0, top_p=top_p)
    _run_case("scd", 1, 64, 64000, 0, seed=47, top_k=0, top_p=top_p)      # the video setting's shape


def test_verify_cfg_temperature_and_allowed_range():
    for it in range(5):
        _run_case("scd", 2, 8, 4099, it, seed=7, temperature=0.7, top_k=300, lam=3.0, lo=101, hi=3000)
        _run_case("scd", 1, 16, 2048, it, seed=8, temperature=1.3, top_k=100, lam=1.5)


def test_verify_fresh_rows_and_forced_tokens():
    for it in range(4):
        _run_case("scd", 2, 12, 777, it, seed=9, top_k=40, q_present=False)
        _run_case("scd", 2, 12, 777, it, seed=10, top_k=40, lo=10, hi=700, row_period=5, eol_id=720,
                  pos_base=0)


def test_verify_ties_and_topk_edges():
    for it in range(4):
        _run_case("scd", 2, 6, 1500, it, seed=11, top_k=100, quantise=0.5)
        _run_case("scd", 1, 6, 600, it, seed=12, top_k=1)          # greedy: one-hot rows
        _run_case("scd", 1, 6, 600, it, seed=13, top_k=600)        # k = n: no threshold
        _run_case("scd", 1, 6, 600, it, seed=14, top_k=5000)       # k > n


def test_verify_large_vocab_and_max_window():
    _run_case("scd", 1, 64, 64000, 0, seed=15, top_k=1000)
    _run_case("scd", 1, 256, 512, 1, seed=16, top_k=20)


def test_verify_rejects_bad_arguments():
    cfg = scd.decode_config(batch=1, window_L=4, allowed_hi=10)
    p = torch.zeros(1, 1, 4, 10, device="cuda")
    d = torch.zeros(1, 4, dtype=torch.int32, device="cuda")
    pos = torch.zeros(1, dtype=torch.int64, device="cuda")
    for bad in (dict(window_L=0), dict(window_L=257), dict(batch=0), dict(temperature=0.0),
                dict(allowed_hi=11), dict(allowed_lo=10), dict(mode=9), dict(row_period=3, eol_id=10),
                dict(mode=scd.SCD_MODE_ALPHA, alpha=1.5), dict(mode=scd.SCD_MODE_ALPHA, alpha=-0.1)):
        kw = dict(batch=1, window_L=4, allowed_hi=10)
        kw.update(bad)
        with pytest.raises(scd.ScdError) as e:
            scd.scd_verify(scd.decode_config(**kw), p, None, d, pos, 0,
                           workspace=torch.zeros(1 << 16, dtype=torch.uint8, device="cuda"))
        assert e.value.code == scd.SCD_ERR_ARG
    # the context is still usable
    scd.scd_verify(cfg, p, None, d, pos, 0)
    torch.cuda.synchronize()


def test_verify_draft_without_mass_is_rejected():
    """Drafts that have no mass under p (outside its top-k; some outside q's as well, which X ~ q rules
    out but a caller can hand in): never accepted, the row's output comes from the residual."""
    B, L, V, top_k, seed = 2, 6, 2000, 20, 51
    p, q = synth.verify_logits(seed, 0, B, L, V, device="cuda")
    drafts = torch.argmin(p[0] + q, dim=-1).to(torch.int32)          # far below both thresholds
    drafts[0, 1] = torch.argmax(q[0, 1]).to(torch.int32)              # one ordinary row in between
    positions = torch.tensor([300, 900], dtype=torch.int64, device="cuda")
    cfg = scd.decode_config(mode=scd.SCD_MODE_SCD_MC, batch=B, window_L=L, top_k=top_k, seed=seed, allowed_hi=V)
    got = [t.cpu().numpy() for t in scd.scd_verify(cfg, p, q, drafts, positions, 3)]
    want = oracle_verify("scd", p.cpu().numpy(), q.cpu().numpy(), drafts.cpu().numpy(), positions.cpu().numpy(),
                         3, seed, 1.0, top_k)
    assert np.array_equal(got[0], want["n_commit"]) and np.array_equal(got[3], want["flags"])
    assert np.array_equal(got[2], want["next_drafts"])
    assert (got[3][:, 0] == 0).all() and (got[0] == 1).all()         # row 0 of both sequences rejects
    for b in range(B):
        assert got[1][b, 0] == want["committed"][b, 0] and got[1][b, 0] != drafts[b, 0].item()
