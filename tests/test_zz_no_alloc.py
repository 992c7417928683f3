"""scd_verify_noalloc: the verify-and-redraft call for hosts that must not allocate.

A serving process that has given all device memory to its own pool, or that sits in a section
where cudaMalloc would stall the device or fail, cannot hand scd_verify a freshly allocated
workspace. scd_verify_noalloc takes its scratch from a 16 MiB buffer built into the library
instead. This file checks, through the C ABI, that it returns exactly what scd_verify returns
(integer outputs: bit-exact, the bar of the other verify tests) on two calls in a row - the
second call finds the first call's leftovers in the shared buffer - and that a request too
large for the buffer is refused without launching anything.

Collected last on purpose (file name), so that a run stopping at the first failure has already
run every other test. It needs no state from other tests: every tensor is created here, before
the calls, and the calls themselves allocate nothing."""
import numpy as np
import pytest
import torch

from helpers import oracle_verify
from paper_2510_24211_b200 import binding as scd
from paper_2510_24211_b200 import synth

pytestmark = pytest.mark.gpu


def _case(seed, iteration, B, L, V, top_k, lam=0.0):
    S = 2 if lam != 0.0 else 1
    p, q = synth.verify_logits(seed, iteration, B, L, V, device="cuda", streams=S)
    drafts = synth.draft_ids_from_logits(q, top_k, seed * 100 + iteration)
    positions = torch.tensor([500 + 41 * b + iteration for b in range(B)], dtype=torch.int64, device="cuda")
    cfg = scd.decode_config(mode=scd.SCD_MODE_SCD_MC, batch=B, window_L=L, temperature=1.0, top_k=top_k,
                            cfg_lambda=lam, seed=seed, allowed_lo=0, allowed_hi=V)
    return cfg, p, q, drafts, positions


def _outputs(B, L):
    return (torch.full((B,), -1, dtype=torch.int32, device="cuda"),
            torch.zeros(B, L, dtype=torch.int32, device="cuda"),
            torch.full((B, L), -1, dtype=torch.int32, device="cuda"),
            torch.zeros(B, L, dtype=torch.uint8, device="cuda"))


def test_noalloc_matches_scd_verify_twice_in_a_row():
    assert scd.scd_verify_noalloc_max_bytes() == 16 << 20
    # two different problems back to back: the second one reuses the buffer the first one dirtied
    for it, (B, L, V, top_k, lam) in enumerate([(2, 32, 16384, 2000, 0.0), (1, 16, 4096, 100, 1.5)]):
        cfg, p, q, drafts, positions = _case(seed=5, iteration=it, B=B, L=L, V=V, top_k=top_k, lam=lam)
        assert scd.scd_verify_workspace_bytes(cfg, V) <= scd.scd_verify_noalloc_max_bytes()
        want = scd.scd_verify(cfg, p, q, drafts, positions, it)
        torch.cuda.synchronize()
        out = _outputs(B, L)
        got = scd.scd_verify_noalloc(cfg, p, q, drafts, positions, it, out)
        torch.cuda.synchronize()
        a = int(want[0][0])
        assert torch.equal(got[0], want[0])                       # tokens committed
        assert torch.equal(got[3], want[3])                       # accept flag of every row
        assert torch.equal(got[2], want[2])                       # next drafts
        for b in range(B):
            a = int(want[0][b])
            assert torch.equal(got[1][b, :a], want[1][b, :a])     # committed ids (first a are defined)
        # same call again on the same inputs: same answer (nothing left over changes it), and - the
        # first call on this device being behind us - no device memory is taken by the call
        out2 = _outputs(B, L)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        got2 = scd.scd_verify_noalloc(cfg, p, q, drafts, positions, it, out2)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before
        assert torch.equal(got2[0], want[0]) and torch.equal(got2[2], want[2]) and torch.equal(got2[3], want[3])
        # and against the CPU oracle, like every other verify test
        ref = oracle_verify("scd", p.cpu().numpy(), q.cpu().numpy(), drafts.cpu().numpy(), positions.cpu().numpy(),
                            it, 5, 1.0, top_k, lam)
        assert np.array_equal(got2[0].cpu().numpy(), ref["n_commit"])
        assert np.array_equal(got2[3].cpu().numpy(), ref["flags"])
        assert np.array_equal(got2[2].cpu().numpy(), ref["next_drafts"])
        for b in range(B):
            a = int(ref["n_commit"][b])
            assert np.array_equal(got2[1][b, :a].cpu().numpy(), ref["committed"][b, :a])


def test_noalloc_refuses_what_does_not_fit():
    B, L, V = 8, 32, 16384                                        # 16 MiB of rows alone, plus bookkeeping
    cfg, p, q, drafts, positions = _case(seed=1, iteration=0, B=B, L=L, V=V, top_k=2000)
    assert scd.scd_verify_workspace_bytes(cfg, V) > scd.scd_verify_noalloc_max_bytes()
    out = _outputs(B, L)
    with pytest.raises(scd.ScdError) as e:
        scd.scd_verify_noalloc(cfg, p, q, drafts, positions, 0, out)
    assert e.value.code == scd.SCD_ERR_CAPACITY
    torch.cuda.synchronize()
    assert int(out[0][0]) == -1                                   # nothing ran
    # the context is still usable and the buffer still works
    cfg, p, q, drafts, positions = _case(seed=2, iteration=0, B=1, L=8, V=1024, top_k=0)
    want = scd.scd_verify(cfg, p, q, drafts, positions, 0)
    got = scd.scd_verify_noalloc(cfg, p, q, drafts, positions, 0, _outputs(1, 8))
    torch.cuda.synchronize()
    assert torch.equal(got[0], want[0]) and torch.equal(got[3], want[3])
