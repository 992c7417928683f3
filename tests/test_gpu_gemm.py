"""GPU numerics of the tcgen05 weight-streaming GEMM hook against an fp64 library matmul of the
same bf16 operands (products of bf16 values are exact in fp32; only the fp32 accumulation order
differs, so the tolerance is a few fp32 ulps of the accumulated magnitude)."""
import pytest
import torch

from paper_2510_24211_b200 import binding as scd

pytestmark = pytest.mark.gpu


def _check(M, N, K, seed=0, k_splits=0, stages=0):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    x = torch.randn(M, K, generator=g, device="cuda").to(torch.bfloat16)
    w = (torch.randn(N, K, generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    y = scd.scd_gemm_bf16(x, w, k_splits=k_splits, stages=stages)
    torch.cuda.synchronize()
    ref = x.double() @ w.double().T
    scale = (x.double().abs() @ w.double().abs().T).max().item()
    err = (y.double() - ref).abs().max().item()
    assert err <= 2e-6 * scale, (M, N, K, err, scale)
    # deterministic: split-K partials are added in a fixed order
    y2 = scd.scd_gemm_bf16(x, w, k_splits=k_splits, stages=stages)
    assert torch.equal(y, y2)


@pytest.mark.parametrize("M,N,K", [
    (64, 256, 128), (1, 128, 64), (16, 128, 4096), (37, 1000, 320), (64, 12288, 4096),
    (256, 512, 704), (17, 4096, 11008), (2, 16384, 1280), (64, 4096, 4096), (100, 8, 64),
])
def test_gemm_matches_fp64_matmul(M, N, K):
    _check(M, N, K)


@pytest.mark.parametrize("splits,stages", [(1, 2), (2, 3), (7, 4), (8, 2), (3, 12), (5, 3)])
def test_gemm_forced_slices_and_stages(splits, stages):
    _check(64, 1024, 2048, seed=splits, k_splits=splits, stages=stages)
    _check(48, 384, 512, seed=stages, k_splits=splits, stages=stages)


def test_gemm_rejects_bad_shapes():
    x = torch.zeros(4, 64, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(16, 64, dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    for (M, N, K) in [(0, 16, 64), (300, 16, 64), (4, 12, 64), (4, 16, 32), (4, 16, 96)]:
        rc = scd.lib().scd_gemm_bf16(x.data_ptr(), w.data_ptr(), ws.data_ptr(), M, N, K, ws.data_ptr(), None)
        assert rc == scd.SCD_ERR_SHAPE
    assert scd.scd_gemm_workspace_bytes(64, 4096, 4096) > 0
