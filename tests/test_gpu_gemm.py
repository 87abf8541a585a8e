"""The tensor-core matrix product on its own, against a float64 product of the same bf16 inputs."""
import numpy as np
import pytest
import torch

from paper_2204_04179_b200 import binding

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def ctx():
    cfg = binding.GramConfig()
    cfg.n_items = 8
    cfg.P_max = 8
    cfg.d = 8
    return binding.Gram(cfg)


CASES = [  # M, N, K
    (128, 256, 64), (128, 64, 128), (256, 128, 192), (1000, 768, 768), (2048, 2304, 768), (777 * 8, 3072, 768),
    (520, 192, 64), (64, 64, 1024), (8, 8, 8), (768, 768, 40_000), (2304, 768, 20_000), (136, 1032, 72),
]


@pytest.mark.parametrize("a_k,b_k", [(1, 1), (1, 0), (0, 1), (0, 0)])
@pytest.mark.parametrize("M,N,K", CASES)
def test_gemm_bf16_all_layouts(M, N, K, a_k, b_k):
    g = ctx()
    gen = torch.Generator(device="cpu").manual_seed(M * 31 + N * 7 + K)
    A = (torch.randn(M, K, generator=gen) * 0.5).to(torch.bfloat16)
    B = (torch.randn(N, K, generator=gen) * 0.5).to(torch.bfloat16)
    bias = torch.randn(N, generator=gen)
    want = A.double() @ B.double().T + bias.double()
    Ad = (A if a_k else A.T.contiguous()).to(DEV)
    Bd = (B if b_k else B.T.contiguous()).to(DEV)
    for c_dtype in (torch.float32, torch.bfloat16):
        Cd = torch.full((M, N), float("nan"), dtype=c_dtype, device=DEV)
        g.gemm_bf16(Ad, a_k, Bd, b_k, Cd, bias.to(DEV), 0, M, N, K)
        g.sync()
        got = Cd.double().cpu()
        # fp32 accumulation of K products of bf16 values: error ~ K * 2^-24 * |a||b| plus the output rounding
        tol = 1e-4 * np.sqrt(K) + (0.0 if c_dtype == torch.float32 else 2.0 ** -8 * want.abs().max().item())
        assert torch.isfinite(got).all()
        assert (got - want).abs().max().item() <= tol, (c_dtype, (got - want).abs().max().item(), tol)
    # accumulate into fp32 C, twice, bit-identical across runs
    C1 = torch.ones(M, N, device=DEV)
    g.gemm_bf16(Ad, a_k, Bd, b_k, C1, None, 1, M, N, K)
    C2 = torch.ones(M, N, device=DEV)
    g.gemm_bf16(Ad, a_k, Bd, b_k, C2, None, 1, M, N, K)
    g.sync()
    assert torch.equal(C1, C2)
    assert (C1.double().cpu() - (want - bias.double() + 1.0)).abs().max().item() <= 1e-4 * np.sqrt(K)
    g.close()
