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


def _erf_gelu(v):
    import math
    phi = 0.5 * (1.0 + torch.erf(v / math.sqrt(2.0)))
    pdf = torch.exp(-0.5 * v * v) / math.sqrt(2.0 * math.pi)
    return v * phi, phi + v * pdf


# (M, N, K): full 256 x 256 pair tiles, ragged rows and columns, a small single-CTA shape, a wide N
EPI_SHAPES = [(512, 768, 768), (1000, 768, 3072), (296, 3072, 768), (136, 200, 72), (2048, 2304, 768), (264, 264, 64), (520, 1032, 128), (1288, 1096, 192)]


@pytest.mark.parametrize("M,N,K", EPI_SHAPES)
@pytest.mark.parametrize("kind", ["gelu", "dgelu", "res", "res_ln", "res_ln_copy", "bias_f32", "plain_bf16"])
def test_gemm_epilogues_against_float64(M, N, K, kind):
    """Every fused epilogue the layers use, element by element against float64 arithmetic on the same bf16 inputs."""
    g = ctx()
    gen = torch.Generator(device="cpu").manual_seed(M + 3 * N + 7 * K)
    A = (torch.randn(M, K, generator=gen) * 0.5).to(torch.bfloat16)
    b_k = 0 if kind in ("dgelu", "res") else 1            # the input-gradient products read W as [K, N]
    B = (torch.randn(N, K, generator=gen) * (2.0 / np.sqrt(K))).to(torch.bfloat16)
    acc = A.double() @ B.double().T
    Bd = (B if b_k else B.T.contiguous()).to(DEV)
    Ad = A.to(DEV)
    bias = torch.randn(N, generator=gen) * 0.3
    kw, want, want2 = {}, None, None
    c_f32 = kind in ("res", "res_ln", "res_ln_copy", "bias_f32")
    Cd = torch.full((M, N), float("nan"), dtype=torch.float32 if c_f32 else torch.bfloat16, device=DEV)
    out2 = None
    if kind == "gelu":
        out2 = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=DEV)
        kw = dict(bias=bias.to(DEV), gelu=True, gelu_grad_out=out2)
        want, want2 = _erf_gelu(acc + bias.double())
    elif kind == "dgelu":
        dg = torch.rand(M, N, generator=gen).to(torch.bfloat16)
        kw = dict(gelu_grad_in=dg.to(DEV))
        want = acc * dg.double()
    elif kind == "res":
        res = torch.randn(M, N, generator=gen)
        kw = dict(res=res.to(DEV))
        want = acc + res.double()
    elif kind in ("res_ln", "res_ln_copy"):
        res = torch.randn(M, N, generator=gen) * 2 + 0.5
        mean = res.double().mean(1); rstd = 1.0 / torch.sqrt(res.double().var(1, unbiased=False) + 1e-5)
        gamma = torch.rand(N, generator=gen) + 0.5; beta = torch.randn(N, generator=gen) * 0.2
        kw = dict(bias=bias.to(DEV), res=res.to(DEV), res_ln=(mean.float().to(DEV), rstd.float().to(DEV), gamma.to(DEV), beta.to(DEV)))
        want = acc + bias.double() + (res.double() - mean.float().double()[:, None]) * rstd.float().double()[:, None] * gamma.double() + beta.double()
        if kind == "res_ln_copy":
            out2 = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=DEV)
            kw["copy_bf16"] = out2
            want2 = want
    elif kind == "bias_f32":
        kw = dict(bias=bias.to(DEV))
        want = acc + bias.double()
    else:
        want = acc
    g.gemm_bf16_epilogue(Ad, 1, Bd, b_k, Cd, M, N, K, **kw)
    g.sync()
    got = Cd.double().cpu()
    assert torch.isfinite(got).all()
    scale = want.abs().max().item()
    tol = 1e-4 * np.sqrt(K) + 2e-6 * scale + (0.0 if c_f32 else 2.0 ** -8 * scale)
    if kind == "gelu":
        tol += 4e-7 * scale + 2e-6            # the kernel's erf is a rational approximation good to 1.5e-7
    assert (got - want).abs().max().item() <= tol, ((got - want).abs().max().item(), tol)
    if want2 is not None:
        got2 = out2.double().cpu()
        s2 = want2.abs().max().item()
        assert torch.isfinite(got2).all()
        assert (got2 - want2).abs().max().item() <= 1e-4 * np.sqrt(K) + 2.0 ** -8 * s2 + 1e-5, (got2 - want2).abs().max().item()
    # a second launch gives bit-identical results
    Ce = torch.empty_like(Cd)
    kw2 = dict(kw)
    if "gelu_grad_out" in kw2:
        kw2["gelu_grad_out"] = torch.empty_like(out2)
    if "copy_bf16" in kw2:
        kw2["copy_bf16"] = torch.empty_like(out2)
    g.gemm_bf16_epilogue(Ad, 1, Bd, b_k, Ce, M, N, K, **kw2)
    g.sync()
    assert torch.equal(Cd, Ce)
    g.close()
