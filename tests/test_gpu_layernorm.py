"""GPU parity of laga_layernorm / laga_layernorm_backward (Algorithm 1 step 1: LayerNorm of the latent) against
the float64 oracle."""
import pytest
import torch

from parity import rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def laga():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2607_17644_b200 import laga as _laga
    _laga.lib()
    return _laga


def draw(M, D, seed):
    """The latent before its norm: rows of order one with a per-row offset and spread (what a projection of a
    residual stream gives); gamma near one, beta near zero; upstream gradient ~ N(0,1)."""
    g = torch.Generator().manual_seed(seed)
    x = (torch.randn(M, D, generator=g) * (0.5 + torch.rand(M, 1, generator=g) * 2) + torch.randn(M, 1, generator=g)).to(torch.bfloat16)
    gamma = (1 + 0.2 * torch.randn(D, generator=g)).to(torch.bfloat16)
    beta = (0.1 * torch.randn(D, generator=g)).to(torch.bfloat16)
    dy = torch.randn(M, D, generator=g).to(torch.bfloat16)
    return x, gamma, beta, dy


@pytest.mark.parametrize("M,D,with_beta", [(4096, 512, True), (1000, 512, False), (1, 512, True), (77, 8, True),
                                           (300, 1024, True), (513, 264, True), (20000, 512, True)])
def test_layernorm_forward_and_backward(laga, oracle, M, D, with_beta):
    x, gamma, beta, dy = draw(M, D, 8000 + M + D)
    eps = 1e-5
    rows = slice(None) if M <= 4096 else torch.randperm(M, generator=torch.Generator().manual_seed(1))[:512]
    y, mean, rstd = laga.layernorm(x.cuda(), gamma.cuda(), beta.cuda() if with_beta else None, eps,
                                   y=torch.full((M, D), float("nan"), dtype=torch.bfloat16, device="cuda"))
    dx, dgamma, dbeta = laga.layernorm_backward(dy.cuda(), x.cuda(), gamma.cuda(), mean, rstd, with_beta=with_beta,
                                                dx=torch.full((M, D), float("nan"), dtype=torch.bfloat16, device="cuda"))
    ry, rmean, rrstd = oracle.layernorm(x[rows], gamma, beta if with_beta else None, eps)
    # bf16 outputs of order one: one rounding (2^-9 relative) on top of fp32 arithmetic
    assert float((y.cpu().double()[rows] - ry).abs().max()) <= 2e-2 and rel_l2(y.cpu().double()[rows], ry) <= 3e-3
    assert float((mean.cpu().double()[rows] - rmean).abs().max()) <= 1e-5
    assert float(((rstd.cpu().double()[rows] - rrstd) / rrstd).abs().max()) <= 1e-5
    rdx, rdgamma, rdbeta = oracle.layernorm_bwd(dy[rows], x[rows], gamma, eps)
    assert rel_l2(dx.cpu().double()[rows], rdx) <= 3e-3
    assert float((dx.cpu().double()[rows] - rdx).abs().max()) <= 2e-2 * max(1.0, float(rdx.abs().max()))
    if M <= 4096:                                    # the column sums need every row
        assert rel_l2(dgamma.cpu().double(), rdgamma) <= 1e-5
        if with_beta:
            assert rel_l2(dbeta.cpu().double(), rdbeta) <= 1e-5
        else:
            assert dbeta is None
    assert not torch.isnan(y.float()).any() and not torch.isnan(dx.float()).any()


def test_layernorm_rejects_unsupported_widths(laga):
    x = torch.zeros(4, 2048, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(laga.LagaError):
        laga.layernorm(x, torch.ones(2048, dtype=torch.bfloat16, device="cuda"))
    x = torch.zeros(4, 20, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(laga.LagaError):
        laga.layernorm(x, torch.ones(20, dtype=torch.bfloat16, device="cuda"))
