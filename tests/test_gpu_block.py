"""Algorithm 1 as one differentiable block (SP degree 1) on the library's kernels, against the float64 oracle
functions chained stage by stage.  The reference rounds to bf16 exactly where the block hands a bf16 tensor
from one entry point to the next, so that what is compared is the arithmetic inside the stages."""
import pytest
import torch

from parity import rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def block_mod():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2607_17644_b200 import laga
    laga.lib()
    from paper_2607_17644_b200 import block
    return block


def bf(t):
    return t.to(torch.float32).to(torch.bfloat16)


def reference(oracle, hidden, d_out, blk, cu, causal):
    """Forward and backward of Algorithm 1 (P = 1) from the oracle's pieces, float64 inside each stage."""
    H, DQK, DC, DV = blk.n_heads, 192, 512, 128
    w_q, w_kv_a, w_kv_b, w_o = (p.detach().cpu() for p in (blk.w_q, blk.w_kv_a, blk.w_kv_b, blk.w_o))
    gamma, beta = blk.ln_gamma.detach().cpu(), blk.ln_beta.detach().cpu()
    S = hidden.shape[0]
    scale = DQK ** -0.5
    q = bf(oracle.linear(hidden, w_q))
    kv_a = bf(oracle.linear(hidden, w_kv_a))
    pre = kv_a[:, :DC].contiguous()
    latent = bf(oracle.layernorm(pre, gamma, beta, blk.eps)[0])
    k_pe = kv_a[:, DC:].contiguous()
    q3 = q.view(S, H, DQK)
    out = torch.zeros(S, H, DV, dtype=torch.float64)
    seqs = list(zip(cu[:-1], cu[1:]))
    for a, b in seqs:
        out[a:b] = oracle.fwd(q3[a:b], latent[a:b], k_pe[a:b], w_kv_b, DV, scale, causal=causal, kv_round_bf16=True)[0]
    out_b = bf(out).reshape(S, H * DV)
    y = oracle.linear(out_b, w_o)
    # backward
    d_out2, d_w_o = oracle.linear_bwd(d_out, out_b, w_o)
    d_out3 = bf(d_out2).view(S, H, DV)
    dq = torch.zeros(S, H, DQK, dtype=torch.float64)
    dlat = torch.zeros(S, DC, dtype=torch.float64)
    dkpe = torch.zeros(S, 64, dtype=torch.float64)
    d_w_kv_b = torch.zeros_like(w_kv_b, dtype=torch.float64)
    for a, b in seqs:
        r = oracle.bwd(q3[a:b], latent[a:b], k_pe[a:b], w_kv_b, d_out3[a:b], DV, scale, causal=causal, kv_round_bf16=True)
        dq[a:b], dlat[a:b], dkpe[a:b] = r["dq"], r["dc_kv"], r["dk_pe"]
        d_w_kv_b += r["dw"]
    dpre, dgamma, dbeta = oracle.layernorm_bwd(bf(dlat), pre, gamma, blk.eps)
    d_kv_a = torch.cat([bf(dpre), bf(dkpe)], dim=1)
    dh1, d_w_q = oracle.linear_bwd(bf(dq).reshape(S, H * DQK), hidden, w_q)
    dh2, d_w_kv_a = oracle.linear_bwd(d_kv_a, hidden, w_kv_a)
    return {"y": y, "dh": bf(dh1).double() + bf(dh2).double(), "w_q": d_w_q, "w_kv_a": d_w_kv_a, "w_kv_b": d_w_kv_b,
            "w_o": d_w_o, "ln_gamma": dgamma, "ln_beta": dbeta}


@pytest.mark.parametrize("S,cu,causal", [(700, None, True), (900, [0, 300, 301, 900], True), (256, None, False)])
def test_block_forward_and_backward(block_mod, oracle, S, cu, causal):
    d_model, heads = 1024, 4
    blk = block_mod.LagaBlock(d_model, heads, seed=5)
    with torch.no_grad():                                   # non-trivial affine parameters of the norm
        g = torch.Generator().manual_seed(6)
        blk.ln_gamma.copy_((1 + 0.2 * torch.randn(512, generator=g)).to(torch.bfloat16))
        blk.ln_beta.copy_((0.1 * torch.randn(512, generator=g)).to(torch.bfloat16))
    g = torch.Generator().manual_seed(7 + S)
    hidden = torch.randn(S, d_model, generator=g).to(torch.bfloat16)
    d_out = torch.randn(S, d_model, generator=g).to(torch.bfloat16)
    h_dev = hidden.cuda().requires_grad_(True)
    y = blk(h_dev, cu_seqlens=cu, causal=causal)
    y.backward(d_out.cuda())
    ref = reference(oracle, hidden, d_out, blk, cu if cu is not None else [0, S], causal)
    assert rel_l2(y.detach().cpu().double(), ref["y"]) <= 1e-2
    assert rel_l2(h_dev.grad.cpu().double(), ref["dh"]) <= 1.5e-2
    for name in ("w_q", "w_kv_a", "w_kv_b", "w_o", "ln_gamma", "ln_beta"):
        got = getattr(blk, name).grad.cpu().double()
        # weight gradients reach autograd rounded to the bf16 of the weight
        assert rel_l2(got, ref[name]) <= 2e-2, name
    assert not torch.isnan(y.float()).any() and not torch.isnan(h_dev.grad.float()).any()
