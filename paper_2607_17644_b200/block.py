"""Algorithm 1 of the paper as one differentiable block for SP degree 1 (no exchange steps), with every
step executed by the library's kernels:

  step 1   q = W_q(h);  latent, k_pe = W_kv_a(h);  latent = LayerNorm(latent)      laga_linear x2, laga_layernorm
  step 4-5 K_nope/V up-projection of the head shard and causal softmax attention   laga_fwd / laga_bwd
  step 7   W_o(reshape(out))                                                        laga_linear

Steps 2, 3 and 6 are the sequence-parallel exchanges (``sp.py``); with one rank they are the identity.
This module is torch.autograd plumbing only: three ``autograd.Function``s that hand tensors to the C ABI
entry points and a module that owns the block's weights.  As in Algorithm 1, q_rope and k_pe are taken as
the projections deliver them (the paper's algorithm has no rotary step of its own).

Weights are stored as [in_features, out_features] (y = x W), the layout ``W_kv_b`` already has.  Weight
gradients leave the kernels in fp32 and are handed to autograd in the weight's dtype.
"""
from __future__ import annotations

import torch

from . import laga
from .autograd import laga_attention


class _Linear(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, w):
        y, status = laga.linear(x, w)
        ctx.save_for_backward(x, w)
        return y

    @staticmethod
    def backward(ctx, dy):
        x, w = ctx.saved_tensors
        dx, dw, _ = laga.linear_backward(dy.contiguous(), x, w)
        return dx, dw.to(w.dtype)


class _LayerNorm(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, gamma, beta, eps):
        y, mean, rstd = laga.layernorm(x, gamma, beta, eps)
        ctx.save_for_backward(x, gamma, mean, rstd)
        ctx.has_beta = beta is not None
        return y

    @staticmethod
    def backward(ctx, dy):
        x, gamma, mean, rstd = ctx.saved_tensors
        dx, dgamma, dbeta = laga.layernorm_backward(dy.contiguous(), x, gamma, mean, rstd, with_beta=ctx.has_beta)
        return dx, dgamma.to(gamma.dtype), (dbeta.to(gamma.dtype) if ctx.has_beta else None), None


def linear(x: torch.Tensor, w: torch.Tensor) -> torch.Tensor:
    """y[M, N] = x[M, K] . w[K, N] through laga_linear / laga_linear_backward (bf16 CUDA tensors)."""
    return _Linear.apply(x, w)


def layernorm(x: torch.Tensor, gamma: torch.Tensor, beta=None, eps: float = 1e-5) -> torch.Tensor:
    """LayerNorm over the last axis through laga_layernorm / laga_layernorm_backward (bf16 CUDA tensors)."""
    return _LayerNorm.apply(x, gamma, beta, eps)


class LagaBlock(torch.nn.Module):
    """hidden [S, d_model] -> [S, d_model]: Algorithm 1 with P = 1 for ``n_heads`` heads of the DeepSeek-V3
    geometry (d_nope 128, d_rope 64, d_v 128, d_c 512).  ``forward(hidden, cu_seqlens=None)``: with
    ``cu_seqlens`` the rows are packed sequences and attention stays inside each."""

    D_NOPE, D_ROPE, D_V, D_C = 128, 64, 128, 512

    def __init__(self, d_model: int, n_heads: int, eps: float = 1e-5, device="cuda", seed: int = 0):
        super().__init__()
        g = torch.Generator().manual_seed(seed)

        def weight(k, n):     # variance-preserving draw, rounded once to bf16
            return torch.nn.Parameter((torch.randn(k, n, generator=g) * k ** -0.5).to(torch.bfloat16).to(device))

        d_qk = self.D_NOPE + self.D_ROPE
        self.n_heads, self.eps = n_heads, eps
        self.w_q = weight(d_model, n_heads * d_qk)
        self.w_kv_a = weight(d_model, self.D_C + self.D_ROPE)
        self.w_kv_b = weight(self.D_C, n_heads * (self.D_NOPE + self.D_V))
        self.w_o = weight(n_heads * self.D_V, d_model)
        self.ln_gamma = torch.nn.Parameter(torch.ones(self.D_C, dtype=torch.bfloat16, device=device))
        self.ln_beta = torch.nn.Parameter(torch.zeros(self.D_C, dtype=torch.bfloat16, device=device))

    def forward(self, hidden: torch.Tensor, cu_seqlens=None, causal: bool = True) -> torch.Tensor:
        S = hidden.shape[0]
        q = linear(hidden, self.w_q).view(S, self.n_heads, self.D_NOPE + self.D_ROPE)            # step 1
        kv_a = linear(hidden, self.w_kv_a)
        latent = layernorm(kv_a[:, :self.D_C].contiguous(), self.ln_gamma, self.ln_beta, self.eps)
        k_pe = kv_a[:, self.D_C:].contiguous()
        out = laga_attention(q, latent, k_pe, self.w_kv_b, causal=causal, cu_seqlens=cu_seqlens)   # steps 4-5
        return linear(out.reshape(S, self.n_heads * self.D_V), self.w_o)                          # step 7
