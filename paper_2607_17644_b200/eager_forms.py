"""Comparison forms of the same attention block in plain PyTorch ops -- COMPARATORS, not the product.

The paper contrasts three ways of running MLA attention under sequence parallelism (Section 3.2):
the explicit form B1 (per-head K/V materialised), the absorbed form B2 (W_uk folded into the query,
attention in latent space, W_uv applied last) and LAGA, whose per-rank compute equals B1's.  Its
memory study ran B1 and B2 as eager PyTorch (full S x S scores).  This module does the same on one
GPU with library kernels (torch.matmul / softmax, i.e. cuBLAS and ATen) and autograd, so that
``bench.py --compare-eager`` can report their time and peak activation memory beside the CUDA path.
Nothing here is used by laga_fwd / laga_bwd.

Both forms take the hot path's inputs (same layouts as the C ABI; any float dtype, so the CPU test
can run them in fp64) and return out [S,h,d_v]; ``run_form`` adds the backward through autograd.
"""
from __future__ import annotations

import torch


def _split_w(w_kv_b: torch.Tensor, h: int, d_nope: int, d_v: int):
    w3 = w_kv_b.view(w_kv_b.shape[0], h, d_nope + d_v)
    return w3[:, :, :d_nope], w3[:, :, d_nope:]          # W_uk [d_c,h,d_nope], W_uv [d_c,h,d_v]


def _causal_softmax(scores: torch.Tensor, causal: bool) -> torch.Tensor:
    if causal:
        S = scores.shape[-1]
        mask = torch.ones(S, S, dtype=torch.bool, device=scores.device).triu_(1)
        scores = scores.masked_fill(mask, float("-inf"))
    return torch.softmax(scores, dim=-1)


def explicit_form(q, c_kv, k_pe, w_kv_b, d_v: int, softmax_scale: float, causal: bool = True):
    """B1's per-rank compute in eager ops: K_nope, V per head, full score matrix."""
    S, h, d_qk = q.shape
    d_rope = k_pe.shape[1]
    d_nope = d_qk - d_rope
    w_uk, w_uv = _split_w(w_kv_b, h, d_nope, d_v)
    k_nope = torch.einsum("tc,chd->htd", c_kv, w_uk)
    v = torch.einsum("tc,chd->htd", c_kv, w_uv)
    k = torch.cat([k_nope, k_pe.unsqueeze(0).expand(h, -1, -1)], dim=-1)
    scores = torch.matmul(q.transpose(0, 1), k.transpose(1, 2)) * softmax_scale      # [h,S,S]
    p = _causal_softmax(scores, causal)
    return torch.matmul(p, v).transpose(0, 1)                                        # [S,h,d_v]


def absorbed_form(q, c_kv, k_pe, w_kv_b, d_v: int, softmax_scale: float, causal: bool = True):
    """B2 in eager ops: q_abs = W_uk q_nope lives in h*d_c dims, scores are taken against the latent
    itself, the accumulator is h*d_c wide and W_uv comes last."""
    S, h, d_qk = q.shape
    d_rope = k_pe.shape[1]
    d_nope = d_qk - d_rope
    w_uk, w_uv = _split_w(w_kv_b, h, d_nope, d_v)
    q_abs = torch.einsum("shd,chd->hsc", q[..., :d_nope], w_uk)                       # [h,S,d_c]
    scores = (torch.matmul(q_abs, c_kv.t()) +
              torch.matmul(q[..., d_nope:].transpose(0, 1), k_pe.t())) * softmax_scale  # [h,S,S]
    p = _causal_softmax(scores, causal)
    latent_acc = torch.matmul(p, c_kv)                                                # [h,S,d_c]
    return torch.einsum("hsc,chd->shd", latent_acc, w_uv)


def run_form(form, q, c_kv, k_pe, w_kv_b, dout, d_v: int, softmax_scale: float, causal: bool = True):
    """Forward + backward of one form with autograd.  Returns (out, dq, dc_kv, dk_pe, dw_kv_b)."""
    leaves = [t.detach().clone().requires_grad_(True) for t in (q, c_kv, k_pe, w_kv_b)]
    out = form(*leaves, d_v, softmax_scale, causal)
    out.backward(dout)
    return (out.detach(),) + tuple(t.grad for t in leaves)
