"""torch.autograd plumbing around the C-ABI entry points: ``laga_attention(q, c_kv, k_pe, w_kv_b)`` is a
differentiable call whose forward is laga_fwd and whose backward is laga_bwd (Algorithm 1 steps 4-5 and
Section 5.2).  Nothing is computed here; the Function only keeps what the backward needs (the inputs, out
and LSE -- K_nope / V are recomputed, as in the library) and hands tensors over.

The weight gradient leaves the library in fp32 (it is a sum over the whole sequence that the SP group
reduces further); it is returned in the weight's dtype, as autograd requires, unless ``dw_fp32_out`` is
given, in which case the fp32 gradient is ADDED into that buffer (gradient accumulation across micro-batches
without a bf16 round trip) and autograd gets no gradient for the weight.
"""
from __future__ import annotations

import torch

from . import laga


class _LagaAttention(torch.autograd.Function):
    @staticmethod
    def forward(ctx, q, c_kv, k_pe, w_kv_b, causal, softmax_scale, dw_fp32_out, cu_seqlens, bwd_flags):
        out, lse, _ = laga.fwd(q, c_kv, k_pe, w_kv_b, softmax_scale=softmax_scale, causal=causal, cu_seqlens=cu_seqlens)
        ctx.save_for_backward(q, c_kv, k_pe, w_kv_b, out, lse)
        ctx.causal, ctx.softmax_scale, ctx.dw_fp32_out, ctx.cu_seqlens = causal, softmax_scale, dw_fp32_out, cu_seqlens
        ctx.bwd_flags = int(bwd_flags)
        ctx.mark_non_differentiable(lse)
        return out, lse

    @staticmethod
    def backward(ctx, dout, _dlse):
        q, c_kv, k_pe, w_kv_b, out, lse = ctx.saved_tensors
        acc = ctx.dw_fp32_out
        dq, dc_kv, dk_pe, dw, _ = laga.bwd(q, c_kv, k_pe, w_kv_b, out, lse, dout.contiguous(), softmax_scale=ctx.softmax_scale,
                                           causal=ctx.causal, dw_kv_b=acc,
                                           flags=ctx.bwd_flags | (laga.FLAG_ACCUM_DW if acc is not None else 0),
                                           cu_seqlens=ctx.cu_seqlens)
        return dq, dc_kv, dk_pe, (None if acc is not None else dw.to(w_kv_b.dtype)), None, None, None, None, None


def laga_attention(q, c_kv, k_pe, w_kv_b, causal=True, softmax_scale=None, dw_fp32_out=None, return_lse=False,
                   cu_seqlens=None, bwd_flags=0):
    """out[S,h,d_v] (and LSE) of one SP rank's head shard after the latent all-gather; differentiable in q, c_kv,
    k_pe and w_kv_b.  Inputs are contiguous bf16 CUDA tensors with the shapes of ``laga.fwd``.  With
    ``cu_seqlens`` (n_seqs + 1 host integers) the rows are packed sequences and attention stays inside each.
    ``bwd_flags``: flags for laga_bwd (``laga.FLAG_DETERMINISTIC``, ``laga.FLAG_FUSED_KV_REBUILD``, ...)."""
    cu = None if cu_seqlens is None else tuple(int(v) for v in (cu_seqlens.tolist() if isinstance(cu_seqlens, torch.Tensor)
                                                                  else cu_seqlens))
    out, lse = _LagaAttention.apply(q, c_kv, k_pe, w_kv_b, bool(causal), softmax_scale, dw_fp32_out, cu, int(bwd_flags))
    return (out, lse) if return_lse else out
