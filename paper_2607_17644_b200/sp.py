"""The sequence-parallel exchanges around the per-rank hot path (Algorithm 1 steps 2, 3 and 6, and the
backward duals of Section 5.2), over ``torch.distributed``.

Rank r of P owns S/P consecutive tokens of every tensor outside the attention block and the head
shard H_r = {r n_h/P, ..., (r+1) n_h/P - 1} inside it:

  step 2   head-scatter all-to-all of q            [S/P, n_h, d_qk]   -> [S, n_h/P, d_qk]
  step 3   sequence all-gather of latent, k_pe     [S/P, d_c], [S/P, d_rope] -> [S, d_c], [S, d_rope]
  step 4-5 the hot path on the rank's head shard   (``compute.fwd``: laga_fwd on the GPU)
  step 6   sequence-scatter all-to-all of out      [S, n_h/P, d_v]    -> [S/P, n_h, d_v]

Backward: the gradient of step 6 is a head-scatter all-to-all of d_out, the gradient of step 2 a
sequence-scatter all-to-all of dq, the gradient of step 3 a reduce-scatter of the ranks' partial
dc_kv and dk_pe, and the W_kv_b gradient -- complete for H_r's columns on rank r, zero elsewhere --
is summed over the group (an all-gather of the column shards).  Only the exchanges are here; every contraction is in ``compute``.

No kernel of this repository reads peer memory: a gathered tensor lands in this GPU's memory first
and the hot path reads it from there.  On this build's single-GPU test pool the exchanges are covered
by world_size-2 ``gloo`` tests on the CPU with a stand-in ``compute``, and with world size 1 on the GPU.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch
import torch.distributed as dist


# ---- communication volume (Section 4, Evaluation: communication-volume table) --------------------
@dataclass(frozen=True)
class CommDims:
    n_h: int = 128
    d_nope: int = 128
    d_rope: int = 64
    d_v: int = 128
    d_c: int = 512


def comm_bytes_per_rank(form: str, S: int, P: int, dims: CommDims = CommDims()) -> int:
    """Bytes one rank sends in one forward pass, by the closed form that reproduces every printed cell
    of the paper's communication table: an all-to-all sends the (P-1)/P part of the rank's S/P tokens
    that belongs to other ranks, counted at 4 bytes per element; the all-gather contributes the
    rank's own S/P x (d_c + d_rope) shard once, at 2 bytes per element.  (The table's numbers need
    exactly these element sizes; the paper does not say why they differ.)

    ``explicit`` (B1): all-to-alls of q, of K as the full d_nope + d_rope key per head, of V and of out.
    ``laga`` and ``absorbed`` (B2): all-to-alls of q and out, all-gather of latent and k_pe.
    """
    tokens = S // P
    d_qk = dims.d_nope + dims.d_rope
    if form == "explicit":
        per_token = dims.n_h * (d_qk + d_qk + dims.d_v + dims.d_v)
        return 4 * tokens * per_token * (P - 1) // P
    if form in ("laga", "absorbed"):
        per_token = dims.n_h * (d_qk + dims.d_v)
        return 4 * tokens * per_token * (P - 1) // P + 2 * tokens * (dims.d_c + dims.d_rope)
    raise ValueError(f"unknown form {form!r}")


# ---- the exchanges -------------------------------------------------------------------------------
def _world(group):
    return dist.get_world_size(group), dist.get_rank(group)


def head_scatter_all_to_all(x: torch.Tensor, group=None) -> torch.Tensor:
    """[S/P, n_h, d] (my tokens, all heads) -> [S, n_h/P, d] (all tokens, my heads).  Step 2; also the
    gradient of step 6."""
    P, _ = _world(group)
    s_loc, n_h, d = x.shape
    assert n_h % P == 0, "the head count must be a multiple of the SP degree"
    h = n_h // P
    send = x.reshape(s_loc, P, h, d).permute(1, 0, 2, 3).contiguous()      # [P (destination), S/P, h, d]
    recv = torch.empty_like(send)                                          # [P (source), S/P, h, d]
    dist.all_to_all_single(recv, send, group=group)
    return recv.reshape(P * s_loc, h, d)


def seq_scatter_all_to_all(x: torch.Tensor, group=None) -> torch.Tensor:
    """[S, n_h/P, d] (all tokens, my heads) -> [S/P, n_h, d] (my tokens, all heads).  Step 6; also the
    gradient of step 2."""
    P, _ = _world(group)
    S, h, d = x.shape
    assert S % P == 0, "the sequence length must be a multiple of the SP degree"
    s_loc = S // P
    send = x.reshape(P, s_loc, h, d).contiguous()                          # [P (destination), S/P, h, d]
    recv = torch.empty_like(send)                                          # [P (source = head shard), S/P, h, d]
    dist.all_to_all_single(recv, send, group=group)
    return recv.permute(1, 0, 2, 3).reshape(s_loc, P * h, d).contiguous()


def seq_all_gather(x: torch.Tensor, group=None) -> torch.Tensor:
    """[S/P, d] -> [S, d].  Step 3."""
    P, _ = _world(group)
    out = torch.empty((P * x.shape[0],) + tuple(x.shape[1:]), dtype=x.dtype, device=x.device)
    dist.all_gather_into_tensor(out, x.contiguous(), group=group)
    return out


def seq_reduce_scatter(x: torch.Tensor, group=None) -> torch.Tensor:
    """[S, d] partial sums on every rank -> [S/P, d] complete sums of my tokens.  Gradient of step 3."""
    P, _ = _world(group)
    assert x.shape[0] % P == 0
    out = torch.empty((x.shape[0] // P,) + tuple(x.shape[1:]), dtype=x.dtype, device=x.device)
    dist.reduce_scatter_tensor(out, x.contiguous(), group=group)
    return out


def shard_columns(w_kv_b: torch.Tensor, n_h: int, group=None) -> torch.Tensor:
    """This rank's head shard of W_kv_b [d_c, n_h (d_nope + d_v)]: heads are interleaved per head, so the
    shard is a contiguous column slice."""
    P, r = _world(group)
    per_head = w_kv_b.shape[1] // n_h
    h = n_h // P
    return w_kv_b[:, r * h * per_head:(r + 1) * h * per_head].contiguous()


def all_gather_dw(dw_shard: torch.Tensor, n_h: int, group=None) -> torch.Tensor:
    """The head-axis reduction of the W_kv_b gradient (Section 5.2).  Rank r's gradient is complete for H_r's
    columns of the replicated W_kv_b and identically zero elsewhere, so the sum over the group is the
    concatenation of the column shards: an all-gather moves 1/P of what an all-reduce of zero-padded full
    matrices would.  Returns the full [d_c, n_h (d_nope + d_v)] gradient (identical on every rank)."""
    P, _ = _world(group)
    d_c, cols = dw_shard.shape
    gathered = torch.empty(P * d_c, cols, dtype=dw_shard.dtype, device=dw_shard.device)   # rank-major row blocks
    dist.all_gather_into_tensor(gathered, dw_shard.contiguous(), group=group)
    return gathered.view(P, d_c, cols).permute(1, 0, 2).reshape(d_c, P * cols).contiguous()


# ---- one attention block under SP ----------------------------------------------------------------
class CudaCompute:
    """Steps 4-5 and their backward on the GPU: the C-ABI entry points laga_fwd / laga_bwd."""

    def __init__(self):
        from . import laga
        self._laga = laga

    def fwd(self, q, c_kv, k_pe, w, causal):
        out, lse, ws = self._laga.fwd(q, c_kv, k_pe, w, causal=causal)
        self._laga.check_status(ws, where="laga_fwd")
        return out, lse

    def bwd(self, q, c_kv, k_pe, w, out, lse, dout, causal):
        dq, dc_kv, dk_pe, dw, ws = self._laga.bwd(q, c_kv, k_pe, w, out, lse, dout, causal=causal)
        self._laga.check_status(ws, where="laga_bwd")
        return dq, dc_kv, dk_pe, dw


def sp_forward(q_local, c_kv_local, k_pe_local, w_kv_b, n_h, compute, causal=True, group=None):
    """Algorithm 1 steps 2-6 on this rank.  Returns out_local [S/P, n_h, d_v] and the context the
    backward needs (the gathered operands, this rank's shard of the weights, out and LSE)."""
    q = head_scatter_all_to_all(q_local, group)
    c_kv = seq_all_gather(c_kv_local, group)
    k_pe = seq_all_gather(k_pe_local, group)
    w = shard_columns(w_kv_b, n_h, group)
    out, lse = compute.fwd(q, c_kv, k_pe, w, causal)
    ctx = (q, c_kv, k_pe, w, out, lse, causal, n_h)
    return seq_scatter_all_to_all(out, group), ctx


def sp_backward(ctx, dout_local, compute, group=None):
    """Backward of ``sp_forward``: returns dq_local [S/P, n_h, d_qk], dc_kv_local [S/P, d_c],
    dk_pe_local [S/P, d_rope] and the full dW_kv_b [d_c, n_h (d_nope + d_v)] (identical on every rank)."""
    q, c_kv, k_pe, w, out, lse, causal, n_h = ctx
    dout = head_scatter_all_to_all(dout_local, group)
    dq, dc_kv, dk_pe, dw = compute.bwd(q, c_kv, k_pe, w, out, lse, dout, causal)
    return (seq_scatter_all_to_all(dq, group), seq_reduce_scatter(dc_kv, group), seq_reduce_scatter(dk_pe, group),
            all_gather_dw(dw, n_h, group))
