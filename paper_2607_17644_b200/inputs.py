"""Seeded synthetic inputs for the LAGA hot path.

This module holds no arithmetic of the method: it only draws random tensors.  It is the one module
that both the CUDA path's tests/benchmark and the CPU oracle's callers use, so that both sides
consume identical bf16 bit patterns.

Recipe: a CPU ``torch.Generator`` seeded with ``seed``; fp32 normal draws in the fixed order
q, c_kv, k_pe, W_kv_b, dO; each rounded once (round-to-nearest-even) to bf16.  q, c_kv, k_pe and dO
are N(0,1); W_kv_b is N(0, variance 1/d_c), which makes the up-projected K_nope, V and the scaled
scores unit-variance.  c_kv stands in for the already-normalised gathered latent and q[..., d_nope:]
/ k_pe for already-rotated rope bands (Algorithm 1 step 1 happens before this path).
"""
from __future__ import annotations

import dataclasses
import math

import torch


@dataclasses.dataclass(frozen=True)
class LagaShape:
    """Problem size of one sequence-parallel rank after the latent all-gather."""
    S: int
    h: int
    d_c: int = 512
    d_nope: int = 128
    d_rope: int = 64
    d_v: int = 128

    @property
    def d_qk(self) -> int:
        return self.d_nope + self.d_rope

    @property
    def n_cols(self) -> int:
        """Columns of the W_kv_b head shard: per head d_nope K columns then d_v V columns."""
        return self.h * (self.d_nope + self.d_v)

    @property
    def softmax_scale(self) -> float:
        return 1.0 / math.sqrt(self.d_qk)


# The benchmark configurations (DeepSeek-V3 per-rank shard dims unless stated).
CONFIGS = {
    "c0": LagaShape(S=512, h=2),        # tiny forward
    "c1": LagaShape(S=4096, h=16),      # V3 shard, SP=8, forward
    "c2": LagaShape(S=16384, h=16),     # V3 shard, SP=8, forward+backward (headline)
    "c3_sp1": LagaShape(S=8192, h=128),
    "c3_sp2": LagaShape(S=8192, h=64),
    "c3_sp4": LagaShape(S=8192, h=32),
    "c3_sp8": LagaShape(S=8192, h=16),
    "c4": LagaShape(S=16384, h=16),     # the absorbed form on c2's inputs (same shapes, same seed)
}
CONFIG_SEEDS = {"c0": 1000, "c1": 1001, "c2": 1002, "c3_sp1": 1003, "c3_sp2": 1003, "c3_sp4": 1003,
                "c3_sp8": 1003, "c4": 1002}


def make_inputs(shape: LagaShape, seed: int, with_dout: bool = True, pin_memory: bool = False,
                h_generate: int | None = None):
    """Draw (q, c_kv, k_pe, w_kv_b, dout) as bf16 CPU tensors.

    ``h_generate`` (>= shape.h) draws the tensors for a wider head count and returns the first
    ``shape.h`` heads of it: that is how one rank's shard at several SP degrees is cut from the same
    full-head draw.
    """
    hg = shape.h if h_generate is None else h_generate
    assert hg >= shape.h
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    per_head = shape.d_nope + shape.d_v
    q = torch.randn(shape.S, hg, shape.d_qk, generator=g, dtype=torch.float32)
    c_kv = torch.randn(shape.S, shape.d_c, generator=g, dtype=torch.float32)
    k_pe = torch.randn(shape.S, shape.d_rope, generator=g, dtype=torch.float32)
    w = torch.randn(shape.d_c, hg * per_head, generator=g, dtype=torch.float32) / math.sqrt(shape.d_c)
    dout = torch.randn(shape.S, hg, shape.d_v, generator=g, dtype=torch.float32) if with_dout else None
    q = q[:, :shape.h].contiguous()
    w = w[:, :shape.h * per_head].contiguous()
    if dout is not None:
        dout = dout[:, :shape.h].contiguous()
    outs = [t.to(torch.bfloat16) if t is not None else None for t in (q, c_kv, k_pe, w, dout)]
    if pin_memory:
        outs = [t.pin_memory() if t is not None else None for t in outs]
    return tuple(outs)
