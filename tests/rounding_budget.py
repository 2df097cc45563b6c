"""How far from the fp64 oracle must ANY bf16-operand tensor-core implementation of the path land?

This script answers that on the CPU, without any GPU code: it evaluates the explicit MLA form of
Algorithm 1 steps 4-5 and the backward of Section 5.2 in float64 and inserts a round-to-bf16 at exactly
the places where a tensor-core path needs a bf16 operand or writes a bf16 result:

    K_nope, V (step 4 output)        P (operand of P V and of dV = P^T dO)      O (output; enters delta)
    dS (operand of dQ and dK)        dK_nope, dV (operands of dc_kv and dW)     dQ, dc_kv, dk_pe (outputs)

Everything else (scores, softmax statistics, all accumulations, dW) stays float64, i.e. BETTER than any
real kernel.  The distance of that model from the oracle (`oracle.bwd`, the only reference this script
calls) is the rounding budget: error that is in the problem statement, not in a kernel.  The tolerances
in tests/parity.py are set from these numbers (see the table this script writes to
tests/golden/rounding_budget.txt) and must stay above them.

    python tests/rounding_budget.py            # prints the table and rewrites tests/golden/rounding_budget.txt
"""
from __future__ import annotations

import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2607_17644_b200.inputs import LagaShape, make_inputs  # noqa: E402  (random draws only)

GOLDEN = os.path.join(ROOT, "tests", "golden", "rounding_budget.txt")
CASES = [(512, 2, 1512), (2048, 2, 3048), (25, 2, 5017), (51, 3, 5003)]     # (S, h, seed)


def bf16(x: torch.Tensor) -> torch.Tensor:
    return x.to(torch.float32).to(torch.bfloat16).to(torch.float64)


def rounded_model(q, c_kv, k_pe, w, dout, sh: LagaShape):
    """The explicit form with the unavoidable bf16 roundings, head by head, full S x S matrices."""
    f = lambda t: t.to(torch.float64)
    q, c_kv, k_pe, w, dout = f(q), f(c_kv), f(k_pe), f(w), f(dout)
    S, h = sh.S, sh.h
    kv = bf16(c_kv @ w).view(S, h, sh.d_nope + sh.d_v)
    mask = torch.ones(S, S, dtype=torch.bool).tril()
    out = torch.empty(S, h, sh.d_v, dtype=torch.float64)
    lse = torch.empty(S, h, dtype=torch.float64)
    dq = torch.empty(S, h, sh.d_qk, dtype=torch.float64)
    dkv = torch.empty(S, h, sh.d_nope + sh.d_v, dtype=torch.float64)
    dk_pe = torch.zeros(S, sh.d_rope, dtype=torch.float64)
    for i in range(h):
        k = torch.cat([kv[:, i, :sh.d_nope], k_pe], dim=1)
        v = kv[:, i, sh.d_nope:]
        s = (q[:, i] @ k.T) * sh.softmax_scale
        s = s.masked_fill(~mask, float("-inf"))
        lse[:, i] = torch.logsumexp(s, dim=1)
        p = torch.exp(s - lse[:, i:i + 1])
        o = bf16(bf16(p) @ v)
        out[:, i] = o
        delta = (dout[:, i] * o).sum(dim=1, keepdim=True)
        dp = dout[:, i] @ v.T
        ds = bf16(p * (dp - delta))
        dq[:, i] = bf16(sh.softmax_scale * (ds @ k))
        dk = sh.softmax_scale * (ds.T @ q[:, i])
        dkv[:, i, :sh.d_nope] = bf16(dk[:, :sh.d_nope])
        dkv[:, i, sh.d_nope:] = bf16(bf16(p).T @ dout[:, i])
        dk_pe += dk[:, sh.d_nope:]
    dkv2 = dkv.reshape(S, -1)
    return {"out": out, "lse": lse, "dq": dq, "dc_kv": bf16(dkv2 @ w.T), "dk_pe": bf16(dk_pe), "dw": c_kv.T @ dkv2}


def metrics(g, r):
    diff = (g - r).abs()
    rms = float(r.pow(2).mean().sqrt())
    row_rms = r.pow(2).mean(dim=-1, keepdim=True).sqrt().clamp_min(1.0)
    return {"max_abs": float(diff.max()), "scaled": float(diff.max()) / max(1.0, rms),
            "row_scaled": float((diff / row_rms).max()), "rel_l2": float((g - r).norm() / r.norm())}


def budget(S, h, seed):
    import oracle
    sh = LagaShape(S=S, h=h)
    tensors = make_inputs(sh, seed)
    model = rounded_model(*tensors, sh)
    rows = {}
    for mode, rounded in (("plain", False), ("kv_round_bf16", True)):
        ref = oracle.bwd(*tensors, sh.d_v, sh.softmax_scale, causal=True, kv_round_bf16=rounded, return_fwd=True)
        rows[mode] = {name: metrics(model[name], ref[name]) for name in ("out", "dq", "dc_kv", "dk_pe", "dw")}
        rows[mode]["lse"] = {"max_abs": float((model["lse"] - ref["lse"]).abs().max())}
    return rows


def table():
    lines = ["# Rounding budget of the LAGA hot path: the explicit form in float64 with the bf16 roundings a",
             "# tensor-core path cannot avoid (K_nope/V, P, O, dS, dK_nope/dV, bf16 outputs), against the fp64 oracle.",
             "# Written by tests/rounding_budget.py (calls only oracle/); inputs: the seeded recipe of inputs.py.",
             "# columns: S h oracle-mode tensor max_abs max_abs/max(1,rms) max(|d|/max(1,row_rms)) rel_l2"]
    for S, h, seed in CASES:
        rows = budget(S, h, seed)
        for mode, per in rows.items():
            for name, m in per.items():
                if name == "lse":
                    lines.append(f"{S} {h} {mode} lse {m['max_abs']:.3e} - - -")
                else:
                    lines.append(f"{S} {h} {mode} {name} {m['max_abs']:.3e} {m['scaled']:.3e} {m['row_scaled']:.3e} {m['rel_l2']:.3e}")
    return "\n".join(lines) + "\n"


if __name__ == "__main__":
    text = table()
    sys.stdout.write(text)
    with open(GOLDEN, "w") as fh:
        fh.write(text)
