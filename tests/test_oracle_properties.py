"""Property tests of the CPU oracle over random small shapes (hypothesis): each property follows from
the definition of the path and is checked against torch's own fp64 arithmetic, not the oracle's."""
import torch
from hypothesis import given, settings, strategies as st

from paper_2607_17644_b200.inputs import LagaShape, make_inputs

shapes = st.builds(LagaShape, S=st.integers(1, 40), h=st.integers(1, 4), d_c=st.sampled_from([4, 8, 16]),
                   d_nope=st.sampled_from([2, 4, 8]), d_rope=st.sampled_from([0, 2, 4]), d_v=st.sampled_from([1, 3, 8]))


def _amax(t):
    return float(t.abs().max()) if t.numel() else 0.0


def _kv(c_kv, k_pe, w, sh):
    w3 = w.double().reshape(sh.d_c, sh.h, sh.d_nope + sh.d_v)
    kv = torch.einsum("tc,chn->thn", c_kv.double(), w3)
    k = torch.cat([kv[..., :sh.d_nope], k_pe.double()[:, None, :].expand(-1, sh.h, -1)], -1)
    return k, kv[..., sh.d_nope:]


@settings(max_examples=30, deadline=None)
@given(sh=shapes, seed=st.integers(0, 10_000), causal=st.booleans())
def test_forward_matches_dense_softmax(oracle, sh, seed, causal):
    q, c_kv, k_pe, w, _ = make_inputs(sh, seed)
    k, v = _kv(c_kv, k_pe, w, sh)
    scores = sh.softmax_scale * torch.einsum("shd,thd->hst", q.double(), k)
    if causal:
        scores = scores.masked_fill(~torch.tril(torch.ones(sh.S, sh.S, dtype=torch.bool)), float("-inf"))
    o_ref = torch.einsum("hst,thd->shd", torch.softmax(scores, -1), v)
    o, lse = oracle.fwd(q, c_kv, k_pe, w, sh.d_v, sh.softmax_scale, causal=causal)
    assert (o - o_ref).abs().max() < 1e-11
    assert (lse - torch.logsumexp(scores, -1).T).abs().max() < 1e-11


@settings(max_examples=20, deadline=None)
@given(sh=shapes, seed=st.integers(0, 10_000))
def test_gradients_are_linear_in_dout_and_shards_add(oracle, sh, seed):
    q, c_kv, k_pe, w, dout = make_inputs(sh, seed)
    r1 = oracle.bwd(q, c_kv, k_pe, w, dout, sh.d_v, sh.softmax_scale)
    # doubling dO (exact in bf16) doubles every gradient
    r2 = oracle.bwd(q, c_kv, k_pe, w, (dout.float() * 2).to(torch.bfloat16), sh.d_v, sh.softmax_scale)
    for name in ("dq", "dc_kv", "dk_pe", "dw"):
        assert _amax(r2[name] - 2 * r1[name]) <= 1e-12 * max(1.0, _amax(r1[name]))
    # per-head runs: dq / dw are per head, dc_kv / dk_pe add up over heads
    per = sh.d_nope + sh.d_v
    acc_dc, acc_dk = torch.zeros_like(r1["dc_kv"]), torch.zeros_like(r1["dk_pe"])
    for i in range(sh.h):
        ri = oracle.bwd(q[:, i:i + 1].contiguous(), c_kv, k_pe, w[:, i * per:(i + 1) * per].contiguous(),
                        dout[:, i:i + 1].contiguous(), sh.d_v, sh.softmax_scale)
        assert torch.equal(ri["dq"], r1["dq"][:, i:i + 1]) and torch.equal(ri["dw"], r1["dw"][:, i * per:(i + 1) * per])
        acc_dc += ri["dc_kv"]
        acc_dk += ri["dk_pe"]
    assert _amax(acc_dc - r1["dc_kv"]) <= 1e-11 * max(1.0, _amax(r1["dc_kv"]))
    assert _amax(acc_dk - r1["dk_pe"]) <= 1e-11 * max(1.0, _amax(r1["dk_pe"]))
