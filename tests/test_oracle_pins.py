"""Pins for the fp64 CPU oracle: every check here is computed by something OTHER than the oracle's
own arithmetic (brute force in numpy, torch's SDPA + autograd in fp64, finite differences, closed
forms, algebraic identities), so that a dropped term, a wrong sign or index, or a transposed operand
in the oracle fails at least one of them.  CPU only.
"""
import math

import numpy as np
import pytest
import torch

from paper_2607_17644_b200.inputs import LagaShape, make_inputs

TOY = LagaShape(S=13, h=3, d_c=8, d_nope=4, d_rope=2, d_v=5)
SMALL = LagaShape(S=96, h=2, d_c=32, d_nope=16, d_rope=8, d_v=16)


def f64(t):
    return t.to(torch.float64)


def split_w(w, sh):
    """W_kv_b shard [d_c, h*(d_nope+d_v)] -> (W_uk [h,d_c,d_nope], W_uv [h,d_c,d_v]); written here
    independently of the oracle: per head, the first d_nope columns make K_nope, the rest V."""
    w3 = f64(w).reshape(sh.d_c, sh.h, sh.d_nope + sh.d_v)
    return w3[:, :, :sh.d_nope].permute(1, 0, 2), w3[:, :, sh.d_nope:].permute(1, 0, 2)


def explicit_kv(c_kv, k_pe, w, sh):
    w_uk, w_uv = split_w(w, sh)
    k_nope = torch.einsum("tc,hcd->thd", f64(c_kv), w_uk)
    v = torch.einsum("tc,hcd->thd", f64(c_kv), w_uv)
    k = torch.cat([k_nope, f64(k_pe)[:, None, :].expand(-1, sh.h, -1)], dim=-1)
    return k, v


def brute_force_fwd(q, c_kv, k_pe, w, sh, scale, causal):
    """Materialise the full S x S score matrix per head in numpy."""
    k, v = explicit_kv(c_kv, k_pe, w, sh)
    qn, kn, vn = f64(q).numpy(), k.numpy(), v.numpy()
    out = np.zeros((sh.S, sh.h, sh.d_v))
    lse = np.zeros((sh.S, sh.h))
    for i in range(sh.h):
        x = scale * qn[:, i, :] @ kn[:, i, :].T
        if causal:
            x = np.where(np.tril(np.ones((sh.S, sh.S), dtype=bool)), x, -np.inf)
        e = np.exp(x)
        lse[:, i] = np.log(e.sum(axis=1))
        out[:, i, :] = (e / e.sum(axis=1, keepdims=True)) @ vn[:, i, :]
    return torch.from_numpy(out), torch.from_numpy(lse)


def autograd_reference(q, c_kv, k_pe, w, dout, sh, scale, causal):
    """torch SDPA + autograd in fp64 on leaves q, c_kv, k_pe, W."""
    ql, cl, kl, wl = (f64(t).clone().requires_grad_(True) for t in (q, c_kv, k_pe, w))
    w3 = wl.reshape(sh.d_c, sh.h, sh.d_nope + sh.d_v)
    kv = torch.einsum("tc,chn->htn", cl, w3)
    k = torch.cat([kv[..., :sh.d_nope], kl[None].expand(sh.h, -1, -1)], dim=-1)
    v = kv[..., sh.d_nope:]
    o = torch.nn.functional.scaled_dot_product_attention(ql.permute(1, 0, 2)[None], k[None], v[None],
                                                         is_causal=causal, scale=scale)[0]
    o = o.permute(1, 0, 2)
    (o * f64(dout)).sum().backward()
    return o.detach(), ql.grad, cl.grad, kl.grad, wl.grad


@pytest.mark.parametrize("sh", [TOY, SMALL], ids=["toy", "small"])
@pytest.mark.parametrize("causal", [True, False])
def test_brute_force_forward(oracle, sh, causal):
    q, c_kv, k_pe, w, _ = make_inputs(sh, 11)
    o, lse = oracle.fwd(q, c_kv, k_pe, w, sh.d_v, sh.softmax_scale, causal=causal)
    o_ref, lse_ref = brute_force_fwd(q, c_kv, k_pe, w, sh, sh.softmax_scale, causal)
    assert (o - o_ref).abs().max() < 1e-12
    assert (lse - lse_ref).abs().max() < 1e-12


def test_row_subset_matches_full(oracle):
    sh = SMALL
    q, c_kv, k_pe, w, _ = make_inputs(sh, 12)
    o, lse = oracle.fwd(q, c_kv, k_pe, w, sh.d_v, sh.softmax_scale)
    rows = [0, 5, 95, 31]
    o_r, lse_r = oracle.fwd(q, c_kv, k_pe, w, sh.d_v, sh.softmax_scale, rows=rows)
    assert torch.equal(o_r, o[rows]) and torch.equal(lse_r, lse[rows])


def test_row_zero_is_v0(oracle):
    """Causal row 0 attends to key 0 only: O[0]=V[0] and LSE[0]=scale*q[0].K[0], exactly."""
    sh = SMALL
    q, c_kv, k_pe, w, _ = make_inputs(sh, 13)
    o, lse = oracle.fwd(q, c_kv, k_pe, w, sh.d_v, sh.softmax_scale, rows=[0])
    k, v = explicit_kv(c_kv, k_pe, w, sh)
    assert (o[0] - v[0]).abs().max() < 1e-13
    ref = sh.softmax_scale * (f64(q)[0] * k[0]).sum(-1)
    assert (lse[0] - ref).abs().max() < 1e-13


def test_up_projection_and_bf16_rounding(oracle):
    sh = SMALL
    q, c_kv, k_pe, w, _ = make_inputs(sh, 14)
    k_ref, v_ref = explicit_kv(c_kv, k_pe, w, sh)
    _, _, kn, v = oracle.fwd(q, c_kv, k_pe, w, sh.d_v, sh.softmax_scale, rows=[0], return_kv=True)
    assert (kn - k_ref[..., :sh.d_nope]).abs().max() < 1e-13 and (v - v_ref).abs().max() < 1e-13
    _, _, kn_r, v_r = oracle.fwd(q, c_kv, k_pe, w, sh.d_v, sh.softmax_scale, rows=[0], return_kv=True,
                                 kv_round_bf16=True)
    # rounded values are bf16-representable and within half a bf16 ulp (at most 2^-8 relative) of the exact
    assert torch.equal(kn_r.to(torch.bfloat16).to(torch.float64), kn_r)
    assert torch.equal(v_r.to(torch.bfloat16).to(torch.float64), v_r)
    assert ((kn_r - kn).abs() <= kn.abs() * 2.0 ** -8 + 1e-300).all()
    assert ((v_r - v).abs() <= v.abs() * 2.0 ** -8 + 1e-300).all()


def test_round_bf16_matches_single_rounding(oracle):
    """For doubles that are exact in fp32, one fp32->bf16 rounding (torch, RNE) is the reference."""
    g = torch.Generator().manual_seed(5)
    x = torch.cat([torch.randn(2000, generator=g), torch.randn(500, generator=g) * 1e-20,
                   torch.randn(500, generator=g) * 1e20,
                   torch.tensor([1.00390625, 1.01171875, -1.00390625, 0.0, 3.0e38, 1e-40])])
    ref = x.to(torch.bfloat16).to(torch.float64)
    got = torch.tensor([oracle.round_bf16(float(v)) for v in x.to(torch.float64)], dtype=torch.float64)
    assert torch.equal(got, ref)
    # a double just above a tie must round up although fp32 would first collapse it onto the tie
    assert oracle.round_bf16(1.00390625 + 1e-12) == 1.0078125


@pytest.mark.parametrize("sh", [TOY, SMALL], ids=["toy", "small"])
def test_head_shard_concatenation(oracle, sh):
    """Section 5.1: step 4 computes, for the heads of a shard, the same per-head linear maps as the full
    up-projection, i.e. a head shard's up-projection is a column slice of the full one, so running the
    shards separately reproduces the full-head run; shared-tensor gradients add across shards."""
    sh = LagaShape(S=sh.S, h=4, d_c=sh.d_c, d_nope=sh.d_nope, d_rope=sh.d_rope, d_v=sh.d_v)
    q, c_kv, k_pe, w, dout = make_inputs(sh, 15)
    full = oracle.bwd(q, c_kv, k_pe, w, dout, sh.d_v, sh.softmax_scale, return_fwd=True)
    per = sh.d_nope + sh.d_v
    acc_dc, acc_dk = 0, 0
    for lo, hi in [(0, 1), (1, 4)]:
        r = oracle.bwd(q[:, lo:hi].contiguous(), c_kv, k_pe, w[:, lo * per:hi * per].contiguous(),
                       dout[:, lo:hi].contiguous(), sh.d_v, sh.softmax_scale, return_fwd=True)
        assert torch.equal(r["out"], full["out"][:, lo:hi]) and torch.equal(r["lse"], full["lse"][:, lo:hi])
        assert torch.equal(r["dq"], full["dq"][:, lo:hi])
        assert torch.equal(r["dw"], full["dw"][:, lo * per:hi * per])
        acc_dc, acc_dk = acc_dc + r["dc_kv"], acc_dk + r["dk_pe"]
    assert (acc_dc - full["dc_kv"]).abs().max() < 1e-12
    assert (acc_dk - full["dk_pe"]).abs().max() < 1e-12


@pytest.mark.parametrize("causal", [True, False])
def test_absorbed_form_equals_explicit(oracle, causal):
    """Section 3.2's absorbed form: q_abs = W_uk q_nope scores against the latent itself, the
    accumulator lives in latent space and W_uv is applied last.  Same function as the explicit form."""
    sh = SMALL
    q, c_kv, k_pe, w, _ = make_inputs(sh, 16)
    w_uk, w_uv = split_w(w, sh)
    qd, cd, kd = f64(q), f64(c_kv), f64(k_pe)
    q_abs = torch.einsum("shd,hcd->shc", qd[..., :sh.d_nope], w_uk)
    scores = sh.softmax_scale * (torch.einsum("shc,tc->hst", q_abs, cd)
                                 + torch.einsum("shr,tr->hst", qd[..., sh.d_nope:], kd))
    if causal:
        scores = scores.masked_fill(~torch.tril(torch.ones(sh.S, sh.S, dtype=torch.bool)), -math.inf)
    p = torch.softmax(scores, dim=-1)
    latent_acc = torch.einsum("hst,tc->shc", p, cd)
    o_abs = torch.einsum("shc,hcd->shd", latent_acc, w_uv)
    o, lse = oracle.fwd(q, c_kv, k_pe, w, sh.d_v, sh.softmax_scale, causal=causal)
    assert (o - o_abs).abs().max() < 1e-12
    assert (lse - torch.logsumexp(scores, dim=-1).T).abs().max() < 1e-12


@pytest.mark.parametrize("sh", [TOY, SMALL, LagaShape(S=200, h=2)], ids=["toy", "small", "v3dims"])
@pytest.mark.parametrize("causal", [True, False])
def test_library_sdpa_and_autograd(oracle, sh, causal):
    q, c_kv, k_pe, w, dout = make_inputs(sh, 17)
    o_ref, dq, dc, dk, dw = autograd_reference(q, c_kv, k_pe, w, dout, sh, sh.softmax_scale, causal)
    r = oracle.bwd(q, c_kv, k_pe, w, dout, sh.d_v, sh.softmax_scale, causal=causal, return_fwd=True)
    assert (r["out"] - o_ref).abs().max() < 1e-12
    for name, ref in [("dq", dq), ("dc_kv", dc), ("dk_pe", dk), ("dw", dw)]:
        err = (r[name] - ref).abs().max() / max(1.0, ref.abs().max())
        assert err < 1e-11, (name, float(err))


def test_finite_differences(oracle):
    """Central differences of L = sum(O * dO) in fp64.  Inputs must stay bf16-representable for the
    oracle, so each probe moves one entry by a bf16-exact step and the quadratic term cancels."""
    sh = TOY
    q, c_kv, k_pe, w, dout = make_inputs(sh, 18)
    r = oracle.bwd(q, c_kv, k_pe, w, dout, sh.d_v, sh.softmax_scale)
    tensors = {"dq": q, "dc_kv": c_kv, "dk_pe": k_pe, "dw": w}
    order = ["dq", "dc_kv", "dk_pe", "dw"]

    def loss(args):
        o, _ = oracle.fwd(args[0], args[1], args[2], args[3], sh.d_v, sh.softmax_scale)
        return float((o * f64(dout)).sum())

    rng = np.random.default_rng(0)
    for name in order:
        base = tensors[name]
        for _ in range(6):
            idx = tuple(int(rng.integers(0, n)) for n in base.shape)
            # Richardson on two bf16-exact steps removes the cubic term of the central difference
            x0 = float(base[idx])
            ulp = 2.0 ** (math.floor(math.log2(abs(x0))) - 7) if x0 != 0 else 2.0 ** -10
            vals = []
            for step in (ulp, 2 * ulp):
                fs = []
                for sign in (+1, -1):
                    pert = base.clone()
                    pert[idx] = x0 + sign * step
                    assert float(pert[idx]) == x0 + sign * step, "step must be bf16-exact"
                    args = [pert if n == name else tensors[n] for n in order]
                    fs.append(loss(args))
                vals.append((fs[0] - fs[1]) / (2 * step))
            fd = (4 * vals[0] - vals[1]) / 3
            an = float(r[name][idx])
            assert abs(fd - an) <= 1e-5 * max(1.0, abs(an)), (name, idx, fd, an)


def test_zero_query_closed_form(oracle):
    """q = 0 makes every allowed key equally likely: O[s] is the running mean of V, LSE = ln(#keys)."""
    sh = SMALL
    q, c_kv, k_pe, w, _ = make_inputs(sh, 19)
    q = torch.zeros_like(q)
    _, v = explicit_kv(c_kv, k_pe, w, sh)
    o, lse = oracle.fwd(q, c_kv, k_pe, w, sh.d_v, sh.softmax_scale)
    counts = torch.arange(1, sh.S + 1, dtype=torch.float64)
    assert (o - v.cumsum(0) / counts[:, None, None]).abs().max() < 1e-12
    assert (lse - counts.log()[:, None]).abs().max() < 1e-12
    o_nc, lse_nc = oracle.fwd(q, c_kv, k_pe, w, sh.d_v, sh.softmax_scale, causal=False)
    assert (o_nc - v.mean(0)[None]).abs().max() < 1e-12 and (lse_nc - math.log(sh.S)).abs().max() < 1e-12


def test_identical_latent_rows_give_v(oracle):
    sh = SMALL
    q, c_kv, k_pe, w, _ = make_inputs(sh, 20)
    c_kv = c_kv[:1].expand(sh.S, -1).contiguous()
    _, v = explicit_kv(c_kv, k_pe, w, sh)
    o, _ = oracle.fwd(q, c_kv, k_pe, w, sh.d_v, sh.softmax_scale)
    assert (o - v).abs().max() < 1e-12


def test_rope_key_shift_property(oracle):
    """Adding u to every k_pe row adds scale*<q_rope,u> to every allowed score of that row: softmax is
    unchanged, LSE moves by exactly that amount (so the rope band and the scale are both in the LSE)."""
    sh = SMALL
    q, c_kv, k_pe, w, _ = make_inputs(sh, 21)
    # k_pe on a 1/8 grid so that k_pe + u is exact in bf16 (no re-rounding of the shifted keys)
    k_pe = (k_pe.to(torch.float32).clamp(-4, 4) * 8).round().div(8).to(torch.bfloat16)
    u = torch.tensor([0.5, -0.25, 1.0, 0.125, -2.0, 0.75, 0.0, 1.5])[:sh.d_rope]
    k_shift = (k_pe.to(torch.float32) + u).to(torch.bfloat16)
    du = f64(k_shift) - f64(k_pe)
    assert (du == f64(u)[None]).all()
    o0, l0 = oracle.fwd(q, c_kv, k_pe, w, sh.d_v, sh.softmax_scale)
    o1, l1 = oracle.fwd(q, c_kv, k_shift, w, sh.d_v, sh.softmax_scale)
    assert (o0 - o1).abs().max() < 1e-12
    expect = sh.softmax_scale * torch.einsum("shr,r->sh", f64(q)[..., sh.d_nope:], du[0])
    assert ((l1 - l0) - expect).abs().max() < 1e-12


def test_output_is_convex_combination(oracle):
    sh = SMALL
    q, c_kv, k_pe, w, _ = make_inputs(sh, 22)
    _, v = explicit_kv(c_kv, k_pe, w, sh)
    o, _ = oracle.fwd(q, c_kv, k_pe, w, sh.d_v, sh.softmax_scale)
    run_max = torch.cummax(v, dim=0).values
    run_min = torch.cummin(v, dim=0).values
    assert (o <= run_max + 1e-12).all() and (o >= run_min - 1e-12).all()


def test_trace_identities(oracle):
    """Bilinearity: <W,dW> = <c_kv,dc_kv> = <(K_nope|V),(dK_nope|dV)>; per head sum_s q.dQ = sum_t K.dK
    (both equal scale*sum dS*scores); dS rows sum to zero so sum_t K.dK needs the scale factor right."""
    sh = SMALL
    q, c_kv, k_pe, w, dout = make_inputs(sh, 23)
    r = oracle.bwd(q, c_kv, k_pe, w, dout, sh.d_v, sh.softmax_scale, return_dkv=True)
    k, v = explicit_kv(c_kv, k_pe, w, sh)
    a = (f64(w) * r["dw"]).sum()
    b = (f64(c_kv) * r["dc_kv"]).sum()
    c = (k[..., :sh.d_nope] * r["dk"][..., :sh.d_nope]).sum() + (v * r["dv"]).sum()
    assert abs(a - b) < 1e-9 * abs(a) and abs(a - c) < 1e-9 * abs(a)
    lhs = (f64(q) * r["dq"]).sum(dim=(0, 2))
    rhs = (k * r["dk"]).sum(dim=(0, 2))
    assert ((lhs - rhs).abs() < 1e-9 * lhs.abs().clamp_min(1.0)).all()
    assert (r["dk_pe"] - r["dk"][..., sh.d_nope:].sum(1)).abs().max() < 1e-12


def test_single_token(oracle):
    sh = LagaShape(S=1, h=3, d_c=8, d_nope=4, d_rope=2, d_v=5)
    q, c_kv, k_pe, w, dout = make_inputs(sh, 24)
    r = oracle.bwd(q, c_kv, k_pe, w, dout, sh.d_v, sh.softmax_scale, return_fwd=True, return_dkv=True)
    _, v = explicit_kv(c_kv, k_pe, w, sh)
    w_uk, w_uv = split_w(w, sh)
    assert (r["out"] - v).abs().max() < 1e-13
    assert r["dq"].abs().max() == 0 and r["dk"].abs().max() == 0 and r["dk_pe"].abs().max() == 0
    assert (r["dv"] - f64(dout)).abs().max() == 0
    dc_ref = torch.einsum("shd,hcd->sc", f64(dout), w_uv)
    assert (r["dc_kv"] - dc_ref).abs().max() < 1e-13
    dw3 = r["dw"].reshape(sh.d_c, sh.h, sh.d_nope + sh.d_v)
    assert dw3[..., :sh.d_nope].abs().max() == 0
    dwv_ref = torch.einsum("sc,shd->chd", f64(c_kv), f64(dout))
    assert (dw3[..., sh.d_nope:] - dwv_ref).abs().max() < 1e-13


def test_single_head_and_last_row(oracle):
    sh = LagaShape(S=40, h=1, d_c=16, d_nope=8, d_rope=4, d_v=8)
    q, c_kv, k_pe, w, dout = make_inputs(sh, 25)
    r = oracle.bwd(q, c_kv, k_pe, w, dout, sh.d_v, sh.softmax_scale, return_dkv=True)
    assert torch.equal(r["dk_pe"], r["dk"][:, 0, sh.d_nope:])
    o_c, l_c = oracle.fwd(q, c_kv, k_pe, w, sh.d_v, sh.softmax_scale, causal=True)
    o_n, l_n = oracle.fwd(q, c_kv, k_pe, w, sh.d_v, sh.softmax_scale, causal=False)
    assert torch.equal(o_c[-1], o_n[-1]) and torch.equal(l_c[-1], l_n[-1])
    assert not torch.equal(o_c[0], o_n[0])


def test_config_distribution_statistics(oracle):
    """Loose sanity of the input recipe at the V3 dims: K_nope, V ~ unit variance, scaled scores ~ N(0,1)
    so LSE[s] - ln(s+1) averages about 1/2 on late rows (log-normal mean)."""
    sh = LagaShape(S=768, h=2)
    q, c_kv, k_pe, w, _ = make_inputs(sh, 1000)
    rows = list(range(512, 768, 4))
    _, lse, kn, v = oracle.fwd(q, c_kv, k_pe, w, sh.d_v, sh.softmax_scale, rows=rows, return_kv=True)
    assert 0.9 < float(kn.std()) < 1.1 and 0.9 < float(v.std()) < 1.1
    excess = lse - torch.tensor(rows, dtype=torch.float64).add(1).log()[:, None]
    assert 0.4 < float(excess.mean()) < 0.6


@pytest.mark.parametrize("causal", [True, False])
def test_row_and_key_subsets_match_full_backward(oracle, causal):
    """The spot-check entry points return exactly what the (autograd-pinned) full backward returns."""
    sh = LagaShape(S=70, h=3, d_c=16, d_nope=8, d_rope=4, d_v=8)
    q, c_kv, k_pe, w, dout = make_inputs(sh, 26)
    full = oracle.bwd(q, c_kv, k_pe, w, dout, sh.d_v, sh.softmax_scale, causal=causal, return_fwd=True,
                      return_dkv=True)
    rows = [0, 69, 17, 40]
    r = oracle.bwd_rows(q, c_kv, k_pe, w, dout, sh.d_v, sh.softmax_scale, rows, causal=causal)
    assert torch.equal(r["dq"], full["dq"][rows]) and torch.equal(r["out"], full["out"][rows])
    assert torch.equal(r["lse"], full["lse"][rows])
    keys = [69, 33, 50, 68]
    k = oracle.bwd_keys(q, c_kv, k_pe, w, dout, sh.d_v, sh.softmax_scale, keys, causal=causal)
    assert (k["dk"] - full["dk"][keys]).abs().max() < 1e-13 and (k["dv"] - full["dv"][keys]).abs().max() < 1e-13
    assert (k["dk_pe"] - full["dk_pe"][keys]).abs().max() < 1e-13
    assert (k["dc_kv"] - full["dc_kv"][keys]).abs().max() < 1e-12


def test_linear_oracle_against_loops_closed_forms_and_autograd(oracle):
    """The dense projections (Algorithm 1 steps 1 and 7).  The oracle calls a library matrix product, so it is
    pinned by things that are not that call: an explicit triple loop on a tiny case (a transposed operand or a
    swapped index fails it), closed forms (identity weight; all-ones weight = row sums), the bilinear trace
    identity between the two gradients, and torch.autograd on an elementwise restatement."""
    g = torch.Generator().manual_seed(31)
    M, K, N = 5, 4, 3
    x = torch.randn(M, K, generator=g).to(torch.bfloat16)
    w = torch.randn(K, N, generator=g).to(torch.bfloat16)
    dy = torch.randn(M, N, generator=g).to(torch.bfloat16)
    y = oracle.linear(x, w)
    dx, dw = oracle.linear_bwd(dy, x, w)
    xs, ws, dys = x.double().tolist(), w.double().tolist(), dy.double().tolist()
    for m in range(M):
        for n in range(N):
            assert abs(float(y[m, n]) - sum(xs[m][k] * ws[k][n] for k in range(K))) < 1e-12
        for k in range(K):
            assert abs(float(dx[m, k]) - sum(dys[m][n] * ws[k][n] for n in range(N))) < 1e-12
    for k in range(K):
        for n in range(N):
            assert abs(float(dw[k, n]) - sum(xs[m][k] * dys[m][n] for m in range(M))) < 1e-12
    # closed forms
    eye = torch.eye(K).to(torch.bfloat16)
    assert torch.equal(oracle.linear(x, eye), x.double())
    ones = torch.ones(K, 2).to(torch.bfloat16)
    assert torch.allclose(oracle.linear(x, ones), x.double().sum(dim=1, keepdim=True).expand(M, 2), atol=1e-12)
    # <dy, y> = <dx, x> = <dw, w>
    t = float((dy.double() * y).sum())
    assert abs(t - float((dx * x.double()).sum())) < 1e-10 and abs(t - float((dw * w.double()).sum())) < 1e-10
    # autograd of sum_mn dy[m,n] * sum_k x[m,k] w[k,n], written with broadcasting (no matmul)
    xa, wa = x.double().requires_grad_(True), w.double().requires_grad_(True)
    ((xa[:, :, None] * wa[None, :, :]).sum(dim=1) * dy.double()).sum().backward()
    assert torch.allclose(xa.grad, dx, atol=1e-12) and torch.allclose(wa.grad, dw, atol=1e-12)


def test_layernorm_oracle_against_library_closed_forms_and_finite_differences(oracle):
    """LayerNorm of the latent (Algorithm 1 step 1).  Pins: torch.nn.functional.layer_norm with float64 autograd
    (a library routine the oracle does not call), closed forms (a constant row normalises to beta; a two-valued
    row to +-gamma), invariance to a shift and -- with eps = 0 -- to a positive scale of the row, the identities
    sum_c dx = 0 and sum_c dx * xhat = 0, and central finite differences."""
    g = torch.Generator().manual_seed(41)
    M, D, eps = 6, 16, 1e-5
    x = (torch.randn(M, D, generator=g) * 2 + 0.5).to(torch.bfloat16)
    gamma = (1 + 0.3 * torch.randn(D, generator=g)).to(torch.bfloat16)
    beta = (0.2 * torch.randn(D, generator=g)).to(torch.bfloat16)
    dy = torch.randn(M, D, generator=g).to(torch.bfloat16)
    y, mean, rstd = oracle.layernorm(x, gamma, beta, eps)
    dx, dgamma, dbeta = oracle.layernorm_bwd(dy, x, gamma, eps)
    xa, ga, ba = x.double().requires_grad_(True), gamma.double().requires_grad_(True), beta.double().requires_grad_(True)
    ya = torch.nn.functional.layer_norm(xa, (D,), ga, ba, eps)
    assert torch.allclose(ya, y, atol=1e-12)
    (ya * dy.double()).sum().backward()
    assert torch.allclose(xa.grad, dx, atol=1e-11) and torch.allclose(ga.grad, dgamma, atol=1e-11)
    assert torch.allclose(ba.grad, dbeta, atol=1e-12)
    assert torch.allclose(mean, x.double().mean(dim=1), atol=1e-13)
    assert torch.allclose(rstd, 1 / torch.sqrt(x.double().var(dim=1, unbiased=False) + eps), atol=1e-12)
    # closed forms
    const = torch.full((1, D), 3.0).to(torch.bfloat16)
    assert torch.allclose(oracle.layernorm(const, gamma, beta, eps)[0], beta.double().expand(1, D), atol=1e-12)
    two = torch.tensor([[1.0, -1.0] * (D // 2)]).to(torch.bfloat16)        # mean 0, variance 1
    assert torch.allclose(oracle.layernorm(two, gamma, None, 0.0)[0], two.double() * gamma.double(), atol=1e-12)
    # shift invariance; scale invariance without eps
    assert torch.allclose(oracle.layernorm(x.double() + 7.0, gamma, beta, eps)[0], y, atol=1e-10)
    assert torch.allclose(oracle.layernorm(x.double() * 4.0, gamma, beta, 0.0)[0], oracle.layernorm(x, gamma, beta, 0.0)[0], atol=1e-10)
    # dx is orthogonal to the constant and to xhat (the two directions the normalisation removes), up to eps
    xhat = (x.double() - mean[:, None]) * rstd[:, None]
    assert float(dx.sum(dim=1).abs().max()) < 1e-10
    assert float((dx * xhat).sum(dim=1).abs().max()) < 1e-3
    # finite differences of L = sum(dy * y) in a few entries of x and gamma
    def loss(xv, gv):
        return float((oracle.layernorm(xv, gv, beta, eps)[0] * dy.double()).sum())
    for (m, c) in [(0, 0), (3, 7), (5, 15)]:
        h = 1e-5
        xp, xm = x.double().clone(), x.double().clone()
        xp[m, c] += h
        xm[m, c] -= h
        assert abs((loss(xp, gamma) - loss(xm, gamma)) / (2 * h) - float(dx[m, c])) < 1e-6
        gp, gmn = gamma.double().clone(), gamma.double().clone()
        gp[c] += h
        gmn[c] -= h
        assert abs((loss(x, gp) - loss(x, gmn)) / (2 * h) - float(dgamma[c])) < 1e-6
