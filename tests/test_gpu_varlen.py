"""GPU parity of the packed variable-length entry points (laga_fwd_varlen / laga_bwd_varlen).

The reference is the single-sequence fp64 oracle applied to every sequence on its own: attention is confined
to a sequence, the projections are token-wise, dW sums over the sequences.  Composition only; no arithmetic
of the method lives here.
"""
import pytest
import torch

from paper_2607_17644_b200.inputs import LagaShape, make_inputs
from parity import TOL_LSE, check_dw, check_tensor, max_abs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def laga():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2607_17644_b200 import laga as _laga
    _laga.lib()
    return _laga


def nan_like(shape, dtype):
    return torch.full(shape, float("nan"), dtype=dtype, device="cuda")


def cu_of(lengths):
    cu = [0]
    for n in lengths:
        cu.append(cu[-1] + n)
    return cu


def oracle_packed(oracle, tensors, sh, cu, causal):
    """The oracle, sequence by sequence, stitched back into the packed layout."""
    q, c_kv, k_pe, w, dout = tensors
    S = q.shape[0]
    ref = {"out": torch.zeros(S, sh.h, sh.d_v, dtype=torch.float64), "lse": torch.zeros(S, sh.h, dtype=torch.float64),
           "dq": torch.zeros(S, sh.h, sh.d_qk, dtype=torch.float64), "dc_kv": torch.zeros(S, sh.d_c, dtype=torch.float64),
           "dk_pe": torch.zeros(S, sh.d_rope, dtype=torch.float64), "dw": torch.zeros(sh.d_c, sh.n_cols, dtype=torch.float64)}
    for a, b in zip(cu[:-1], cu[1:]):
        if b == a:
            continue
        r = oracle.bwd(q[a:b], c_kv[a:b], k_pe[a:b], w, dout[a:b], sh.d_v, sh.softmax_scale, causal=causal,
                       kv_round_bf16=True, return_fwd=True)
        for name in ("out", "lse", "dq", "dc_kv", "dk_pe"):
            ref[name][a:b] = r[name]
        ref["dw"] += r["dw"]
    return ref


def run_packed(laga, tensors, cu, causal, flags=0):
    q, c_kv, k_pe, w, dout = (t.cuda() for t in tensors)
    S, h = q.shape[0], q.shape[1]
    out, lse, ws = laga.fwd(q, c_kv, k_pe, w, causal=causal, out=nan_like((S, h, 128), torch.bfloat16),
                            lse=nan_like((S, h), torch.float32), cu_seqlens=cu)
    laga.check_status(ws, where="laga_fwd_varlen")
    dq, dc_kv, dk_pe, dw, ws2 = laga.bwd(q, c_kv, k_pe, w, out, lse, dout, causal=causal, cu_seqlens=cu, flags=flags,
                                         dq=nan_like(tuple(q.shape), torch.bfloat16),
                                         dc_kv=nan_like(tuple(c_kv.shape), torch.bfloat16),
                                         dk_pe=nan_like(tuple(k_pe.shape), torch.bfloat16),
                                         dw_kv_b=nan_like(tuple(w.shape), torch.float32))
    laga.check_status(ws2, where="laga_bwd_varlen")
    return {k: v.cpu() for k, v in dict(out=out, lse=lse, dq=dq, dc_kv=dc_kv, dk_pe=dk_pe, dw=dw).items()}


CASES = [
    # lengths, h, causal
    ([300, 212], 2, True),                   # two ragged sequences
    ([128, 128, 128], 3, True),              # a batch of equal, tile-aligned sequences
    ([1, 129, 64, 500], 2, True),            # one token; one row past a tile; less than a tile; several tiles
    ([100, 0, 260], 1, True),                # an empty sequence in the middle
    ([97, 385, 30], 2, False),               # non-causal, forward key tiles of 96 with tails
    ([1000, 2048, 77], 4, True),             # long and short mixed: the longest-first order interleaves them
    ([5] * 40, 1, True),                     # many tiny sequences: forty tiles of five rows
]


@pytest.mark.parametrize("lengths,h,causal", CASES)
def test_packed_sequences_elementwise(laga, oracle, lengths, h, causal):
    cu = cu_of(lengths)
    sh = LagaShape(S=cu[-1], h=h)
    tensors = make_inputs(sh, 4000 + cu[-1] + h)
    g = run_packed(laga, tensors, cu, causal)
    r = oracle_packed(oracle, tensors, sh, cu, causal)
    check_tensor("out", g["out"], r["out"])
    assert max_abs(g["lse"], r["lse"]) <= TOL_LSE
    check_tensor("dq", g["dq"], r["dq"])
    check_tensor("dk_pe", g["dk_pe"], r["dk_pe"])
    check_tensor("dc_kv", g["dc_kv"], r["dc_kv"])
    check_dw(g["dw"], r["dw"])


def test_one_packed_sequence_is_the_single_sequence_path_bit_for_bit(laga):
    """cu_seqlens = {0, S}: same tiles in the same order through the same kernels."""
    sh = LagaShape(S=700, h=2)
    tensors = make_inputs(sh, 4100)
    q, c_kv, k_pe, w, dout = (t.cuda() for t in tensors)
    det = laga.FLAG_DETERMINISTIC
    out, lse, ws = laga.fwd(q, c_kv, k_pe, w)
    single = laga.bwd(q, c_kv, k_pe, w, out, lse, dout, flags=det)[:4]
    out_v, lse_v, ws_v = laga.fwd(q, c_kv, k_pe, w, cu_seqlens=[0, sh.S])
    packed = laga.bwd(q, c_kv, k_pe, w, out_v, lse_v, dout, flags=det, cu_seqlens=[0, sh.S])[:4]
    laga.check_status(ws_v)
    assert torch.equal(out, out_v) and torch.equal(lse, lse_v)
    for a, b in zip(single, packed):
        assert torch.equal(a, b)


def test_a_batch_equals_its_sequences_run_one_by_one(laga):
    """Sequences do not see each other: every packed row equals the same row of a single-sequence call (the
    projections are token-wise and the attention tiles of a sequence are computed in the same order)."""
    lengths = [260, 513, 64]
    cu = cu_of(lengths)
    sh = LagaShape(S=cu[-1], h=2)
    tensors = make_inputs(sh, 4200)
    q, c_kv, k_pe, w, dout = (t.cuda() for t in tensors)
    out, lse, ws = laga.fwd(q, c_kv, k_pe, w, cu_seqlens=cu)
    dq, dc_kv, dk_pe, dw, ws2 = laga.bwd(q, c_kv, k_pe, w, out, lse, dout, cu_seqlens=cu, flags=laga.FLAG_DETERMINISTIC)
    laga.check_status(ws2)
    dw_sum = torch.zeros_like(dw)
    for a, b in zip(cu[:-1], cu[1:]):
        o1, l1, _ = laga.fwd(q[a:b].contiguous(), c_kv[a:b].contiguous(), k_pe[a:b].contiguous(), w)
        g1 = laga.bwd(q[a:b].contiguous(), c_kv[a:b].contiguous(), k_pe[a:b].contiguous(), w, o1, l1,
                      dout[a:b].contiguous(), flags=laga.FLAG_DETERMINISTIC)
        assert torch.equal(out[a:b], o1) and torch.equal(lse[a:b], l1)
        assert torch.equal(dq[a:b], g1[0]) and torch.equal(dk_pe[a:b], g1[2])
        # dc_kv rows come from the same dKV rows through a GEMM whose row tiles differ in position only
        assert torch.equal(dc_kv[a:b], g1[1])
        dw_sum += g1[3]
    assert float((dw - dw_sum).norm() / dw_sum.norm()) < 1e-5       # summed in a different order


def test_kv_saved_pairs_the_varlen_calls(laga):
    lengths = [400, 150, 300]
    cu = cu_of(lengths)
    sh = LagaShape(S=cu[-1], h=2)
    q, c_kv, k_pe, w, dout = (t.cuda() for t in make_inputs(sh, 4300))
    det = laga.FLAG_DETERMINISTIC
    ws = laga.alloc_workspace(laga.bwd_varlen_workspace_bytes(sh.S, len(lengths), sh.h, flags=det))
    out, lse, _ = laga.fwd(q, c_kv, k_pe, w, workspace=ws, cu_seqlens=cu)
    saved = laga.bwd(q, c_kv, k_pe, w, out, lse, dout, workspace=ws, flags=det | laga.FLAG_KV_SAVED, cu_seqlens=cu)[:4]
    laga.check_status(ws)
    saved = [t.clone() for t in saved]
    ws.zero_()
    recomputed = laga.bwd(q, c_kv, k_pe, w, out, lse, dout, workspace=ws, flags=det, cu_seqlens=cu)[:4]
    laga.check_status(ws)
    for a, b in zip(saved, recomputed):
        assert torch.equal(a, b)


def test_malformed_cu_seqlens_is_refused(laga):
    sh = LagaShape(S=256, h=1)
    q, c_kv, k_pe, w, dout = (t.cuda() for t in make_inputs(sh, 4400))
    with pytest.raises(laga.LagaError):
        laga.fwd(q, c_kv, k_pe, w, cu_seqlens=[0, 100, 255])
    with pytest.raises(laga.LagaError):
        laga.fwd(q, c_kv, k_pe, w, cu_seqlens=[0, 200, 100, 256])
    out, lse, ws = laga.fwd(q, c_kv, k_pe, w, cu_seqlens=[0, 100, 256])
    laga.check_status(ws)                                                # the context is fine afterwards


def test_autograd_wrapper_takes_packed_sequences(laga):
    from paper_2607_17644_b200 import laga_attention
    cu = cu_of([200, 330])
    sh = LagaShape(S=cu[-1], h=2)
    q, c_kv, k_pe, w, dout = (t.cuda() for t in make_inputs(sh, 4500))
    out, lse, _ = laga.fwd(q, c_kv, k_pe, w, cu_seqlens=cu)
    dq, dc_kv, dk_pe, dw, ws = laga.bwd(q, c_kv, k_pe, w, out, lse, dout, cu_seqlens=cu, flags=laga.FLAG_DETERMINISTIC)
    laga.check_status(ws)
    leaves = [t.clone().requires_grad_(True) for t in (q, c_kv, k_pe, w)]
    o = laga_attention(*leaves, cu_seqlens=torch.tensor(cu, dtype=torch.int32))
    assert torch.equal(o, out)
    o.backward(dout)
    assert torch.equal(leaves[0].grad, dq) and torch.equal(leaves[1].grad, dc_kv)
    assert float((leaves[2].grad.float() - dk_pe.float()).abs().max()) <= 2e-2 * max(1.0, float(dk_pe.float().abs().max()))
    assert float((leaves[3].grad.float() - dw).norm() / dw.norm()) < 1e-2      # bf16 copy of an fp32 gradient


def test_random_packings(laga, oracle):
    """Seeded random packings (two to six sequences of 1..700 tokens, one to three heads, either mask): the
    longest-first tile order and the per-sequence padding change with every draw."""
    rng = torch.Generator().manual_seed(4600)
    for trial in range(6):
        n_seqs = int(torch.randint(2, 7, (1,), generator=rng))
        lengths = [int(torch.randint(1, 701, (1,), generator=rng)) for _ in range(n_seqs)]
        h = int(torch.randint(1, 4, (1,), generator=rng))
        causal = bool(torch.randint(0, 2, (1,), generator=rng))
        cu = cu_of(lengths)
        sh = LagaShape(S=cu[-1], h=h)
        tensors = make_inputs(sh, 4600 + trial)
        g = run_packed(laga, tensors, cu, causal)
        r = oracle_packed(oracle, tensors, sh, cu, causal)
        for name in ("out", "dq", "dk_pe", "dc_kv"):
            check_tensor(f"{name} (lengths {lengths}, h={h}, causal={causal})", g[name], r[name])
        assert max_abs(g["lse"], r["lse"]) <= TOL_LSE
        check_dw(g["dw"], r["dw"])
