"""The absorbed form (Section 3.2, baseline B2) as hand-written kernels, against the SAME fp64 oracle as
the explicit path: the two forms are algebraically identical (q_nope . (W_uk^T c) = (W_uk q_nope) . c), so
out and LSE must agree with the oracle within the same bounds.  The absorbed path never forms K_nope / V
(it rounds q_abs and the latent accumulator to bf16 instead), so it is compared with the plain oracle."""
import pytest
import torch

from paper_2607_17644_b200.inputs import CONFIGS, CONFIG_SEEDS, LagaShape, make_inputs
from parity import TOL_LSE_UNROUNDED, check_row_bands, check_tensor, max_abs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def laga():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2607_17644_b200 import laga as _laga
    _laga.lib()
    return _laga


def run(laga, tensors, causal):
    q, c_kv, k_pe, w = (t.cuda() for t in tensors[:4])
    S, h = q.shape[0], q.shape[1]
    out = torch.full((S, h, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((S, h), float("nan"), dtype=torch.float32, device="cuda")
    out, lse, ws = laga.absorbed_fwd(q, c_kv, k_pe, w, causal=causal, out=out, lse=lse)
    laga.check_status(ws, where="laga_absorbed_fwd")
    return out.cpu(), lse.cpu()


@pytest.mark.parametrize("S,h,causal", [(512, 2, True), (300, 3, True), (300, 3, False), (1, 1, True), (64, 1, True),
                                        (65, 2, True), (129, 2, True), (1024, 4, True), (200, 1, False), (700, 1, True)])
def test_absorbed_forward_elementwise(laga, oracle, S, h, causal):
    sh = LagaShape(S=S, h=h)
    tensors = make_inputs(sh, 2000 + S + h, with_dout=False)
    out, lse = run(laga, tensors, causal)
    ref_out, ref_lse = oracle.fwd(*tensors[:4], sh.d_v, sh.softmax_scale, causal=causal)
    check_tensor("out", out, ref_out)
    assert max_abs(lse, ref_lse) <= TOL_LSE_UNROUNDED
    if S >= 64:
        check_row_bands("out", out, ref_out)


def test_absorbed_and_explicit_paths_agree(laga):
    """Both CUDA paths on the same inputs: two bf16 evaluations of the same function."""
    sh = LagaShape(S=2048, h=4)
    q, c_kv, k_pe, w, _ = (t.cuda() if t is not None else None for t in make_inputs(sh, 44, with_dout=False))
    out_e, lse_e, ws_e = laga.fwd(q, c_kv, k_pe, w)
    out_a, lse_a, ws_a = laga.absorbed_fwd(q, c_kv, k_pe, w)
    laga.check_status(ws_e), laga.check_status(ws_a)
    assert float((out_a.float() - out_e.float()).abs().max()) <= 2e-2
    # each path is within TOL_LSE_UNROUNDED of the plain oracle (their roundings differ: K_nope/V there, q_abs here)
    assert float((lse_a - lse_e).abs().max()) <= 2 * TOL_LSE_UNROUNDED
    # the memory trap: q_abs and the latent accumulator against the explicit form's K_nope / V
    assert laga.absorbed_fwd_workspace_bytes(sh.S, sh.h) >= 4 * laga.fwd_workspace_bytes(sh.S, sh.h) - 4096


def test_absorbed_headline_inputs_sampled(laga, oracle):
    """Benchmark configuration 4: the absorbed form on configuration 2's inputs at full size, checked on
    sampled query rows against the oracle."""
    sh = CONFIGS["c2"]
    tensors = make_inputs(sh, CONFIG_SEEDS["c4"], with_dout=False)
    out, lse = run(laga, tensors, True)
    rows = sorted({0, 1, 63, 64, 127, 128, 129, 4095, 4096, 9000, sh.S - 129, sh.S - 128, sh.S - 1})
    ref_out, ref_lse = oracle.fwd(*tensors[:4], sh.d_v, sh.softmax_scale, causal=True, rows=rows)
    check_tensor("out[rows]", out[rows], ref_out)
    assert max_abs(lse[rows], ref_lse) <= TOL_LSE_UNROUNDED
    assert bool(torch.isfinite(out.float()).all()) and bool(torch.isfinite(lse).all())
