"""The eager comparison forms (explicit B1 and absorbed B2, Section 3.2) against the fp64 oracle.

The absorbed form reaches the same output and gradients by a different association of the same
products (W_uk folded into the query, W_uv applied after the latent accumulator), so agreement in
fp64 both validates the comparator the bench times and pins the oracle to an identity it does not
use itself.  CPU only.
"""
import pytest
import torch

from paper_2607_17644_b200 import eager_forms
from paper_2607_17644_b200.inputs import LagaShape, make_inputs

SHAPES = [LagaShape(S=13, h=3, d_c=8, d_nope=4, d_rope=2, d_v=5),
          LagaShape(S=70, h=2, d_c=32, d_nope=16, d_rope=8, d_v=16)]


@pytest.mark.parametrize("sh", SHAPES, ids=lambda s: f"S{s.S}h{s.h}")
@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("form", [eager_forms.explicit_form, eager_forms.absorbed_form],
                         ids=["explicit", "absorbed"])
def test_eager_form_matches_oracle_fp64(oracle, sh, causal, form):
    q, c_kv, k_pe, w, dout = make_inputs(sh, seed=77)
    ref_o, _ = oracle.fwd(q, c_kv, k_pe, w, sh.d_v, sh.softmax_scale, causal=causal)
    ref_g = oracle.bwd(q, c_kv, k_pe, w, dout, sh.d_v, sh.softmax_scale, causal=causal)
    got = eager_forms.run_form(form, *(t.to(torch.float64) for t in (q, c_kv, k_pe, w, dout)),
                               sh.d_v, sh.softmax_scale, causal)
    refs = (ref_o, ref_g["dq"], ref_g["dc_kv"], ref_g["dk_pe"], ref_g["dw"])
    for name, g, r in zip(("out", "dq", "dc_kv", "dk_pe", "dw_kv_b"), got, refs):
        assert g.shape == r.shape, name
        assert (g - r).abs().max().item() <= 1e-10 * max(1.0, r.abs().max().item()), name
