"""The tolerances of tests/parity.py against the rounding budget: the error of an idealised bf16-operand
evaluation of the path (float64 everywhere except the roundings a tensor-core path cannot avoid) from the
fp64 oracle, stored in tests/golden/rounding_budget.txt by tests/rounding_budget.py.  Every bound the GPU
path is held to must lie above that budget (else it would ask for more than the arithmetic allows), and the
stored table must be what the script produces."""
import os

import parity
import rounding_budget

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "rounding_budget.txt")


def rows():
    out = []
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        S, h, mode, name, *vals = line.split()
        out.append((int(S), int(h), mode, name, [None if v == "-" else float(v) for v in vals]))
    return out


def test_every_bound_lies_above_the_rounding_budget():
    worst_dw = 0.0
    for S, h, mode, name, (max_abs, scaled, row_scaled, rel_l2) in rows():
        if name == "lse":
            assert max_abs <= (parity.TOL_LSE if mode == "kv_round_bf16" else parity.TOL_LSE_UNROUNDED), (S, mode, max_abs)
            continue
        assert rel_l2 <= parity.TOL_REL_L2, (S, mode, name, rel_l2)
        if name == "dw":
            assert scaled <= parity.TOL_DW_SCALED, (S, mode, scaled)
            worst_dw = max(worst_dw, scaled)
        else:
            assert row_scaled <= parity.TOL_MAX_ABS, (S, mode, name, row_scaled)
        if name in ("out", "dq"):
            assert max_abs <= parity.TOL_MAX_ABS, (S, mode, name, max_abs)       # the plain bound binds these
    # a dW bound of 2e-2 on the scaled error would sit BELOW what the roundings alone produce on short sequences
    assert 2e-2 < worst_dw <= parity.TOL_DW_SCALED


def test_stored_table_is_what_the_script_writes(oracle):
    S, h, seed = rounding_budget.CASES[2]                 # the 25-token case: a fraction of a second
    fresh = rounding_budget.budget(S, h, seed)
    stored = {(mode, name): vals for s_, h_, mode, name, vals in rows() if (s_, h_) == (S, h)}
    for mode, per in fresh.items():
        for name, m in per.items():
            want = stored[(mode, name)][0]
            assert abs(m["max_abs"] - want) <= 1e-3 * max(want, 1e-12) + 1e-15, (mode, name, m["max_abs"], want)
