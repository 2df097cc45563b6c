"""laga_fwd_builtin_scratch: the forward for callers that cannot allocate device memory (plug-ins and
callbacks where allocation calls are off-limits, processes whose memory belongs to another pool,
latency-critical loops).  It must give what laga_fwd gives, using only the library's fixed scratch
array, on repeated calls, and refuse problems larger than that array.

Collected last on purpose: a failure here cannot hide a failure of any other test under `-x`.
The file stands alone too: it does not depend on anything another test ran before it.
"""
import pytest
import torch

from paper_2607_17644_b200.inputs import LagaShape, make_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def laga():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2607_17644_b200 import laga as _laga
    _laga.lib()
    return _laga


def _both_ways(laga, sh, seed, causal):
    q, c_kv, k_pe, w, _ = (t.cuda() if t is not None else None for t in make_inputs(sh, seed, with_dout=False))
    ref_out, ref_lse, ws = laga.fwd(q, c_kv, k_pe, w, causal=causal)
    laga.check_status(ws, where="laga_fwd")
    out = torch.full_like(ref_out, float("nan"))
    lse = torch.full_like(ref_lse, float("nan"))
    laga.fwd_builtin_scratch(q, c_kv, k_pe, w, out, lse, causal=causal)
    torch.cuda.synchronize()
    return out, lse, ref_out, ref_lse


def _check_same(out, lse, ref_out, ref_lse):
    assert torch.isfinite(out.float()).all() and torch.isfinite(lse).all()
    # same kernels on the same inputs: the tolerance of the parity tests (2e-2 / 1e-3) is met with
    # room to spare -- the results are in fact identical
    assert float((out.float() - ref_out.float()).abs().max()) <= 2e-2
    assert float((lse - ref_lse).abs().max()) <= 1e-3
    assert torch.equal(out, ref_out) and torch.equal(lse, ref_lse)


def test_two_calls_in_a_row_match_laga_fwd(laga):
    """Second call: a smaller, differently shaped problem on the same (now dirty) built-in scratch."""
    first = _both_ways(laga, LagaShape(S=1024, h=4), seed=31, causal=True)
    _check_same(*first)
    second = _both_ways(laga, LagaShape(S=300, h=3), seed=32, causal=False)
    _check_same(*second)


def test_matches_the_oracle_directly(laga, oracle):
    """One comparison that does not go through laga_fwd at all: the entry point against the fp64 oracle."""
    from parity import TOL_LSE, check_tensor, max_abs
    sh = LagaShape(S=700, h=3)
    tensors = make_inputs(sh, 36, with_dout=False)
    q, c_kv, k_pe, w = (t.cuda() for t in tensors[:4])
    out = torch.full((sh.S, sh.h, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((sh.S, sh.h), float("nan"), dtype=torch.float32, device="cuda")
    laga.fwd_builtin_scratch(q, c_kv, k_pe, w, out, lse)
    torch.cuda.synchronize()
    ref_out, ref_lse = oracle.fwd(*tensors[:4], sh.d_v, sh.softmax_scale, causal=True, kv_round_bf16=True)
    check_tensor("out", out, ref_out)
    assert max_abs(lse, ref_lse) <= TOL_LSE


def test_the_call_allocates_no_device_memory(laga):
    """After one warm call (which may make the CUDA runtime load the library's device code, the scratch
    array included), further calls must leave the device's free memory and torch's allocator untouched,
    at two different shapes."""
    shapes = [LagaShape(S=512, h=4), LagaShape(S=1000, h=2)]
    cases = []
    for i, sh in enumerate(shapes):
        q, c_kv, k_pe, w = (t.cuda() for t in make_inputs(sh, 40 + i, with_dout=False)[:4])
        out = torch.empty(sh.S, sh.h, 128, dtype=torch.bfloat16, device="cuda")
        lse = torch.empty(sh.S, sh.h, dtype=torch.float32, device="cuda")
        cases.append((q, c_kv, k_pe, w, out, lse))
    laga.fwd_builtin_scratch(*cases[0])                      # warm: module load, address lookup
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    allocated_before, reserved_before = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for case in cases + cases:
        laga.fwd_builtin_scratch(*case)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert torch.cuda.memory_allocated() == allocated_before and torch.cuda.memory_reserved() == reserved_before
    assert free_after == free_before, f"device free memory moved by {free_before - free_after} bytes"


def test_back_to_back_on_one_stream_without_sync(laga):
    """Two enqueues with no host synchronisation between them: stream order alone must be enough."""
    sh_a, sh_b = LagaShape(S=640, h=2), LagaShape(S=512, h=5)
    a = [t.cuda() for t in make_inputs(sh_a, 33, with_dout=False)[:4]]
    b = [t.cuda() for t in make_inputs(sh_b, 34, with_dout=False)[:4]]
    out_a = torch.empty(sh_a.S, sh_a.h, 128, dtype=torch.bfloat16, device="cuda")
    lse_a = torch.empty(sh_a.S, sh_a.h, dtype=torch.float32, device="cuda")
    out_b = torch.empty(sh_b.S, sh_b.h, 128, dtype=torch.bfloat16, device="cuda")
    lse_b = torch.empty(sh_b.S, sh_b.h, dtype=torch.float32, device="cuda")
    laga.fwd_builtin_scratch(*a, out_a, lse_a)
    laga.fwd_builtin_scratch(*b, out_b, lse_b)
    torch.cuda.synchronize()
    ref_a = laga.fwd(*a)
    ref_b = laga.fwd(*b)
    torch.cuda.synchronize()
    assert torch.equal(out_a, ref_a[0]) and torch.equal(lse_a, ref_a[1])
    assert torch.equal(out_b, ref_b[0]) and torch.equal(lse_b, ref_b[1])


def test_limit_is_enforced_and_nothing_is_written(laga):
    limit = laga.BUILTIN_SCRATCH_MAX_TOKEN_HEADS
    sh = LagaShape(S=limit // 16, h=16)                       # exactly at the limit: accepted
    q, c_kv, k_pe, w, _ = (t.cuda() if t is not None else None for t in make_inputs(sh, 35, with_dout=False))
    out = torch.empty(sh.S, sh.h, 128, dtype=torch.bfloat16, device="cuda")
    lse = torch.empty(sh.S, sh.h, dtype=torch.float32, device="cuda")
    laga.fwd_builtin_scratch(q, c_kv, k_pe, w, out, lse)
    ref_out, ref_lse, _ = laga.fwd(q, c_kv, k_pe, w)
    torch.cuda.synchronize()
    assert torch.equal(out, ref_out) and torch.equal(lse, ref_lse)

    big = LagaShape(S=limit // 16 + 1, h=16)                  # one token past it: refused
    qb = torch.zeros(big.S, big.h, 192, dtype=torch.bfloat16, device="cuda")
    cb = torch.zeros(big.S, 512, dtype=torch.bfloat16, device="cuda")
    kb = torch.zeros(big.S, 64, dtype=torch.bfloat16, device="cuda")
    ob = torch.full((big.S, big.h, 128), 7.0, dtype=torch.bfloat16, device="cuda")
    lb = torch.full((big.S, big.h), 7.0, dtype=torch.float32, device="cuda")
    with pytest.raises(laga.LagaError) as err:
        laga.fwd_builtin_scratch(qb, cb, kb, w, ob, lb)
    assert err.value.code == laga.ERR_WORKSPACE_TOO_SMALL
    torch.cuda.synchronize()
    assert bool((ob == 7.0).all()) and bool((lb == 7.0).all())
