"""The SP wrapper on the GPU with world size 1 (NCCL): every exchange is then the identity, so the
block must return exactly what the C-ABI entry points return when called directly."""
import pytest
import torch

from paper_2607_17644_b200.inputs import LagaShape, make_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def laga():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2607_17644_b200 import laga as _laga
    _laga.lib()          # must load: there is no fallback
    return _laga


def test_sp_block_world_size_one_equals_direct_calls(laga):
    import torch.distributed as dist
    from paper_2607_17644_b200 import sp
    sh = LagaShape(S=640, h=4)
    q, c_kv, k_pe, w, dout = (t.cuda() for t in make_inputs(sh, 97))
    from conftest import free_port
    dist.init_process_group(backend="nccl", init_method=f"tcp://127.0.0.1:{free_port()}", rank=0, world_size=1)
    try:
        compute = sp.CudaCompute()
        out_local, ctx = sp.sp_forward(q, c_kv, k_pe, w, sh.h, compute)
        dq, dc, dk, dw = sp.sp_backward(ctx, dout, compute)
        torch.cuda.synchronize()
    finally:
        dist.destroy_process_group()
    out, lse, _ = laga.fwd(q, c_kv, k_pe, w)
    dq2, dc2, dk2, dw2, _ = laga.bwd(q, c_kv, k_pe, w, out, lse, dout)
    assert torch.equal(out_local, out) and torch.equal(dq, dq2)
    # dk_pe, dc_kv and dW pass through fp32 atomics whose order varies from run to run
    assert (dk.float() - dk2.float()).abs().max() <= 2e-2
    assert (dc.float() - dc2.float()).abs().max() <= 2e-2 * max(1.0, float(dc2.float().abs().max()) / 4)
    assert (dw - dw2).abs().max() <= 1e-2 * float(dw2.abs().max())
