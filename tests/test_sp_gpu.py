"""The sequence-parallel block wrapper on the GPU with world size 1 (NCCL).  Every exchange is then the
identity, so the block's results are the hot path's results: they are held to the fp64 oracle with the
same bounds as the direct C-ABI calls (a wrapper that scrambled tokens, heads or the W_kv_b columns on
its way through the exchanges would fail here)."""
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
    _laga.lib()          # must load: there is no fallback
    return _laga


def test_sp_block_world_size_one_against_the_oracle(laga, oracle):
    import torch.distributed as dist
    from paper_2607_17644_b200 import sp
    sh = LagaShape(S=640, h=4)
    tensors = make_inputs(sh, 97)
    q, c_kv, k_pe, w, dout = (t.cuda() for t in tensors)
    from conftest import free_port
    dist.init_process_group(backend="nccl", init_method=f"tcp://127.0.0.1:{free_port()}", rank=0, world_size=1)
    try:
        compute = sp.CudaCompute()
        out_local, ctx = sp.sp_forward(q, c_kv, k_pe, w, sh.h, compute)
        dq, dc, dk, dw = sp.sp_backward(ctx, dout, compute)
        lse = ctx[5]
        torch.cuda.synchronize()
    finally:
        dist.destroy_process_group()
    ref = oracle.bwd(*tensors, sh.d_v, sh.softmax_scale, causal=True, kv_round_bf16=True, return_fwd=True)
    check_tensor("out", out_local, ref["out"])
    assert max_abs(lse, ref["lse"]) <= TOL_LSE
    check_tensor("dq", dq, ref["dq"])
    check_tensor("dc_kv", dc, ref["dc_kv"])
    check_tensor("dk_pe", dk, ref["dk_pe"])
    check_dw(dw, ref["dw"])
