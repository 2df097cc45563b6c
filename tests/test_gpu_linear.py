"""GPU parity of laga_linear / laga_linear_backward (the dense projections of Algorithm 1 steps 1 and 7 on the
CTA-pair tcgen05 GEMM) against the float64 oracle, at the DeepSeek-V3 projection shapes and at ragged ones."""
import pytest
import torch

from parity import check_tensor, rel_l2, scaled_max_abs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def laga():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2607_17644_b200 import laga as _laga
    _laga.lib()
    return _laga


def draw(M, K, N, seed):
    """x, dy ~ N(0,1); w ~ N(0, 1/K) so that y has unit variance: the value distributions of the path's own
    projections (hidden states and upstream gradients of order one, variance-preserving weights)."""
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(M, K, generator=g).to(torch.bfloat16)
    w = (torch.randn(K, N, generator=g) * K ** -0.5).to(torch.bfloat16)
    dy = torch.randn(M, N, generator=g).to(torch.bfloat16)
    return x, w, dy


CASES = [
    # M, K, N
    (300, 512, 576),      # ragged rows; N = 576 = d_c + d_rope (W_kv_a's output): two full column tiles and a quarter
    (1000, 1536, 768),    # the query up-projection from the 1536-wide low-rank query, four heads of 192
    (257, 7168, 576),     # W_kv_a at the DeepSeek-V3 hidden size, one row past a row tile
    (512, 2048, 7168),    # W_o for a 16-head shard: 16 x 128 -> hidden
    (64, 72, 40),         # everything smaller than one tile, K and N only multiples of 8
    (1, 512, 256),        # a single token
    (4096, 512, 4096),    # Algorithm 1 step 4 at benchmark configuration 1, through this entry point
]


@pytest.mark.parametrize("M,K,N", CASES)
def test_linear_forward_and_backward(laga, oracle, M, K, N):
    x, w, dy = draw(M, K, N, 9000 + M + K + N)
    y, st = laga.linear(x.cuda(), w.cuda(), y=torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda"))
    assert laga.query_status(st)[0] == laga.OK
    dx, dw, st2 = laga.linear_backward(dy.cuda(), x.cuda(), w.cuda(),
                                       dx=torch.full((M, K), float("nan"), dtype=torch.bfloat16, device="cuda"),
                                       dw=torch.full((K, N), float("nan"), dtype=torch.float32, device="cuda"))
    assert laga.query_status(st2)[0] == laga.OK
    ry = oracle.linear(x, w)
    rdx, rdw = oracle.linear_bwd(dy, x, w)
    check_tensor("y", y.cpu(), ry)
    check_tensor("dx", dx.cpu(), rdx)
    # dw stays fp32: only accumulation order separates it from the oracle
    assert rel_l2(dw.cpu().double(), rdw) <= 1e-5 and scaled_max_abs(dw.cpu().double(), rdw) <= 1e-4


def test_linear_backward_flags(laga, oracle):
    M, K, N = 700, 512, 576
    x, w, dy = draw(M, K, N, 9100)
    xg, wg, dyg = x.cuda(), w.cuda(), dy.cuda()
    det = laga.FLAG_DETERMINISTIC
    a = laga.linear_backward(dyg, xg, wg, flags=det)[1]
    b = laga.linear_backward(dyg, xg, wg, flags=det)[1]
    assert torch.equal(a, b)                                              # one addition per element: repeatable
    acc = a.clone()
    laga.linear_backward(dyg, xg, wg, dw=acc, flags=det | laga.FLAG_ACCUM_DW)
    assert rel_l2(acc.cpu().double(), 2 * oracle.linear_bwd(dy, x, w)[1]) <= 1e-5
    with pytest.raises(laga.LagaError):
        laga.linear(torch.zeros(8, 12, dtype=torch.bfloat16, device="cuda"), torch.zeros(12, 16, dtype=torch.bfloat16, device="cuda"))


def test_step_four_is_this_gemm(laga):
    """laga_up_project (Algorithm 1 step 4) and laga_linear with K = d_c are the same launch."""
    g = torch.Generator().manual_seed(9200)
    c_kv = torch.randn(900, 512, generator=g).to(torch.bfloat16).cuda()
    w = (torch.randn(512, 512, generator=g) * 512 ** -0.5).to(torch.bfloat16).cuda()
    assert torch.equal(laga.up_project(c_kv, w, 2)[0], laga.linear(c_kv, w)[0])
