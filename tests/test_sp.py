"""The sequence-parallel exchanges around the hot path (Algorithm 1 steps 2, 3, 6 and the backward
duals of Section 5.2), on the CPU: the communication-volume closed form against the values the paper
prints, and a world_size-2 and -4 ``gloo`` run of the whole block with the fp64 oracle standing in for
the per-rank compute, checked against one single-process run over the full sequence and all heads
(Proposition 2: the sharded form reorders the same arithmetic)."""
import os

import pytest
import torch

from paper_2607_17644_b200 import sp
from paper_2607_17644_b200.inputs import LagaShape, make_inputs

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "comm_table.txt")


def _golden():
    table, ratios = [], []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        parts = line.split()
        if parts[0] == "ratio":
            ratios.append((int(parts[1]), float(parts[2])))
        else:
            table.append((int(parts[0]), int(parts[1]), float(parts[2]), float(parts[3]), float(parts[4])))
    return table, ratios


def test_comm_volume_matches_every_printed_cell():
    table, ratios = _golden()
    assert len(table) == 8 and len(ratios) == 4
    for P, S, b1, b2, laga in table:
        for form, printed in (("explicit", b1), ("absorbed", b2), ("laga", laga)):
            mb = sp.comm_bytes_per_rank(form, S, P) / 1e6
            assert abs(mb - printed) <= 0.05 + 1e-9, (form, P, S, mb, printed)   # one printed decimal
    for n_h, printed in ratios:
        dims = sp.CommDims(n_h=n_h)
        r = sp.comm_bytes_per_rank("explicit", 8192, 8, dims) / sp.comm_bytes_per_rank("laga", 8192, 8, dims)
        assert abs(r - printed) <= 0.005 + 1e-9, (n_h, r, printed)


class OracleCompute:
    """Stand-in for the GPU entry points in the CPU tests: the fp64 oracle on the rank's head shard."""

    def __init__(self, d_v, scale):
        import oracle
        self.oracle, self.d_v, self.scale = oracle, d_v, scale

    def fwd(self, q, c_kv, k_pe, w, causal):
        return self.oracle.fwd(q, c_kv, k_pe, w, self.d_v, self.scale, causal=causal)

    def bwd(self, q, c_kv, k_pe, w, out, lse, dout, causal):
        g = self.oracle.bwd(q, c_kv, k_pe, w, dout, self.d_v, self.scale, causal=causal)
        return g["dq"], g["dc_kv"], g["dk_pe"], g["dw"]


FULL = LagaShape(S=48, h=4, d_c=16, d_nope=8, d_rope=4, d_v=8)


def _rank_main(rank, world, port, failures):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch.distributed as dist
    import oracle
    dist.init_process_group(backend="gloo", rank=rank, world_size=world)
    try:
        sh = FULL
        q, c_kv, k_pe, w, dout = make_inputs(sh, seed=4242)           # every rank draws the same full tensors
        ref_o, _ = oracle.fwd(q, c_kv, k_pe, w, sh.d_v, sh.softmax_scale)
        ref = oracle.bwd(q, c_kv, k_pe, w, dout, sh.d_v, sh.softmax_scale)
        n = sh.S // world
        rows = slice(rank * n, (rank + 1) * n)
        compute = OracleCompute(sh.d_v, sh.softmax_scale)
        out_local, ctx = sp.sp_forward(q[rows].contiguous(), c_kv[rows].contiguous(), k_pe[rows].contiguous(), w, sh.h,
                                       compute)
        dq, dc, dk, dw = sp.sp_backward(ctx, dout[rows].contiguous(), compute)
        checks = {"out": (out_local, ref_o[rows]), "dq": (dq, ref["dq"][rows]), "dc_kv": (dc, ref["dc_kv"][rows]),
                  "dk_pe": (dk, ref["dk_pe"][rows]), "dw": (dw, ref["dw"])}
        for name, (got, want) in checks.items():
            if got.shape != want.shape:
                failures.append(f"rank {rank}: {name} shape {tuple(got.shape)} vs {tuple(want.shape)}")
                continue
            err = float((got.to(torch.float64) - want).abs().max())
            if err > 1e-9 * max(1.0, float(want.abs().max())):
                failures.append(f"rank {rank}: {name} max-abs {err:.3e}")
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 4])
def test_sp_block_with_gloo_ranks_matches_the_single_process_result(oracle, world):
    import torch.multiprocessing as mp
    from conftest import free_port
    port = free_port()
    ctx = mp.get_context("spawn")
    failures = ctx.Manager().list()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, failures)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(180)
        assert p.exitcode == 0
    assert list(failures) == []
