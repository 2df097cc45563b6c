"""Stand-in for a memory checker: run the hot path with every output and every workspace carved out of one
arena and fenced by guard bands of a known byte pattern, then verify that (1) the device status word is
clean, (2) the results agree with the fp64 oracle, (3) no guard byte changed.  Run as a script (the GPU test
test_gpu_debug_build.py starts it once against the normal library and once with LAGA_DEBUG=1, the checked
build whose kernels verify their own index arithmetic).  Prints GUARD_BANDS_OK on success."""
import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

from paper_2607_17644_b200 import laga  # noqa: E402
from paper_2607_17644_b200.inputs import LagaShape, make_inputs  # noqa: E402
import oracle  # noqa: E402

GUARD = 4096
PATTERN = 0xC3


class Arena:
    def __init__(self, n_bytes):
        self.buf = torch.full((n_bytes,), PATTERN, dtype=torch.uint8, device="cuda")
        self.base = (-self.buf.data_ptr()) % 1024
        self.pos = self.base
        self.used = []

    def take(self, n_bytes, dtype=torch.uint8, shape=None):
        self.pos += GUARD
        start = self.pos
        size = (n_bytes + 1023) // 1024 * 1024
        self.pos += size
        self.used.append((start, start + n_bytes))
        t = self.buf[start:start + n_bytes]
        return t if shape is None else t.view(dtype).view(shape)

    def guards_intact(self):
        mask = torch.ones_like(self.buf, dtype=torch.bool)
        for lo, hi in self.used:
            mask[lo:hi] = False
        return bool((self.buf[mask] == PATTERN).all())


def rel_l2(g, r):
    g = g.double().cpu()
    if float(r.norm()) == 0.0:            # one token: the exact dq and dk_pe are zero
        return float((g - r).abs().max())
    return float((g - r).norm() / r.norm())


def run_case(S, h, causal):
    sh = LagaShape(S=S, h=h)
    tensors = make_inputs(sh, 900 + S + h)
    q, c_kv, k_pe, w, dout = (t.cuda() for t in tensors)
    bf, f32 = torch.bfloat16, torch.float32
    ws_sizes = [laga.fwd_workspace_bytes(S, h), laga.bwd_workspace_bytes(S, h), laga.absorbed_fwd_workspace_bytes(S, h),
                laga.bwd_workspace_bytes(S, h, flags=laga.FLAG_FUSED_BWD)]
    arena = Arena(sum(ws_sizes) + 16 * S * h * 192 * 4 + 64 * GUARD + 512 * h * 256 * 4 + (1 << 20))
    out = arena.take(S * h * 128 * 2, bf, (S, h, 128))
    lse = arena.take(S * h * 4, f32, (S, h))
    dq = arena.take(S * h * 192 * 2, bf, (S, h, 192))
    dc_kv = arena.take(S * 512 * 2, bf, (S, 512))
    dk_pe = arena.take(S * 64 * 2, bf, (S, 64))
    dw = arena.take(512 * h * 256 * 4, f32, (512, h * 256))
    out_a = arena.take(S * h * 128 * 2, bf, (S, h, 128))
    lse_a = arena.take(S * h * 4, f32, (S, h))
    dq_1 = arena.take(S * h * 192 * 2, bf, (S, h, 192))
    dc_kv_1 = arena.take(S * 512 * 2, bf, (S, 512))
    dk_pe_1 = arena.take(S * 64 * 2, bf, (S, 64))
    dw_1 = arena.take(512 * h * 256 * 4, f32, (512, h * 256))
    ws_f, ws_b, ws_a, ws_1 = (arena.take(n) for n in ws_sizes)
    laga.fwd(q, c_kv, k_pe, w, causal=causal, out=out, lse=lse, workspace=ws_f)
    laga.check_status(ws_f, where="laga_fwd")
    laga.bwd(q, c_kv, k_pe, w, out, lse, dout, causal=causal, dq=dq, dc_kv=dc_kv, dk_pe=dk_pe, dw_kv_b=dw, workspace=ws_b)
    laga.check_status(ws_b, where="laga_bwd")
    laga.bwd(q, c_kv, k_pe, w, out, lse, dout, causal=causal, dq=dq_1, dc_kv=dc_kv_1, dk_pe=dk_pe_1, dw_kv_b=dw_1,
             workspace=ws_1, flags=laga.FLAG_FUSED_BWD)
    laga.check_status(ws_1, where="laga_bwd (one-pass backward)")
    laga.absorbed_fwd(q, c_kv, k_pe, w, causal=causal, out=out_a, lse=lse_a, workspace=ws_a)
    laga.check_status(ws_a, where="laga_absorbed_fwd")
    torch.cuda.synchronize()
    assert arena.guards_intact(), f"a guard band was overwritten (S={S}, h={h})"
    ref = oracle.bwd(*tensors, sh.d_v, sh.softmax_scale, causal=causal, kv_round_bf16=True, return_fwd=True)
    for name, got in (("out", out), ("dq", dq), ("dc_kv", dc_kv), ("dk_pe", dk_pe), ("dw", dw), ("out", out_a),
                      ("dq", dq_1), ("dc_kv", dc_kv_1), ("dk_pe", dk_pe_1), ("dw", dw_1)):
        err = rel_l2(got, ref[name])
        assert err <= 5e-3, (name, err)
    assert float((lse.double().cpu() - ref["lse"]).abs().max()) <= 1e-3
    assert float((lse_a.double().cpu() - ref["lse"]).abs().max()) <= 5e-3
    # step 4 rebuilt inside the dK/dV kernel (its TMA stores of the K/V tiles end at the last row): same buffers again
    for t in (dq_1, dc_kv_1, dk_pe_1, dw_1):
        t.fill_(float("nan"))
    laga.bwd(q, c_kv, k_pe, w, out, lse, dout, causal=causal, dq=dq_1, dc_kv=dc_kv_1, dk_pe=dk_pe_1, dw_kv_b=dw_1,
             workspace=ws_b, flags=laga.FLAG_FUSED_KV_REBUILD)
    laga.check_status(ws_b, where="laga_bwd (K/V rebuilt in the dK/dV kernel)")
    torch.cuda.synchronize()
    assert arena.guards_intact(), f"a guard band was overwritten by the rebuild path (S={S}, h={h})"
    for name, got in (("dq", dq_1), ("dc_kv", dc_kv_1), ("dk_pe", dk_pe_1), ("dw", dw_1)):
        err = rel_l2(got, ref[name])
        assert err <= 5e-3, ("rebuild", name, err)


def run_packed_case(lengths, h, causal):
    """The packed variable-length entry points between guard bands, against the oracle sequence by sequence."""
    cu = [0]
    for n in lengths:
        cu.append(cu[-1] + n)
    S = cu[-1]
    sh = LagaShape(S=S, h=h)
    tensors = make_inputs(sh, 950 + S + h)
    q, c_kv, k_pe, w, dout = (t.cuda() for t in tensors)
    bf, f32 = torch.bfloat16, torch.float32
    ws_sizes = [laga.fwd_varlen_workspace_bytes(S, len(lengths), h), laga.bwd_varlen_workspace_bytes(S, len(lengths), h)]
    arena = Arena(sum(ws_sizes) + 8 * S * h * 192 * 4 + 32 * GUARD + 512 * h * 256 * 4 + (1 << 20))
    out = arena.take(S * h * 128 * 2, bf, (S, h, 128))
    lse = arena.take(S * h * 4, f32, (S, h))
    dq = arena.take(S * h * 192 * 2, bf, (S, h, 192))
    dc_kv = arena.take(S * 512 * 2, bf, (S, 512))
    dk_pe = arena.take(S * 64 * 2, bf, (S, 64))
    dw = arena.take(512 * h * 256 * 4, f32, (512, h * 256))
    ws_f, ws_b = (arena.take(n) for n in ws_sizes)
    laga.fwd(q, c_kv, k_pe, w, causal=causal, out=out, lse=lse, workspace=ws_f, cu_seqlens=cu)
    laga.check_status(ws_f, where="laga_fwd_varlen")
    laga.bwd(q, c_kv, k_pe, w, out, lse, dout, causal=causal, dq=dq, dc_kv=dc_kv, dk_pe=dk_pe, dw_kv_b=dw, workspace=ws_b,
             cu_seqlens=cu)
    laga.check_status(ws_b, where="laga_bwd_varlen")
    torch.cuda.synchronize()
    assert arena.guards_intact(), f"a guard band was overwritten (packed {lengths}, h={h})"
    dw_ref = torch.zeros(512, h * 256, dtype=torch.float64)
    for a, b in zip(cu[:-1], cu[1:]):
        if a == b:
            continue
        tq, tc, tk, tw, tdo = tensors
        ref = oracle.bwd(tq[a:b], tc[a:b], tk[a:b], tw, tdo[a:b], sh.d_v, sh.softmax_scale, causal=causal,
                         kv_round_bf16=True, return_fwd=True)
        dw_ref += ref["dw"]
        if b - a > 1:
            for name, got in (("out", out), ("dq", dq), ("dc_kv", dc_kv), ("dk_pe", dk_pe)):
                assert rel_l2(got[a:b], ref[name]) <= 5e-3, (name, a, b)
        assert float((lse[a:b].double().cpu() - ref["lse"]).abs().max()) <= 1e-3
    assert rel_l2(dw, dw_ref) <= 5e-3


if __name__ == "__main__":
    laga.lib()
    expect_debug = os.environ.get("LAGA_DEBUG", "0") not in ("", "0")
    assert laga.DEBUG == expect_debug and laga.LIB_PATH.endswith("liblaga_debug.so" if expect_debug else "liblaga.so")
    for S, h, causal in ((300, 3, True), (1024, 4, True), (129, 2, False), (1, 1, True), (2500, 1, True)):
        run_case(S, h, causal)
    for lengths, h, causal in (([300, 1, 140], 2, True), ([129, 0, 700], 1, False)):
        run_packed_case(lengths, h, causal)
    print("GUARD_BANDS_OK", "checked build" if expect_debug else "normal build")
