"""Host-side checks of the C ABI that need no GPU: the library builds and loads, exports exactly the
entry points include/laga.h declares, sizes workspaces as documented and rejects bad arguments
before touching a device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "laga.h")


@pytest.fixture(scope="module")
def laga():
    from paper_2607_17644_b200 import build
    build.build()
    from paper_2607_17644_b200 import laga as _laga
    _laga.lib()
    return _laga


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(laga_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_expected_entry_points():
    names = declared_functions()
    for required in ["laga_fwd", "laga_bwd", "laga_fwd_workspace_bytes", "laga_bwd_workspace_bytes",
                     "laga_status_string", "laga_query_status", "laga_version", "laga_up_project",
                     "laga_kv_backward"]:
        assert required in names


def test_library_exports_every_declared_symbol(laga):
    handle = ctypes.CDLL(laga.LIB_PATH)
    for name in declared_functions():
        assert hasattr(handle, name), f"{name} declared in include/laga.h but not exported"
    assert set(declared_functions()) == set(laga.SIGNATURES), "binding and header list different entry points"


def test_library_has_no_driver_link_dependency(laga):
    """It must load on a machine without the NVIDIA driver (this one): libcuda is resolved at run time."""
    import subprocess
    needed = subprocess.run(["readelf", "-d", laga.LIB_PATH], capture_output=True, text=True).stdout
    assert "libcuda.so" not in needed


def test_version_and_status_strings(laga):
    assert laga.version() >= 100
    assert laga.status_string(0) == "LAGA_OK"
    assert laga.status_string(laga.ERR_INVALID_ARG) == "LAGA_ERR_INVALID_ARG"
    assert laga.status_string(laga.ERR_UNSUPPORTED) == "LAGA_ERR_UNSUPPORTED"
    assert laga.status_string(laga.ERR_WORKSPACE_TOO_SMALL) == "LAGA_ERR_WORKSPACE_TOO_SMALL"
    assert laga.status_string(laga.ERR_DEVICE_TIMEOUT) == "LAGA_ERR_DEVICE_TIMEOUT"
    assert laga.status_string(-99) == "LAGA_ERR_UNKNOWN"


def test_workspace_sizes(laga):
    S, h = 16384, 16
    kv_bytes = S * h * 256 * 2
    assert laga.fwd_workspace_bytes(S, h) == 1024 + kv_bytes
    bwd = laga.bwd_workspace_bytes(S, h)
    assert bwd >= 1024 + 2 * kv_bytes              # recomputed KV and dKV, both bf16
    assert bwd <= 1024 + 2 * kv_bytes + S * h * 2 * 4 + S * 64 * 4 + 8192
    assert laga.bwd_workspace_bytes(S, h, flags=laga.FLAG_DETERMINISTIC) >= bwd + S * h * 64 * 4
    # the one-pass backward adds an fp32 dQ accumulator for a window of heads, at most 64 MB of it
    fused = laga.bwd_workspace_bytes(S, h, flags=laga.FLAG_FUSED_BWD)
    assert bwd + S * 192 * 4 <= fused <= bwd + (64 << 20) + 1024
    assert laga.bwd_workspace_bytes(512, 2, flags=laga.FLAG_FUSED_BWD) == laga.bwd_workspace_bytes(512, 2) + 512 * 2 * 192 * 4
    assert laga.fwd_workspace_bytes(300, 3) % 1024 == 0 and laga.bwd_workspace_bytes(300, 3) % 1024 == 0
    # unsupported geometry or empty problem: 0
    assert laga.fwd_workspace_bytes(128, 2, d_c=256) == laga.fwd_workspace_bytes(128, 2)      # the latent width is free
    assert laga.fwd_workspace_bytes(128, 2, d_c=260) == 0                                   # ... in multiples of 8
    assert laga.fwd_workspace_bytes(128, 2, d_nope=64) == 0
    assert laga.bwd_workspace_bytes(128, 2, d_rope=32) == 0
    assert laga.fwd_workspace_bytes(0, 2) == 0 and laga.fwd_workspace_bytes(128, 0) == 0


def test_argument_validation_happens_before_any_device_work(laga):
    lib = laga.lib()
    p = ctypes.c_void_p
    good = p(1024)                                   # never dereferenced on these paths
    args = dict(S=128, h=2, d_c=512, d_nope=128, d_rope=64, d_v=128)

    def fwd(q=good, c=good, k=good, w=good, out=good, lse=good, ws=good, ws_bytes=1 << 40, flags=0, scale=0.07,
            **over):
        a = {**args, **over}
        return lib.laga_fwd(q, c, k, w, a["S"], a["h"], a["d_c"], a["d_nope"], a["d_rope"], a["d_v"], scale, 1,
                            out, lse, ws, ws_bytes, flags, None)

    assert fwd(q=None) == laga.ERR_INVALID_ARG
    assert fwd(lse=None) == laga.ERR_INVALID_ARG
    assert fwd(S=0) == laga.ERR_INVALID_ARG
    assert fwd(h=-1) == laga.ERR_INVALID_ARG
    assert fwd(q=p(1032)) == laga.ERR_INVALID_ARG    # not 16-byte aligned
    assert fwd(ws=p(1040)) == laga.ERR_INVALID_ARG   # workspace not 1024-byte aligned
    assert fwd(flags=8) == laga.ERR_INVALID_ARG
    assert fwd(scale=0.0) == laga.ERR_INVALID_ARG
    assert fwd(d_c=260) == laga.ERR_UNSUPPORTED
    assert fwd(d_nope=64) == laga.ERR_UNSUPPORTED
    assert fwd(d_rope=32) == laga.ERR_UNSUPPORTED
    assert fwd(ws_bytes=1024) == laga.ERR_WORKSPACE_TOO_SMALL

    def bwd(dq=good, ws_bytes=1 << 40, flags=0, **over):
        a = {**args, **over}
        return lib.laga_bwd(good, good, good, good, good, good, good, a["S"], a["h"], a["d_c"], a["d_nope"],
                            a["d_rope"], a["d_v"], 0.07, 1, dq, good, good, good, good, ws_bytes, flags, None)

    assert bwd(dq=None) == laga.ERR_INVALID_ARG
    assert bwd(flags=32) == laga.ERR_INVALID_ARG    # 1, 2, 4, 8 and 16 are defined
    assert bwd(flags=laga.FLAG_FUSED_KV_REBUILD | laga.FLAG_KV_SAVED) == laga.ERR_INVALID_ARG
    assert bwd(flags=laga.FLAG_FUSED_KV_REBUILD | laga.FLAG_FUSED_BWD) == laga.ERR_INVALID_ARG
    assert bwd(flags=laga.FLAG_FUSED_BWD | laga.FLAG_DETERMINISTIC) == laga.ERR_INVALID_ARG
    assert bwd(d_v=64) == laga.ERR_UNSUPPORTED
    assert bwd(ws_bytes=4096) == laga.ERR_WORKSPACE_TOO_SMALL
    assert lib.laga_up_project(None, good, 128, 2, 512, 128, 128, good, good, None) == laga.ERR_INVALID_ARG
    assert lib.laga_kv_backward(good, good, good, 128, 2, 512, 128, 128, good, good, 4, good, None) == laga.ERR_INVALID_ARG
    assert lib.laga_query_status(None, None, None) == laga.ERR_INVALID_ARG
    assert lib.laga_linear(good, good, 128, 512, 260, good, good, None) == laga.ERR_INVALID_ARG      # N not a multiple of 8
    assert lib.laga_linear(good, good, 128, 4, 256, good, good, None) == laga.ERR_INVALID_ARG        # K < 8
    assert lib.laga_linear(good, None, 128, 512, 256, good, good, None) == laga.ERR_INVALID_ARG
    assert lib.laga_linear_backward(good, good, good, 0, 512, 256, good, good, 0, good, None) == laga.ERR_INVALID_ARG
    assert lib.laga_linear_backward(good, good, good, 8, 512, 256, good, good, 4, good, None) == laga.ERR_INVALID_ARG   # KV_SAVED means nothing here


def test_varlen_entry_points_validate_cu_seqlens_before_any_device_work(laga):
    lib = laga.lib()
    p = ctypes.c_void_p
    good = p(1024)

    def cu(*v):
        return (ctypes.c_int * len(v))(*v)

    def fwd(cu_seqlens, n_seqs, S_total=256, ws_bytes=1 << 40):
        return lib.laga_fwd_varlen(good, good, good, good, cu_seqlens, n_seqs, S_total, 2, 512, 128, 64, 128, 0.07, 1,
                                   good, good, good, ws_bytes, 0, None)

    def bwd(cu_seqlens, n_seqs, S_total=256, flags=0, ws_bytes=1 << 40):
        return lib.laga_bwd_varlen(good, good, good, good, good, good, good, cu_seqlens, n_seqs, S_total, 2, 512, 128,
                                   64, 128, 0.07, 1, good, good, good, good, good, ws_bytes, flags, None)

    for call in (fwd, bwd):
        assert call(None, 2) == laga.ERR_INVALID_ARG
        assert call(cu(0, 100, 256), 0) == laga.ERR_INVALID_ARG          # no sequence
        assert call(cu(1, 100, 256), 2) == laga.ERR_INVALID_ARG          # does not start at 0
        assert call(cu(0, 100, 255), 2) == laga.ERR_INVALID_ARG          # does not end at S_total
        assert call(cu(0, 200, 100, 256), 3) == laga.ERR_INVALID_ARG     # decreasing
        assert call(cu(0, 100, 256), 2, ws_bytes=4096) == laga.ERR_WORKSPACE_TOO_SMALL
    assert bwd(cu(0, 100, 256), 2, flags=laga.FLAG_FUSED_BWD) == laga.ERR_INVALID_ARG
    # sizes: the single-sequence figure plus the tile tables, whatever the lengths are
    S, n, h = 5000, 7, 4
    assert laga.fwd_varlen_workspace_bytes(S, n, h) >= laga.fwd_workspace_bytes(S, h) + 32 * (S // 128 + n)
    assert laga.fwd_varlen_workspace_bytes(S, n, h) <= laga.fwd_workspace_bytes(S, h) + 32 * (S // 128 + n) + 8 * n + 2048
    assert laga.bwd_varlen_workspace_bytes(S, n, h) >= laga.bwd_workspace_bytes(S, h) + 2 * h * 127 * n * 4
    assert laga.bwd_varlen_workspace_bytes(S, n, h, flags=laga.FLAG_FUSED_BWD) == 0
    assert laga.fwd_varlen_workspace_bytes(S, 0, h) == 0 and laga.bwd_varlen_workspace_bytes(S, 0, h) == 0


def test_binding_rejects_cpu_tensors(laga):
    import torch
    q = torch.zeros(128, 2, 192, dtype=torch.bfloat16)
    c = torch.zeros(128, 512, dtype=torch.bfloat16)
    k = torch.zeros(128, 64, dtype=torch.bfloat16)
    w = torch.zeros(512, 512, dtype=torch.bfloat16)
    with pytest.raises(ValueError):
        laga.fwd(q, c, k, w)


def test_binding_refuses_tensors_on_different_devices(laga):
    """One call, one device: the check runs before anything reaches the C side (here with a CPU and a
    meta tensor, which need no GPU)."""
    import torch
    a = torch.zeros(4)
    b = torch.zeros(4, device="meta")
    with pytest.raises(ValueError, match="different devices"):
        laga.same_device(a, b)
    assert laga.same_device(a, None, torch.ones(2)) == a.device


def test_checked_build_exports_the_same_entry_points():
    """liblaga_debug.so (-DLAGA_DEBUG: kernels that verify their own index arithmetic) is the same ABI."""
    from paper_2607_17644_b200 import build
    path = build.build(debug=True)
    handle = ctypes.CDLL(path)
    for name in declared_functions():
        assert hasattr(handle, name), f"{name} missing from the checked build"
    handle.laga_status_string.restype = ctypes.c_char_p
    assert handle.laga_status_string(-6) == b"LAGA_ERR_DEVICE_CHECK"
