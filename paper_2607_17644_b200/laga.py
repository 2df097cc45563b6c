"""ctypes binding of the LAGA C ABI (``include/laga.h``): argument marshalling only.

PyTorch appears here for device memory and the current CUDA stream; every step of the path runs in
the library's CUDA kernels.  The shared library must exist (``python -m paper_2607_17644_b200.build``):
there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes
import os

import torch

OK = 0
ERR_INVALID_ARG = -1
ERR_UNSUPPORTED = -2
ERR_WORKSPACE_TOO_SMALL = -3
ERR_CUDA = -4
ERR_DEVICE_TIMEOUT = -5
ERR_DEVICE_CHECK = -6
FLAG_ACCUM_DW = 1
FLAG_DETERMINISTIC = 2
FLAG_KV_SAVED = 4
FLAG_FUSED_BWD = 8
FLAG_FUSED_KV_REBUILD = 16

# LAGA_DEBUG=1 selects the checked build of the same kernels (liblaga_debug.so): every TMA issue and global
# store verifies its index arithmetic first and reports LAGA_ERR_DEVICE_CHECK instead of a bad access.
DEBUG = os.environ.get("LAGA_DEBUG", "0") not in ("", "0")
LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "liblaga_debug.so" if DEBUG else "liblaga.so")
_lib = None

# name -> (restype, argtypes); mirrors include/laga.h one to one
_vp, _ci, _cf, _cu, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_uint, ctypes.c_size_t
SIGNATURES = {
    "laga_version": (_ci, []),
    "laga_status_string": (ctypes.c_char_p, [_ci]),
    "laga_fwd_workspace_bytes": (_sz, [_ci] * 6),
    "laga_bwd_workspace_bytes": (_sz, [_ci] * 6 + [_cu]),
    "laga_fwd": (_ci, [_vp] * 4 + [_ci] * 6 + [_cf, _ci, _vp, _vp, _vp, _sz, _cu, _vp]),
    "laga_bwd": (_ci, [_vp] * 7 + [_ci] * 6 + [_cf, _ci] + [_vp] * 4 + [_vp, _sz, _cu, _vp]),
    "laga_fwd_varlen_workspace_bytes": (_sz, [_ci] * 7),
    "laga_bwd_varlen_workspace_bytes": (_sz, [_ci] * 7 + [_cu]),
    "laga_fwd_varlen": (_ci, [_vp] * 4 + [ctypes.POINTER(_ci)] + [_ci] * 7 + [_cf, _ci, _vp, _vp, _vp, _sz, _cu, _vp]),
    "laga_bwd_varlen": (_ci, [_vp] * 7 + [ctypes.POINTER(_ci)] + [_ci] * 7 + [_cf, _ci] + [_vp] * 4 + [_vp, _sz, _cu, _vp]),
    "laga_absorbed_fwd_workspace_bytes": (_sz, [_ci] * 6),
    "laga_absorbed_fwd": (_ci, [_vp] * 4 + [_ci] * 6 + [_cf, _ci, _vp, _vp, _vp, _sz, _cu, _vp]),
    "laga_linear": (_ci, [_vp, _vp, _ci, _ci, _ci, _vp, _vp, _vp]),
    "laga_linear_backward": (_ci, [_vp, _vp, _vp, _ci, _ci, _ci, _vp, _vp, _cu, _vp, _vp]),
    "laga_layernorm": (_ci, [_vp, _vp, _vp, _ci, _ci, _cf, _vp, _vp, _vp, _vp]),
    "laga_layernorm_backward": (_ci, [_vp] * 5 + [_ci, _ci] + [_vp] * 4),
    "laga_up_project": (_ci, [_vp, _vp] + [_ci] * 5 + [_vp, _vp, _vp]),
    "laga_kv_backward": (_ci, [_vp] * 3 + [_ci] * 5 + [_vp, _vp, _cu, _vp, _vp]),
    "laga_query_status": (_ci, [_vp, _vp, ctypes.POINTER(_cu)]),
    "laga_profile_kernel": (_ci, [_ci, ctypes.POINTER(_vp), ctypes.POINTER(_vp), _ci]),
    "laga_query_kernel_clocks": (_ci, [_vp, _vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]),
    "laga_selftest_bounded_wait": (_ci, [_vp, _cu, _vp]),
    "laga_fwd_builtin_scratch": (_ci, [_vp] * 4 + [_ci] * 6 + [_cf, _ci, _vp, _vp, _vp]),
}
BUILTIN_SCRATCH_MAX_TOKEN_HEADS = 32768   # S * h limit of laga_fwd_builtin_scratch (16 MiB of bf16 KV)
KERNELS = {"up_project": 0, "attn_fwd": 1, "bwd_delta": 2, "attn_bwd_dkv": 3, "attn_bwd_dq": 4,
           "dkpe_reduce": 5, "dckv_gemm": 6, "dw_gemm": 7, "q_absorb": 8, "attn_absorbed": 9, "v_project": 10,
           "attn_bwd_fused": 11, "dq_convert": 12}


class LagaError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


def lib():
    """Load liblaga.so once.  Raises if it has not been built: the product has no other path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_17644_b200.build`")
        handle = ctypes.CDLL(LIB_PATH)
        for name, (restype, argtypes) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = restype, argtypes
        _lib = handle
    return _lib


def version() -> int:
    return int(lib().laga_version())


def status_string(code: int) -> str:
    return lib().laga_status_string(int(code)).decode()


def _check(code: int, where: str):
    if code != OK:
        raise LagaError(code, where)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream, device):
    s = torch.cuda.current_stream(device) if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _dev(t: torch.Tensor, dtype, shape, name):
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous() and tuple(t.shape) == tuple(shape)):
        raise ValueError(f"{name}: expected contiguous CUDA {dtype} tensor of shape {tuple(shape)}, "
                         f"got {t.dtype} {tuple(t.shape)} on {t.device}")
    return t


def same_device(*tensors) -> torch.device:
    """All tensors of a call must live on ONE device: the library launches on the current device, so the
    call runs under that device (see ``_on``) and a tensor from anywhere else is refused here, before the
    C side would refuse its pointer."""
    present = [t for t in tensors if t is not None]
    dev = present[0].device
    for t in present[1:]:
        if t.device != dev:
            raise ValueError(f"tensors of one call are on different devices: {dev} and {t.device}")
    return dev


def _on(device):
    """Context that makes `device` current for the duration of a library call."""
    return torch.cuda.device(device)


def _geometry(q, c_kv, k_pe, w_kv_b, d_v):
    S, h, d_qk = q.shape
    d_c, d_rope = c_kv.shape[1], k_pe.shape[1]
    d_nope = d_qk - d_rope
    _dev(c_kv, torch.bfloat16, (S, d_c), "c_kv")
    _dev(k_pe, torch.bfloat16, (S, d_rope), "k_pe")
    _dev(w_kv_b, torch.bfloat16, (d_c, h * (d_nope + d_v)), "w_kv_b")
    _dev(q, torch.bfloat16, (S, h, d_qk), "q")
    return S, h, d_c, d_nope, d_rope


def fwd_workspace_bytes(S, h, d_c=512, d_nope=128, d_rope=64, d_v=128) -> int:
    return int(lib().laga_fwd_workspace_bytes(S, h, d_c, d_nope, d_rope, d_v))


def bwd_workspace_bytes(S, h, d_c=512, d_nope=128, d_rope=64, d_v=128, flags=0) -> int:
    return int(lib().laga_bwd_workspace_bytes(S, h, d_c, d_nope, d_rope, d_v, flags))


def fwd_varlen_workspace_bytes(S_total, n_seqs, h, d_c=512, d_nope=128, d_rope=64, d_v=128) -> int:
    return int(lib().laga_fwd_varlen_workspace_bytes(S_total, n_seqs, h, d_c, d_nope, d_rope, d_v))


def bwd_varlen_workspace_bytes(S_total, n_seqs, h, d_c=512, d_nope=128, d_rope=64, d_v=128, flags=0) -> int:
    return int(lib().laga_bwd_varlen_workspace_bytes(S_total, n_seqs, h, d_c, d_nope, d_rope, d_v, flags))


def _cu_seqlens(cu_seqlens):
    """The host array laga_*_varlen takes: n_seqs + 1 C ints from a list or a CPU tensor."""
    values = [int(v) for v in (cu_seqlens.tolist() if isinstance(cu_seqlens, torch.Tensor) else cu_seqlens)]
    if len(values) < 2:
        raise ValueError("cu_seqlens needs at least two entries (one sequence)")
    return (ctypes.c_int * len(values))(*values), len(values) - 1


def alloc_workspace(n_bytes: int, device="cuda") -> torch.Tensor:
    """A 1024-byte aligned byte buffer (torch's caching allocator aligns to at least 512; over-allocate)."""
    buf = torch.empty(n_bytes + 1024, dtype=torch.uint8, device=device)
    off = (-buf.data_ptr()) % 1024
    return buf[off:off + n_bytes]


def fwd(q, c_kv, k_pe, w_kv_b, d_v=128, softmax_scale=None, causal=True, out=None, lse=None, workspace=None,
        stream=None, cu_seqlens=None):
    """laga_fwd: returns (out bf16 [S,h,d_v], lse fp32 [S,h], workspace).  Enqueues only.
    With cu_seqlens (list or CPU tensor, n_seqs + 1 entries): laga_fwd_varlen over packed sequences."""
    S, h, d_c, d_nope, d_rope = _geometry(q, c_kv, k_pe, w_kv_b, d_v)
    dev = same_device(q, c_kv, k_pe, w_kv_b, out, lse, workspace)
    if softmax_scale is None:
        softmax_scale = (d_nope + d_rope) ** -0.5
    if out is None:
        out = torch.empty(S, h, d_v, dtype=torch.bfloat16, device=dev)
    if lse is None:
        lse = torch.empty(S, h, dtype=torch.float32, device=dev)
    _dev(out, torch.bfloat16, (S, h, d_v), "out")
    _dev(lse, torch.float32, (S, h), "lse")
    cu, n_seqs = _cu_seqlens(cu_seqlens) if cu_seqlens is not None else (None, 0)
    need = (fwd_workspace_bytes(S, h, d_c, d_nope, d_rope, d_v) if cu is None else
            fwd_varlen_workspace_bytes(S, n_seqs, h, d_c, d_nope, d_rope, d_v))
    if need == 0:
        raise LagaError(ERR_UNSUPPORTED, "laga_fwd_workspace_bytes")
    if workspace is None:
        workspace = alloc_workspace(need, dev)
    with _on(dev):
        if cu is None:
            rc = lib().laga_fwd(_ptr(q), _ptr(c_kv), _ptr(k_pe), _ptr(w_kv_b), S, h, d_c, d_nope, d_rope, d_v,
                                float(softmax_scale), int(bool(causal)), _ptr(out), _ptr(lse), _ptr(workspace),
                                workspace.numel(), 0, _stream(stream, dev))
        else:
            rc = lib().laga_fwd_varlen(_ptr(q), _ptr(c_kv), _ptr(k_pe), _ptr(w_kv_b), cu, n_seqs, S, h, d_c, d_nope,
                                       d_rope, d_v, float(softmax_scale), int(bool(causal)), _ptr(out), _ptr(lse),
                                       _ptr(workspace), workspace.numel(), 0, _stream(stream, dev))
    _check(rc, "laga_fwd" if cu is None else "laga_fwd_varlen")
    return out, lse, workspace


def absorbed_fwd_workspace_bytes(S, h, d_c=512, d_nope=128, d_rope=64, d_v=128) -> int:
    return int(lib().laga_absorbed_fwd_workspace_bytes(S, h, d_c, d_nope, d_rope, d_v))


def absorbed_fwd(q, c_kv, k_pe, w_kv_b, d_v=128, softmax_scale=None, causal=True, out=None, lse=None, workspace=None,
                 stream=None):
    """laga_absorbed_fwd: the absorbed form of the forward (comparison path).  Returns (out, lse, workspace)."""
    S, h, d_c, d_nope, d_rope = _geometry(q, c_kv, k_pe, w_kv_b, d_v)
    dev = same_device(q, c_kv, k_pe, w_kv_b, out, lse, workspace)
    if softmax_scale is None:
        softmax_scale = (d_nope + d_rope) ** -0.5
    if out is None:
        out = torch.empty(S, h, d_v, dtype=torch.bfloat16, device=dev)
    if lse is None:
        lse = torch.empty(S, h, dtype=torch.float32, device=dev)
    _dev(out, torch.bfloat16, (S, h, d_v), "out")
    _dev(lse, torch.float32, (S, h), "lse")
    need = absorbed_fwd_workspace_bytes(S, h, d_c, d_nope, d_rope, d_v)
    if need == 0:
        raise LagaError(ERR_UNSUPPORTED, "laga_absorbed_fwd_workspace_bytes")
    if workspace is None:
        workspace = alloc_workspace(need, dev)
    with _on(dev):
        rc = lib().laga_absorbed_fwd(_ptr(q), _ptr(c_kv), _ptr(k_pe), _ptr(w_kv_b), S, h, d_c, d_nope, d_rope, d_v,
                                     float(softmax_scale), int(bool(causal)), _ptr(out), _ptr(lse), _ptr(workspace),
                                     workspace.numel(), 0, _stream(stream, dev))
    _check(rc, "laga_absorbed_fwd")
    return out, lse, workspace


def fwd_builtin_scratch(q, c_kv, k_pe, w_kv_b, out, lse, d_v=128, softmax_scale=None, causal=True, stream=None):
    """laga_fwd_builtin_scratch: the forward for callers that cannot obtain scratch memory.

    `out` and `lse` are written in place (the caller passes them: this wrapper, like the entry point,
    allocates nothing).  The up-projection lives in a fixed 16 MiB array inside the library, so
    S * h must not exceed BUILTIN_SCRATCH_MAX_TOKEN_HEADS; larger problems raise
    LAGA_ERR_WORKSPACE_TOO_SMALL.  Calls on one stream may follow each other freely; calls that could
    overlap on the GPU share the array and must be ordered by the caller.  The first call on a device
    resolves the array's address (and may be the call that makes the CUDA runtime load the library's
    device code, array included): it belongs in initialisation, outside any stream capture.
    """
    S, h, d_c, d_nope, d_rope = _geometry(q, c_kv, k_pe, w_kv_b, d_v)
    dev = same_device(q, c_kv, k_pe, w_kv_b, out, lse)
    if softmax_scale is None:
        softmax_scale = (d_nope + d_rope) ** -0.5
    _dev(out, torch.bfloat16, (S, h, d_v), "out")
    _dev(lse, torch.float32, (S, h), "lse")
    with _on(dev):
        rc = lib().laga_fwd_builtin_scratch(_ptr(q), _ptr(c_kv), _ptr(k_pe), _ptr(w_kv_b), S, h, d_c, d_nope,
                                            d_rope, d_v, float(softmax_scale), int(bool(causal)), _ptr(out),
                                            _ptr(lse), _stream(stream, dev))
    _check(rc, "laga_fwd_builtin_scratch")


def bwd(q, c_kv, k_pe, w_kv_b, out, lse, dout, d_v=128, softmax_scale=None, causal=True, dq=None, dc_kv=None,
        dk_pe=None, dw_kv_b=None, workspace=None, flags=0, stream=None, cu_seqlens=None):
    """laga_bwd: returns (dq, dc_kv, dk_pe, dw_kv_b, workspace).  Enqueues only.
    With cu_seqlens (list or CPU tensor, n_seqs + 1 entries): laga_bwd_varlen over packed sequences."""
    S, h, d_c, d_nope, d_rope = _geometry(q, c_kv, k_pe, w_kv_b, d_v)
    dev = same_device(q, c_kv, k_pe, w_kv_b, out, lse, dout, dq, dc_kv, dk_pe, dw_kv_b, workspace)
    if softmax_scale is None:
        softmax_scale = (d_nope + d_rope) ** -0.5
    _dev(out, torch.bfloat16, (S, h, d_v), "out")
    _dev(lse, torch.float32, (S, h), "lse")
    _dev(dout, torch.bfloat16, (S, h, d_v), "dout")
    dq = torch.empty_like(q) if dq is None else _dev(dq, torch.bfloat16, q.shape, "dq")
    dc_kv = torch.empty_like(c_kv) if dc_kv is None else _dev(dc_kv, torch.bfloat16, c_kv.shape, "dc_kv")
    dk_pe = torch.empty_like(k_pe) if dk_pe is None else _dev(dk_pe, torch.bfloat16, k_pe.shape, "dk_pe")
    if dw_kv_b is None:
        if flags & FLAG_ACCUM_DW:
            raise ValueError("LAGA_FLAG_ACCUM_DW needs an existing dw_kv_b to add into")
        dw_kv_b = torch.empty(w_kv_b.shape, dtype=torch.float32, device=dev)
    _dev(dw_kv_b, torch.float32, w_kv_b.shape, "dw_kv_b")
    cu, n_seqs = _cu_seqlens(cu_seqlens) if cu_seqlens is not None else (None, 0)
    need = (bwd_workspace_bytes(S, h, d_c, d_nope, d_rope, d_v, flags) if cu is None else
            bwd_varlen_workspace_bytes(S, n_seqs, h, d_c, d_nope, d_rope, d_v, flags))
    if need == 0:
        raise LagaError(ERR_UNSUPPORTED, "laga_bwd_workspace_bytes")
    if workspace is None:
        workspace = alloc_workspace(need, dev)
    with _on(dev):
        if cu is None:
            rc = lib().laga_bwd(_ptr(q), _ptr(c_kv), _ptr(k_pe), _ptr(w_kv_b), _ptr(out), _ptr(lse), _ptr(dout), S, h,
                                d_c, d_nope, d_rope, d_v, float(softmax_scale), int(bool(causal)), _ptr(dq), _ptr(dc_kv),
                                _ptr(dk_pe), _ptr(dw_kv_b), _ptr(workspace), workspace.numel(), flags,
                                _stream(stream, dev))
        else:
            rc = lib().laga_bwd_varlen(_ptr(q), _ptr(c_kv), _ptr(k_pe), _ptr(w_kv_b), _ptr(out), _ptr(lse), _ptr(dout),
                                       cu, n_seqs, S, h, d_c, d_nope, d_rope, d_v, float(softmax_scale),
                                       int(bool(causal)), _ptr(dq), _ptr(dc_kv), _ptr(dk_pe), _ptr(dw_kv_b),
                                       _ptr(workspace), workspace.numel(), flags, _stream(stream, dev))
    _check(rc, "laga_bwd" if cu is None else "laga_bwd_varlen")
    return dq, dc_kv, dk_pe, dw_kv_b, workspace


def linear(x, w, y=None, status_word=None, stream=None):
    """laga_linear: y bf16 [M, N] = x [M, K] . w [K, N] (Algorithm 1 steps 1 and 7).  Returns (y, status_word)."""
    M, K = x.shape
    N = w.shape[1]
    _dev(x, torch.bfloat16, (M, K), "x")
    _dev(w, torch.bfloat16, (K, N), "w")
    dev = same_device(x, w, y, status_word)
    y = torch.empty(M, N, dtype=torch.bfloat16, device=dev) if y is None else _dev(y, torch.bfloat16, (M, N), "y")
    if status_word is None:
        status_word = torch.zeros(1, dtype=torch.int32, device=dev)
    with _on(dev):
        rc = lib().laga_linear(_ptr(x), _ptr(w), M, K, N, _ptr(y), _ptr(status_word), _stream(stream, dev))
    _check(rc, "laga_linear")
    return y, status_word


def linear_backward(dy, x, w, dx=None, dw=None, flags=0, status_word=None, stream=None):
    """laga_linear_backward: dx bf16 [M, K] = dy . w^T, dw fp32 [K, N] (+)= x^T . dy.  Returns (dx, dw, status_word)."""
    M, K = x.shape
    N = w.shape[1]
    _dev(x, torch.bfloat16, (M, K), "x")
    _dev(w, torch.bfloat16, (K, N), "w")
    _dev(dy, torch.bfloat16, (M, N), "dy")
    dev = same_device(dy, x, w, dx, dw, status_word)
    dx = torch.empty(M, K, dtype=torch.bfloat16, device=dev) if dx is None else _dev(dx, torch.bfloat16, (M, K), "dx")
    if dw is None:
        if flags & FLAG_ACCUM_DW:
            raise ValueError("LAGA_FLAG_ACCUM_DW needs an existing dw to add into")
        dw = torch.empty(K, N, dtype=torch.float32, device=dev)
    _dev(dw, torch.float32, (K, N), "dw")
    if status_word is None:
        status_word = torch.zeros(1, dtype=torch.int32, device=dev)
    with _on(dev):
        rc = lib().laga_linear_backward(_ptr(dy), _ptr(x), _ptr(w), M, K, N, _ptr(dx), _ptr(dw), flags, _ptr(status_word),
                                        _stream(stream, dev))
    _check(rc, "laga_linear_backward")
    return dx, dw, status_word


def layernorm(x, gamma, beta=None, eps=1e-5, y=None, stream=None):
    """laga_layernorm: returns (y bf16 [M, D], mean fp32 [M], rstd fp32 [M])."""
    M, D = x.shape
    _dev(x, torch.bfloat16, (M, D), "x")
    _dev(gamma, torch.bfloat16, (D,), "gamma")
    if beta is not None:
        _dev(beta, torch.bfloat16, (D,), "beta")
    dev = same_device(x, gamma, beta, y)
    y = torch.empty_like(x) if y is None else _dev(y, torch.bfloat16, (M, D), "y")
    mean = torch.empty(M, dtype=torch.float32, device=dev)
    rstd = torch.empty(M, dtype=torch.float32, device=dev)
    with _on(dev):
        rc = lib().laga_layernorm(_ptr(x), _ptr(gamma), _ptr(beta) if beta is not None else None, M, D, float(eps), _ptr(y),
                                  _ptr(mean), _ptr(rstd), _stream(stream, dev))
    _check(rc, "laga_layernorm")
    return y, mean, rstd


def layernorm_backward(dy, x, gamma, mean, rstd, with_beta=True, dx=None, stream=None):
    """laga_layernorm_backward: returns (dx bf16 [M, D], dgamma fp32 [D], dbeta fp32 [D] or None)."""
    M, D = x.shape
    _dev(x, torch.bfloat16, (M, D), "x")
    _dev(dy, torch.bfloat16, (M, D), "dy")
    _dev(gamma, torch.bfloat16, (D,), "gamma")
    _dev(mean, torch.float32, (M,), "mean")
    _dev(rstd, torch.float32, (M,), "rstd")
    dev = same_device(dy, x, gamma, mean, rstd, dx)
    dx = torch.empty_like(x) if dx is None else _dev(dx, torch.bfloat16, (M, D), "dx")
    dgamma = torch.empty(D, dtype=torch.float32, device=dev)
    dbeta = torch.empty(D, dtype=torch.float32, device=dev) if with_beta else None
    with _on(dev):
        rc = lib().laga_layernorm_backward(_ptr(dy), _ptr(x), _ptr(gamma), _ptr(mean), _ptr(rstd), M, D, _ptr(dx), _ptr(dgamma),
                                           _ptr(dbeta) if dbeta is not None else None, _stream(stream, dev))
    _check(rc, "laga_layernorm_backward")
    return dx, dgamma, dbeta


def up_project(c_kv, w_kv_b, h, d_nope=128, d_v=128, kv=None, status_word=None, stream=None):
    """laga_up_project: kv bf16 [S, h*(d_nope+d_v)] = c_kv . w_kv_b.  Returns (kv, status_word)."""
    S, d_c = c_kv.shape
    n = h * (d_nope + d_v)
    _dev(c_kv, torch.bfloat16, (S, d_c), "c_kv")
    _dev(w_kv_b, torch.bfloat16, (d_c, n), "w_kv_b")
    dev = same_device(c_kv, w_kv_b, kv, status_word)
    kv = torch.empty(S, n, dtype=torch.bfloat16, device=dev) if kv is None else kv
    _dev(kv, torch.bfloat16, (S, n), "kv")
    if status_word is None:
        status_word = torch.zeros(1, dtype=torch.int32, device=dev)
    with _on(dev):
        rc = lib().laga_up_project(_ptr(c_kv), _ptr(w_kv_b), S, h, d_c, d_nope, d_v, _ptr(kv), _ptr(status_word),
                                   _stream(stream, dev))
    _check(rc, "laga_up_project")
    return kv, status_word


def kv_backward(dkv, c_kv, w_kv_b, h, d_nope=128, d_v=128, dc_kv=None, dw_kv_b=None, flags=0, status_word=None,
                stream=None):
    """laga_kv_backward: dc_kv = dkv . w_kv_b^T (bf16), dw_kv_b (+)= c_kv^T . dkv (fp32)."""
    S, d_c = c_kv.shape
    n = h * (d_nope + d_v)
    _dev(dkv, torch.bfloat16, (S, n), "dkv")
    _dev(c_kv, torch.bfloat16, (S, d_c), "c_kv")
    _dev(w_kv_b, torch.bfloat16, (d_c, n), "w_kv_b")
    dev = same_device(dkv, c_kv, w_kv_b, dc_kv, dw_kv_b, status_word)
    dc_kv = torch.empty_like(c_kv) if dc_kv is None else _dev(dc_kv, torch.bfloat16, c_kv.shape, "dc_kv")
    if dw_kv_b is None:
        dw_kv_b = torch.empty(d_c, n, dtype=torch.float32, device=dev)
    _dev(dw_kv_b, torch.float32, (d_c, n), "dw_kv_b")
    if status_word is None:
        status_word = torch.zeros(1, dtype=torch.int32, device=dev)
    with _on(dev):
        rc = lib().laga_kv_backward(_ptr(dkv), _ptr(c_kv), _ptr(w_kv_b), S, h, d_c, d_nope, d_v, _ptr(dc_kv),
                                    _ptr(dw_kv_b), flags, _ptr(status_word), _stream(stream, dev))
    _check(rc, "laga_kv_backward")
    return dc_kv, dw_kv_b, status_word


def profile_kernel(kernel: str, start_events=(), stop_events=()):
    """laga_profile_kernel: record the given torch.cuda.Event pairs around every launch of `kernel`
    (cycling through them); call with no events to stop.  Events must have been created with
    enable_timing=True and recorded once already (torch creates the CUDA event lazily)."""
    n = len(start_events)
    assert n == len(stop_events)
    starts = (_vp * max(n, 1))(*[e.cuda_event for e in start_events])
    stops = (_vp * max(n, 1))(*[e.cuda_event for e in stop_events])
    _check(lib().laga_profile_kernel(KERNELS[kernel], starts, stops, n), "laga_profile_kernel")


def query_kernel_clocks(workspace, stream=None) -> dict:
    """laga_query_kernel_clocks: synchronises the stream; returns {kernel name: (SM MHz, kernel ms)} for
    the attention kernels the last call on `workspace` ran (measured inside the kernels themselves)."""
    mhz = (ctypes.c_double * len(KERNELS))()
    ms = (ctypes.c_double * len(KERNELS))()
    with _on(workspace.device):
        rc = lib().laga_query_kernel_clocks(_ptr(workspace), _stream(stream, workspace.device), mhz, ms)
    _check(rc, "laga_query_kernel_clocks")
    return {name: (float(mhz[i]), float(ms[i])) for name, i in KERNELS.items() if mhz[i] > 0.0}


def selftest_bounded_wait(budget_us: int = 1000, stream=None):
    """laga_selftest_bounded_wait: run the kernel whose waits cannot complete; returns the status word
    tensor to pass to query_status (expected: ERR_DEVICE_TIMEOUT, detail 0x54007e57)."""
    word = torch.zeros(1, dtype=torch.int32, device="cuda")
    with _on(word.device):
        rc = lib().laga_selftest_bounded_wait(_ptr(word), int(budget_us), _stream(stream, word.device))
    _check(rc, "laga_selftest_bounded_wait")
    return word


def query_status(workspace_or_word, stream=None) -> tuple[int, int]:
    """laga_query_status: synchronises the stream; returns (status code, raw device word)."""
    detail = ctypes.c_uint(0)
    dev = workspace_or_word.device
    with _on(dev):
        rc = lib().laga_query_status(_ptr(workspace_or_word), _stream(stream, dev), ctypes.byref(detail))
    return int(rc), int(detail.value)


def check_status(workspace_or_word, stream=None, where="laga"):
    rc, detail = query_status(workspace_or_word, stream)
    if rc != OK:
        raise LagaError(rc, f"{where} (device word 0x{detail:08x})")
