"""fp64 CPU oracle of the LAGA per-rank hot path -- TEST INFRASTRUCTURE ONLY.

Thin ctypes loader around ``laga_oracle.c`` (plain C, double precision, OpenMP over rows).  Only the
tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the product
package never does, and the two share no code.

What it computes: Algorithm 1 steps 4-5 of the paper (head-shard up-projection of the gathered
latent, key assembly with the shared rope band, explicit softmax attention) and the backward of
Section 5.2, written out as the explicit MLA definition (Section 5.1 shows LAGA equals it).

All functions take torch CPU tensors (bf16 inputs) and return float64 torch tensors.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "laga_oracle.c")
_LIB_PATH = os.path.join(_HERE, "liblaga_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2 -fopenmp, strict IEEE: no fast-math) if stale."""
    with _lock:
        stale = (force or not os.path.exists(_LIB_PATH)
                 or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC))
        if stale:
            tmp = _LIB_PATH + f".tmp{os.getpid()}"
            subprocess.run(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC,
                            "-lm"], check=True)
            os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u16p = ctypes.POINTER(ctypes.c_uint16)
        f64p = ctypes.POINTER(ctypes.c_double)
        i32p = ctypes.POINTER(ctypes.c_int)
        ci, cd = ctypes.c_int, ctypes.c_double
        lib.laga_oracle_fwd_rows.argtypes = [u16p, u16p, u16p, u16p, ci, ci, ci, ci, ci, ci, cd, ci, ci,
                                             i32p, ci, f64p, f64p, f64p, f64p]
        lib.laga_oracle_fwd_rows.restype = ci
        lib.laga_oracle_bwd.argtypes = [u16p, u16p, u16p, u16p, u16p, ci, ci, ci, ci, ci, ci, cd, ci, ci,
                                        f64p, f64p, f64p, f64p, f64p, f64p, f64p, f64p]
        lib.laga_oracle_bwd.restype = ci
        lib.laga_oracle_round_bf16.argtypes = [cd]
        lib.laga_oracle_round_bf16.restype = cd
        lib.laga_oracle_threads.restype = ci
        _lib = lib
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle will use."""
    return int(_load().laga_oracle_threads())


def round_bf16(x: float) -> float:
    """Nearest bf16-representable value of a double (ties to even), as the oracle rounds K/V."""
    return float(_load().laga_oracle_round_bf16(float(x)))


def _bits(t: torch.Tensor) -> np.ndarray:
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu", "oracle inputs are bf16 CPU tensors"
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def _u16(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16))


def _f64(a):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _dims(q, c_kv, k_pe, w_kv_b, d_v):
    S, h, d_qk = q.shape
    d_c = c_kv.shape[1]
    d_rope = k_pe.shape[1]
    d_nope = d_qk - d_rope
    assert c_kv.shape[0] == S and k_pe.shape[0] == S
    assert tuple(w_kv_b.shape) == (d_c, h * (d_nope + d_v)), "W_kv_b shard is [d_c, h*(d_nope+d_v)]"
    return S, h, d_c, d_nope, d_rope


def fwd(q, c_kv, k_pe, w_kv_b, d_v, softmax_scale, causal=True, kv_round_bf16=False, rows=None,
        return_kv=False):
    """Forward (Algorithm 1 steps 4-5).  Returns (O[R,h,d_v], LSE[R,h]) for the query rows in
    ``rows`` (all S rows when None); with ``return_kv`` also (K_nope[S,h,d_nope], V[S,h,d_v])."""
    lib = _load()
    S, h, d_c, d_nope, d_rope = _dims(q, c_kv, k_pe, w_kv_b, d_v)
    if rows is None:
        rows_arr, n_rows, rows_p = None, S, None
    else:
        rows_arr = np.ascontiguousarray(np.asarray(rows, dtype=np.int32))
        assert rows_arr.ndim == 1 and (rows_arr >= 0).all() and (rows_arr < S).all()
        n_rows = rows_arr.shape[0]
        rows_p = rows_arr.ctypes.data_as(ctypes.POINTER(ctypes.c_int))
    out = np.empty((n_rows, h, d_v), dtype=np.float64)
    lse = np.empty((n_rows, h), dtype=np.float64)
    kn = np.empty((S, h, d_nope), dtype=np.float64) if return_kv else None
    vv = np.empty((S, h, d_v), dtype=np.float64) if return_kv else None
    qb, cb, kb, wb = _bits(q), _bits(c_kv), _bits(k_pe), _bits(w_kv_b)
    rc = lib.laga_oracle_fwd_rows(_u16(qb), _u16(cb), _u16(kb), _u16(wb), S, h, d_c, d_nope, d_rope, d_v,
                                  float(softmax_scale), int(bool(causal)), int(bool(kv_round_bf16)),
                                  rows_p, n_rows, _f64(out), _f64(lse), _f64(kn), _f64(vv))
    if rc != 0:
        raise RuntimeError(f"laga_oracle_fwd_rows failed with code {rc}")
    res = (torch.from_numpy(out), torch.from_numpy(lse))
    if return_kv:
        res = res + (torch.from_numpy(kn), torch.from_numpy(vv))
    return res


def bwd(q, c_kv, k_pe, w_kv_b, dout, d_v, softmax_scale, causal=True, kv_round_bf16=False,
        return_fwd=False, return_dkv=False):
    """Backward (Section 5.2).  Returns a dict with dq, dc_kv, dk_pe, dw (float64); optionally the
    forward it differentiates (out, lse) and the per-head dk [S,h,d_qk], dv [S,h,d_v]."""
    lib = _load()
    S, h, d_c, d_nope, d_rope = _dims(q, c_kv, k_pe, w_kv_b, d_v)
    assert tuple(dout.shape) == (S, h, d_v)
    d_qk = d_nope + d_rope
    dq = np.empty((S, h, d_qk), dtype=np.float64)
    dc = np.empty((S, d_c), dtype=np.float64)
    dkpe = np.empty((S, d_rope), dtype=np.float64)
    dw = np.empty((d_c, h * (d_nope + d_v)), dtype=np.float64)
    out = np.empty((S, h, d_v), dtype=np.float64) if return_fwd else None
    lse = np.empty((S, h), dtype=np.float64) if return_fwd else None
    dk = np.empty((S, h, d_qk), dtype=np.float64) if return_dkv else None
    dv = np.empty((S, h, d_v), dtype=np.float64) if return_dkv else None
    qb, cb, kb, wb, db = _bits(q), _bits(c_kv), _bits(k_pe), _bits(w_kv_b), _bits(dout)
    rc = lib.laga_oracle_bwd(_u16(qb), _u16(cb), _u16(kb), _u16(wb), _u16(db), S, h, d_c, d_nope, d_rope,
                             d_v, float(softmax_scale), int(bool(causal)), int(bool(kv_round_bf16)),
                             _f64(dq), _f64(dc), _f64(dkpe), _f64(dw), _f64(out), _f64(lse), _f64(dk),
                             _f64(dv))
    if rc != 0:
        raise RuntimeError(f"laga_oracle_bwd failed with code {rc}")
    res = {"dq": torch.from_numpy(dq), "dc_kv": torch.from_numpy(dc), "dk_pe": torch.from_numpy(dkpe),
           "dw": torch.from_numpy(dw)}
    if return_fwd:
        res["out"], res["lse"] = torch.from_numpy(out), torch.from_numpy(lse)
    if return_dkv:
        res["dk"], res["dv"] = torch.from_numpy(dk), torch.from_numpy(dv)
    return res


def _int_list(values, upper):
    arr = np.ascontiguousarray(np.asarray(values, dtype=np.int32))
    assert arr.ndim == 1 and arr.size > 0 and (arr >= 0).all() and (arr < upper).all()
    return arr, arr.ctypes.data_as(ctypes.POINTER(ctypes.c_int))


def bwd_rows(q, c_kv, k_pe, w_kv_b, dout, d_v, softmax_scale, rows, causal=True, kv_round_bf16=False):
    """dQ for the listed query rows (a dQ row depends on its own query row only), with the forward
    values it used.  Returns dict: dq [R,h,d_qk], out [R,h,d_v], lse [R,h]."""
    lib = _load()
    lib.laga_oracle_bwd_rows.argtypes = ([ctypes.POINTER(ctypes.c_uint16)] * 5 + [ctypes.c_int] * 6
                                         + [ctypes.c_double, ctypes.c_int, ctypes.c_int,
                                            ctypes.POINTER(ctypes.c_int), ctypes.c_int]
                                         + [ctypes.POINTER(ctypes.c_double)] * 3)
    lib.laga_oracle_bwd_rows.restype = ctypes.c_int
    S, h, d_c, d_nope, d_rope = _dims(q, c_kv, k_pe, w_kv_b, d_v)
    rows_arr, rows_p = _int_list(rows, S)
    n = rows_arr.shape[0]
    dq = np.empty((n, h, d_nope + d_rope), dtype=np.float64)
    out = np.empty((n, h, d_v), dtype=np.float64)
    lse = np.empty((n, h), dtype=np.float64)
    qb, cb, kb, wb, db = _bits(q), _bits(c_kv), _bits(k_pe), _bits(w_kv_b), _bits(dout)
    rc = lib.laga_oracle_bwd_rows(_u16(qb), _u16(cb), _u16(kb), _u16(wb), _u16(db), S, h, d_c, d_nope, d_rope,
                                  d_v, float(softmax_scale), int(bool(causal)), int(bool(kv_round_bf16)),
                                  rows_p, n, _f64(dq), _f64(out), _f64(lse))
    if rc != 0:
        raise RuntimeError(f"laga_oracle_bwd_rows failed with code {rc}")
    return {"dq": torch.from_numpy(dq), "out": torch.from_numpy(out), "lse": torch.from_numpy(lse)}


def bwd_keys(q, c_kv, k_pe, w_kv_b, dout, d_v, softmax_scale, keys, causal=True, kv_round_bf16=False):
    """Key-side gradients for the listed key positions only.  Returns dict: dk [T,h,d_qk],
    dv [T,h,d_v], dk_pe [T,d_rope], dc_kv [T,d_c] (the same numbers the full backward gives there)."""
    lib = _load()
    lib.laga_oracle_bwd_keys.argtypes = ([ctypes.POINTER(ctypes.c_uint16)] * 5 + [ctypes.c_int] * 6
                                         + [ctypes.c_double, ctypes.c_int, ctypes.c_int,
                                            ctypes.POINTER(ctypes.c_int), ctypes.c_int]
                                         + [ctypes.POINTER(ctypes.c_double)] * 4)
    lib.laga_oracle_bwd_keys.restype = ctypes.c_int
    S, h, d_c, d_nope, d_rope = _dims(q, c_kv, k_pe, w_kv_b, d_v)
    keys_arr, keys_p = _int_list(keys, S)
    n = keys_arr.shape[0]
    dk = np.empty((n, h, d_nope + d_rope), dtype=np.float64)
    dv = np.empty((n, h, d_v), dtype=np.float64)
    dkpe = np.empty((n, d_rope), dtype=np.float64)
    dc = np.empty((n, d_c), dtype=np.float64)
    qb, cb, kb, wb, db = _bits(q), _bits(c_kv), _bits(k_pe), _bits(w_kv_b), _bits(dout)
    rc = lib.laga_oracle_bwd_keys(_u16(qb), _u16(cb), _u16(kb), _u16(wb), _u16(db), S, h, d_c, d_nope, d_rope,
                                  d_v, float(softmax_scale), int(bool(causal)), int(bool(kv_round_bf16)),
                                  keys_p, n, _f64(dk), _f64(dv), _f64(dkpe), _f64(dc))
    if rc != 0:
        raise RuntimeError(f"laga_oracle_bwd_keys failed with code {rc}")
    return {"dk": torch.from_numpy(dk), "dv": torch.from_numpy(dv), "dk_pe": torch.from_numpy(dkpe),
            "dc_kv": torch.from_numpy(dc)}


# ---- the dense projections around the path (Algorithm 1 steps 1 and 7) ------------------------------
# Their definition IS the matrix product, so the oracle is that product in float64 through the library
# routine (torch.matmul on CPU tensors), nothing else.

def linear(x: torch.Tensor, w: torch.Tensor) -> torch.Tensor:
    """y[M, N] = x[M, K] . w[K, N] in float64 (Algorithm 1 steps 1 and 7: W_q, W_kv_a, W_o)."""
    return x.to(torch.float64) @ w.to(torch.float64)


def linear_bwd(dy: torch.Tensor, x: torch.Tensor, w: torch.Tensor):
    """Gradients of ``linear`` for an upstream dy[M, N]: dx[M, K] = dy . w^T and dw[K, N] = x^T . dy, float64."""
    dy64 = dy.to(torch.float64)
    return dy64 @ w.to(torch.float64).T, x.to(torch.float64).T @ dy64


# ---- LayerNorm of the latent (Algorithm 1 step 1) ---------------------------------------------------
# The paper names the operation only; the definition written out here is the usual one: statistics over the
# last axis, biased variance, scale gamma, optional shift beta.  float64 throughout, one row at a time.

def layernorm(x: torch.Tensor, gamma: torch.Tensor, beta, eps: float):
    """y = (x - mean) / sqrt(var + eps) * gamma + beta, row by row.  Returns (y, mean, rstd) in float64."""
    x64, g64 = x.to(torch.float64), gamma.to(torch.float64)
    b64 = torch.zeros_like(g64) if beta is None else beta.to(torch.float64)
    M, D = x64.shape
    y = torch.empty_like(x64)
    mean = torch.empty(M, dtype=torch.float64)
    rstd = torch.empty(M, dtype=torch.float64)
    for m in range(M):
        mu = x64[m].sum() / D
        var = ((x64[m] - mu) ** 2).sum() / D
        r = 1.0 / torch.sqrt(var + eps)
        y[m] = (x64[m] - mu) * r * g64 + b64
        mean[m], rstd[m] = mu, r
    return y, mean, rstd


def layernorm_bwd(dy: torch.Tensor, x: torch.Tensor, gamma: torch.Tensor, eps: float):
    """Gradients of ``layernorm`` for an upstream dy: (dx [M, D], dgamma [D], dbeta [D]) in float64, from the chain
    rule through mean and variance written out row by row."""
    dy64, x64, g64 = dy.to(torch.float64), x.to(torch.float64), gamma.to(torch.float64)
    M, D = x64.shape
    dx = torch.empty_like(x64)
    dgamma = torch.zeros(D, dtype=torch.float64)
    dbeta = torch.zeros(D, dtype=torch.float64)
    for m in range(M):
        mu = x64[m].sum() / D
        var = ((x64[m] - mu) ** 2).sum() / D
        r = 1.0 / torch.sqrt(var + eps)
        xhat = (x64[m] - mu) * r
        g = dy64[m] * g64
        dx[m] = r * (g - g.sum() / D - xhat * (g * xhat).sum() / D)
        dgamma += dy64[m] * xhat
        dbeta += dy64[m]
    return dx, dgamma, dbeta
