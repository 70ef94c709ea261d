"""fp64 CPU oracle for the rank-r delta-rule recurrence -- TEST INFRASTRUCTURE, not the product.

Only ``tests/``, ``__graft_entry__.smoke()`` and ``bench.py``'s CPU-baseline leg may import this
package.  It never imports the CUDA package and shares no code with it.

``deltanet_fwd`` wraps the C routine in ``pf_oracle.c`` (the token-by-token recurrence of
Section 1.1 with the rank-R delta-rule drivers of Section 3.1, written out in fp64).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pf_oracle.c")
_LIB = os.path.join(_HERE, "libpf_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile pf_oracle.c into libpf_oracle.so (gcc, -O2, OpenMP).  Returns the library path."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp%d" % os.getpid()
            cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        for fn in (lib.pf_oracle_deltanet_fwd_f64, lib.pf_oracle_deltanet_product_fwd_f64):
            fn.restype = ctypes.c_int
            fn.argtypes = [ctypes.c_void_p] * 5 + [ctypes.c_int] * 6 + [ctypes.c_void_p] * 2 + [
                ctypes.c_int, ctypes.POINTER(ctypes.c_int)]
        lib.pf_oracle_deltanet_exact_fwd_f64.restype = ctypes.c_int
        lib.pf_oracle_deltanet_exact_fwd_f64.argtypes = [ctypes.c_int] + [ctypes.c_void_p] * 5 + [ctypes.c_int] * 6 + [
            ctypes.c_void_p] * 2 + [ctypes.c_int, ctypes.POINTER(ctypes.c_int)]
        _lib = lib
    return _lib


def _as_f32(x, shape):
    a = np.ascontiguousarray(_to_numpy(x), dtype=np.float32)
    if a.shape != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {a.shape}")
    return a


def _to_numpy(x):
    if isinstance(x, np.ndarray):
        return x
    # torch tensor (possibly bf16): widen exactly to fp32 first
    import torch  # local import: the oracle itself needs only numpy
    if isinstance(x, torch.Tensor):
        x = x.detach().cpu()
        if x.dtype in (torch.bfloat16, torch.float16):
            x = x.float()
        return x.numpy()
    return np.asarray(x)


def deltanet_fwd(q, k, v, beta, S0=None, num_threads: int = 0, return_threads: bool = False, mode: str = "sum",
                 exact: bool = False):
    """Run the recurrence.  ``mode``: "sum" (all r factors of a token read the same old state: the paper's
    rank-R form) or "product" (the factors act one after another: rank-1 delta rule r times per token).
    ``exact``: every rank-1 factor takes the exact step exp(-beta k k^T) instead of the Euler step I - beta k k^T
    (r = 1, or the product form).  Shapes: q [B,H,L,d_k], k [B,H,L,r,d_k], v [B,H,L,r,d_v], beta [B,H,L,r],
    S0 [B,H,d_k,d_v] or None.  Inputs may be numpy or torch (bf16/fp16/fp32); they are widened
    exactly, the arithmetic is fp64.  Returns (O [B,H,L,d_v] float64, S_final [B,H,d_k,d_v] float64)
    and, if ``return_threads``, the number of host threads used."""
    kk = _to_numpy(k)
    if kk.ndim != 5:
        raise ValueError("k must be [B,H,L,r,d_k]")
    B, H, L, r, d_k = kk.shape
    d_v = _to_numpy(v).shape[-1]
    qa = _as_f32(q, (B, H, L, d_k))
    ka = _as_f32(kk, (B, H, L, r, d_k))
    va = _as_f32(v, (B, H, L, r, d_v))
    ba = _as_f32(beta, (B, H, L, r))
    s0 = None
    if S0 is not None:
        s0 = np.ascontiguousarray(_to_numpy(S0), dtype=np.float64)
        if s0.shape != (B, H, d_k, d_v):
            raise ValueError(f"S0 must be {(B, H, d_k, d_v)}, got {s0.shape}")
    O = np.empty((B, H, L, d_v), dtype=np.float64)
    Sf = np.empty((B, H, d_k, d_v), dtype=np.float64)
    used = ctypes.c_int(0)
    if mode not in ("sum", "product"):
        raise ValueError("mode must be 'sum' or 'product'")
    fn = _load().pf_oracle_deltanet_fwd_f64 if mode == "sum" else _load().pf_oracle_deltanet_product_fwd_f64
    if exact:
        base = _load().pf_oracle_deltanet_exact_fwd_f64
        fn = lambda *a: base(1 if mode == "product" else 0, *a)
    rc = fn(
        qa.ctypes.data, ka.ctypes.data, va.ctypes.data, ba.ctypes.data,
        s0.ctypes.data if s0 is not None else None,
        B, H, L, d_k, d_v, r, O.ctypes.data, Sf.ctypes.data, int(num_threads), ctypes.byref(used))
    if rc != 0:
        raise RuntimeError(f"pf_oracle_deltanet_fwd_f64 failed with code {rc}")
    if return_threads:
        return O, Sf, used.value
    return O, Sf
