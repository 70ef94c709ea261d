"""ctypes binding of libpf.so: argument marshalling only -- every step runs in the CUDA kernels.

The function names mirror the C ABI in include/pf.h.  Tensors are torch CUDA tensors (torch is
used for device memory and streams only).  If the library is missing or cannot be loaded the
import of this module fails loudly; there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libpf.so")

PF_DTYPE_BF16, PF_DTYPE_F32 = 0, 1
PF_IMPL_AUTO, PF_IMPL_SIMT, PF_IMPL_TC = 0, 1, 2
PF_IMPL_TC_REFFLOW = 3
PF_IMPL_TC_SPLIT = 4
PF_MODE_SUM, PF_MODE_PRODUCT = 0, 1
MODE_BY_NAME = {"sum": PF_MODE_SUM, "product": PF_MODE_PRODUCT}
PF_STEP_EULER, PF_STEP_EXACT = 0, 1
STEP_BY_NAME = {"euler": PF_STEP_EULER, "exact": PF_STEP_EXACT}
IMPL_BY_NAME = {"auto": PF_IMPL_AUTO, "simt": PF_IMPL_SIMT, "tc": PF_IMPL_TC, "tc_refflow": PF_IMPL_TC_REFFLOW,
                "tc_split": PF_IMPL_TC_SPLIT}

# every symbol include/pf.h declares
EXPORTS = [
    "pf_deltanet_fwd", "pf_deltanet_fwd_f32", "pf_deltanet_fwd_ex", "pf_workspace_bytes", "pf_select_impl",
    "pf_last_launch_count", "pf_status_string", "pf_last_error_string", "pf_version",
    "pf_profile_enable", "pf_profile_count", "pf_profile_read", "pf_tc_selftest",
    "pf_deltanet_fwd_f32_static", "pf_static_scratch_bytes", "pf_static_scratch_need",
    "pf_workspace_bytes_ex", "pf_select_chunk", "pf_read_status", "pf_last_wait_code", "pf_wait_selftest",
]


class PfParams(ctypes.Structure):
    _fields_ = [
        ("q", ctypes.c_void_p), ("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("beta", ctypes.c_void_p),
        ("S0", ctypes.c_void_p),
        ("B", ctypes.c_int), ("H", ctypes.c_int), ("L", ctypes.c_int), ("d_k", ctypes.c_int),
        ("d_v", ctypes.c_int), ("r", ctypes.c_int), ("chunk", ctypes.c_int),
        ("O", ctypes.c_void_p), ("S_final", ctypes.c_void_p),
        ("in_dtype", ctypes.c_int), ("impl", ctypes.c_int),
        ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
        ("stream", ctypes.c_void_p),
        ("mode", ctypes.c_int),
        ("step", ctypes.c_int),
        ("segments", ctypes.c_int),
        ("wu_builder", ctypes.c_int),
        ("ring_depth", ctypes.c_int),
        ("status", ctypes.c_void_p),
    ]


class PfError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().pf_status_string(status).decode()
        detail = lib().pf_last_error_string().decode()
        super().__init__(f"{where}: {msg} ({status})" + (f": {detail}" if status == -5 and detail else ""))


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2504_00492_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, ci = ctypes.c_void_p, ctypes.c_int
        L.pf_deltanet_fwd.restype = ci
        L.pf_deltanet_fwd.argtypes = [vp] * 5 + [ci] * 7 + [vp, vp, vp]
        L.pf_deltanet_fwd_f32.restype = ci
        L.pf_deltanet_fwd_f32.argtypes = [vp] * 5 + [ci] * 7 + [vp, vp, vp]
        L.pf_deltanet_fwd_ex.restype = ci
        L.pf_deltanet_fwd_ex.argtypes = [ctypes.POINTER(PfParams)]
        L.pf_workspace_bytes.restype = ctypes.c_size_t
        L.pf_workspace_bytes.argtypes = [ci] * 9
        L.pf_select_impl.restype = ci
        L.pf_select_impl.argtypes = [ci] * 9
        L.pf_last_launch_count.restype = ci
        L.pf_last_launch_count.argtypes = []
        L.pf_status_string.restype = ctypes.c_char_p
        L.pf_status_string.argtypes = [ci]
        L.pf_last_error_string.restype = ctypes.c_char_p
        L.pf_last_error_string.argtypes = []
        L.pf_version.restype = ci
        L.pf_version.argtypes = []
        L.pf_profile_enable.restype = None
        L.pf_profile_enable.argtypes = [ci]
        L.pf_profile_count.restype = ci
        L.pf_profile_count.argtypes = []
        L.pf_profile_read.restype = ci
        L.pf_profile_read.argtypes = [ci, ctypes.c_char_p, ci, ctypes.POINTER(ctypes.c_float)]
        L.pf_deltanet_fwd_f32_static.restype = ci
        L.pf_deltanet_fwd_f32_static.argtypes = [vp] * 5 + [ci] * 7 + [vp, vp, vp]
        L.pf_static_scratch_bytes.restype = ctypes.c_size_t
        L.pf_static_scratch_bytes.argtypes = []
        L.pf_static_scratch_need.restype = ctypes.c_size_t
        L.pf_static_scratch_need.argtypes = [ci] * 7
        L.pf_workspace_bytes_ex.restype = ctypes.c_size_t
        L.pf_workspace_bytes_ex.argtypes = [ctypes.POINTER(PfParams)]
        L.pf_select_chunk.restype = ci
        L.pf_select_chunk.argtypes = [ci] * 9
        L.pf_read_status.restype = ci
        L.pf_read_status.argtypes = [vp, vp]
        L.pf_last_wait_code.restype = ci
        L.pf_last_wait_code.argtypes = []
        L.pf_wait_selftest.restype = ci
        L.pf_wait_selftest.argtypes = [vp, ci, vp]
        L.pf_tc_selftest.restype = ci
        L.pf_tc_selftest.argtypes = [ci, vp, vp, vp, ci, vp]
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _check_inputs(q, k, v, beta, S0, dtype) -> Tuple[int, int, int, int, int, int]:
    if k.dim() != 5 or q.dim() != 4 or v.dim() != 5 or beta.dim() != 4:
        raise ValueError("expected q [B,H,L,d_k], k [B,H,L,r,d_k], v [B,H,L,r,d_v], beta [B,H,L,r]")
    B, H, L, r, d_k = k.shape
    d_v = v.shape[-1]
    if tuple(q.shape) != (B, H, L, d_k) or tuple(v.shape) != (B, H, L, r, d_v) or tuple(beta.shape) != (B, H, L, r):
        raise ValueError("inconsistent input shapes")
    for name, t in (("q", q), ("k", k), ("v", v), ("beta", beta)):
        if t.dtype != dtype:
            raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
        if not t.is_cuda:
            raise ValueError(f"{name} must be a CUDA tensor")
        if not t.is_contiguous():
            raise ValueError(f"{name} must be contiguous")
    if S0 is not None:
        if S0.dtype != torch.float32 or tuple(S0.shape) != (B, H, d_k, d_v) or not S0.is_cuda or not S0.is_contiguous():
            raise ValueError("S0 must be a contiguous fp32 CUDA tensor [B,H,d_k,d_v]")
    return B, H, L, d_k, d_v, r


def _outputs(q, B, H, L, d_k, d_v, O, S_final, want_state):
    if O is None:
        O = torch.empty(B, H, L, d_v, dtype=torch.float32, device=q.device)
    if S_final is None and want_state:
        S_final = torch.empty(B, H, d_k, d_v, dtype=torch.float32, device=q.device)
    return O, S_final


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def pf_deltanet_fwd(q, k, v, beta, S0, chunk: int, O=None, S_final=None, stream=None, want_state: bool = True):
    """bf16 q/k/v/beta -> (O fp32 [B,H,L,d_v], S_final fp32 [B,H,d_k,d_v] or None)."""
    B, H, L, d_k, d_v, r = _check_inputs(q, k, v, beta, S0, torch.bfloat16)
    O, S_final = _outputs(q, B, H, L, d_k, d_v, O, S_final, want_state)
    with torch.cuda.device(q.device):
        st = lib().pf_deltanet_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(S0), B, H, L, d_k, d_v, r, chunk,
                                   _ptr(O), _ptr(S_final), _stream(stream))
    if st != 0:
        raise PfError(st, "pf_deltanet_fwd")
    return O, S_final


def pf_deltanet_fwd_f32(q, k, v, beta, S0, chunk: int, O=None, S_final=None, stream=None, want_state: bool = True):
    """fp32 q/k/v/beta -> (O, S_final), all arithmetic fp32."""
    B, H, L, d_k, d_v, r = _check_inputs(q, k, v, beta, S0, torch.float32)
    O, S_final = _outputs(q, B, H, L, d_k, d_v, O, S_final, want_state)
    with torch.cuda.device(q.device):
        st = lib().pf_deltanet_fwd_f32(_ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(S0), B, H, L, d_k, d_v, r, chunk,
                                       _ptr(O), _ptr(S_final), _stream(stream))
    if st != 0:
        raise PfError(st, "pf_deltanet_fwd_f32")
    return O, S_final


def pf_deltanet_fwd_f32_static(q, k, v, beta, S0, chunk: int, O=None, S_final=None, stream=None,
                               want_state: bool = True):
    """pf_deltanet_fwd_f32 without any device allocation inside the library: the per-chunk scratch is a
    fixed array of pf_static_scratch_bytes() built into libpf.so.  Pass O (and S_final) if the caller
    must not allocate either; otherwise they are created here with torch.  Problems too large for the
    fixed array raise PfError with status -6.  Calls on one device must not overlap on the GPU."""
    B, H, L, d_k, d_v, r = _check_inputs(q, k, v, beta, S0, torch.float32)
    O, S_final = _outputs(q, B, H, L, d_k, d_v, O, S_final, want_state)
    with torch.cuda.device(q.device):
        st = lib().pf_deltanet_fwd_f32_static(_ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(S0), B, H, L, d_k, d_v, r,
                                              chunk, _ptr(O), _ptr(S_final), _stream(stream))
    if st != 0:
        raise PfError(st, "pf_deltanet_fwd_f32_static")
    return O, S_final


def pf_static_scratch_bytes() -> int:
    return int(lib().pf_static_scratch_bytes())


def pf_deltanet_fwd_ex(q, k, v, beta, S0, chunk: int, impl="auto", workspace: Optional[torch.Tensor] = None,
                       O=None, S_final=None, stream=None, want_state: bool = True, mode="sum", step="euler",
                       segments: int = 0, wu_builder: int = 0, ring_depth: int = 0,
                       status: Optional[torch.Tensor] = None):
    """Same operation with an explicit implementation and (optionally) a caller-owned workspace
    (a uint8 CUDA tensor of at least pf_workspace_bytes_ex(...) bytes).  mode: "sum" (the r factors of a token
    read the same previous state) or "product" (they act one after another).  step: "euler" (the paper's
    discretisation) or "exact" (each rank-1 factor takes exp(-beta k k^T); r = 1 or the product form).
    segments / wu_builder / ring_depth: the options of pf_params (0 = default).  status: an int32 CUDA tensor of one
    element that receives the code of the first device-side wait that expired (see pf_read_status)."""
    dtype = q.dtype
    if dtype not in (torch.bfloat16, torch.float32):
        raise TypeError("q/k/v/beta must be bf16 or fp32")
    B, H, L, d_k, d_v, r = _check_inputs(q, k, v, beta, S0, dtype)
    O, S_final = _outputs(q, B, H, L, d_k, d_v, O, S_final, want_state)
    p = PfParams()
    p.q, p.k, p.v, p.beta, p.S0 = _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(S0)
    p.B, p.H, p.L, p.d_k, p.d_v, p.r, p.chunk = B, H, L, d_k, d_v, r, chunk
    p.O, p.S_final = _ptr(O), _ptr(S_final)
    p.in_dtype = PF_DTYPE_F32 if dtype == torch.float32 else PF_DTYPE_BF16
    p.impl = IMPL_BY_NAME[impl] if isinstance(impl, str) else int(impl)
    if workspace is not None:
        p.workspace, p.workspace_bytes = workspace.data_ptr(), workspace.numel() * workspace.element_size()
    p.stream = _stream(stream)
    p.mode = MODE_BY_NAME[mode] if isinstance(mode, str) else int(mode)
    p.step = STEP_BY_NAME[step] if isinstance(step, str) else int(step)
    p.segments, p.wu_builder, p.ring_depth = int(segments), int(wu_builder), int(ring_depth)
    if status is not None:
        if status.dtype != torch.int32 or not status.is_cuda or status.numel() < 1:
            raise ValueError("status must be an int32 CUDA tensor")
        p.status = status.data_ptr()
    with torch.cuda.device(q.device):
        st = lib().pf_deltanet_fwd_ex(ctypes.byref(p))
    if st != 0:
        raise PfError(st, "pf_deltanet_fwd_ex")
    return O, S_final


def pf_workspace_bytes_ex(B, H, L, d_k, d_v, r, chunk, in_dtype=PF_DTYPE_BF16, impl="auto", mode="sum", segments=0,
                          wu_builder=0, ring_depth=0) -> int:
    """pf_workspace_bytes with the options of pf_params taken into account."""
    p = PfParams()
    p.B, p.H, p.L, p.d_k, p.d_v, p.r, p.chunk = B, H, L, d_k, d_v, r, chunk
    p.in_dtype = in_dtype
    p.impl = IMPL_BY_NAME[impl] if isinstance(impl, str) else int(impl)
    p.mode = MODE_BY_NAME[mode] if isinstance(mode, str) else int(mode)
    p.segments, p.wu_builder, p.ring_depth = int(segments), int(wu_builder), int(ring_depth)
    return int(lib().pf_workspace_bytes_ex(ctypes.byref(p)))


def pf_select_chunk(B, H, L, d_k, d_v, r, chunk, in_dtype=PF_DTYPE_BF16, impl="auto") -> int:
    impl = IMPL_BY_NAME[impl] if isinstance(impl, str) else int(impl)
    return int(lib().pf_select_chunk(B, H, L, d_k, d_v, r, chunk, in_dtype, impl))


def pf_read_status(word=None, stream=None) -> int:
    """Synchronises the stream and returns 0 or -7 (PF_ERR_TIMEOUT).  `word`: the status tensor, the workspace tensor
    (its word 0), or None for the library's own word on the current device."""
    return int(lib().pf_read_status(None if word is None else word.data_ptr(), _stream(stream)))


def pf_last_wait_code() -> int:
    return int(lib().pf_last_wait_code())


def pf_wait_selftest(status=None, limit_us: int = 1000, stream=None) -> None:
    st = lib().pf_wait_selftest(None if status is None else status.data_ptr(), int(limit_us), _stream(stream))
    if st != 0:
        raise PfError(st, "pf_wait_selftest")


def pf_static_scratch_need(B, H, L, d_k, d_v, r, chunk) -> int:
    return int(lib().pf_static_scratch_need(B, H, L, d_k, d_v, r, chunk))


def pf_workspace_bytes(B, H, L, d_k, d_v, r, chunk, in_dtype=PF_DTYPE_BF16, impl="auto") -> int:
    impl = IMPL_BY_NAME[impl] if isinstance(impl, str) else int(impl)
    return int(lib().pf_workspace_bytes(B, H, L, d_k, d_v, r, chunk, in_dtype, impl))


def pf_select_impl(B, H, L, d_k, d_v, r, chunk, in_dtype=PF_DTYPE_BF16, impl="auto") -> int:
    impl = IMPL_BY_NAME[impl] if isinstance(impl, str) else int(impl)
    return int(lib().pf_select_impl(B, H, L, d_k, d_v, r, chunk, in_dtype, impl))


def pf_last_launch_count() -> int:
    return int(lib().pf_last_launch_count())


def pf_status_string(status: int) -> str:
    return lib().pf_status_string(status).decode()


def pf_last_error_string() -> str:
    return lib().pf_last_error_string().decode()


def pf_version() -> int:
    return int(lib().pf_version())
