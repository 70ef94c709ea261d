"""CPU-side checks of the C-ABI library: it loads, exports what include/pf.h declares, and its
host-only logic (shape checks, workspace arithmetic, status strings) behaves."""
import ctypes
import os
import re

import pytest

import paper_2504_00492_b200 as pf
from paper_2504_00492_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "pf.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pf_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(binding.LIB_PATH)
    syms = declared_symbols()
    assert "pf_deltanet_fwd" in syms and "pf_deltanet_fwd_f32" in syms and "pf_deltanet_fwd_ex" in syms
    for s in syms:
        assert hasattr(lib, s), f"libpf.so does not export {s}"
    assert sorted(binding.EXPORTS) == syms


def test_version_and_status_strings():
    assert pf.pf_version() >= 100
    assert pf.pf_status_string(0) == "ok"
    for code in range(-7, 0):
        assert pf.pf_status_string(code) not in ("", "unknown status")
    assert pf.pf_status_string(-99) == "unknown status"


@pytest.mark.parametrize("kw,code", [
    (dict(d_k=96), -2), (dict(d_v=32), -2), (dict(r=5), -2), (dict(r=0), -2), (dict(chunk=48), -2),
    (dict(chunk=128), -2), (dict(B=0), -1), (dict(L=-1), -1),
])
def test_shape_checks_need_no_gpu(kw, code):
    args = dict(B=1, H=1, L=64, d_k=64, d_v=64, r=1, chunk=64)
    args.update(kw)
    assert pf.pf_select_impl(**args) == code
    assert pf.pf_workspace_bytes(**args) == 0
    # the forward call itself must refuse before touching CUDA
    p = binding.PfParams()
    for k_, v_ in args.items():
        setattr(p, k_, v_)
    assert binding.lib().pf_deltanet_fwd_ex(ctypes.byref(p)) == code
    assert binding.lib().pf_deltanet_fwd_ex(None) == -1


def test_simt_workspace_arithmetic():
    # T [G][n][n] + W [G][n][d_k] + U [G][n][d_v] + P [G][C][n], fp32, each 256-byte aligned, then room for the fp32
    # step sizes of PF_STEP_EXACT [B,H,L,r]
    B, H, L, d_k, d_v, r, C = 2, 3, 100, 64, 128, 3, 32
    G, n = B * H * ((L + C - 1) // C), C * r
    al = lambda x: (x + 255) // 256 * 256
    want = al(G * n * n * 4) + al(G * n * d_k * 4) + al(G * n * d_v * 4) + al(G * C * n * 4) + 256 + al(B * H * L * r * 4)
    assert pf.pf_workspace_bytes(B, H, L, d_k, d_v, r, C, binding.PF_DTYPE_F32, "simt") == want
    assert pf.pf_select_impl(B, H, L, d_k, d_v, r, C, binding.PF_DTYPE_F32, "auto") == binding.PF_IMPL_SIMT
    assert pf.pf_select_impl(B, H, L, d_k, d_v, r, C, binding.PF_DTYPE_F32, "tc") == -2
