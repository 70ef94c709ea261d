"""Times the two ways the fp32 SIMT kernels obtain W and Uh of a chunk, on synthetic inputs:

    python -m paper_2504_00492_b200.compare_builders

builder 0: triangular inverse T' (Theorem 3.2), then W = T'K, Uh = T'V   (kernels simt_solve + simt_wu)
builder 1: the two-index system of Theorem 3.3 swept along its antidiagonals (kernel simt_sigdelta)

Per-kernel device times come from the library's own CUDA-event profiling (pf_profile_*); the third of three calls
is reported.  Needs a GPU."""
import ctypes
import os
import sys

import torch

sys.path.insert(0, os.path.join(os.path.dirname(os.path.abspath(__file__)), ".."))
import pf_synth  # noqa: E402
import paper_2504_00492_b200 as pf  # noqa: E402
from paper_2504_00492_b200 import binding  # noqa: E402


def kernel_times(w, builder: int) -> dict:
    lib = binding.lib()
    pf.pf_set_option("wu_builder", builder)
    try:
        d = pf_synth.make_inputs(w).to("cuda")
        lib.pf_profile_enable(1)
        out = {}
        for _ in range(3):
            pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, impl="simt")
            torch.cuda.synchronize()
            out = {}
            for i in range(lib.pf_profile_count()):
                name, ms = ctypes.create_string_buffer(64), ctypes.c_float()
                lib.pf_profile_read(i, name, 64, ctypes.byref(ms))
                out[name.value.decode()] = ms.value
        return out
    finally:
        lib.pf_profile_enable(0)
        pf.pf_set_option("wu_builder", 0)


def main():
    base = pf_synth.CONFIGS["c2"]
    print("rows per chunk | chunks | inverse + products (solve, wu) | Theorem 3.3 wavefront | gram | scan   [ms]")
    for (B, H, L, r, C) in [(1, 8, 2048, 1, 64), (1, 8, 2048, 2, 64), (1, 8, 2048, 4, 64), (1, 8, 2048, 4, 32)]:
        w = base.with_(B=B, H=H, L=L, r=r, chunk=C)
        a, b = kernel_times(w, 0), kernel_times(w, 1)
        print(f"n={C * r:3d} (C={C}, r={r}) | {B * H * L // C:4d} | {a['simt_solve'] + a['simt_wu']:.3f} "
              f"({a['simt_solve']:.3f}, {a['simt_wu']:.3f}) | {b['simt_sigdelta']:.3f} | {a['simt_gram']:.3f} | "
              f"{a['simt_scan']:.3f}")


if __name__ == "__main__":
    main()
