"""Two measurements of the single-launch kernel on the headline workload (config 2), for profiles/:

    python -m paper_2504_00492_b200.diag build       # once, anywhere nvcc is: libpf_diag.so with -DPF_ENDS
    python -m paper_2504_00492_b200.diag ends         # when each CTA of one launch starts and ends (device clock)
    python -m paper_2504_00492_b200.diag flow-ctas    # time per call against the number of flow-building CTAs

`ends` needs the diagnostic library (thread 0 of every CTA stamps the global timer into the status block of the
workspace); `flow-ctas` runs on the ordinary library through pf_set_option("flow_ctas", n)."""
import os
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
DIAG_LIB = os.path.join(PKG, "libpf_diag.so")


def _setup(lib_path=None):
    sys.path.insert(0, os.path.dirname(PKG))
    from paper_2504_00492_b200 import binding
    if lib_path:
        binding.LIB_PATH = lib_path
    import torch
    import pf_synth
    import paper_2504_00492_b200 as pf
    w = pf_synth.CONFIGS["c2"]
    d = pf_synth.make_inputs(w).to("cuda")
    O = torch.empty(w.B, w.H, w.L, w.d_v, device="cuda")
    Sf = torch.empty(w.B, w.H, w.d_k, w.d_v, device="cuda")
    nb = pf.pf_workspace_bytes(w.B, w.H, w.L, w.d_k, w.d_v, w.r, w.chunk, impl="tc")
    ws = torch.zeros(nb, dtype=torch.uint8, device="cuda")

    def call():
        pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, impl="tc", workspace=ws, O=O, S_final=Sf)
    return torch, pf, w, ws, call


def _time(torch, call, n=10):
    for _ in range(3):
        call()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n):
        call()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / n * 1e3


def ends():
    import numpy as np
    if not os.path.exists(DIAG_LIB):
        raise SystemExit("build the diagnostic library first: python -m paper_2504_00492_b200.diag build")
    torch, pf, w, ws, call = _setup(DIAG_LIB)
    us = _time(torch, call)
    ws[:4096].zero_()
    call()
    torch.cuda.synchronize()
    t = np.array(ws[1024:1024 + 8 * 384].view(torch.int64).cpu().tolist(), dtype=np.int64)
    ns = w.B * w.H
    st, en = t[:148], t[160:308]
    t0 = st.min()
    se, fe = (en[:ns] - t0) / 1e3, (en[ns:148] - t0) / 1e3
    print(f"{us:.1f} us per call (CUDA events, 10 calls back to back); CTA starts within {(st.max() - t0) / 1e3:.1f} us")
    print(f"flow CTAs end: min {fe.min():.1f}  median {np.median(fe):.1f}  max {fe.max():.1f} us")
    print(f"scan CTAs end: min {se.min():.1f}  median {np.median(se):.1f}  max {se.max():.1f} us")


def flow_ctas():
    torch, pf, w, ws, call = _setup()
    try:
        for n in (0, 108, 100, 90, 80, 64):
            pf.pf_set_option("flow_ctas", n)
            us = _time(torch, call)
            shown = n if n else 148 - w.B * w.H
            print(f"flow CTAs {shown:3d}: {us:6.1f} us per call   (us x CTAs = {us * shown:7.0f})")
    finally:
        pf.pf_set_option("flow_ctas", 0)


if __name__ == "__main__":
    what = sys.argv[1] if len(sys.argv) > 1 else ""
    if what == "build":
        sys.path.insert(0, os.path.dirname(PKG))
        from paper_2504_00492_b200 import build as _b
        print(_b.build(force=True, extra_flags=("-DPF_ENDS",), out=DIAG_LIB))
    elif what == "ends":
        ends()
    elif what == "flow-ctas":
        flow_ctas()
    else:
        raise SystemExit(__doc__)
