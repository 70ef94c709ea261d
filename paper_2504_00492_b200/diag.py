"""Two measurements of the single-launch kernel on the headline workload (config 2), for profiles/:

    python -m paper_2504_00492_b200.diag build       # once, anywhere nvcc is: libpf_diag.so with -DPF_ENDS
    python -m paper_2504_00492_b200.diag ends         # when each CTA of one launch starts and ends (device clock)
    python -m paper_2504_00492_b200.diag flow-ctas    # time per call against the number of flow-building CTAs
    python -m paper_2504_00492_b200.diag build-delays # anywhere nvcc is: 17 libraries, each with a 2000-cycle spin at
                                                      # one hand-off of the pipeline (-DPF_DELAY_SITE=n)
    python -m paper_2504_00492_b200.diag sensitivity  # time per call of each of them against the ordinary library

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


DELAY_SITES = {
    0: "solve warps, after the Gram epilogue", 1: "solve warps, after the inverse (before X is ready)",
    2: "mid warps, after the Uh epilogue", 3: "mid warps, before the Xi^T drain", 4: "mid warps, before converting V",
    5: "out warps, after the W epilogue", 6: "out warps, after the P^T epilogue", 7: "out warps, before the E drain",
    8: "out warps, after the Qt / OI drain", 9: "out warps, before preparing Q", 10: "MMA warp, before [Uh|W] = X [V|K]",
    11: "MMA warp, before E and Xi^T", 12: "MMA warp, before Qt^T and OI^T", 13: "MMA warp, before the next Gram product",
    14: "TMA warp, before loading K", 15: "flag warp, before the release of the ready flag",
    16: "scan CTAs: chain warps, before publishing the state (128 steps per sequence)",
}


def _delay_lib(site: int) -> str:
    return os.path.join(PKG, "_build_diag", f"libpf_delay{site}.so")


def build_delays():
    """Only pf_fused.cu differs between the variants: its object is rebuilt, the others come from the ordinary build."""
    import glob
    import subprocess
    sys.path.insert(0, os.path.dirname(PKG))
    from paper_2504_00492_b200 import build as _b
    _b.build()
    others = [o for o in glob.glob(os.path.join(PKG, "_build", "*.o")) if os.path.basename(o) != "pf_fused.o"]
    os.makedirs(os.path.join(PKG, "_build_diag"), exist_ok=True)
    procs = []
    for site in DELAY_SITES:
        obj = os.path.join(PKG, "_build_diag", f"pf_fused_delay{site}.o")
        cmd = ["nvcc", *_b.NVCC_FLAGS, f"-DPF_DELAY_SITE={site}", "-I", os.path.join(_b.ROOT, "include"), "-I", _b.CSRC,
               "-c", os.path.join(_b.CSRC, "pf_fused.cu"), "-o", obj]
        procs.append((site, obj, subprocess.Popen(cmd)))
        if len(procs) % 6 == 0:
            for _, _, pr in procs[-6:]:
                pr.wait()
    for site, obj, pr in procs:
        if pr.wait() != 0:
            raise RuntimeError(f"nvcc failed for site {site}")
        subprocess.run(["nvcc", "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", _delay_lib(site), obj,
                        *others], check=True)
    print("built", len(procs), "libraries under", os.path.join(PKG, "_build_diag"))


def sensitivity():
    """Each variant in a process of its own (one library per process)."""
    import subprocess
    def run(lib):
        code = ("import sys; sys.argv=['x']; from paper_2504_00492_b200 import diag; "
                f"t,pf,w,ws,call = diag._setup({lib!r}); print(diag._time(t, call))")
        out = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, cwd=os.path.dirname(PKG))
        return float(out.stdout.strip().splitlines()[-1])
    base = sorted(run(None) for _ in range(3))[1]
    print(f"ordinary library: {base:.1f} us per call (median of 3)")
    for site, name in DELAY_SITES.items():
        us = run(_delay_lib(site))
        per = 128 if site == 16 else 36       # delays per CTA: chunks per flow CTA / steps per scan CTA at config 2
        injected = per * 2000 / 1965.0
        print(f"site {site:2d} {name:62s}: {us:6.1f} us  +{us - base:5.1f} us = {100 * (us - base) / injected:4.0f} % of "
              f"the {injected:.0f} us injected")


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
    elif what == "build-delays":
        build_delays()
    elif what == "sensitivity":
        sensitivity()
    else:
        raise SystemExit(__doc__)
