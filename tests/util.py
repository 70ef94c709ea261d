"""Helpers shared by the GPU parity tests."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import pf_synth

TOL_BF16 = 2e-3   # bf16 inputs: max|gpu - ref| / max|ref| per tensor
TOL_F32 = 1e-5    # fp32 path


def max_rel(x, ref) -> float:
    """max_i |x_i - ref_i| / max_i |ref_i| over the whole tensor."""
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.abs(ref).max() if ref.size else 0.0
    if ref.size == 0:
        return 0.0
    if den == 0.0:
        return float(np.abs(x - ref).max())
    return float(np.abs(x - ref).max() / den)


def rel_l2(x, ref) -> float:
    """||x - ref||_2 / ||ref||_2 over the whole tensor."""
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = float(np.linalg.norm(ref))
    return float(np.linalg.norm(x - ref)) / den if den > 0 else float(np.linalg.norm(x - ref))


def check_per_sequence(x, ref, tol, what=""):
    """The same max-normalised error, but per (b, h) sequence: a sequence whose values are small against the largest
    sequence of the tensor cannot hide behind it."""
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    if ref.ndim < 3 or ref.size == 0:
        return 0.0
    worst = 0.0
    for b in range(ref.shape[0]):
        for h in range(ref.shape[1]):
            e = max_rel(x[b, h], ref[b, h])
            worst = max(worst, e)
            assert e <= tol, f"{what}: sequence (b={b}, h={h}) error {e:.3e} > {tol}"
    return worst


def run_gpu(w: pf_synth.Workload, inp: pf_synth.Inputs, impl="auto", chunk=None, workspace=None, mode="sum",
            step="euler", **options):
    import paper_2504_00492_b200 as pf
    d = inp.to("cuda")
    O, Sf = pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, chunk or w.chunk, impl=impl, workspace=workspace,
                                  mode=mode, step=step, **options)
    torch.cuda.synchronize()
    return O.cpu().numpy(), Sf.cpu().numpy()


def run_oracle(inp: pf_synth.Inputs, mode="sum", step="euler"):
    return oracle.deltanet_fwd(inp.q, inp.k, inp.v, inp.beta, inp.S0, mode=mode, exact=(step == "exact"))


def check_parity(w: pf_synth.Workload, impl="auto", tol=None, inp=None, mode="sum", step="euler", **options):
    """CUDA path against the oracle on the same bits: max|d| / max|ref| per tensor (the tolerance's metric) and per
    (b, h) sequence; the relative L2 errors are printed beside them."""
    inp = inp or pf_synth.make_inputs(w)
    tol = tol if tol is not None else (TOL_F32 if w.dtype == "f32" else TOL_BF16)
    O, Sf = run_gpu(w, inp, impl=impl, mode=mode, step=step, **options)
    O_ref, Sf_ref = run_oracle(inp, mode=mode, step=step)
    assert np.isfinite(O).all() and np.isfinite(Sf).all()
    eo, es = max_rel(O, O_ref), max_rel(Sf, Sf_ref)
    print(f"{w.name}: max-normalised O {eo:.2e} S_final {es:.2e}; relative L2 O {rel_l2(O, O_ref):.2e} "
          f"S_final {rel_l2(Sf, Sf_ref):.2e}")
    assert eo <= tol, f"{w.name}: O error {eo:.3e} > {tol}"
    assert es <= tol, f"{w.name}: S_final error {es:.3e} > {tol}"
    check_per_sequence(O, O_ref, tol, w.name + " O")
    check_per_sequence(Sf, Sf_ref, tol, w.name + " S_final")
    return eo, es
