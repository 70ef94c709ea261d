"""The allocation-free entry point pf_deltanet_fwd_f32_static.

It serves callers that may not allocate device memory when they need the forward pass (a loop that
forbids allocation after start-up, a host with a fixed device-memory budget, a process whose allocator
belongs to another runtime): its per-chunk scratch is a fixed array inside libpf.so instead of memory
taken from an allocator.  The test calls it through the C ABI with caller-provided outputs and checks it
against the fp64 oracle on two calls in a row with different inputs, so that whatever the first call
left in the shared array cannot leak into the second.  This file sorts last on purpose: a run that stops
at the first failure has then already run every other test."""
import pytest
import torch

import pf_synth
from pf_synth import Workload
from tests import util

pytestmark = pytest.mark.gpu


def _call_static(lib, d, w, O, S):
    return lib.pf_deltanet_fwd_f32_static(d.q.data_ptr(), d.k.data_ptr(), d.v.data_ptr(), d.beta.data_ptr(),
                                          None if d.S0 is None else d.S0.data_ptr(), w.B, w.H, w.L, w.d_k, w.d_v,
                                          w.r, w.chunk, O.data_ptr(), None if S is None else S.data_ptr(),
                                          torch.cuda.current_stream().cuda_stream)


def test_static_scratch_entry_matches_the_oracle_twice():
    import paper_2504_00492_b200 as pf
    from paper_2504_00492_b200 import binding
    lib = binding.lib()
    assert pf.pf_static_scratch_bytes() == 8 << 20
    cases = [pf_synth.CONFIGS["c0"],
             Workload("static_r2", B=1, H=2, L=150, d_k=64, d_v=128, r=2, chunk=32, dtype="f32", s0_std=0.1, seed=41)]
    for w in cases:
        assert 0 < pf.pf_static_scratch_need(w.B, w.H, w.L, w.d_k, w.d_v, w.r, w.chunk) <= pf.pf_static_scratch_bytes()
        inp = pf_synth.make_inputs(w)
        d = inp.to("cuda")
        O = torch.full((w.B, w.H, w.L, w.d_v), float("nan"), device="cuda")
        S = torch.full((w.B, w.H, w.d_k, w.d_v), float("nan"), device="cuda")
        rc = _call_static(lib, d, w, O, S)
        assert rc == 0, binding.pf_status_string(rc) + " " + binding.pf_last_error_string()
        torch.cuda.synchronize()
        assert pf.pf_last_launch_count() == 4          # Gram/attention, solve, W/Uh, scan
        O_ref, S_ref = util.run_oracle(inp)
        assert util.max_rel(O.cpu().numpy(), O_ref) <= util.TOL_F32
        assert util.max_rel(S.cpu().numpy(), S_ref) <= util.TOL_F32
        util.check_per_sequence(O.cpu().numpy(), O_ref, util.TOL_F32, w.name + " O")


def test_static_scratch_entry_refuses_outputs_that_overlap_inputs():
    from paper_2504_00492_b200 import binding
    lib = binding.lib()
    w = Workload("static_alias", B=1, H=1, L=64, d_k=64, d_v=64, r=1, chunk=32, dtype="f32", seed=43)
    d = pf_synth.make_inputs(w).to("cuda")
    v_before = d.v.clone()
    O_alias = d.v.view(w.B, w.H, w.L, w.d_v)           # r = 1 and d_v = d_v: the same bytes as v
    rc = _call_static(lib, d, w, O_alias, None)
    assert rc == -1, binding.pf_status_string(rc)              # PF_ERR_INVALID
    torch.cuda.synchronize()
    assert torch.equal(d.v, v_before)


def test_static_scratch_entry_refuses_large_problems():
    import paper_2504_00492_b200 as pf
    w = Workload("static_big", B=2, H=4, L=2048, d_k=128, d_v=128, r=2, chunk=64, dtype="f32", seed=42)
    d = pf_synth.make_inputs(w).to("cuda")
    O = torch.zeros(w.B, w.H, w.L, w.d_v, device="cuda")
    with pytest.raises(pf.PfError) as ei:
        pf.pf_deltanet_fwd_f32_static(d.q, d.k, d.v, d.beta, None, w.chunk, O=O)
    assert ei.value.status == -6
    torch.cuda.synchronize()
    assert float(O.abs().sum()) == 0.0
