"""GPU parity: the CUDA path against the fp64 oracle on the same seeded inputs, through the C ABI."""
import numpy as np
import pytest
import torch

import pf_synth
from pf_synth import Workload
from tests import util

pytestmark = pytest.mark.gpu

SMALL = [
    # several chunks + ragged tail, d_k != d_v, every r, every chunk size
    Workload("s_r1", B=2, H=2, L=200, d_k=64, d_v=128, r=1, chunk=64, s0_std=0.1, seed=11),
    Workload("s_r2", B=1, H=3, L=150, d_k=128, d_v=64, r=2, chunk=32, s0_std=0.1, seed=12),
    Workload("s_r3", B=2, H=1, L=97, d_k=64, d_v=64, r=3, chunk=16, beta_scale=2.0, seed=13),
    Workload("s_r4", B=1, H=2, L=260, d_k=128, d_v=128, r=4, chunk=64, beta_scale=2.0, s0_std=0.1, seed=14),
    Workload("s_one_token", B=1, H=1, L=1, d_k=64, d_v=64, r=2, chunk=64, s0_std=0.1, seed=15),
    Workload("s_exact_chunks", B=1, H=2, L=128, d_k=64, d_v=64, r=1, chunk=64, seed=16),
]


@pytest.mark.parametrize("w", SMALL, ids=lambda w: w.name)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_small_cases_simt(w, dtype):
    util.check_parity(w.with_(dtype=dtype), impl="simt")


@pytest.mark.parametrize("w", SMALL, ids=lambda w: w.name)
def test_small_cases_default_impl(w):
    util.check_parity(w, impl="auto")


def test_config0_fp32():
    import paper_2504_00492_b200 as pf
    w = pf_synth.CONFIGS["c0"]
    inp = pf_synth.make_inputs(w)
    d = inp.to("cuda")
    O, Sf = pf.pf_deltanet_fwd_f32(d.q, d.k, d.v, d.beta, None, w.chunk)
    O_ref, Sf_ref = util.run_oracle(inp)
    assert util.max_rel(O.cpu().numpy(), O_ref) <= util.TOL_F32
    assert util.max_rel(Sf.cpu().numpy(), Sf_ref) <= util.TOL_F32
    assert pf.pf_last_launch_count() > 0


def _full_size_parity(w):
    """One call of the plain entry point at full size against the oracle over every (b, h) sequence."""
    import paper_2504_00492_b200 as pf
    inp = pf_synth.make_inputs(w)
    d = inp.to("cuda")
    O, Sf = pf.pf_deltanet_fwd(d.q, d.k, d.v, d.beta, d.S0, w.chunk)
    assert pf.pf_read_status() == 0, pf.pf_last_wait_code()
    assert torch.isfinite(O).all() and torch.isfinite(Sf).all()
    O_ref, Sf_ref = util.run_oracle(inp)
    O, Sf = O.cpu().numpy(), Sf.cpu().numpy()
    eo, es = util.max_rel(O, O_ref), util.max_rel(Sf, Sf_ref)
    print(f"{w.name}: max-normalised O {eo:.2e} S_final {es:.2e}; relative L2 O {util.rel_l2(O, O_ref):.2e} "
          f"S_final {util.rel_l2(Sf, Sf_ref):.2e}")
    assert eo <= util.TOL_BF16 and es <= util.TOL_BF16, (eo, es)
    util.check_per_sequence(O, O_ref, util.TOL_BF16, w.name + " O")
    util.check_per_sequence(Sf, Sf_ref, util.TOL_BF16, w.name + " S_final")


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c3_chunk32"])
def test_full_configs(name):
    """Full benchmark sizes through the central call, in the configuration bench.py times."""
    _full_size_parity(pf_synth.CONFIGS[name])


def test_long_context_all_heads():
    """L = 65536 at full size; the oracle recomputes every one of the 32 heads over all tokens."""
    _full_size_parity(pf_synth.CONFIGS["c4"])


# --- properties that hold at any size -------------------------------------------------------------

@pytest.mark.parametrize("impl", ["simt", "auto"])
def test_split_invariance_and_state_carry(impl):
    """Proposition 2.1: running [0,L1) then [L1,L) with S_final -> S0 equals one call."""
    import paper_2504_00492_b200 as pf
    w = Workload("split", B=1, H=2, L=256, d_k=64, d_v=128, r=2, chunk=32, s0_std=0.1, seed=21)
    d = pf_synth.make_inputs(w).to("cuda")
    O, Sf = pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, impl=impl)
    L1 = 96
    O1, S1 = pf.pf_deltanet_fwd_ex(d.q[:, :, :L1].contiguous(), d.k[:, :, :L1].contiguous(),
                                   d.v[:, :, :L1].contiguous(), d.beta[:, :, :L1].contiguous(), d.S0, w.chunk, impl=impl)
    O2, S2 = pf.pf_deltanet_fwd_ex(d.q[:, :, L1:].contiguous(), d.k[:, :, L1:].contiguous(),
                                   d.v[:, :, L1:].contiguous(), d.beta[:, :, L1:].contiguous(), S1, w.chunk, impl=impl)
    tol = 2e-3
    assert util.max_rel(torch.cat([O1, O2], 2).cpu().numpy(), O.cpu().numpy()) <= tol
    assert util.max_rel(S2.cpu().numpy(), Sf.cpu().numpy()) <= tol


def test_chunk_size_invariance_fp32():
    import paper_2504_00492_b200 as pf
    w = Workload("chunkinv", B=1, H=2, L=192, d_k=64, d_v=64, r=2, chunk=64, dtype="f32", s0_std=0.1, seed=22)
    d = pf_synth.make_inputs(w).to("cuda")
    outs = [pf.pf_deltanet_fwd_f32(d.q, d.k, d.v, d.beta, d.S0, c) for c in (16, 32, 64)]
    for O, Sf in outs[1:]:
        assert util.max_rel(O.cpu().numpy(), outs[0][0].cpu().numpy()) <= 2e-5
        assert util.max_rel(Sf.cpu().numpy(), outs[0][1].cpu().numpy()) <= 2e-5


def test_beta_zero_and_empty_sequence():
    import paper_2504_00492_b200 as pf
    w = Workload("bz", B=1, H=2, L=70, d_k=64, d_v=64, r=2, chunk=32, s0_std=0.1, seed=23)
    d = pf_synth.make_inputs(w).to("cuda")
    O, Sf = pf.pf_deltanet_fwd(d.q, d.k, d.v, torch.zeros_like(d.beta), d.S0, w.chunk)
    assert torch.equal(Sf, d.S0)
    ref = torch.einsum("bhij,bhti->bhtj", d.S0.double(), d.q.double())
    assert util.max_rel(O.cpu().numpy(), ref.cpu().numpy()) <= util.TOL_BF16
    # L = 0: nothing to do but hand the state through
    e = lambda *s: torch.empty(*s, dtype=torch.bfloat16, device="cuda")
    O0, S0f = pf.pf_deltanet_fwd(e(1, 2, 0, 64), e(1, 2, 0, 2, 64), e(1, 2, 0, 2, 64), e(1, 2, 0, 2), d.S0, 32)
    assert O0.shape == (1, 2, 0, 64) and torch.equal(S0f, d.S0)


@pytest.mark.parametrize("impl", ["simt", "auto"])
def test_deterministic_and_workspace_bounds(impl):
    """No atomics anywhere: two runs are bitwise equal; a caller workspace is never overrun."""
    import paper_2504_00492_b200 as pf
    from paper_2504_00492_b200 import binding
    w = Workload("det", B=2, H=2, L=130, d_k=64, d_v=64, r=3, chunk=32, s0_std=0.1, seed=24)
    d = pf_synth.make_inputs(w).to("cuda")
    need = pf.pf_workspace_bytes(w.B, w.H, w.L, w.d_k, w.d_v, w.r, w.chunk, binding.PF_DTYPE_BF16, impl)
    guard = 4096
    buf = torch.full((need + 2 * guard + 256,), 0x5A, dtype=torch.uint8, device="cuda")
    off = (-buf.data_ptr() - guard) % 256 + guard
    ws = buf[off:off + need]
    assert ws.data_ptr() % 256 == 0
    O1, S1 = pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, impl=impl, workspace=ws)
    O2, S2 = pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, impl=impl)
    torch.cuda.synchronize()
    assert torch.equal(O1, O2) and torch.equal(S1, S2)
    assert bool((buf[:off] == 0x5A).all()) and bool((buf[off + need:] == 0x5A).all())
    with pytest.raises(pf.PfError) as ei:
        pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, impl=impl, workspace=ws[: max(need - 256, 0)])
    assert ei.value.status == -6


def test_argument_errors_launch_nothing():
    import paper_2504_00492_b200 as pf
    from paper_2504_00492_b200 import binding
    w = Workload("err", B=1, H=1, L=64, d_k=64, d_v=64, r=1, chunk=64, seed=25)
    d = pf_synth.make_inputs(w).to("cuda")
    O = torch.zeros(1, 1, 64, 64, device="cuda")
    lib = binding.lib()
    st = torch.cuda.current_stream().cuda_stream
    # misaligned q
    rc = lib.pf_deltanet_fwd(d.q.data_ptr() + 2, d.k.data_ptr(), d.v.data_ptr(), d.beta.data_ptr(), None,
                             1, 1, 64, 64, 64, 1, 64, O.data_ptr(), None, st)
    assert rc == -3
    # null k
    rc = lib.pf_deltanet_fwd(d.q.data_ptr(), None, d.v.data_ptr(), d.beta.data_ptr(), None,
                             1, 1, 64, 64, 64, 1, 64, O.data_ptr(), None, st)
    assert rc == -1
    # O aliasing v
    rc = lib.pf_deltanet_fwd(d.q.data_ptr(), d.k.data_ptr(), d.v.data_ptr(), d.beta.data_ptr(), None,
                             1, 1, 64, 64, 64, 1, 64, d.v.data_ptr(), None, st)
    assert rc == -1
    torch.cuda.synchronize()
    assert float(O.abs().sum()) == 0.0


# --- tensor-core path -------------------------------------------------------------------------------

TC_CASES = [
    Workload("tc_r2_d128", B=1, H=2, L=512, d_k=128, d_v=128, r=2, chunk=64, s0_std=0.1, seed=31),
    Workload("tc_r2_ragged", B=2, H=1, L=333, d_k=128, d_v=128, r=2, chunk=64, s0_std=0.1, seed=32),
    Workload("tc_r1_d128", B=1, H=2, L=300, d_k=128, d_v=128, r=1, chunk=64, s0_std=0.1, seed=33),
    Workload("tc_r4_d64_c32", B=2, H=2, L=200, d_k=64, d_v=64, r=4, chunk=32, beta_scale=2.0, seed=34),
    Workload("tc_dk64_dv128", B=1, H=2, L=256, d_k=64, d_v=128, r=2, chunk=64, s0_std=0.1, seed=35),
    Workload("tc_dk128_dv64", B=1, H=2, L=256, d_k=128, d_v=64, r=2, chunk=32, s0_std=0.1, seed=36),
    Workload("tc_one_token", B=1, H=1, L=1, d_k=128, d_v=128, r=2, chunk=64, s0_std=0.1, seed=37),
    # r = 3: 96 (48) rows per chunk in a tile of 128 (64), the rows past them switched off by beta = 0
    Workload("tc_r3_d64_c32", B=2, H=2, L=333, d_k=64, d_v=64, r=3, chunk=32, beta_scale=2.0, s0_std=0.1, seed=48),
    Workload("tc_r3_d64_c16", B=1, H=2, L=200, d_k=64, d_v=64, r=3, chunk=16, s0_std=0.1, seed=49),
    Workload("tc_r3_dk64_dv128", B=1, H=2, L=256, d_k=64, d_v=128, r=3, chunk=32, s0_std=0.1, seed=50),
]


def _run_with_status(w, impl, mode="sum", step="euler", **options):
    """Runs with a caller workspace, reads the device status word through pf_read_status, compares with the oracle."""
    import paper_2504_00492_b200 as pf
    from paper_2504_00492_b200 import binding
    inp = pf_synth.make_inputs(w)
    d = inp.to("cuda")
    need = pf.pf_workspace_bytes_ex(w.B, w.H, w.L, w.d_k, w.d_v, w.r, w.chunk, binding.PF_DTYPE_BF16, impl, mode=mode,
                                    **options)
    assert need > 0
    ws = torch.zeros(need + 256, dtype=torch.uint8, device="cuda")
    off = (-ws.data_ptr()) % 256
    O, Sf = pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, impl=impl, workspace=ws[off:off + need],
                                  mode=mode, step=step, **options)
    st = pf.pf_read_status(ws[off:off + need])
    assert st == 0, f"device-side wait {pf.pf_last_wait_code()} expired"
    O_ref, Sf_ref = util.run_oracle(inp, mode=mode, step=step)
    util.check_per_sequence(O.cpu().numpy(), O_ref, util.TOL_BF16, w.name + " O")
    return util.max_rel(O.cpu().numpy(), O_ref), util.max_rel(Sf.cpu().numpy(), Sf_ref)


@pytest.mark.parametrize("w", TC_CASES, ids=lambda w: w.name)
def test_tc_scan_with_reference_flows(w):
    """tc_scan alone: the per-chunk flows come from the fp32 SIMT kernels."""
    eo, es = _run_with_status(w, "tc_refflow")
    assert eo <= util.TOL_BF16 and es <= util.TOL_BF16, (eo, es)


@pytest.mark.parametrize("w", TC_CASES, ids=lambda w: w.name)
def test_tc_full_path(w):
    """tc_flow + tc_scan: everything on tensor cores."""
    eo, es = _run_with_status(w, "tc")
    assert eo <= util.TOL_BF16 and es <= util.TOL_BF16, (eo, es)


def _scaled(inp, factor):
    return pf_synth.Inputs(inp.q, inp.k, inp.v * factor, inp.beta, None if inp.S0 is None else inp.S0 * factor)


@pytest.mark.parametrize("impl", ["tc", "tc_split"])
def test_values_near_the_top_of_the_documented_fp16_range(impl):
    """v and S0 scaled by 2^10 (exact in bf16): the tensor-core paths hold them and the state in fp16, whose range the
    header documents; the result is linear in (v, S0), so the normalised error must stay what it is unscaled."""
    import paper_2504_00492_b200 as pf
    w = Workload("range_1e3", B=1, H=2, L=512, d_k=128, d_v=128, r=2, chunk=64, s0_std=0.1, seed=38)
    inp = _scaled(pf_synth.make_inputs(w), 1024.0)
    d = inp.to("cuda")
    O, Sf = pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, impl=impl)
    assert pf.pf_read_status() == 0
    O_ref, Sf_ref = util.run_oracle(inp)
    assert float(abs(O_ref).max()) > 100.0
    assert torch.isfinite(O).all() and torch.isfinite(Sf).all()
    assert util.max_rel(O.cpu().numpy(), O_ref) <= util.TOL_BF16
    assert util.max_rel(Sf.cpu().numpy(), Sf_ref) <= util.TOL_BF16


def test_values_beyond_the_fp16_range_need_the_fp32_path():
    """Scaled by 2^20 the fp16 operands overflow (documented); PF_IMPL_SIMT keeps fp32 throughout and still agrees."""
    import paper_2504_00492_b200 as pf
    w = Workload("range_1e6", B=1, H=1, L=256, d_k=128, d_v=128, r=2, chunk=64, s0_std=0.1, seed=39)
    inp = _scaled(pf_synth.make_inputs(w), float(2 ** 20))
    d = inp.to("cuda")
    O, Sf = pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, impl="simt")
    O_ref, Sf_ref = util.run_oracle(inp)
    assert util.max_rel(O.cpu().numpy(), O_ref) <= util.TOL_BF16
    assert util.max_rel(Sf.cpu().numpy(), Sf_ref) <= util.TOL_BF16


# --- single-launch tensor-core path (flow builders and state scan side by side) -----------------------

FUSED_CASES = [
    Workload("fu_r2_c64", B=2, H=3, L=1000, d_k=128, d_v=128, r=2, chunk=64, s0_std=0.1, seed=41),       # n = 128, ring wraps
    Workload("fu_r4_c32", B=1, H=2, L=333, d_k=128, d_v=128, r=4, chunk=32, beta_scale=2.0, s0_std=0.1, seed=42),
    Workload("fu_r1_c64", B=2, H=2, L=700, d_k=128, d_v=128, r=1, chunk=64, s0_std=0.1, seed=43),       # n = 64
    Workload("fu_r2_c32", B=1, H=3, L=450, d_k=128, d_v=128, r=2, chunk=32, seed=44),                   # n = 64, no S0
    Workload("fu_r4_c16", B=1, H=2, L=130, d_k=128, d_v=128, r=4, chunk=16, beta_scale=2.0, seed=45),   # n = 64, C = 16
    Workload("fu_short", B=3, H=1, L=17, d_k=128, d_v=128, r=2, chunk=64, s0_std=0.1, seed=46),         # less than a chunk
    Workload("fu_r3_c32", B=2, H=2, L=1000, d_k=128, d_v=128, r=3, chunk=32, s0_std=0.1, seed=51),       # 96 rows in a tile of 128
    Workload("fu_r3_c16", B=1, H=3, L=333, d_k=128, d_v=128, r=3, chunk=16, beta_scale=2.0, seed=52),   # 48 rows in a tile of 64
    Workload("fu_many_seq", B=5, H=28, L=192, d_k=128, d_v=128, r=2, chunk=64, s0_std=0.1, seed=47),    # 140 scan CTAs, 8 flow CTAs
]


@pytest.mark.parametrize("w", FUSED_CASES, ids=lambda w: w.name)
def test_fused_path_against_oracle(w):
    eo, es = _run_with_status(w, "tc")
    assert eo <= util.TOL_BF16 and es <= util.TOL_BF16, (eo, es)


def test_fused_and_split_agree_and_ring_depth_is_invisible():
    """The single-launch and the two-launch forms compute the same chunk algebra (different accumulation
    orders and operand roundings: they agree to the bf16 tolerance); the ring depth changes only the
    schedule, so results are bitwise identical across depths and across repeated runs."""
    import paper_2504_00492_b200 as pf
    w = Workload("fu_vs_split", B=2, H=2, L=1500, d_k=128, d_v=128, r=2, chunk=64, s0_std=0.1, seed=48)
    d = pf_synth.make_inputs(w).to("cuda")
    outs = []
    for depth in (3, 5, 8, 0, 21):
        O, Sf = pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, impl="tc", ring_depth=depth)
        assert pf.pf_read_status() == 0, pf.pf_last_wait_code()      # (no workspace, no status pointer: the library's word)
        outs.append((O.clone(), Sf.clone()))
    for O, Sf in outs[1:]:
        assert torch.equal(O, outs[0][0]) and torch.equal(Sf, outs[0][1])
    O2, S2 = pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, impl="tc_split")
    assert util.max_rel(outs[0][0].cpu().numpy(), O2.cpu().numpy()) <= util.TOL_BF16
    assert util.max_rel(outs[0][1].cpu().numpy(), S2.cpu().numpy()) <= util.TOL_BF16


def test_too_many_sequences_take_the_two_launch_form():
    """More sequences than scan CTAs can be placed: PF_IMPL_TC still works (two launches)."""
    w = Workload("fu_fallback", B=6, H=25, L=130, d_k=128, d_v=128, r=2, chunk=64, s0_std=0.1, seed=49)   # 150 sequences
    eo, es = _run_with_status(w, "tc")
    assert eo <= util.TOL_BF16 and es <= util.TOL_BF16, (eo, es)


def test_options_reject_bad_values():
    import paper_2504_00492_b200 as pf
    w = FUSED_CASES[5]
    d = pf_synth.make_inputs(w).to("cuda")
    for bad in (dict(ring_depth=2), dict(ring_depth=65), dict(wu_builder=2), dict(segments=-1), dict(segments=65)):
        with pytest.raises(pf.PfError) as ei:
            pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, impl="tc", **bad)
        assert ei.value.status == -1, bad
        assert pf.pf_workspace_bytes_ex(w.B, w.H, w.L, w.d_k, w.d_v, w.r, w.chunk, impl="tc", **bad) == 0


def test_an_expired_device_wait_is_reported():
    """A wait that runs out: one warp waits (bounded, 200 us) for a flag that nothing sets.  The kernel returns, the
    status word holds the code, pf_read_status reports PF_ERR_TIMEOUT, and the next forward call clears the word and
    works -- nothing hangs or faults on the way."""
    import paper_2504_00492_b200 as pf
    for own in (False, True):
        word = torch.zeros(1, dtype=torch.int32, device="cuda") if own else None
        pf.pf_wait_selftest(word, limit_us=200)
        assert pf.pf_read_status(word) == -7
        assert pf.pf_last_wait_code() == 900
        assert pf.pf_status_string(-7) == "device-side wait timed out"
        w = FUSED_CASES[5]
        inp = pf_synth.make_inputs(w)
        d = inp.to("cuda")
        O, Sf = pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, impl="tc", status=word)
        assert pf.pf_read_status(word) == 0 and pf.pf_last_wait_code() == 0
        O_ref, Sf_ref = util.run_oracle(inp)
        assert util.max_rel(O.cpu().numpy(), O_ref) <= util.TOL_BF16
        assert util.max_rel(Sf.cpu().numpy(), Sf_ref) <= util.TOL_BF16


def test_chunk_length_that_auto_evaluates_with_is_reported():
    import paper_2504_00492_b200 as pf
    from paper_2504_00492_b200 import binding
    assert pf.pf_select_chunk(8, 16, 4096, 64, 64, 4, 64) == 32                 # 256 rows per chunk: evaluated as chunk 32
    assert pf.pf_select_chunk(8, 16, 4096, 64, 64, 4, 64, impl="simt") == 64    # explicit implementations keep it
    assert pf.pf_select_chunk(2, 16, 8192, 128, 128, 2, 64) == 64
    assert pf.pf_select_chunk(2, 16, 8192, 128, 128, 2, 48) == -2


def test_back_to_back_launches_without_synchronisation():
    """Several calls queued on one stream with a shared caller workspace: flags are reset in stream order."""
    import paper_2504_00492_b200 as pf
    from paper_2504_00492_b200 import binding
    w = Workload("fu_b2b", B=1, H=8, L=4096, d_k=128, d_v=128, r=2, chunk=64, s0_std=0.1, seed=50)
    d = pf_synth.make_inputs(w).to("cuda")
    need = pf.pf_workspace_bytes(w.B, w.H, w.L, w.d_k, w.d_v, w.r, w.chunk, binding.PF_DTYPE_BF16, "tc")
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    first = None
    for rep in range(6):
        for _ in range(3):
            O, Sf = pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, impl="tc", workspace=ws)
        torch.cuda.synchronize()
        assert int(ws[:4].view(torch.int32).item()) == 0
        if first is None:
            first = (O.clone(), Sf.clone())
        else:
            assert torch.equal(O, first[0]) and torch.equal(Sf, first[1])


# --- product form: the r factors of a token act one after another (mask strict in the flattened row index) -------

@pytest.mark.parametrize("w", [w for w in SMALL if w.r > 1], ids=lambda w: w.name)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_product_mode_simt(w, dtype):
    util.check_parity(w.with_(dtype=dtype), impl="simt", mode="product")


@pytest.mark.parametrize("w", [w for w in TC_CASES if w.r > 1], ids=lambda w: w.name)
@pytest.mark.parametrize("impl", ["tc_split", "tc_refflow"])
def test_product_mode_two_launch_tensor_core_path(w, impl):
    eo, es = _run_with_status(w, impl, mode="product")
    assert eo <= util.TOL_BF16 and es <= util.TOL_BF16, (eo, es)


@pytest.mark.parametrize("w", [w for w in FUSED_CASES if w.r > 1], ids=lambda w: w.name)
def test_product_mode_single_launch_path(w):
    eo, es = _run_with_status(w, "tc", mode="product")
    assert eo <= util.TOL_BF16 and es <= util.TOL_BF16, (eo, es)


def test_product_mode_differs_from_sum_and_r1_does_not():
    """The mode reaches the kernels (the two forms differ by far more than the tolerance for r = 2), and for
    r = 1 the two are the same computation, bit for bit."""
    import paper_2504_00492_b200 as pf
    w = Workload("pm_r2", B=1, H=2, L=300, d_k=128, d_v=128, r=2, chunk=64, s0_std=0.1, seed=51)
    d = pf_synth.make_inputs(w).to("cuda")
    for impl in ("simt", "tc"):
        Os, Ss = pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, impl=impl)
        Op, Sp = pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, impl=impl, mode="product")
        assert util.max_rel(Op.cpu().numpy(), Os.cpu().numpy()) > 10 * util.TOL_BF16
    w1 = w.with_(r=1)
    d1 = pf_synth.make_inputs(w1).to("cuda")
    for impl in ("simt", "tc"):
        Os, Ss = pf.pf_deltanet_fwd_ex(d1.q, d1.k, d1.v, d1.beta, d1.S0, w1.chunk, impl=impl)
        Op, Sp = pf.pf_deltanet_fwd_ex(d1.q, d1.k, d1.v, d1.beta, d1.S0, w1.chunk, impl=impl, mode="product")
        assert torch.equal(Os, Op) and torch.equal(Ss, Sp)


def test_unknown_mode_is_rejected():
    import paper_2504_00492_b200 as pf
    w = SMALL[1]
    d = pf_synth.make_inputs(w).to("cuda")
    with pytest.raises(pf.PfError) as e:
        pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, mode=7)
    assert e.value.status == -1


# --- exact step of a rank-1 factor: exp(-beta k k^T) instead of I - beta k k^T ---------------------------------------

EXACT_CASES = [   # (workload, impl, mode): r = 1 in the sum form, any r in the product form; beta up to 2
    (SMALL[0].with_(dtype="f32"), "simt", "sum"),
    (SMALL[0], "simt", "sum"),
    (SMALL[3], "simt", "product"),
    (SMALL[2].with_(dtype="f32"), "simt", "product"),
    (TC_CASES[2], "tc_split", "sum"),
    (TC_CASES[3], "tc_split", "product"),
    (TC_CASES[4], "tc_refflow", "product"),
    (FUSED_CASES[2], "tc", "sum"),
    (FUSED_CASES[0], "tc", "product"),
    (FUSED_CASES[1], "tc", "product"),
    ([w for w in TC_CASES if w.name == "tc_r3_d64_c32"][0], "tc_split", "product"),      # rank 3: 96 rows in a tile of 128
    ([w for w in FUSED_CASES if w.name == "fu_r3_c32"][0], "tc", "product"),
]


@pytest.mark.parametrize("w,impl,mode", EXACT_CASES, ids=lambda x: getattr(x, "name", x))
def test_exact_step(w, impl, mode):
    if impl == "simt":
        util.check_parity(w, impl=impl, mode=mode, step="exact")
    else:
        eo, es = _run_with_status(w, impl, mode=mode, step="exact")
        assert eo <= util.TOL_BF16 and es <= util.TOL_BF16, (eo, es)


def test_exact_step_changes_the_result_and_needs_rank_one_factors():
    import paper_2504_00492_b200 as pf
    w = TC_CASES[2]                                    # r = 1
    d = pf_synth.make_inputs(w).to("cuda")
    O1, _ = pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk)
    O2, _ = pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, step="exact")
    assert util.max_rel(O2.cpu().numpy(), O1.cpu().numpy()) > 10 * util.TOL_BF16
    w2 = TC_CASES[0]                                   # r = 2, sum form: not rank 1
    d2 = pf_synth.make_inputs(w2).to("cuda")
    with pytest.raises(pf.PfError) as e:
        pf.pf_deltanet_fwd_ex(d2.q, d2.k, d2.v, d2.beta, d2.S0, w2.chunk, step="exact")
    assert e.value.status == -2
    with pytest.raises(pf.PfError) as e:
        pf.pf_deltanet_fwd_ex(d2.q, d2.k, d2.v, d2.beta, d2.S0, w2.chunk, step=5)
    assert e.value.status == -1


# --- W and Uh from the two-index system of Theorem 3.3 (pf_params.wu_builder = 1) instead of the triangular inverse ----

@pytest.mark.parametrize("w", SMALL, ids=lambda w: w.name)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_theorem_3_3_builder_simt(w, dtype):
    util.check_parity(w.with_(dtype=dtype), impl="simt", wu_builder=1)


@pytest.mark.parametrize("w", [SMALL[1], SMALL[3]], ids=lambda w: w.name)
def test_theorem_3_3_builder_product_form_and_exact_step(w):
    util.check_parity(w.with_(dtype="f32"), impl="simt", mode="product", wu_builder=1)
    util.check_parity(w, impl="simt", mode="product", step="exact", wu_builder=1)


def test_theorem_3_3_builder_feeds_the_tensor_core_scan():
    eo, es = _run_with_status(TC_CASES[0], "tc_refflow", wu_builder=1)
    assert eo <= util.TOL_BF16 and es <= util.TOL_BF16, (eo, es)


def test_the_two_builders_agree_closely_and_need_different_workspaces():
    import paper_2504_00492_b200 as pf
    w = SMALL[3].with_(dtype="f32")
    d = pf_synth.make_inputs(w).to("cuda")
    O0, S0_ = pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, impl="simt")
    need0 = pf.pf_workspace_bytes(w.B, w.H, w.L, w.d_k, w.d_v, w.r, w.chunk, 1, "simt")
    O1, S1_ = pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, impl="simt", wu_builder=1)
    need1 = pf.pf_workspace_bytes_ex(w.B, w.H, w.L, w.d_k, w.d_v, w.r, w.chunk, 1, "simt", wu_builder=1)
    assert need1 > need0
    assert pf.pf_workspace_bytes(w.B, w.H, w.L, w.d_k, w.d_v, w.r, w.chunk, 1, "simt") == need0      # (no hidden state)
    assert util.max_rel(O1.cpu().numpy(), O0.cpu().numpy()) < 2 * util.TOL_F32
    assert util.max_rel(S1_.cpu().numpy(), S0_.cpu().numpy()) < 2 * util.TOL_F32


# --- segments evaluated side by side, flows composed (pf_params.segments) -----------------------------------------------

SEGMENT_CASES = [
    (Workload("sg_simt_f32", B=1, H=2, L=256, d_k=64, d_v=64, r=2, chunk=32, s0_std=0.1, seed=61, dtype="f32"), "simt", 4),
    (Workload("sg_simt_r3", B=2, H=1, L=120, d_k=128, d_v=128, r=3, chunk=16, beta_scale=2.0, seed=62, dtype="f32"), "simt", 3),
    (Workload("sg_fused", B=1, H=2, L=2048, d_k=128, d_v=128, r=2, chunk=64, s0_std=0.1, seed=63), "tc", 8),
    (Workload("sg_fused_ragged", B=1, H=1, L=1000, d_k=128, d_v=128, r=2, chunk=64, s0_std=0.1, seed=64), "tc", 2),
    (Workload("sg_split_d64", B=1, H=2, L=512, d_k=64, d_v=64, r=4, chunk=32, beta_scale=2.0, seed=65), "tc_split", 4),
    (Workload("sg_fused_r3", B=1, H=2, L=1536, d_k=128, d_v=128, r=3, chunk=64, s0_std=0.1, seed=68), "auto", 4),   # chunks of 42 tokens
]


@pytest.mark.parametrize("w,impl,S", SEGMENT_CASES, ids=lambda x: getattr(x, "name", x))
def test_segmented_evaluation(w, impl, S):
    if impl == "simt":
        util.check_parity(w, impl=impl, segments=S)
    else:
        eo, es = _run_with_status(w, impl, segments=S)
        assert eo <= util.TOL_BF16 and es <= util.TOL_BF16, (eo, es)


def test_segmented_product_form_exact_step_and_library_workspace():
    import paper_2504_00492_b200 as pf
    w = Workload("sg_modes", B=1, H=2, L=512, d_k=128, d_v=128, r=2, chunk=64, s0_std=0.1, seed=66)
    eo, es = _run_with_status(w, "tc", mode="product", step="exact", segments=4)
    assert eo <= util.TOL_BF16 and es <= util.TOL_BF16, (eo, es)
    inp = pf_synth.make_inputs(w)
    d = inp.to("cuda")
    O, Sf = pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, segments=4)      # library-owned workspace
    assert pf.pf_read_status() == 0
    O_ref, Sf_ref = util.run_oracle(inp)
    assert util.max_rel(O.cpu().numpy(), O_ref) <= util.TOL_BF16 and util.max_rel(Sf.cpu().numpy(), Sf_ref) <= util.TOL_BF16
    # the plain entry points are not affected by anything an earlier call asked for
    O2, _ = pf.pf_deltanet_fwd(d.q, d.k, d.v, d.beta, d.S0, w.chunk)
    torch.cuda.synchronize()
    assert pf.pf_last_launch_count() == 1


def test_segments_that_do_not_fit_are_refused():
    import paper_2504_00492_b200 as pf
    w = SMALL[0]                                   # d_k != d_v
    d = pf_synth.make_inputs(w).to("cuda")
    with pytest.raises(pf.PfError) as e:
        pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, segments=4)
    assert e.value.status == -2
    w2 = Workload("sg_bad_L", B=1, H=1, L=130, d_k=64, d_v=64, r=1, chunk=32, seed=67)     # 130 % 4 != 0
    d2 = pf_synth.make_inputs(w2).to("cuda")
    with pytest.raises(pf.PfError) as e:
        pf.pf_deltanet_fwd_ex(d2.q, d2.k, d2.v, d2.beta, d2.S0, w2.chunk, segments=4)
    assert e.value.status == -2
    assert pf.pf_workspace_bytes_ex(w2.B, w2.H, w2.L, w2.d_k, w2.d_v, w2.r, w2.chunk, 0, "auto", segments=4) == 0
    assert pf.pf_workspace_bytes(w2.B, w2.H, w2.L, w2.d_k, w2.d_v, w2.r, w2.chunk, 0, "auto") > 0


# --- PF_IMPL_AUTO may evaluate with another chunk length to reach the tensor-core kernels ---------------------------------

def test_auto_rechunks_onto_the_tensor_core_path():
    import paper_2504_00492_b200 as pf
    from paper_2504_00492_b200 import binding
    # r = 4 with chunk 64 is 256 rows per chunk; chunk 32 gives the 128 the kernels take
    w = Workload("auto_r4_c64", B=2, H=2, L=500, d_k=64, d_v=64, r=4, chunk=64, beta_scale=2.0, s0_std=0.1, seed=71)
    assert pf.pf_select_impl(w.B, w.H, w.L, w.d_k, w.d_v, w.r, w.chunk, binding.PF_DTYPE_BF16, "auto") == binding.PF_IMPL_TC
    # an explicit tensor-core choice splits the 256-row chunk into two blocks of 128 rows as well
    assert pf.pf_select_impl(w.B, w.H, w.L, w.d_k, w.d_v, w.r, w.chunk, binding.PF_DTYPE_BF16, "tc") == binding.PF_IMPL_TC
    assert pf.pf_select_chunk(w.B, w.H, w.L, w.d_k, w.d_v, w.r, w.chunk, impl="tc") == 32
    util.check_parity(w, impl="auto")
    for impl in ("auto", "tc", "tc_split"):
        eo, es = _run_with_status(w, impl)
        assert eo <= util.TOL_BF16 and es <= util.TOL_BF16, (impl, eo, es)
    eo, es = _run_with_status(w.with_(d_k=128, d_v=128, name="tc_r4_c64_d128"), "tc")        # the single launch
    assert eo <= util.TOL_BF16 and es <= util.TOL_BF16, (eo, es)
    # r = 1 with chunk 32 is 32 rows: chunk 64 gives 64
    w2 = Workload("auto_r1_c32", B=1, H=2, L=300, d_k=128, d_v=128, r=1, chunk=32, s0_std=0.1, seed=72)
    assert pf.pf_select_impl(w2.B, w2.H, w2.L, w2.d_k, w2.d_v, w2.r, w2.chunk, binding.PF_DTYPE_BF16, "auto") == binding.PF_IMPL_TC
    util.check_parity(w2, impl="auto")
    # r = 3 never gives 64 or 128 rows: its chunks sit in the next larger tile (48 rows in 64, 96 in 128); 192 rows
    # do not fit, so chunk 64 is evaluated with a shorter chunk
    w3 = SMALL[2]
    assert pf.pf_select_impl(w3.B, w3.H, w3.L, w3.d_k, w3.d_v, w3.r, w3.chunk, binding.PF_DTYPE_BF16, "auto") == binding.PF_IMPL_TC
    assert pf.pf_select_impl(w3.B, w3.H, w3.L, w3.d_k, w3.d_v, w3.r, w3.chunk, binding.PF_DTYPE_BF16, "tc") == binding.PF_IMPL_TC
    w4 = Workload("auto_r3_c64", B=2, H=2, L=700, d_k=128, d_v=128, r=3, chunk=64, s0_std=0.1, seed=73)
    assert pf.pf_select_impl(w4.B, w4.H, w4.L, w4.d_k, w4.d_v, w4.r, w4.chunk, binding.PF_DTYPE_BF16, "tc") == binding.PF_IMPL_TC
    # ... but an explicit choice never lengthens a chunk: r = 1 with chunk 32 (32 rows) stays outside the tensor-core set
    assert pf.pf_select_impl(w2.B, w2.H, w2.L, w2.d_k, w2.d_v, w2.r, w2.chunk, binding.PF_DTYPE_BF16, "tc") == -2
    assert pf.pf_select_chunk(w4.B, w4.H, w4.L, w4.d_k, w4.d_v, w4.r, w4.chunk) == 42         # 126 of a tile's 128 rows
    util.check_parity(w4, impl="auto")
    util.check_parity(w4.with_(d_k=64, d_v=64, name="auto_r3_c64_d64"), impl="auto")


def test_auto_leaves_the_single_launch_when_few_sms_remain_for_flows():
    """Up to 0.7 x SM count sequences PF_IMPL_AUTO takes the single launch, beyond that the two-launch form; an
    explicit PF_IMPL_TC takes the single launch whenever it can run.  Told apart by the number of kernels launched."""
    import paper_2504_00492_b200 as pf
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    many = Workload("auto_many_seq", B=4, H=(sms * 8 // 10 + 3) // 4, L=192, d_k=128, d_v=128, r=2, chunk=64, s0_std=0.1, seed=73)
    few = many.with_(B=1, H=8)
    assert many.B * many.H * 10 > sms * 7 and many.B * many.H <= sms - 8
    for w, impl, launches in ((many, "auto", 2), (many, "tc", 1), (few, "auto", 1)):
        inp = pf_synth.make_inputs(w)
        d = inp.to("cuda")
        O, Sf = pf.pf_deltanet_fwd_ex(d.q, d.k, d.v, d.beta, d.S0, w.chunk, impl=impl)
        torch.cuda.synchronize()
        assert pf.pf_last_launch_count() == launches, (w.name, impl, pf.pf_last_launch_count())
        O_ref, Sf_ref = util.run_oracle(inp)
        assert util.max_rel(O.cpu().numpy(), O_ref) <= util.TOL_BF16 and util.max_rel(Sf.cpu().numpy(), Sf_ref) <= util.TOL_BF16
