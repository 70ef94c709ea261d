"""tcgen05 building blocks: one GEMM in every operand-major combination against a host matmul."""
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("variant", list(range(8)) + [8, 9, 16, 18, 24, 27, 10, 17, 32, 34, 36, 48, 50])
@pytest.mark.parametrize("N", [32, 64, 128, 192, 256])
def test_tcgen05_gemm_variants(variant, N):
    from paper_2504_00492_b200 import binding
    g = torch.Generator().manual_seed(100 * variant + N)
    a_mn, b_mn, neg = bool(variant & 1), bool(variant & 2), bool(variant & 4)   # bits 3, 4: unswizzled staging
    A = (torch.randn(128, 128, generator=g) * 0.1).half()        # [m][k] or [k][m]
    Bm = (torch.randn(N, 128, generator=g) * 0.1).half()         # logical B[n][k]
    A_log = A.t() if a_mn else A                                  # logical A[m][k]
    B_dev = Bm.t().contiguous() if b_mn else Bm
    ref = (A_log.double() @ Bm.double().t()) * (-1.0 if neg else 1.0)
    Ad, Bd = A.cuda(), B_dev.cuda()
    D = torch.full((128, N), float("nan"), device="cuda")
    rc = binding.lib().pf_tc_selftest(variant, Ad.data_ptr(), Bd.data_ptr(), D.data_ptr(), N,
                                      torch.cuda.current_stream().cuda_stream)
    assert rc == 0, binding.pf_status_string(rc) + " " + binding.pf_last_error_string()
    err = (D.cpu().double() - ref).abs().max().item()
    assert err < 1e-5, f"variant {variant} N {N}: max abs err {err}"
