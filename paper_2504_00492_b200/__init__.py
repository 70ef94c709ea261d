"""B200-native chunkwise-parallel forward pass of the rank-r generalized delta rule.

The product is the C-ABI library ``libpf.so`` (CUDA kernels for sm_100a, declared in
``include/pf.h``); ``binding`` marshals torch tensors into it.  Build the library with
``python -m paper_2504_00492_b200.build``.
"""
from .binding import (  # noqa: F401
    PF_DTYPE_BF16, PF_DTYPE_F32, PF_IMPL_AUTO, PF_IMPL_SIMT, PF_IMPL_TC, PfError, lib,
    pf_deltanet_fwd, pf_deltanet_fwd_ex, pf_deltanet_fwd_f32, pf_deltanet_fwd_f32_static, pf_static_scratch_bytes, pf_last_error_string, pf_last_launch_count,
    pf_select_impl, pf_select_chunk, pf_status_string, pf_version, pf_workspace_bytes, pf_workspace_bytes_ex,
    pf_read_status, pf_last_wait_code, pf_wait_selftest, pf_static_scratch_need,
)
