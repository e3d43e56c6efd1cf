"""Monarch matrix multiply for NVIDIA B200: Python binding over the C-ABI library libmonarch.

The functions here marshal arguments only; every step of the computation runs in the CUDA
kernels of ``libmonarch.so`` (built in-tree by ``paper_2204_00595_b200.build``).  There is no
CPU fallback: a missing library or device raises.
"""
from .binding import (  # noqa: F401
    BF16, F32, IMPL_AUTO, IMPL_FUSED, IMPL_STAGED, OP_BWD, OP_BWD_DW, OP_BWD_DX, OP_FWD, OP_CPLX, OP_MLP_BWD,
    OP_MLP_FWD,
    HostContext, MonarchError, Workspace, lib, monarch_bwd, monarch_bwd_dw, monarch_bwd_dx, monarch_fwd, monarch_fwd_noalloc, monarch_impl_name,
    monarch_last_device_status, monarch_launch_count, monarch_cplx_fwd, monarch_dense, monarch_mlp_bwd, monarch_mlp_fwd, monarch_project, monarch_rect_bwd, monarch_rect_bwd_workspace_bytes,
    monarch_rect_fwd, monarch_rect_workspace_bytes,
    monarch_rectw_fwd, monarch_rectw_bwd, monarch_rectw_workspace_bytes, monarch_rectw_bwd_workspace_bytes,
    monarch_set_impl, monarch_set_deterministic, monarch_debug_set_wait_limit, monarch_debug_skip_load,
    monarch_status_string, monarch_workspace_bytes, monarch_workspace_init,
)
