"""LBP-WHT linear-layer backward for NVIDIA B200: Python binding of liblbp.so.

The package is a thin wrapper over the C ABI declared in include/lbp.h; see
binding.py.  The shared library is built in-tree by `build.build_library()`.
"""
from .binding import (  # noqa: F401
    LBP_BF16, LBP_F32, SEL_L1, SEL_LINF, SEL_PREFIX, EXPORTED, LIB_PATH, LbpError,
    alloc_workspace, lbp_backward, lbp_backward_fullrank, lbp_basis_matrix, lbp_expand,
    lbp_flops, lbp_poll_status, lbp_project, lbp_select_bases, lbp_status_bytes,
    lbp_status_string, lbp_workspace_bytes, lbp_launch_count, lbp_phase_count, lbp_phase_name,
    lbp_set_phase_events, lbp_backward_static, STATIC_SCRATCH_BYTES,
    lbp_select_lhe, lbp_spectrum, lbp_spectrum_workspace_bytes, lbp_backward_batch,
    lbp_test_stall_products, lbp_test_reload_env, lbp_test_tile_plan,
    lbp_backward_ex, lbp_backward_projected, lbp_workspace_bytes_ex,
)
from .autograd import LbpLinear, LbpLinearFunction  # noqa: F401,E402
