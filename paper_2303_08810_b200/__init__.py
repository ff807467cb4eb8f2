"""B200 (sm_100a) Bi-Level Routing Attention: CUDA library and its thin Python binding.

The compute runs in libbra_b200.so (hand-written CUDA behind a C boundary,
include/bra.h).  There is no CPU or PyTorch fallback: calling an op without
the built library raises.
"""
from .binding import (  # noqa: F401
    BraProblem, BraError, load_library, make_problem, workspace, workspace_bytes, workspace_init,
    bra_route, bra_route_static, bra_attend, bra_forward, bra_backward, bra_device_status,
    last_launch_count, status_string, version,
    IMPL_AUTO, IMPL_SIMT, IMPL_MMA, IMPL_TC, IMPL_IMG, IMPL_TC_FUSED,
)
