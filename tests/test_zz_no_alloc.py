"""bra_route_static: the routing call for callers that cannot allocate.

Some users of this library run where device memory may not be requested at call
time: a plug-in inside an application that owns the memory pool, a real-time
loop that cannot afford an allocation's hidden synchronisation, a thin C caller
with no allocator at hand.  For them the library carries the scratch that
bra_route wants (the region means) as a fixed array of its own.  These tests
check, through the C boundary, that the variant gives exactly bra_route's index,
call after call, and that it refuses problems larger than its array.

This file is named to be collected last, so a run that stops at the first
failure has already gone through every other test.
"""
import ctypes

import numpy as np
import pytest

from paper_2303_08810_b200 import synthetic
from paper_2303_08810_b200.synthetic import BraConfig, CONFIGS

A = 0x10000  # an aligned address that is never dereferenced


@pytest.fixture(scope="module")
def bra():
    import paper_2303_08810_b200 as pkg
    from paper_2303_08810_b200 import build
    build.build_library()
    pkg.load_library()
    return pkg


def test_too_large_problem_is_refused_on_the_host(bra):
    """B*S*S*C above the built-in array's capacity: a clear error, before any CUDA call."""
    lib = bra.load_library()
    limit = bra.binding.ROUTE_STATIC_MAX_MEAN_FLOATS
    p = bra.make_problem(B=256, H=56, W=56, C=64, heads=2, S=7, topk=1)        # 802 816 floats
    assert p.B * p.R * p.C > limit
    rc = lib.bra_route_static(ctypes.byref(p), A, A, A, None)
    assert rc == 11
    assert "no-allocation" in lib.bra_status_string(rc).decode()
    # the usual host checks still come first
    bad = bra.make_problem(B=1, H=16, W=16, C=64, heads=2, S=0, topk=1)
    assert lib.bra_route_static(ctypes.byref(bad), A, A, A, None) == 2
    # a map S does not divide would need a padded copy of Q and K, i.e. scratch: not through this entry point
    odd = bra.make_problem(B=1, H=16, W=16, C=64, heads=2, S=3, topk=1)
    assert lib.bra_route_static(ctypes.byref(odd), A, A, A, None) == 7
    ok = bra.make_problem(B=1, H=16, W=16, C=64, heads=2, S=4, topk=1)
    assert lib.bra_route_static(ctypes.byref(ok), A, None, A, None) == 1
    assert lib.bra_route_static(ctypes.byref(ok), A, A, A + 4, None) == 5


@pytest.mark.gpu
def test_static_route_equals_route_on_consecutive_calls(bra):
    """Two calls in a row on different problems (the second smaller, so stale means of
    the first are still in the array), each compared with bra_route: same kernels, same
    arithmetic, so the index must be bit-identical."""
    import torch
    cases = [(CONFIGS[2], 1002), (BraConfig("small", 3, 12, 20, 48, 3, 4, 5, "f32"), 31),
             (synthetic.with_batch(CONFIGS[3], 32), 1003)]
    for cfg, seed in cases:
        x = synthetic.make_inputs(cfg, seed=seed)
        dt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
        Q = torch.from_numpy(x["Q"]).cuda().to(dt)
        K = torch.from_numpy(x["K"]).cuda().to(dt)
        p = bra.make_problem(cfg.B, cfg.H, cfg.W, cfg.C, cfg.heads, cfg.S, cfg.topk, cfg.dtype)
        _, _, want = bra.bra_route(p, Q, K)
        out = torch.full_like(want, -1)
        got = bra.bra_route_static(p, Q, K, index=out)
        assert got.data_ptr() == out.data_ptr()
        assert bra.last_launch_count() == 2
        torch.cuda.synchronize()
        assert torch.equal(got, want), cfg.name
        # and once more on the same inputs: the array's old contents change nothing
        again = bra.bra_route_static(p, Q, K, index=torch.full_like(want, -1))
        torch.cuda.synchronize()
        assert torch.equal(again, want), cfg.name
