"""The C boundary without a GPU: the library loads, exports every symbol the
header declares, and rejects bad arguments on the host before touching CUDA."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2303_08810_b200 import build, binding
    build.build_library()
    return binding.load_library()


def declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(bra_[a-z_]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol(lib):
    names = declared_symbols()
    assert {"bra_route", "bra_attend", "bra_forward", "bra_backward", "bra_workspace_bytes",
            "bra_device_status", "bra_status_string", "bra_version"} <= names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/ but not exported"


def test_version_and_status_strings(lib):
    assert lib.bra_version() >= 100
    seen = set()
    for code in range(0, 12):                     # BRA_OK .. BRA_ERR_STATIC_LIMIT
        s = lib.bra_status_string(code).decode()
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 12
    assert lib.bra_status_string(99).decode() == "unknown status"


def problem(**kw):
    from paper_2303_08810_b200 import binding
    base = dict(B=2, H=16, W=16, C=64, heads=2, S=4, topk=2, dtype="bf16")
    base.update(kw)
    return binding.make_problem(**base)


def test_workspace_bytes(lib):
    from paper_2303_08810_b200 import binding
    p = problem()
    n = binding.workspace_bytes(p)
    assert n > 0 and n % 256 == 0
    # holds at least the two mean tensors and the index
    assert n >= 2 * 4 * p.B * 16 * p.C + 4 * p.B * p.heads * 16 * p.topk
    assert binding.workspace_bytes(problem(B=4)) > n
    assert binding.workspace_bytes(problem(S=0)) == 0          # invalid problem
    assert binding.workspace_bytes(problem(S=3)) > n           # S does not divide the map: room for the padded copies


A = 0x10000  # a fake, aligned, never dereferenced device address


@pytest.mark.parametrize("kw,code", [
    (dict(B=0), 2), (dict(H=-1), 2), (dict(S=0), 2), (dict(heads=3), 2),
    (dict(topk=0), 3), (dict(topk=17), 3),
])
def test_route_rejects_bad_problems(lib, kw, code):
    from paper_2303_08810_b200 import binding
    p = problem(**kw)
    rc = lib.bra_route(ctypes.byref(p), A, A, A, A, A, A, 1 << 30, None)
    assert rc == code


def test_bad_dtype_lce_impl(lib):
    p = problem()
    p.dtype = 7
    assert lib.bra_route(ctypes.byref(p), A, A, A, A, A, A, 1 << 30, None) == 4
    p = problem()
    p.lce_ksize = 3
    assert lib.bra_attend(ctypes.byref(p), A, A, A, A, A, None, A, None, A, 1 << 30, None) == 7
    p = problem()
    p.impl = 9
    assert lib.bra_attend(ctypes.byref(p), A, A, A, A, A, None, A, None, A, 1 << 30, None) == 7
    p = problem(C=24, heads=2)           # head dim 12: no 16-byte channel vectors
    assert lib.bra_attend(ctypes.byref(p), A, A, A, A, A, None, A, None, A, 1 << 30, None) == 7


def test_null_alignment_workspace_checks(lib):
    from paper_2303_08810_b200 import binding
    p = problem()
    need = binding.workspace_bytes(p)
    ref = ctypes.byref(p)
    assert lib.bra_route(None, A, A, A, A, A, A, need, None) == 1
    assert lib.bra_route(ref, None, A, A, A, A, A, need, None) == 1
    assert lib.bra_route(ref, A, A, A, A, None, A, need, None) == 1            # index is required
    assert lib.bra_route(ref, A, A, A, A, A, None, need, None) == 1            # ws is required
    assert lib.bra_route(ref, A + 8, A, A, A, A, A, need, None) == 5
    assert lib.bra_route(ref, A, A, A, A, A, A + 16, need, None) == 5          # ws wants 256
    assert lib.bra_route(ref, A, A, A, A, A, A, need - 1, None) == 6
    # attend: LCE weights required unless LCE is off; O required
    assert lib.bra_attend(ref, A, A, A, A, None, None, A, None, A, need, None) == 1
    assert lib.bra_attend(ref, A, A, A, A, A, None, None, None, A, need, None) == 1
    assert lib.bra_attend(ref, A, A, A + 2, A, A, None, A, None, A, need, None) == 5
    assert lib.bra_forward(ref, A, A, None, A, None, A, None, None, A, need, None) == 1
    assert lib.bra_forward(ref, A, A, A, A, None, A, None, None, A, 16, None) == 6
    # backward: lse and dO required
    args = [A] * 12
    bad = list(args); bad[5] = None                                           # lse
    assert lib.bra_backward(ref, *bad, A, need, None) == 1
    bad = list(args); bad[6] = None                                           # dO
    assert lib.bra_backward(ref, *bad, A, need, None) == 1
    assert lib.bra_device_status(None, None) == 1


def test_workspace_init_checks_its_arguments(lib):
    from paper_2303_08810_b200 import binding
    p = problem()
    need = binding.workspace_bytes(p)
    assert lib.bra_workspace_init(ctypes.byref(p), None, need, None) == 1
    assert lib.bra_workspace_init(ctypes.byref(p), A + 8, need, None) == 5
    assert lib.bra_workspace_init(ctypes.byref(p), A, need - 1, None) == 6
    bad = problem(S=0)
    assert lib.bra_workspace_init(ctypes.byref(bad), A, need, None) == 2


def test_injection_switch_is_validated(lib):
    p = problem()
    p.inject = 5
    assert lib.bra_attend(ctypes.byref(p), A, A, A, A, A, None, A, None, A, 1 << 30, None) == 7


def test_unsupported_impl_for_problem(lib):
    from paper_2303_08810_b200 import binding
    p = problem(dtype="f32", impl=binding.IMPL_MMA)      # tensor-core paths are bf16 only
    need = binding.workspace_bytes(p)
    assert lib.bra_attend(ctypes.byref(p), A, A, A, A, A, None, A, None, A, need, None) == 7


def test_binding_fails_loudly_without_gpu():
    import torch
    from paper_2303_08810_b200 import binding
    if torch.cuda.is_available():
        pytest.skip("has a GPU")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.workspace(problem())
