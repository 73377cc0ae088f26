"""The C-ABI library builds, loads, and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "invconv.h")


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b([a-z_][a-z0-9_]*)\s*\([^;{]*\)\s*;", text)
    return sorted(set(names))


@pytest.fixture(scope="module")
def library():
    from paper_2410_14634_b200 import build
    path = build.build()
    return ctypes.CDLL(path)


def test_header_declares_the_four_hot_path_calls():
    names = declared_functions()
    for required in ("invconv_forward", "invconv_backward", "masked_conv_forward", "invconv_logdet"):
        assert required in names


def test_library_exports_every_declared_symbol(library):
    names = declared_functions()
    assert len(names) >= 12
    for name in names:
        assert hasattr(library, name), f"{name} declared in invconv.h but not exported"


def test_status_strings_and_version(library):
    library.invconv_status_string.restype = ctypes.c_char_p
    seen = {library.invconv_status_string(i) for i in range(6)}
    assert len(seen) == 6 and b"ok" in seen
    assert library.invconv_version() >= 100


def test_argument_checks_need_no_device(library):
    # shape validation happens before any CUDA call
    library.invconv_workspace_bytes.restype = ctypes.c_size_t
    assert library.invconv_forward(None, None, None, 1, 1, 4, 4, 3, None) == 1       # NULL pointers
    assert library.invconv_forward(None, None, None, 1, 1, 4, 4, 12, None) == 2      # k beyond the limit
    assert library.invconv_forward(None, None, None, 1, 200, 4, 4, 3, None) == 2     # C beyond the limit
    assert library.invconv_forward(None, None, None, 1, 1, 0, 4, 3, None) == 1       # empty image
    assert library.invconv_logdet(None, None, 1, 4, 4, 3, None) == 1
    assert library.invconv_set_path(99) == -1


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    from paper_2410_14634_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError):
        binding.lib()


def test_dispatch_and_workspace_planning_need_no_device(library):
    """Host logic only: the family AUTO picks and the scratch a call needs, for the ten benchmark shapes and a
    few edge shapes (planning falls back to 148 SMs when no device is present)."""
    from paper_2410_14634_b200 import workloads
    library.invconv_workspace_bytes.restype = ctypes.c_size_t
    library.invconv_workspace_bytes.argtypes = [ctypes.c_int] * 5
    library.invconv_path_for.argtypes = [ctypes.c_int] * 5
    GENERIC, WARP, TEAM, TENSOR = 1, 2, 3, 4
    want = {"pr1": WARP, "mnist": WARP, "cifar": WARP, "large64": WARP, "large256": WARP,
            "cifar_sq": TEAM, "wide48_k3": TENSOR, "wide48_k5": TENSOR, "wide96_k3": TEAM, "wide96_k5": TEAM}
    for s in workloads.SHAPES:
        assert library.invconv_path_for(s.B, s.C, s.H, s.W, s.k) == want[s.name], s.name
        need = library.invconv_workspace_bytes(s.B, s.C, s.H, s.W, s.k)
        na = 4 * s.C * s.C * s.k * s.k
        assert need >= 256 + na, s.name                      # control block + at least one set of partial sums
        assert need < (64 << 20), s.name
    # shapes outside the specialised families fall to the generic kernels, which need no scratch
    assert library.invconv_path_for(1, 3, 8, 8, 7) in (TEAM, GENERIC)
    assert library.invconv_path_for(1, 128, 64, 64, 3) == GENERIC
    assert library.invconv_workspace_bytes(1, 128, 64, 64, 3) == 0
    # invalid shapes report no scratch instead of failing
    assert library.invconv_workspace_bytes(1, 1, 0, 4, 3) == 0
    assert library.invconv_workspace_bytes(1, 1, 4, 4, 12) == 0
    # the scratch of the no-allocation entry point covers every few-channel benchmark shape
    for s in workloads.SHAPES:
        if want[s.name] == WARP:
            assert library.invconv_workspace_bytes(s.B, s.C, s.H, s.W, s.k) <= (1 << 20), s.name

