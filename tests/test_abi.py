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
