"""CPU-only checks of the C-ABI library: it builds, loads, and exports every
symbol that include/ghd.h declares; host-side validation works without a GPU."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    from paper_2505_23219_b200 import build
    return ctypes.CDLL(str(build.build()))


def declared_functions():
    text = (ROOT / "include" / "ghd.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ghd_[a-z_0-9]+)\s*\(", text)))


def test_header_and_binding_agree():
    from paper_2505_23219_b200 import binding
    assert declared_functions() == sorted(binding.EXPORTS)


def test_library_exports_every_declared_symbol(lib):
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_host_side_validation_needs_no_gpu(lib):
    lib.ghd_status_str.restype = ctypes.c_char_p
    assert lib.ghd_status_str(0) == b"ok" and lib.ghd_status_str(3) == b"invalid tree"
    out = ctypes.c_void_p()
    assert lib.ghd_create(None, None, ctypes.byref(out)) == 1           # GHD_EINVAL
    assert lib.ghd_set_option(None, 0, 0) == 1
    assert lib.ghd_sync_status(None) == 1
    lib.ghd_workspace_bytes.restype = ctypes.c_size_t
    assert lib.ghd_workspace_bytes(None) == 0
    lib.ghd_destroy(None)


def test_binding_refuses_a_missing_library(tmp_path):
    from paper_2505_23219_b200 import binding
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.load_library(tmp_path / "libghd.so")
