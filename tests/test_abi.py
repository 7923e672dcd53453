"""The C-ABI library builds for sm_100a, loads, and exports every symbol include/gls.h declares.
No kernel is launched here (CPU only); compute is covered by the gpu-marked parity tests."""
import ctypes
import os
import re
import shutil

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    import paper_2506_05632_b200 as pkg

    if shutil.which("nvcc") is None and not os.path.exists(pkg.lib_path()):
        pytest.skip("no nvcc and no prebuilt libgls.so")
    if shutil.which("nvcc") is not None:
        pkg.build()
    return ctypes.CDLL(pkg.lib_path())


def _declared():
    text = open(os.path.join(ROOT, "include", "gls.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gls_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_entry_points():
    names = _declared()
    for want in ("gls_draft_sample", "gls_target_sample_verify", "gls_compress_select",
                 "gls_workspace_bytes", "gls_status_string", "gls_version"):
        assert want in names


def test_every_declared_symbol_is_exported(lib):
    for name in _declared():
        assert hasattr(lib, name), "libgls.so does not export %s" % name


def test_host_only_calls(lib):
    lib.gls_version.restype = ctypes.c_int
    assert lib.gls_version() >= 100
    lib.gls_status_string.restype = ctypes.c_char_p
    seen = set()
    for code in range(0, 7):
        s = lib.gls_status_string(code)
        assert s and len(s) > 3
        seen.add(s)
    assert len(seen) >= 6
    lib.gls_workspace_bytes.restype = ctypes.c_size_t
    lib.gls_workspace_bytes.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int64]
    small = lib.gls_workspace_bytes(8, 4, 5, 32000)
    big = lib.gls_workspace_bytes(256, 8, 9, 152064)
    assert 0 < small < big < (1 << 30)
    assert lib.gls_workspace_bytes(0, 4, 5, 32000) == 0      # invalid sizes
    assert lib.gls_workspace_bytes(8, 65, 5, 32000) == 0     # K > GLS_MAX_K
    assert lib.gls_workspace_bytes(8, 4, 5, 1 << 31) == 0    # V too large


def test_product_has_no_cpu_fallback():
    """The binding refuses host tensors instead of computing anything on the CPU, and the package
    never imports the oracle."""
    import torch

    import paper_2506_05632_b200 as pkg

    with pytest.raises(pkg.GlsError):
        pkg.binding._rows(torch.zeros(1, 1, 1, 8), 3)
    src_dir = os.path.join(ROOT, "paper_2506_05632_b200")
    pat = re.compile(r"^\s*(from|import)\s+oracle|gls_oracle|libgls_oracle|glso_", re.M)
    for dirpath, _, files in os.walk(src_dir):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                assert not pat.search(open(os.path.join(dirpath, f)).read()), f
