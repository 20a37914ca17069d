"""The C-ABI shared library loads and exports every function include/rcp.h declares (no GPU needed)."""
import ctypes
import os
import re
import shutil

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "rcp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rcp_[a-z0-9_]+)\s*\(", text)))


@pytest.fixture(scope="module")
def libpath():
    from paper_2502_15779_b200 import build
    if not os.path.exists(build.LIB) and shutil.which("nvcc") is None and not os.path.exists("/usr/local/cuda/bin/nvcc"):
        pytest.skip("no nvcc and no prebuilt library")
    return build.build()


def test_header_declares_the_three_hot_path_calls():
    names = _declared_functions()
    for required in ("rcp_pack_weights", "rcp_quantize_act", "rcp_gemv_w2a4"):
        assert required in names


def test_library_exports_every_declared_symbol(libpath):
    L = ctypes.CDLL(libpath)
    for name in _declared_functions():
        assert hasattr(L, name), name


def test_status_strings_and_workspace_query_run_without_gpu(libpath):
    L = ctypes.CDLL(libpath)
    L.rcp_status_str.restype = ctypes.c_char_p
    for code in range(0, -9, -1):
        assert L.rcp_status_str(code) not in (None, b"")
    L.rcp_gemv_workspace_bytes.restype = ctypes.c_size_t
    assert L.rcp_gemv_workspace_bytes(1, 0, 4096) == 0      # bad shape -> 0
    assert L.rcp_gemv_workspace_bytes(1, 4096, 100) == 0    # K % 64 != 0 -> 0
    assert L.rcp_gemv_workspace_bytes(1, 4096, 4096) % 16 == 0


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    from paper_2502_15779_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        binding.lib()
