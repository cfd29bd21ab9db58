"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_2501_19309_b200 import build as B
from paper_2501_19309_b200 import jd

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    src = open(os.path.join(ROOT, "include", "jd.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    names = re.findall(r"\b(jd_[a-z_0-9]+)\s*\(", src)
    return sorted(set(names))


def test_library_builds_and_exports_every_declared_symbol():
    path = B.build()
    assert os.path.exists(path) and path == jd.library_path()
    lib = ctypes.CDLL(path)
    names = declared_functions()
    assert set(jd.EXPORTS) <= set(names)
    assert len(names) >= 11
    for n in names:
        assert hasattr(lib, n), n


def test_calls_that_need_no_device():
    assert jd.jd_version() >= 100
    assert jd.jd_status_string(jd.JD_OK) == "ok"
    assert "wait" in jd.jd_status_string(jd.JD_ERR_TIMEOUT)
    cfg = jd.jd_config_t(4, 16, 8192, 128256, jd.JD_DTYPE_BF16, 0)
    n = jd.jd_workspace_bytes(cfg)
    assert 1 << 20 < n < 1 << 30
    bad = jd.jd_config_t(0, 16, 8192, 128256, jd.JD_DTYPE_BF16, 0)
    assert jd.jd_workspace_bytes(bad) == 0
    # the normal build records no phase stamps and says so; bad arguments are refused first
    buf = (ctypes.c_uint64 * 4096)()
    assert jd.jd_debug_phase_stamps(ctypes.addressof(buf), 4096) == jd.JD_ERR_UNSUPPORTED
    assert jd.jd_debug_phase_stamps(ctypes.addressof(buf), 100) == jd.JD_ERR_INVALID_ARG
    assert jd.jd_debug_phase_stamps(0, 4096) == jd.JD_ERR_INVALID_ARG


def test_struct_layout_matches_header_order():
    src = open(os.path.join(ROOT, "include", "jd.h")).read()
    body = src[src.index("typedef struct {\n  int32_t B;"):src.index("} jd_verify_args_t;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = re.findall(r"([A-Za-z_0-9]+)\s*;", body)
    assert fields == [f[0] for f in jd.jd_verify_args_t._fields_]


def test_header_and_c_caller_compile_as_plain_c():
    """include/jd.h is a C header: the C99 caller under tests/c_abi builds with gcc, warnings as errors."""
    import shutil
    import subprocess
    import tempfile
    cuda_inc = "/usr/local/cuda/include"
    if shutil.which("gcc") is None or not os.path.exists(os.path.join(cuda_inc, "cuda_runtime_api.h")):
        import pytest
        pytest.skip("gcc or the CUDA runtime header is not installed")
    with tempfile.TemporaryDirectory() as tmp:
        cmd = ["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-I", os.path.join(ROOT, "include"), "-I", cuda_inc,
               "-c", os.path.join(ROOT, "tests", "c_abi", "jd_c_caller.c"), "-o", os.path.join(tmp, "caller.o")]
        proc = subprocess.run(cmd, capture_output=True, text=True)
        assert proc.returncode == 0, proc.stderr
