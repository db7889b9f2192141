"""The C-ABI libraries load without a GPU and export every function their headers declare."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared(header):
    src = open(os.path.join(ROOT, "include", header)).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(frog_[a-z_0-9]+)\s*\(", src)))


def test_search_library_exports_every_declared_symbol(libs):
    from paper_2608_16491_b200 import build
    lib = ctypes.CDLL(build.LIB_SEARCH)
    names = sorted(set(_declared("frog.h")) | {"frog_index_build_gpu"})
    assert "frog_index_build_gpu" in _declared("frog_build_gpu.h")
    assert {"frog_index_load", "frog_index_free", "frog_index_info", "frog_search", "frog_search_ex",
            "frog_exact_search", "frog_search_host", "frog_strerror"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_builder_library_exports_every_declared_symbol(libs):
    from paper_2608_16491_b200 import build
    lib = ctypes.CDLL(build.LIB_BUILD)
    names = _declared("frog_build.h")
    assert "frog_index_build" in names
    for n in names:
        assert hasattr(lib, n), n


def test_error_strings_and_argument_checks_need_no_gpu(libs):
    assert libs.strerror(0) == "ok"
    assert "argument" in libs.strerror(1)
    import paper_2608_16491_b200 as frog
    h = ctypes.c_void_p()
    assert frog._lib.frog_index_load(None, 0, ctypes.byref(h)) == 1
    assert frog._lib.frog_index_load(b"/nonexistent/file.idx", 0, ctypes.byref(h)) == 2
    assert frog._lib.frog_search(None, None, None, None, 0, 1, 1, None, None, None) == 1


def test_loader_rejects_malformed_files(libs, tmp_path):
    import paper_2608_16491_b200 as frog
    p = tmp_path / "bad.idx"
    p.write_bytes(b"NOTANIDX" + b"\0" * 300)
    h = ctypes.c_void_p()
    assert frog._lib.frog_index_load(str(p).encode(), 0, ctypes.byref(h)) == 3
    p.write_bytes(b"FROG")
    assert frog._lib.frog_index_load(str(p).encode(), 0, ctypes.byref(h)) == 3


def test_missing_library_fails_loudly_at_first_use(tmp_path):
    """The package imports without the compiled search library (its build step lives in it), but
    every call into the search path then raises: there is no fallback implementation."""
    import subprocess
    import sys
    code = (
        "import os, sys\n"
        "sys.path.insert(0, %r)\n"
        "os.environ['FROG_LIBFROG'] = %r\n"
        "import paper_2608_16491_b200 as frog\n"
        "from paper_2608_16491_b200 import build\n"
        "try:\n"
        "    frog.strerror(0)\n"
        "except ImportError as e:\n"
        "    print('LOUD', 'no fallback' in str(e))\n"
        "else:\n"
        "    print('SILENT')\n"
    ) % (os.path.dirname(os.path.dirname(os.path.abspath(__file__))), str(tmp_path / "nowhere" / "libfrog.so"))
    out = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0, out.stderr
    assert out.stdout.strip() == "LOUD True"
