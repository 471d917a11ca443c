"""No-GPU checks of the C ABI: the library builds, loads, exports every declared symbol, and the
entry points that need no device behave (no compute call is made here)."""
import ctypes
import os
import re

import pytest

from paper_2503_20591_b200 import binding, build as lib_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    lib_build.build()
    return binding.load_library()


def declared_functions():
    names = []
    for hdr in ("nbos.h", "nbos_probe.h"):
        text = open(os.path.join(ROOT, "include", hdr)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b(nbos_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 13
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ but not exported"
    assert sorted(binding.EXPORTED_SYMBOLS) == names


def test_binding_constants_match_the_header():
    """Every NBOS_* constant of the binding has the value include/nbos.h defines."""
    import re
    text = open(os.path.join(ROOT, "include", "nbos.h")).read() + open(os.path.join(ROOT, "include", "nbos_probe.h")).read()
    defines = {m.group(1): m.group(2).strip() for m in re.finditer(r"#define\s+(NBOS_[A-Z0-9_]+)\s+([^/\n]+)", text)}
    enums = {m.group(1): m.group(2).strip() for m in re.finditer(r"\b(NBOS_[A-Z0-9_]+)\s*=\s*(-?\d+)", text)}
    known = {**enums, **defines}
    checked = 0
    for name in dir(binding):
        if name.startswith("NBOS_") and isinstance(getattr(binding, name), int) and name in known:
            assert getattr(binding, name) == eval(known[name].strip("()").replace("u", "")), name
            checked += 1
    assert checked >= 12
    assert binding.NBOS_MAX_HOSTS == 1 << 20 and binding.NBOS_SEQUENTIAL_MAX_HOSTS == 65536


def test_strerror(lib):
    assert binding.nbos_strerror(0) == "ok"
    for code in range(-6, 0):
        assert binding.nbos_strerror(code) not in ("ok", "unknown status")
    assert binding.nbos_strerror(-99) == "unknown status"


def test_workspace_bytes_grows_with_the_table(lib):
    a = binding.nbos_snapshot_workspace_bytes(1, 32)
    b = binding.nbos_snapshot_workspace_bytes(1, 4096)
    c = binding.nbos_snapshot_workspace_bytes(256, 1024)
    assert 0 < a < b < c
    assert b >= 4096 * 32 and c >= 256 * 1024 * 32
    assert a % 256 == 0


def test_argument_errors_need_no_device(lib):
    out = ctypes.c_size_t(0)
    d = binding.nbos_snapshot_desc(0, 32, 3, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0)
    assert lib.nbos_snapshot_workspace_bytes(ctypes.byref(d), ctypes.byref(out)) == binding.NBOS_ERR_INVALID_ARG
    assert "n_snapshots" in binding.nbos_last_error_detail()
    d = binding.nbos_snapshot_desc(1, (1 << 20) + 1, 3, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0)
    assert lib.nbos_snapshot_workspace_bytes(ctypes.byref(d), ctypes.byref(out)) == binding.NBOS_ERR_INVALID_ARG
    d = binding.nbos_snapshot_desc(1, 32, 3, 0, 64, 0, 0, 0, 0, 0, 0, 0, 0, 0)
    assert lib.nbos_snapshot_workspace_bytes(ctypes.byref(d), ctypes.byref(out)) == binding.NBOS_ERR_INVALID_ARG
    handle = ctypes.c_void_p(1)
    # NULL arrays are rejected before any CUDA call
    d = binding.nbos_snapshot_desc(1, 32, 3, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0)
    assert lib.nbos_snapshot_create(ctypes.byref(d), None, 0, None, ctypes.byref(handle)) == binding.NBOS_ERR_INVALID_ARG
    assert handle.value is None
    assert lib.nbos_snapshot_destroy(None) == binding.NBOS_OK
    assert lib.nbos_place_batch(None, None, 1, None, None, None) == binding.NBOS_ERR_INVALID_ARG


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "libnbos.so"))
    with pytest.raises(binding.NbosError, match="no CPU fallback"):
        binding.load_library()


def test_product_code_never_touches_the_checker():
    """The package and its CUDA sources must not import, link or mention the CPU checker."""
    pkg = os.path.join(ROOT, "paper_2503_20591_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f"{f} mentions the checker"
