"""The C-ABI library loads and exports every entry point that include/nolo.h
declares; argument validation that needs no device works.  No GPU needed."""

import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2506_10911_b200 import build
    build.build()
    from paper_2506_10911_b200 import binding
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "nolo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(nolo_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_four_core_calls():
    names = declared_functions()
    for core in ("nolo_create", "nolo_outer_step", "nolo_route", "nolo_destroy"):
        assert core in names
    assert len(names) >= 10


def test_every_declared_symbol_is_exported_and_bound(lib):
    raw = ctypes.CDLL(lib.LIB_PATH)
    for name in declared_functions():
        assert hasattr(raw, name), f"{name} not exported by libnolo.so"
        assert name in lib.SIGNATURES, f"{name} has no ctypes signature"
        assert callable(getattr(lib, name)), f"{name} has no Python wrapper"
    assert sorted(lib.SIGNATURES) == declared_functions()


def test_strerror_and_version(lib):
    assert lib.nolo_version() >= 100
    assert lib.nolo_strerror(0) == "ok"
    texts = {lib.nolo_strerror(c) for c in (-1, -2, -3, -4, -5)}
    assert len(texts) == 5 and "unknown status" not in texts
    assert lib.nolo_strerror(-99) == "unknown status"
    assert lib.nolo_last_error(None) == ""


@pytest.mark.parametrize("args", [
    (0, 1, 8, 1), (4, 0, 8, 1), (4, 3, 8, 1), (4, 8, 8, 1), (4, 2, 0, 1), (4, 2, 8, 0),
    (4097, 1, 8, 1),
])
def test_create_rejects_bad_sizes_before_touching_the_device(lib, args):
    W, n, P, stages = args
    with pytest.raises(lib.NoloError) as e:
        lib.nolo_create(W, n, P, stages, 0.5, 0.7, 0.5)
    assert e.value.status == lib.NOLO_EINVAL


def test_create_rejects_non_finite_hyperparameters(lib):
    for bad in (float("nan"), float("inf")):
        for pos in range(3):
            hp = [0.5, 0.7, 0.5]
            hp[pos] = bad
            with pytest.raises(lib.NoloError) as e:
                lib.nolo_create(4, 2, 8, 1, *hp)
            assert e.value.status == lib.NOLO_EINVAL


def test_null_handle_is_an_error_not_a_crash(lib):
    raw = ctypes.CDLL(lib.LIB_PATH)
    raw.nolo_outer_step.argtypes = [ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint64]
    assert raw.nolo_outer_step(None, 0, 0) == lib.NOLO_EINVAL
    raw.nolo_destroy.argtypes = [ctypes.c_void_p]
    assert raw.nolo_destroy(None) == lib.NOLO_OK
    raw.nolo_create.argtypes = lib.SIGNATURES["nolo_create"]
    assert raw.nolo_create(4, 2, 8, 1, 0.5, 0.7, 0.5, None) == lib.NOLO_EINVAL


def test_missing_library_fails_loudly(tmp_path):
    """There is no fallback path: without the shared library the binding cannot be imported."""
    import glob
    import shutil
    import subprocess
    import sys
    pkg = tmp_path / "paper_2506_10911_b200"          # a copy of the package without its built library
    pkg.mkdir()
    for f in glob.glob(os.path.join(ROOT, "paper_2506_10911_b200", "*.py")):
        shutil.copy(f, pkg)
    env = {k: v for k, v in os.environ.items() if k != "PYTHONPATH"}
    res = subprocess.run([sys.executable, "-c", "from paper_2506_10911_b200 import binding"], cwd=tmp_path, env=env,
                         capture_output=True, text=True)
    assert res.returncode != 0 and "ImportError" in res.stderr and "no CPU or PyTorch fallback" in res.stderr
