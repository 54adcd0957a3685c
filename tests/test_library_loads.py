"""CPU-side checks of the boundary: the library builds/loads and exports what include/sar.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2111_06483_b200 import build
    path = build.build()
    return ctypes.CDLL(path)


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "sar.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sar_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_entry_point_is_exported(lib):
    names = _declared_functions()
    assert len(names) >= 18
    for name in names:
        assert hasattr(lib, name), f"{name} declared in sar.h but not exported"


def test_binding_lists_the_same_entry_points():
    from paper_2111_06483_b200 import binding
    assert sorted(binding.EXPORTS) == _declared_functions()
    for name in binding.EXPORTS:
        assert hasattr(binding, name) or name == "sar_status_string"


def test_host_only_calls(lib):
    lib.sar_status_string.restype = ctypes.c_char_p
    assert lib.sar_status_string(0) == b"ok"
    assert b"invalid" in lib.sar_status_string(-1)
    assert lib.sar_built_for_sm() == 100
    from paper_2111_06483_b200 import binding
    assert binding.sar_partition_bounds(10, 3) == [0, 3, 6, 10]
    assert binding.sar_partition_bounds(20_000_000, 16)[5] == 5 * 20_000_000 // 16
    # argument errors are caught on the host, before anything touches a device
    assert lib.sar_partition_bounds(ctypes.c_int64(5), ctypes.c_int32(0), None) == -1
    assert lib.sar_gat_fwd(None, None, None, None, 1, 1, 0, ctypes.c_float(0.2), 3, None, None, None, None, None,
                           ctypes.c_size_t(0), None) == -1


def test_oracle_and_cuda_package_do_not_import_each_other():
    import oracle
    src = open(oracle.__file__).read() + open(os.path.join(os.path.dirname(oracle.__file__), "sar_oracle.c")).read()
    assert "paper_2111_06483_b200" not in src and "libsar.so" not in src and "sar.h" not in src
    pkg = os.path.join(ROOT, "paper_2111_06483_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text and "sar_oracle" not in text, f
