"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_2509_15038_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "curdkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(curdkv_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib_path = build.build_library()
    lib = ctypes.CDLL(str(lib_path))
    names = declared_functions()
    assert len(names) >= 7
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in curdkv.h but not exported"
    assert set(binding.EXPORTS) == set(names)


def test_host_only_calls_work_without_a_device():
    lib = binding.load()
    assert binding.status_string(0) == "ok"
    assert "workspace" in binding.status_string(3)
    desc = binding.Desc(4, 8, 32, 1000, 128, 32, 0, 0, 128, 0, 0, 128, None, 0, 1)
    # 256 status bytes + four fp32 partials per 128-row tile, rounded to 256 bytes
    assert binding.workspace_bytes(desc) == 256 + 4 * 8 * 8 * 4 * 4
    bad = binding.Desc(4, 8, 12, 1000, 128, 32, 0, 0, 128, 0, 0, 128, None, 0, 1)
    assert binding.workspace_bytes(bad) == 0
    assert lib.curdkv_score(None, None, None, 0, None, None, None, None, 0, None) == 1
