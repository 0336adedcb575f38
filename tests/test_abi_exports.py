"""The C-ABI library builds, loads without a GPU, and exports what include/spec_attn.h declares."""
import ctypes
import os
import re

from paper_2607_27735_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "spec_attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(spec_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    build.build()
    lib = ctypes.CDLL(binding.LIB_PATH)
    names = declared_functions()
    assert "spec_verify_attn" in names and "spec_select_recall" in names
    assert "spec_sparse_draft_attn" in names
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTS) == names


def test_host_only_calls_work_without_a_gpu():
    lib = binding.load()
    assert lib.spec_version() >= 100
    assert binding.strerror(-3) == "workspace too small"
    assert binding.strerror(0) == "ok"
    assert lib.spec_set_verify_impl(99) == -1
