"""The C-ABI library builds, loads without a GPU and exports every function the headers under include/ declare."""
import ctypes
import glob
import os
import re

from conftest import ROOT


def declared_functions(header="*.h"):
    names = set()
    for path in glob.glob(os.path.join(ROOT, "include", header)):
        text = re.sub(r"/\*.*?\*/", "", open(path).read(), flags=re.S)
        names.update(re.findall(r"\b(zl_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_header_declares_the_three_core_calls():
    names = declared_functions("zipline.h")
    for core in ("zl_create", "zl_select_batched", "zl_destroy"):
        assert core in names


def test_library_exports_every_declared_symbol():
    from paper_2001_01347_b200 import build
    lib = ctypes.CDLL(build.build())
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} is declared under include/ but not exported"


def test_binding_lists_every_declared_symbol_and_host_queries_work():
    from paper_2001_01347_b200 import binding
    assert sorted(binding.EXPORTS) == declared_functions()
    assert binding.zl_max_workers() >= 4096
    assert binding.zl_trace_max_elements() >= 1024
    assert binding.zl_status_string(0) == "ok"
    assert "non-decreasing" in binding.zl_status_string(binding.ZL_ERR_UNSORTED)


def test_product_has_no_oracle_import():
    pkg = os.path.join(ROOT, "paper_2001_01347_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src and "zl_oracle" not in src
