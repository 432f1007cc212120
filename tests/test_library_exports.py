"""The C-ABI library builds, loads and exports every symbol include/cod.h declares
(no compute calls: this runs without a GPU)."""
import os
import re

import __graft_entry__ as entry
from paper_2609_14717_b200 import binding


def test_library_builds_loads_and_exports_all_declared_symbols():
    entry.build()
    lib = binding.load_library()
    header = open(os.path.join(entry.ROOT, "include", "cod.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(cod_[a-z_0-9]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_error_strings_and_null_arguments_without_gpu():
    lib = binding.load_library()
    assert lib.cod_error_string(0) == b"ok"
    assert lib.cod_error_string(-1) == b"invalid argument"
    assert lib.cod_create(None, None) == -1
    assert lib.cod_destroy(None) == -1
    assert lib.cod_launch_count(None) == 0
