"""The C-ABI library loads without a GPU and exports every function include/tarflow.h declares."""
import ctypes
import os
import re

import __graft_entry__ as entry

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "tarflow.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tf_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    entry.build()
    lib = ctypes.CDLL(entry.LIB)
    names = declared_functions()
    assert {"tf_load", "tf_free", "tf_forward", "tf_inverse_sequential", "tf_inverse_jacobi",
            "tf_last_error"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in tarflow.h but not exported"


def test_binding_covers_every_declared_symbol():
    from paper_2505_24791_b200 import binding
    for n in declared_functions():
        assert hasattr(binding, n), f"binding lacks {n}"


def test_last_error_is_empty_string_initially_and_null_model_is_rejected():
    from paper_2505_24791_b200 import binding
    lib = binding.lib()
    lib.tf_free(None)                                  # no-op by contract
    assert lib.tf_launch_count(None) == 0
    rc = lib.tf_inverse_sequential(None, None, None, 1, None, None)
    assert rc == binding.TF_EINVAL and b"NULL" in lib.tf_last_error()
