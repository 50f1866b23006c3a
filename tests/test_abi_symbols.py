"""The shared library loads without a GPU and exports every function that include/siso.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "siso.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(siso_[a-z_0-9]+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_entry_point():
    from paper_2508_18736_b200 import build
    lib_path = build.build()                      # compiles only if sources are newer than the library
    lib = ctypes.CDLL(lib_path)
    names = declared_functions()
    assert len(names) >= 19 and "siso_lookup" in names and "siso_cache_create" in names
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in siso.h but not exported"
    lib.siso_status_string.restype = ctypes.c_char_p
    assert lib.siso_status_string(0) == b"ok" and lib.siso_status_string(5) == b"merge candidate buffer overflow"


def test_binding_lists_the_same_entry_points_and_refuses_to_run_without_a_gpu():
    import pytest
    import torch

    import paper_2508_18736_b200 as siso
    assert sorted(siso.binding.EXPORTS) == declared_functions()
    if not torch.cuda.is_available():
        with pytest.raises(RuntimeError):
            siso.SisoCache(16, 8)                 # no CPU fallback
