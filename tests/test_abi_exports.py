"""The C-ABI library loads without a GPU and exports every function mono.h declares."""
import ctypes
import os
import re

import pytest

from paper_2209_07663_b200 import binding as mb
from paper_2209_07663_b200 import build as mbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "mono.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mono_[a-z_]+)\s*\(", text)))


def test_header_declares_the_four_named_calls():
    names = declared_functions()
    for n in ("mono_table_create", "mono_lookup_pool", "mono_apply_grads", "mono_expire"):
        assert n in names


def test_library_builds_and_exports_every_declared_symbol():
    path = mbuild.build()
    lib = ctypes.CDLL(path)
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} declared in mono.h but not exported"
    assert sorted(mb.EXPORTS) == declared_functions()


def test_binding_has_a_function_per_abi_call_and_no_cpu_fallback():
    for name in declared_functions():
        if name in ("mono_last_cuda_error", "mono_error_string"):
            continue
        assert callable(getattr(mb, name)), name
    assert mb.error_string(mb.MONO_ERR_TIME) == "MONO_ERR_TIME"
    import torch
    if not torch.cuda.is_available():
        # without a device the product path refuses to run instead of falling back
        with pytest.raises(mb.MonoError):
            mb.mono_table_create(1024, 16, 2, 10)
        with pytest.raises(RuntimeError):
            mb.MonoTable(1024, 16, 2, 10)


def test_struct_layouts_match_the_header():
    # sizes implied by the field lists in mono.h (natural alignment)
    assert ctypes.sizeof(mb.mono_opt) == 72
    assert ctypes.sizeof(mb.mono_status_t) == 144
    assert ctypes.sizeof(mb.mono_audit_t) == 72


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(RuntimeError):
        mb.load_library(str(tmp_path / "nope.so"))
