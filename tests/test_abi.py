"""The C-ABI library loads without a GPU and exports every symbol include/dropmatch.h declares,
with the binding mirroring it; host-side argument checks that need no device."""
import ctypes
import re
from pathlib import Path

import pytest

import paper_2603_03333_b200 as pk
from paper_2603_03333_b200 import binding

HEADER = Path(__file__).resolve().parent.parent / "include" / "dropmatch.h"


def _declared():
    text = re.sub(r"/\*.*?\*/", "", HEADER.read_text(), flags=re.S)
    return sorted(set(re.findall(r"\b(dm_[a-z_0-9]+|dropmatch_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    names = _declared()
    assert "dropmatch_verify" in names and "dropmatch_verify_tree" in names and len(names) >= 15
    L = binding.lib()
    for n in names:
        assert hasattr(L, n), f"{n} declared in the header but not exported"
        assert n in binding.SIGNATURES, f"{n} has no binding signature"
    assert sorted(binding.SIGNATURES) == names


def test_status_strings_and_null_checks():
    L = binding.lib()
    for code in range(0, -7, -1):
        assert L.dm_strerror(code) not in (None, b"unknown status")
    assert L.dm_strerror(-99) == b"unknown status"
    assert L.dm_create(None, 0) == binding.EINVAL
    assert L.dm_destroy(None) == binding.OK
    assert L.dm_set_impl(None, 0) == binding.EINVAL
    assert L.dm_workspace_bytes(None) == 0
    assert L.dm_set_head(None, None, 1, 8, 0, 1, 1) == binding.EINVAL
    assert L.dropmatch_verify(None, None, None, 1, 1, 0.1, 0, 0, None, None, None, None) == binding.EINVAL


def test_create_without_gpu_reports_an_error_not_a_crash():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    h = ctypes.c_void_p()
    assert binding.lib().dm_create(ctypes.byref(h), 0) in (binding.ECUDA, binding.EINVAL)
    assert not h
    with pytest.raises(pk.DropMatchError):
        pk.Context(0)
