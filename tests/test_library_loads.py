"""Host-side checks that need no GPU: the library builds for sm_100a, loads, and exports every
symbol the header declares; the binding refuses to run without a device."""
import os
import re

import pytest
import torch

import paper_2202_02365_b200 as mg
from paper_2202_02365_b200 import api

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "mgdense.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mg_[a-z0-9_]+)\s*\(", text)))


def test_builds_and_exports_every_declared_symbol():
    import __graft_entry__ as ge
    ge.build()
    lib = mg.load_library()
    names = _declared()
    assert len(names) >= 20
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(api.EXPORTS) == names


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU behaviour")
def test_no_cpu_fallback():
    with pytest.raises(RuntimeError):
        mg.Context(0)
    import ctypes as C
    lib = mg.load_library()
    h = C.c_void_p(0)
    assert lib.mg_create(C.byref(h), 0, None) != 0      # fails cleanly, no crash
    assert not h.value
