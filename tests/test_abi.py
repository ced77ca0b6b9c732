"""The C-ABI library loads and exports every symbol the public header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(e2egrec_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_header_declares_the_four_entry_points():
    names = _declared()
    for n in ("e2egrec_sample_khop", "e2egrec_sage_forward", "e2egrec_sage_backward"):
        assert n in names


def test_library_exports_every_declared_symbol():
    from paper_2511_20564_b200 import build
    so = build.build()
    lib = ctypes.CDLL(so)
    for n in _declared():
        assert hasattr(lib, n), f"{n} declared in include/ but not exported"


def test_status_strings_and_size_queries_work_without_a_gpu():
    import paper_2511_20564_b200 as E
    assert E.status_string(0) == "ok" and "NULL" in E.status_string(-1)
    cd, cs, ce, nbytes = E.sample_khop_workspace(500_000, 4096, [15, 10])
    assert cd == [4096, 65536] and ce == [61440, 655360] and cs == [65536, 500000] and nbytes > 0
    with pytest.raises(E.E2EGrecError):
        E.sample_khop_workspace(1 << 31, 4, [3])
