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


def test_host_side_argument_checks_of_the_newer_entry_points_need_no_gpu():
    """Every entry point validates on the host before it enqueues anything: bad sizes, missing pointers and size
    queries answer without touching a device."""
    import ctypes as C
    from paper_2511_20564_b200 import binding as B
    L = B.lib()
    ERR_NULL, ERR_ARG, ERR_UNSUPPORTED = -1, -2, -6
    # running sums of the weighted sampler
    assert L.e2egrec_edge_cumulate(-1, 0, None, None, None, None) == ERR_ARG
    assert L.e2egrec_edge_cumulate(4, 8, None, None, None, None) == ERR_NULL
    assert L.e2egrec_edge_cumulate(0, 0, C.c_void_p(256), None, None, None) == 0
    # LightGCN on sampled blocks: size queries from capacities alone
    blocks = (B.Block * 2)()
    blocks[0] = B.Block(64, 704, 640, *([None] * 10))
    blocks[1] = B.Block(704, 4224, 3520, *([None] * 10))
    x = B.Mat(None, 5000, 64, 64, B.BF16)
    n = C.c_size_t(0)
    assert L.e2egrec_lightgcn_sampled_forward(blocks, 2, C.byref(x), None, None, C.byref(n), None, None) == 0 and n.value > 0
    m = C.c_size_t(0)
    assert L.e2egrec_lightgcn_sampled_backward(blocks, 2, None, C.byref(x), None, None, C.byref(m), None) == 0 and m.value > 0
    assert L.e2egrec_lightgcn_sampled_forward(blocks, 9, C.byref(x), None, None, C.byref(n), None, None) == ERR_UNSUPPORTED
    assert L.e2egrec_lightgcn_sampled_forward(blocks, 2, C.byref(x), None, None, None, None, None) == ERR_NULL
    bad = B.Mat(None, 5000, 60, 60, B.BF16)            # rows of 120 bytes: not a multiple of 16
    assert L.e2egrec_lightgcn_sampled_forward(blocks, 2, C.byref(bad), None, None, C.byref(n), None, None) == -4
    # the frontier of a hop must fit the destinations of the next one
    blocks[1] = B.Block(100, 4224, 3520, *([None] * 10))
    assert L.e2egrec_lightgcn_sampled_forward(blocks, 2, C.byref(x), None, None, C.byref(n), None, None) == ERR_ARG
    # the transposed form as a call of its own
    blocks[1] = B.Block(704, 4224, 3520, *([None] * 10))
    assert L.e2egrec_blocks_transpose(5000, 2, None, C.c_void_p(256), 1 << 20, None) == ERR_NULL
    assert L.e2egrec_blocks_transpose(5000, 2, blocks, None, 1 << 20, None) == ERR_NULL
    assert L.e2egrec_blocks_transpose(5000, 0, blocks, C.c_void_p(256), 1 << 20, None) == ERR_ARG
    assert L.e2egrec_blocks_transpose(0, 2, blocks, C.c_void_p(256), 1 << 20, None) == ERR_ARG
    assert L.e2egrec_blocks_transpose(5000, 2, blocks, C.c_void_p(264), 1 << 20, None) == -4         # scratch not 256-byte aligned
    assert L.e2egrec_blocks_transpose(5000, 2, blocks, C.c_void_p(256), 1 << 20, None) == ERR_NULL    # blocks without arrays
