import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the sm_100a kernels)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def pytest_terminal_summary(terminalreporter):
    """How much of every compared tensor needed more than the plain tolerance (tests/helpers.py: AUDIT)."""
    try:
        import helpers
    except Exception:
        return
    rows = helpers.AUDIT
    if not rows:
        return
    import json
    terminalreporter.write_line("parity audit: elements outside the plain tolerance (before the terms-scale and outlier allowances)")
    for r in rows:
        if r["outside_plain"]:
            terminalreporter.write_line(f"  {r['test']} {r['tensor']} [{r['dtype']}]: {r['outside_plain']} of {r['elements']} "
                                        f"({r['share']:.2e}), worst {r['worst_ratio']:.2f}x")
    clean = sum(1 for r in rows if not r["outside_plain"])
    terminalreporter.write_line(f"  {clean} of {len(rows)} compared tensors had every element inside the plain tolerance")
    path = os.environ.get("E2EGREC_PARITY_AUDIT")
    if path:
        with open(path, "w") as f:
            json.dump(rows, f, indent=1)
