import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: test needs a CUDA device (B200)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def pytest_sessionfinish(session, exitstatus):
    """With ZC_PARITY_REPORT=<path> set, the figures the GPU parity tests recorded (largest
    output errors, near-tie swaps, units compared code by code) are written there as a
    Markdown table, one row per test case."""
    path = os.environ.get("ZC_PARITY_REPORT")
    if not path:
        return
    try:
        import zc_testlib as tl
    except Exception:
        return
    if not tl.RECORDS:
        return
    keys = []
    for r in tl.RECORDS:
        for k in r:
            if k not in keys:
                keys.append(k)

    def fmt(v):
        if isinstance(v, float):
            return f"{v:.3g}"
        return "" if v is None else str(v)

    lines = ["| " + " | ".join(keys) + " |", "|" + "---|" * len(keys)]
    for r in tl.RECORDS:
        lines.append("| " + " | ".join(fmt(r.get(k)) for k in keys) + " |")
    with open(path, "w") as f:
        f.write("\n".join(lines) + "\n")
