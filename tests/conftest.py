import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def _has_gpu() -> bool:
    try:
        import torch
        return torch.cuda.is_available()
    except Exception:
        return False


def pytest_collection_modifyitems(config, items):
    if _has_gpu():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def pytest_terminal_summary(terminalreporter):
    """Strict statistics of the 16-bit parity checks of this session (see helpers.check_sweep)."""
    try:
        import helpers
    except Exception:
        return
    log = helpers.STATS_LOG
    if not log:
        return
    n = sum(r["n"] for _, r in log)
    wide = sum(r.get("needs_wide", 0) for _, r in log)
    unequal = sum((1.0 - r["equal"]) * r["n"] for _, r in log)
    worst = max(log, key=lambda e: e[1].get("strict_worst_ulp", 0.0))
    terminalreporter.write_line(
        f"16-bit parity checks: {len(log)} checks, {n} elements; not bit-identical {unequal / n:.3e} of them; "
        f"beyond 1 ulp of the oracle's own result (needing the wider reading) {wide} = {wide / n:.3e}; "
        f"worst strict difference {worst[1].get('strict_worst_ulp', 0.0):.2f} ulp in [{worst[0]}]")
