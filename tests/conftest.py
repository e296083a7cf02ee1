import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def pytest_collection_modifyitems(config, items):
    """GPU tests are skipped (not failed) when no device is visible."""
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


def pytest_terminal_summary(terminalreporter, exitstatus, config):
    """Strict elementwise statistics of the programs gated by the row-scaled error only (reported, not gated)."""
    try:
        from tests.parity_util import STRICT_REPORT
    except Exception:
        return
    if not STRICT_REPORT:
        return
    tr = terminalreporter
    tr.section("strict elementwise error vs the fp64 oracle (reported, not gated)")
    tr.write_line("label                               n        R     strict max  n > R   well-cond.  of them > R  max there")
    for st in STRICT_REPORT:
        tr.write_line(f"{st['label'][:34]:34s} {st['n']:9d} {st['r']:.0e}  {st['strict_max']:10.3e} {st['n_over']:7d} "
                      f"{st['n_well']:10d} {st['n_over_well']:11d}  {st['well_max']:.3e}")
