import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


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
    """Kept fractions of the weight comparisons (see util.sign_like_mask): per case and tensor, how many elements
    were compared relatively, how many absolutely, and the worst relative error seen."""
    try:
        import util
    except Exception:
        return
    tr = terminalreporter
    if util.DRIFT:
        tr.write_sep("-", "free-running drift: worst relative error after n steps without re-seeding")
        for (case, steps, kind), worst in sorted(util.DRIFT.items()):
            tr.write_line(f"{case:12s} steps {steps:4d} {kind:8s} {worst:.3e}")
    rows = util.ledger_rows()
    if not rows:
        return
    tr.write_sep("-", "weight comparisons: elements compared relatively / absolutely, worst relative error")
    for (case, name), (kept, masked, worst) in rows:
        frac = kept / max(kept + masked, 1)
        tr.write_line(f"{case:34s} {name:8s} kept {kept:12d} masked {masked:6d} frac {frac:.5f} worst {worst:.3e}")
