import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


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


def pytest_terminal_summary(terminalreporter, exitstatus, config):
    """Ties are reported, not hidden: every kept-set or eviction difference that a parity test
    accepted as a near-tie is listed with how close the oracle's scores were."""
    parity = sys.modules.get("parity")
    if parity is None:          # no parity test was collected in this run
        return
    log = parity.TIE_LOG
    terminalreporter.write_sep("-", f"tie report: {len(log)} accepted near-tie(s)")
    for t in log:
        terminalreporter.write_line(f"  {t['test']}: {t['where']}; {t['pairs']} pair(s) ordered differently, oracle scores "
                                    f"apart by {t['closest_rel_gap']:.2e} to {t['widest_rel_gap']:.2e} (relative)")
