import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


def pytest_collection_modifyitems(config, items):
    """GPU tests are skipped, not failed, on a machine without a device."""
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


@pytest.fixture(scope="session", autouse=True)
def built_libraries():
    """Build libcawn.so (nvcc, sm_100a) and the C oracle (gcc) once per session if they are missing or
    older than their sources; a no-op when they are up to date."""
    import __graft_entry__ as entry
    entry.build()


def pytest_terminal_summary(terminalreporter, exitstatus, config):
    """Parity margins of the run: for every test function that compared something, the largest
    floored error it saw (the quantity the tolerances bound) and the largest unfloored median of
    the element-wise relative error.  Also written as parity_margins.json into the directory the
    environment variable CAWN_REPORT_DIR names, when it is set."""
    import json
    try:
        from helpers import MARGINS
    except Exception:
        return
    if not MARGINS:
        return
    rows = {}
    for test, err, med in MARGINS:
        name = test.split("[")[0]
        n, e, m = rows.get(name, (0, 0.0, 0.0))
        rows[name] = (n + 1, max(e, err), max(m, med))
    terminalreporter.section("parity margins (floored max error | unfloored median error | comparisons)")
    for name in sorted(rows):
        n, e, m = rows[name]
        terminalreporter.write_line("%-96s %.3e  %.3e  %d" % (name, e, m, n))
    out = os.environ.get("CAWN_REPORT_DIR")
    if not out:
        return
    try:
        os.makedirs(out, exist_ok=True)
        with open(os.path.join(out, "parity_margins.json"), "w") as f:
            json.dump({k: {"comparisons": v[0], "floored_max": v[1], "unfloored_median_max": v[2]}
                       for k, v in sorted(rows.items())}, f, indent=1)
    except OSError:
        pass
