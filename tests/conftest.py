import json
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# Worst max|err| / max|ref| seen per (parity case, output), filled by the GPU parity tests
# through `record_margin`, printed at the end of the run and, when the environment
# variable QALORA_PARITY_MARGINS names a file, written there as JSON.
PARITY_MARGINS = {}


def record_margin(case: str, output: str, err: float, tol: float):
    """Notes the error of one output of one parity case and asserts it against `tol`."""
    worst = PARITY_MARGINS.setdefault(case, {})
    worst[output] = max(float(err), worst.get(output, 0.0))
    assert err <= tol, f"{case}: {output} max|err|/max|ref| = {err:.3e} > {tol:.1e}"


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the library's kernels)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        have_gpu = torch.cuda.is_available()
    except Exception:
        have_gpu = False
    if have_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(autouse=True)
def _bounds_check_record(request):
    """With QALORA_LIBRARY=debug (the bounds-check build) every GPU test ends by reading the
    library's record words: a failed index check or an overwritten guard word fails the test."""
    yield
    if os.environ.get("QALORA_LIBRARY") != "debug" or "gpu" not in request.keywords:
        return
    from paper_2309_14717_b200 import binding as Q
    assert Q.qalora_debug_checks(), "QALORA_LIBRARY=debug but the loaded library has no checks"
    words = Q.qalora_debug_report()
    assert not any(words), ("bounds-check build: flags=%d first site=%d index=%d limit=%d failed checks=%d guard=%d"
                            % (words[0], words[1], (words[3] << 32) | (words[2] & 0xffffffff),
                               (words[5] << 32) | (words[4] & 0xffffffff), words[6], words[7]))


def pytest_terminal_summary(terminalreporter):
    if os.environ.get("QALORA_LIBRARY") == "debug":
        terminalreporter.write_line("bounds-check build: record words read after every GPU test")
    if not PARITY_MARGINS:
        return
    tr = terminalreporter
    tr.write_sep("-", "parity margins: worst max|err|/max|ref| per case and output (tolerance 5e-3)")
    for case in sorted(PARITY_MARGINS):
        tr.write_line(case + ": " + ", ".join(f"{k}={v:.2e}" for k, v in sorted(PARITY_MARGINS[case].items())))
    path = os.environ.get("QALORA_PARITY_MARGINS")
    if path:
        with open(path, "w") as f:
            json.dump(PARITY_MARGINS, f, indent=1, sort_keys=True)
