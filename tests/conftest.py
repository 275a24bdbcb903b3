import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


@pytest.fixture(autouse=True)
def _report_output_checks(request):
    """Prints, after every test, what its output comparisons measured: the largest error relative to the RMS and
    how many one-bf16-ulp disagreements the bf16 rule tolerated, with the rows they sit in (`pytest -rP` or `-s`
    shows the lines of passing tests)."""
    try:
        import parity_utils
    except Exception:
        yield
        return
    parity_utils.REPORT.clear()
    yield
    rep = parity_utils.REPORT
    if rep:
        flips = sum(r["flips"] for r in rep)
        worst = max(r["worst_rel"] for r in rep)
        print(f"[parity] {request.node.name}: {len(rep)} output comparisons, worst error {worst:.3e} of RMS, "
              f"{flips} tolerated one-ulp disagreements in {sum(r['elements'] for r in rep)} elements")
        for r in rep:
            if r["flips"]:
                print(f"[parity]   {r['what']}: {r['flips']} flips in {r.get('n_flip_rows', 0)} rows, first rows {r['flip_rows']}")
