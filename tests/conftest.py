import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


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


# Worst element-wise relative error |got - ref| / |ref| seen by the parity tests, per tolerance class, over the
# elements that are not small (|ref| > rms(ref) / 100); the tests' own bound is |got - ref| <= rtol * max(|ref|, rms).
PARITY_WORST = {}


def note_relative_error(rtol, worst_rel, worst_vs_bound):
    cur = PARITY_WORST.setdefault(rtol, [0.0, 0.0, 0, ""])
    cur[0] = max(cur[0], worst_rel)
    if worst_vs_bound > cur[1]:
        cur[1] = worst_vs_bound
        cur[3] = os.environ.get("PYTEST_CURRENT_TEST", "").split(" ")[0]
    cur[2] += 1


def pytest_terminal_summary(terminalreporter):
    if not PARITY_WORST:
        return
    terminalreporter.write_line("parity: worst errors per tolerance class (comparisons; error / bound; pure relative error where |ref| > rms/100)")
    for rtol in sorted(PARITY_WORST):
        rel, vs_bound, count, where = PARITY_WORST[rtol]
        terminalreporter.write_line(f"  rtol {rtol:g}: {count} comparisons, worst {vs_bound:.3f} x the bound ({where}), worst relative error {rel:.3g}")
