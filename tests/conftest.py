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
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def pytest_terminal_summary(terminalreporter, exitstatus, config):
    """Prints the figures the parity gates are read with: for every output check the strict max-abs error and how
    many entries passed only by the one-ulp clause; for every score check the strict (unfloored) relative error."""
    try:
        import gpu_util
    except Exception:  # pragma: no cover
        return
    if gpu_util.REPORT:
        rows = gpu_util.REPORT
        terminalreporter.write_line(f"output parity: {len(rows)} checks, {sum(r['entries'] for r in rows)} entries, "
                                    f"worst rel-Frobenius {max(r['rel_fro'] for r in rows):.3e}, "
                                    f"strict max-abs {max(r['max_abs'] for r in rows):.4f}, "
                                    f"saved by the ulp clause {sum(r['saved_by_ulp'] for r in rows)}")
        for r in sorted(rows, key=lambda r: -r["saved_by_ulp"])[:8]:
            if r["saved_by_ulp"]:
                terminalreporter.write_line(f"  {r['label'] or '(unlabelled)'}: saved {r['saved_by_ulp']} of {r['entries']}, "
                                            f"max-abs {r['max_abs']:.4f}, smallest |ref| saved {r['min_abs_ref_saved']:.2f}")
    if gpu_util.SCORE_REPORT:
        rows = gpu_util.SCORE_REPORT
        terminalreporter.write_line(f"score parity: {len(rows)} checks, worst floored relative error "
                                    f"{max(r['floored'] for r in rows):.3e}, worst strict relative error "
                                    f"{max(r['strict'] for r in rows):.3e} (at |s_ref| = "
                                    f"{max(rows, key=lambda r: r['strict'])['at']:.3e})")
