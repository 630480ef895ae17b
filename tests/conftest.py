import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


def pytest_sessionstart(session):
    """The tests call the CUDA library through its C ABI: compile it (and the C oracle) if a fresh checkout has no
    binaries yet.  nvcc cross-compiles for sm_100a without a GPU."""
    try:
        from paper_2512_04857_b200 import build as lib_build
        from oracle import build as oracle_build
        lib_build.build()
        oracle_build.build()
    except Exception as e:          # the tests that need the library will say so themselves
        print(f"[conftest] build skipped: {e}")


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


def pytest_terminal_summary(terminalreporter, exitstatus, config):
    """What the parity runs compared with the oracle, and how many kept sets differed from it only at score near-ties
    (oracle scores within 1e-5 relative of the eviction boundary): the count is reported, not just bounded."""
    try:
        from _harness import TOTALS
    except Exception:
        return
    if not TOTALS:
        return
    tr = terminalreporter
    tr.write_sep("-", "parity against the CPU oracle")
    tot_c = tot_n = 0
    for where, t in sorted(TOTALS.items()):
        tot_c += t["compressions"]
        tot_n += t["near_ties"]
        tr.write_line(f"{where}: {t['runs']} runs, {t['outputs']} output elements, {t['line_ends']} line ends, "
                      f"{t['compressions']} compressions compared, {t['near_ties']} near-ties, "
                      f"max abs err bf16 {t['max_abs_err_bf16']:.3e} fp32 {t['max_abs_err_fp32']:.3e}")
    tr.write_line(f"near-ties: {tot_n} of {tot_c} compressions compared")
