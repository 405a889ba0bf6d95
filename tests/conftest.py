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
        have = torch.cuda.is_available()
    except Exception:
        have = False
    if have:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


def pytest_terminal_summary(terminalreporter):
    """Margins of the floating-point parity gates seen in this run (tests/_parity.py): the tightest cases."""
    try:
        from tests._parity import MARGINS, TOL
    except Exception:
        return
    if not MARGINS:
        return
    tr = terminalreporter
    tr.write_sep("-", f"parity margins: {len(MARGINS)} gate calls, bar {TOL:g}")
    strict = [m for m in MARGINS if m[1].startswith("strict")]
    if strict:
        tr.write_line(f"fp32 outputs: worst max|err| / rms by the gate's normalisation {max(m[2] for m in strict):.3e}; "
                      f"worst max|err| / GLOBAL rms {max(m[3] for m in strict):.3e}; worst rms(err) / rms {max(m[4] for m in strict):.3e}")
    bf = [m for m in MARGINS if m[1] == "bf16"]
    if bf:
        tr.write_line(f"bf16 outputs: worst rms(err) / rms {max(m[2] for m in bf):.3e}; worst max|err| / GLOBAL rms {max(m[3] for m in bf):.3e}")
    for what, gate, worst, gmax, grms in sorted(MARGINS, key=lambda m: -m[2])[:8]:
        tr.write_line(f"  {worst:.3e} ({gate})  max/global-rms {gmax:.3e}  rms/rms {grms:.3e}  {what}")
