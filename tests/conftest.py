import os
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parents[1]
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture(scope="session")
def golden_dir():
    return ROOT / "tests" / "golden"


def pytest_terminal_summary(terminalreporter):
    """Worst max-abs-err / RMS(O) ratios of the attention parity comparisons (tests/test_gpu_attn.py)."""
    mod = sys.modules.get("test_gpu_attn") or sys.modules.get("tests.test_gpu_attn")
    rows = getattr(mod, "ERR_OVER_RMS", None)
    if not rows:
        return
    rows = sorted(rows, reverse=True)
    terminalreporter.write_line(f"attention parity: {len(rows)} comparisons, worst max-abs-err / RMS(O):")
    for ratio, err, rms, row_ratio, what in rows[:8]:
        terminalreporter.write_line(f"  {ratio:.3e}  (err {err:.3e}, rms {rms:.3e}, per-row excess {row_ratio:.3e})  {what}")
    worst_row = max(r[3] for r in rows)
    terminalreporter.write_line(f"  worst (|err| - 2^-8 |ref|) / rms of the row, over all comparisons: {worst_row:.3e}")
