import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200) and the built library")


def pytest_terminal_summary(terminalreporter):
    """Index-set comparisons of the session: how many selected tokens differed from the oracle's
    and how many of those lay outside the literal / the wide band (see tests/helpers.py)."""
    try:
        from tests import helpers as hp
    except Exception:
        return
    if not hp.BAND_LOG:
        return
    lines = ["case | selected | differing | outside literal band | outside wide band | k-th score | max|r_c|"]
    for r in hp.BAND_LOG:
        lines.append(f"{r.what} | {r.n_sel} | {r.n_diff} | {r.n_outside_literal} | {r.n_outside_wide} | "
                     f"{r.kth:.6g} | {r.scale_r:.6g}")
    tot = (sum(r.n_sel for r in hp.BAND_LOG), sum(r.n_diff for r in hp.BAND_LOG),
           sum(r.n_outside_literal for r in hp.BAND_LOG), sum(r.n_outside_wide for r in hp.BAND_LOG))
    lines.append(f"TOTAL | {tot[0]} | {tot[1]} | {tot[2]} | {tot[3]} | |")
    terminalreporter.write_sep("-", "index-set band report")
    terminalreporter.write_line(lines[0])
    terminalreporter.write_line(lines[-1])
    path = os.environ.get("ESA_BAND_REPORT")
    if path:
        with open(path, "w") as f:
            f.write("\n".join(lines) + "\n")
