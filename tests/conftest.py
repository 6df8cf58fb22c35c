import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the CUDA library through its C ABI)")


@pytest.fixture(scope="session")
def oracle_lib():
    from oracle import build_oracle

    return build_oracle()


def pytest_terminal_summary(terminalreporter, exitstatus, config):
    """Near-tie record of the lock-step runs (also at -q): pair decisions taken, how many were near-ties in the
    oracle (relative score gap below 1e-4) and at how many of those the oracle followed the library's choice."""
    try:
        from lockstep import REPORTS
    except Exception:
        return
    if not REPORTS:
        return
    tr = terminalreporter
    tr.write_line("")
    tr.write_line("lock-step with the fp64 oracle: decisions / near-ties / flips  (max out err, max rel score err)")
    tot = [0, 0, 0]
    for r in REPORTS:
        if r.calls == 0:
            continue
        tr.write_line("  %-88s %8d %5d %5d  (%.2g, %.2g)" % (r.label[-88:], r.decisions, r.near_ties, r.flips,
                                                               r.max_out_err, r.max_score_rel))
        tot[0] += r.decisions; tot[1] += r.near_ties; tot[2] += r.flips
    tr.write_line("  %-88s %8d %5d %5d" % ("TOTAL", tot[0], tot[1], tot[2]))
