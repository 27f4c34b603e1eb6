import os
import sys

import pytest

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session")
def oracle():
    from oracle import gs_oracle
    gs_oracle.build()
    return gs_oracle


# Measured counts behind the parity tolerances (fragile pixels, values outside the literal gradient rule, values that
# need an allowance): tests/gpu_helpers.check_bound appends rows here, the summary prints them, and
# GS_PARITY_REPORT=<file> also stores them (tests/make_parity_bounds.py turns that file into tests/parity_bounds.json).
PARITY_ROWS = []


def record_parity(case, check, **counts):
    PARITY_ROWS.append(dict(case=case, check=check, **counts))


def pytest_terminal_summary(terminalreporter):
    if not PARITY_ROWS:
        return
    tr = terminalreporter
    tr.section("measured parity counts")
    for r in PARITY_ROWS:
        rest = ", ".join(f"{k}={v:.3g}" if isinstance(v, float) else f"{k}={v}" for k, v in r.items() if k not in ("case", "check"))
        tr.write_line(f"{r['case']:<28} {r['check']:<22} {rest}")
    path = os.environ.get("GS_PARITY_REPORT")
    if path:
        import json
        with open(path, "w") as f:
            json.dump(PARITY_ROWS, f, indent=1, default=float)
