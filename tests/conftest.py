import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200, sm_100a)")


def pytest_collection_modifyitems(config, items):
    # GPU tests are deselected by -m "not gpu"; when selected without a device they fail
    # loudly inside the binding rather than being skipped.
    return


def _parity_rows():
    import dataclasses
    try:
        import jd_testlib as T
    except Exception:
        return {}
    return {name: dataclasses.asdict(rep) for name, rep in sorted(T.SESSION_REPORTS.items())}


def pytest_sessionfinish(session, exitstatus):
    """Writes the session's parity counts (one entry per workload) as JSON."""
    import json
    rows = _parity_rows()
    if not rows:
        return
    out_dir = os.environ.get("JD_REPORT_DIR") or os.path.join(ROOT, "parity_reports")
    try:
        os.makedirs(out_dir, exist_ok=True)
        with open(os.path.join(out_dir, "parity_counts.json"), "w") as f:
            json.dump(rows, f, indent=1, sort_keys=True)
    except OSError:
        pass


def pytest_terminal_summary(terminalreporter):
    """Prints the same counts after the test results, so that they survive output capture."""
    rows = _parity_rows()
    if not rows:
        return
    tr = terminalreporter
    tr.write_sep("-", "parity counts against the CPU checker (per workload)")
    tr.write_line("%-28s %5s %6s %7s %7s %6s %7s %8s %9s %9s %9s %9s" % (
        "workload", "seqs", "slots", "ex_acc", "ex_jdg", "ex_len", "tok_eq", "tok_marg", "rel_p", "rel_lse",
        "abs_judge", "rel_logit"))
    for name, r in rows.items():
        tr.write_line("%-28s %5d %6d %7d %7d %6d %7d %8d %9.2e %9.2e %9.2e %9.2e" % (
            name, r["sequences"], r["slots"], r["exempt_accept"], r["exempt_judge"], r["exempt_len"],
            r["token_exact"], r["token_in_margin"], r["max_rel_p"], r["max_rel_lse"], r["max_abs_judge"],
            r["max_rel_logit"]))
