import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")


def pytest_terminal_summary(terminalreporter):
    """Parity report of the bf16 comparisons with the oracle: per test and tensor kind, the worst absolute error
    among elements with |ref| < 4 (bound: plain 2e-2; gradients may hold a share of 1e-4 of elements up to
    2.5e-2, the tail of the operand-rounding error), the worst above (bound: 2e-2 + 2^-8 |ref|), how many
    elements exceed the plain 2e-2, how many of those have |ref| < 4, and the smallest |ref| among them."""
    from tests import _util as U
    recs = [r for r in U.PARITY_REPORT if r["dtype"] == "bf16"]
    if not recs:
        return
    groups = {}
    for r in recs:
        kind = (r["what"].split() or ["?"])[0]
        g = groups.setdefault((r["test"], kind), dict(n=0, max_small=0.0, max_large=0.0, n_large=0, n_over=0, n_over_small=0,
                                                      min_ref_over=None, rel_l2=0.0))
        g["n"] += r["n"]; g["n_large"] += r["n_large"]; g["n_over"] += r["n_over_plain"]; g["n_over_small"] += r["n_over_small"]
        g["max_small"] = max(g["max_small"], r["max_small"]); g["max_large"] = max(g["max_large"], r["max_large"])
        g["rel_l2"] = max(g["rel_l2"], r["rel_l2"])
        if r["min_ref_over_plain"] is not None:
            g["min_ref_over"] = r["min_ref_over_plain"] if g["min_ref_over"] is None else min(g["min_ref_over"],
                                                                                             r["min_ref_over_plain"])
    tr = terminalreporter
    tr.write_line("")
    tr.write_line("bf16 parity report (max |got - oracle|; strict bound 2e-2 where |ref| < 4)")
    tr.write_line(f"{'test':58s} {'tensor':6s} {'elements':>10s} {'max |ref|<4':>12s} {'max |ref|>=4':>12s} "
                  f"{'n |ref|>=4':>10s} {'n > 2e-2':>9s} {'of them <4':>10s} {'min |ref| there':>15s} {'rel-L2':>9s}")
    worst = 0.0
    n_tail = 0
    for (test, kind), g in sorted(groups.items()):
        worst = max(worst, g["max_small"])
        n_tail += g["n_over_small"]
        mro = "-" if g["min_ref_over"] is None else f"{g['min_ref_over']:.2f}"
        tr.write_line(f"{test[:58]:58s} {kind[:6]:6s} {g['n']:10d} {g['max_small']:12.3e} {g['max_large']:12.3e} "
                      f"{g['n_large']:10d} {g['n_over']:9d} {g['n_over_small']:10d} {mro:>15s} {g['rel_l2']:9.2e}")
    tr.write_line(f"worst error among elements with |ref| < 4 over all bf16 comparisons: {worst:.3e} (bound 2e-2); "
                  f"{n_tail} of {sum(g['n'] for g in groups.values())} compared elements with |ref| < 4 exceed 2e-2")
