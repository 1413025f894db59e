"""The plan's decision rules against the clock of this GPU.  The paper ranks candidate plans by measured
runtime (Sec. 3.2-3.3) and prints no thresholds, so nothing in it can pin the constants of the fixed rules;
what can be checked is that the automatic choice is never far slower than the fastest forced alternative.
A constant that is badly off (a block-fill cut-off on the wrong side, the class split at a width where it
loses, a wrong window count) picks a slow alternative at one of these points and fails the bound."""
import os
import sys

import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_automatic_choice_is_within_a_quarter_of_the_fastest_alternative():
    sys.path.insert(0, ROOT)
    import bench
    def slow_points(rows):
        return {(r["rule"], r["point"], r["dtype"], r["N"]): (r["ms"], r["automatic"], r["automatic_ms"]) for r in rows
                if r["regret"] > 0.25}

    rows = bench.regret_rows("test")
    assert len(rows) >= 23
    bad = slow_points(rows)
    if bad:
        # a single timing can be off (plans that use side streams vary by up to 20 % between instances of the same plan):
        # a point counts only when a second, independent sweep finds it slow as well
        again = slow_points(bench.regret_rows("test"))
        bad = {k: (v, again[k]) for k, v in bad.items() if k in again}
    assert not bad, bad
