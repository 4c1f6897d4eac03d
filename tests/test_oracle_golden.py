"""The oracle reproduces its committed values for the `tiny` workload (tests/golden/tiny_oracle.txt,
written by tests/golden/make_golden.py from oracle/ alone)."""
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.join(HERE, "golden"))


def test_oracle_matches_committed_golden_values():
    import make_golden
    want = [l.strip() for l in open(os.path.join(HERE, "golden", "tiny_oracle.txt")) if l.strip() and not l.startswith("#")]
    got = make_golden.compute()
    assert len(got) == len(want)
    for g, w in zip(got, want):
        gn, wn = g.rsplit(" ", 1), w.rsplit(" ", 1)
        assert gn[0] == wn[0]
        a, b = float(gn[1]), float(wn[1])
        assert abs(a - b) <= 1e-12 * max(1.0, abs(b)), (g, w)
