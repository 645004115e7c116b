"""Pins for the integer acceptance rule (LeadingSubstringVerify, Algorithms 1-2)."""
import itertools
import os

from oracle.hispec import leading_substring_verify

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "fig3_scenario.txt")


def test_exhaustive_characterisation():
    """All (S, v) over a 3-letter alphabet, |S| <= 4, with and without the bonus
    entry: the result is the unique list that (i) starts with a prefix of S that
    agrees with v, (ii) is the longest such prefix, (iii) ends with the
    verifier's token at the first disagreement when that token exists."""
    n = 0
    for ls in range(0, 5):
        for S in itertools.product(range(3), repeat=ls):
            for lv in (ls, ls + 1):
                for v in itertools.product(range(3), repeat=lv):
                    out, a = leading_substring_verify(S, v)
                    n += 1
                    assert 0 <= a <= ls
                    assert list(S[:a]) == list(v[:a]) == out[:a]          # accepted prefix agrees with verifier
                    assert a == ls or S[a] != v[a]                          # maximal: next one disagrees
                    if a < lv:
                        assert out == list(S[:a]) + [v[a]]                  # correction / bonus token
                    else:
                        assert out == list(S)                               # all accepted, no bonus computed
                    # every emitted token is the verifier's greedy token at its position
                    assert all(out[i] == v[i] for i in range(len(out)))
    assert n > 5000


def test_paper_scenario_fixture():
    rows = 0
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        S, v, exp, a = [c.split() for c in line.split("|")]
        out, acc = leading_substring_verify([int(t) for t in S], [int(t) for t in v])
        assert out == [int(t) for t in exp] and acc == int(a[0])
        rows += 1
    assert rows == 3
