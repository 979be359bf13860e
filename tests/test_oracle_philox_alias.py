"""Pins for the oracle's random-number generator and alias construction (CPU)."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import ldaref

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]


def test_philox_known_answers():
    for ln in _rows("philox4x32_10_kat.txt"):
        v = [int(x, 16) for x in ln.split()]
        got = ldaref.philox(v[0:4], v[4:6])
        assert [int(x) for x in got] == v[6:10]


def _philox_bigint(ctr, key, rounds=10):
    """The published round function written with Python integers."""
    c = list(ctr)
    k = list(key)
    mask = (1 << 32) - 1
    for _ in range(rounds):
        p0 = 0xD2511F53 * c[0]
        p1 = 0xCD9E8D57 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & mask, (p0 >> 32) ^ c[3] ^ k[1], p0 & mask]
        k = [(k[0] + 0x9E3779B9) & mask, (k[1] + 0xBB67AE85) & mask]
    return c


def test_philox_against_bigint_restatement():
    rng = np.random.default_rng(1)
    for _ in range(200):
        ctr = [int(x) for x in rng.integers(0, 2 ** 32, 4)]
        key = [int(x) for x in rng.integers(0, 2 ** 32, 2)]
        assert [int(x) for x in ldaref.philox(ctr, key)] == _philox_bigint(ctr, key)


def test_alias_hand_tables():
    for ln in _rows("alias_hand_tables.txt"):
        w, thr, al = [[int(x) for x in part.split(",")] for part in ln.split("|")]
        t = ldaref.alias_build(w)
        assert t["shift"] == 0 and t["W"] == sum(w)
        assert [int(x) for x in t["thr"]] == thr
        assert [int(x) for x in t["alias"]] == al


def _masses(t, n):
    """Exact mass routed to each item, in units where a bin holds W."""
    W = t["W"]
    mass = [0] * n
    for b in range(n):
        a = int(t["alias"][b])
        if a == b:
            mass[b] += W
        else:
            assert 0 <= int(t["thr"][b]) <= W
            mass[b] += int(t["thr"][b])
            mass[a] += W - int(t["thr"][b])
    return mass


def _weight_cases():
    rng = np.random.default_rng(7)
    cases = [[5], [3, 3, 3, 3, 3], [1, 1, 1, 1, 10 ** 9], [10 ** 12, 1, 1],
             list(range(1, 40)), [0, 0, 9, 0]]
    for n in (2, 3, 7, 32, 33, 100, 1000):
        cases.append([int(x) for x in rng.integers(1, 2 ** 44, n)])
        cases.append([int(x) for x in rng.integers(1, 50, n)])            # many ties
        cases.append([int(x) for x in (rng.pareto(0.7, n) * 1e6 + 1)])    # heavy tail
    # large totals that force the pre-shift
    cases.append([int(x) for x in rng.integers(2 ** 43, 2 ** 44, 5000)])
    cases.append([2 ** 44] * 4096)
    return cases


@pytest.mark.parametrize("case", range(len(_weight_cases())))
def test_alias_conserves_every_items_mass_exactly(case):
    w = _weight_cases()[case]
    n = len(w)
    t = ldaref.alias_build(w)
    sh = t["shift"]
    assert sh == max(0, sum(w).bit_length() + n.bit_length() - 62)
    ws = [x >> sh for x in w]
    assert t["W"] == sum(ws) and t["W44"] == sum(w)
    assert n * t["W"] < 2 ** 62
    assert _masses(t, n) == [n * x for x in ws]
    # every alias points at a valid item
    assert all(0 <= int(a) < n for a in t["alias"])


def test_alias_draw_law_matches_weights():
    """P(item) from (bin uniform, 32-bit coin) equals w_i / W up to 2^-32 per bin."""
    rng = np.random.default_rng(3)
    w = [int(x) for x in rng.integers(1, 10 ** 6, 37)]
    n = len(w)
    t = ldaref.alias_build(w)
    p = [Fraction(0)] * n
    for b in range(n):
        a = int(t["alias"][b])
        keep = Fraction(1) if a == b else Fraction(int(t["thr32"][b]), 2 ** 32)
        p[b] += keep / n
        if a != b:
            p[a] += (1 - keep) / n
    W = sum(w)
    for i in range(n):
        assert abs(p[i] - Fraction(w[i], W)) < Fraction(2, 2 ** 32)
    # the draw function itself: the bin is floor(r1*n/2^32), the coin compares r2 with thr32
    for _ in range(2000):
        r1, r2 = int(rng.integers(0, 2 ** 32)), int(rng.integers(0, 2 ** 32))
        b = (r1 * n) >> 32
        expect = b if (int(t["alias"][b]) == b or r2 < int(t["thr32"][b])) else int(t["alias"][b])
        assert ldaref.alias_draw(t["thr32"], t["alias"], r1, r2) == expect


def test_alias_split_point_quantisation():
    rng = np.random.default_rng(5)
    w = [int(x) for x in rng.integers(2 ** 30, 2 ** 44, 300)]
    t = ldaref.alias_build(w)
    W = t["W"]
    for b in range(len(w)):
        if int(t["alias"][b]) == b:
            continue
        exact = Fraction(int(t["thr"][b]), W)
        got = Fraction(int(t["thr32"][b]), 2 ** 32)
        assert abs(exact - got) < Fraction(1, 2 ** 30)
