"""Pins of the oracle's correctly rounded merge (exact sum, one rounding to E4M3) against brute force in exact
rational arithmetic, against constructed ties that a floating-point chain cannot see, and against the chain merge
where both must agree."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import falqon_oracle as orc


def _decode_all():
    vals = {}
    for c in range(256):
        v = orc.decode(c, orc.E4M3)
        if np.isfinite(v):
            vals[c] = Fraction(v)
    return vals


VALS = _decode_all()
POS = sorted((v, c) for c, v in VALS.items() if c < 0x80)      # the non-negative values with their codes


def _brute(w: int, d, a) -> int:
    """Exact sum as a Fraction, then the nearest E4M3 value by exhaustive search: ties to the even code, saturation
    at 448, the sign of the exact sum kept when the magnitude rounds to zero, exact zero -> +0."""
    s = VALS[w] + sum(Fraction(float(x)) * VALS[int(c)] for x, c in zip(d, a))
    if s == 0:
        return 0
    mag = abs(s)
    best = None
    for v, c in POS:
        dist = abs(mag - v)
        if best is None or dist < best[0] or (dist == best[0] and c % 2 == 0 and best[1] % 2 == 1):
            best = (dist, c)
    code = best[1]
    if mag > 448:
        code = max(c for _, c in POS)
    return code | (0x80 if s < 0 else 0)


def _rand_codes(rng, size):
    c = rng.integers(0, 256, size=size).astype(np.uint8)
    c[(c & 0x7F) == 0x7F] = 0x3C     # no NaN codes
    return c


def test_exact_merge_matches_rational_brute_force():
    rng = np.random.default_rng(0)
    for trial in range(3000):
        r = int(rng.integers(1, 9))
        a = _rand_codes(rng, r)
        w = int(_rand_codes(rng, 1)[0])
        scale = np.float32(2.0) ** rng.integers(-40, 6)
        d = (rng.standard_normal(r).astype(np.float32) * scale).astype(np.float32)
        if trial % 7 == 0:
            d[rng.integers(0, r)] = np.float32(2.0) ** rng.integers(-149, -100)    # a term far below everything else
        assert orc.exact_merge_element(w, d, a) == _brute(w, d, a), (trial, w, d, a)


def test_ties_and_terms_a_float_chain_cannot_see():
    one, two = orc.encode(1.0, orc.E4M3), orc.encode(2.0, orc.E4M3)
    eight, nine = orc.encode(8.0, orc.E4M3), orc.encode(9.0, orc.E4M3)
    ten = orc.encode(10.0, orc.E4M3)
    a = np.array([one, one], dtype=np.uint8)
    # 8 + 0.5 is a tie between 8 and 9: to the even code (8); 9 + 0.5 is a tie between 9 and 10: to 10
    assert orc.exact_merge_element(eight, np.float32([0.5, 0.0]), a) == eight
    assert orc.exact_merge_element(nine, np.float32([0.5, 0.0]), a) == ten
    # a term of 2^-140 breaks the tie upwards, -2^-140 downwards; fp32 arithmetic loses it
    tiny = np.float32(2.0) ** -140
    assert orc.exact_merge_element(eight, np.float32([0.5, tiny]), a) == nine
    assert orc.exact_merge_element(nine, np.float32([0.5, -tiny]), a) == nine
    # massive cancellation: 2^60 - 2^60 + 0.75 survives
    big = np.float32(2.0) ** 60
    a3 = np.array([one, one, one], dtype=np.uint8)
    assert orc.exact_merge_element(0, np.float32([big, -big, 0.75]), a3) == orc.encode(0.75, orc.E4M3)
    # saturation on both sides, sign of a sum that rounds to zero, exact zero
    assert orc.exact_merge_element(orc.encode(448.0, orc.E4M3), np.float32([100.0, 0.0]), a) == orc.encode(448.0, orc.E4M3)
    assert orc.exact_merge_element(orc.encode(-448.0, orc.E4M3), np.float32([-1e30, 0.0]), a) == orc.encode(-448.0, orc.E4M3)
    assert orc.exact_merge_element(0, np.float32([-tiny, 0.0]), a) == 0x80
    assert orc.exact_merge_element(two, np.float32([-1.0, -1.0]), a) == 0x00


def test_exact_update_agrees_with_chain_update_where_it_must():
    """Same optimizer step, scores, selection and clearing; merged codes equal wherever the chain made no rounding
    error that mattered, and never more than one code apart."""
    rng = np.random.default_rng(3)
    m, n, r, k = 64, 48, 8, 20
    wq = _rand_codes(rng, (m + r, n))
    wq[(wq & 0x7F) > 0x70] &= 0x8F                    # keep clear of saturation so "one code apart" is meaningful
    dbuf = (rng.standard_normal((m, r)) * 0.05).astype(np.float32)
    dB = (rng.standard_normal((m, r)) * 0.5).astype(np.float32)
    w1, d1 = wq.copy(), dbuf.copy()
    w2, d2 = wq.copy(), dbuf.copy()
    idx1, s1 = orc.proxy_update(w1, d1, dB, 0.1, k, m, r)
    idx2, s2 = orc.proxy_update_exact(w2, d2, dB, 0.1, k, m, r)
    assert np.array_equal(idx1, idx2) and np.array_equal(s1.view(np.uint32), s2.view(np.uint32))
    assert np.array_equal(d1.view(np.uint32), d2.view(np.uint32))
    untouched = np.setdiff1d(np.arange(m + r), idx1)
    assert np.array_equal(w2[untouched], wq[untouched])
    v1 = np.vectorize(lambda c: orc.decode(int(c), orc.E4M3))(w1[idx1])
    v2 = np.vectorize(lambda c: orc.decode(int(c), orc.E4M3))(w2[idx1])
    differ = w1[idx1] != w2[idx1]
    assert differ.mean() < 0.05
    # where they differ, they are neighbours on the E4M3 grid
    grid = np.array(sorted(set(float(v) for v in VALS.values())))
    pos1 = np.searchsorted(grid, v1[differ])
    pos2 = np.searchsorted(grid, v2[differ])
    assert np.all(np.abs(pos1 - pos2) <= 1)
    # the exact update of every selected element equals the element-wise pin
    for i in idx1[:5]:
        d_row = np.float32(-0.1) * dB[i] + dbuf[i]     # what the optimizer step left (one fma each)
        d_row = np.array([np.float32(np.float64(np.float32(-0.1)) * np.float64(dB[i, j]) + np.float64(dbuf[i, j])) for j in range(r)],
                         dtype=np.float32)
        for c in range(0, n, 7):
            assert w2[i, c] == orc.exact_merge_element(int(wq[i, c]), d_row, wq[m:, c])


def test_integers_merge_exactly_in_both_variants():
    """Small integers: every partial sum is representable, so the chain makes no rounding and must equal the exact merge."""
    m, n, r = 4, 16, 4
    enc = lambda v: orc.encode(float(v), orc.E4M3)
    wq = np.zeros((m + r, n), dtype=np.uint8)
    wq[:m] = enc(2.0)
    wq[m:] = enc(1.0)
    dbuf = np.ones((m, r), dtype=np.float32)
    w1, d1, w2, d2 = wq.copy(), dbuf.copy(), wq.copy(), dbuf.copy()
    orc.proxy_update(w1, d1, None, 0.0, m, m, r)
    orc.proxy_update_exact(w2, d2, None, 0.0, m, m, r)
    assert np.array_equal(w1, w2) and np.all(w1[:m] == enc(6.0))
