"""Pins for the oracle's random stream: Philox4x32-10, the deterministic -ln(u), the delay law
and the minibatch index draw.  CPU only."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
from scipy import stats

from oracle import core

M32 = 0xFFFFFFFF


def py_philox(key, ctr):
    """Independent restatement with Python integers (10 rounds, key bumped between rounds)."""
    c = list(ctr)
    k = list(key)
    for _ in range(10):
        p0 = 0xD2511F53 * c[0]
        p1 = 0xCD9E8D57 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & M32, (p0 >> 32) ^ c[3] ^ k[1], p0 & M32]
        k = [(k[0] + 0x9E3779B9) & M32, (k[1] + 0xBB67AE85) & M32]
    return c


def test_philox_known_answers(golden_dir):
    rows = [l.split() for l in open(os.path.join(golden_dir, "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        assert core.philox4x32_10(v[4:6], v[0:4]) == v[6:10]
        assert py_philox(v[4:6], v[0:4]) == v[6:10]


def test_philox_matches_python_integers():
    rng = np.random.default_rng(1)
    for _ in range(2000):
        key = [int(x) for x in rng.integers(0, 2**32, 2)]
        ctr = [int(x) for x in rng.integers(0, 2**32, 4)]
        assert core.philox4x32_10(key, ctr) == py_philox(key, ctr)


def test_philox_bytes_are_uniform():
    counts = np.zeros(256)
    for s in range(4000):
        for w in core.philox4x32_10([7, 9], [s, 0, 0, 0]):
            for sh in (0, 8, 16, 24):
                counts[(w >> sh) & 255] += 1
    chi2 = ((counts - counts.mean()) ** 2 / counts.mean()).sum()
    assert chi2 < stats.chi2.ppf(0.9999, 255)


def _u_of(x0, x1):
    k = (x0 << 20) | (x1 >> 12)
    return 2 * k + 1


def test_neg_log_close_to_libm_log():
    rng = np.random.default_rng(2)
    xs = rng.integers(0, 2**32, (20000, 2))
    cases = [(0, 0), (M32, M32), (0x80000000, 0), (0x7FFFFFFF, M32), (1, 0), (0, 1 << 12)]
    cases += [(int(a), int(b)) for a, b in xs]
    # small u as well: zero out leading bits
    cases += [(int(a) >> sh, int(b)) for (a, b), sh in zip(xs[:2000], rng.integers(1, 32, 2000))]
    for x0, x1 in cases:
        n = _u_of(x0, x1)
        ref = -math.log(n / 2.0**53) if n / 2.0**53 < 1.0 else -math.log1p(-(2**53 - n) / 2.0**53)
        got = core.neg_log_uniform(x0, x1)
        assert got > 0.0
        assert abs(got - ref) <= 4 * np.spacing(ref) + 2e-16, (x0, x1, got, ref)


def test_neg_log_exact_against_rational_arithmetic():
    """Each step redone with exact rationals rounded once (what an IEEE op is)."""
    def rn(q):
        return float(q)          # Fraction -> float is correctly rounded, ties to even

    def fma(a, b, c):
        return rn(Fraction(a) * Fraction(b) + Fraction(c))

    rng = np.random.default_rng(3)
    for x0, x1 in rng.integers(0, 2**32, (300, 2)):
        n = _u_of(int(x0), int(x1))
        b = n.bit_length() - 1
        f = Fraction(n, 2**b)
        if f > Fraction(0x16A09E667F3BCD, 2**52):
            f, b = f / 2, b + 1
        f = float(f)
        s = rn(Fraction(rn(Fraction(f) - 1)) / Fraction(rn(Fraction(f) + 1)))
        z = rn(Fraction(s) * Fraction(s))
        p = rn(Fraction(1, 23))
        for i in range(10, -1, -1):
            p = fma(p, z, rn(Fraction(1, 2 * i + 1)))
        lnf = rn(Fraction(rn(Fraction(2) * Fraction(s))) * Fraction(p))
        want = fma(float(53 - b), float.fromhex("0x1.62e42fefa39efp-1"), -lnf)
        assert core.neg_log_uniform(int(x0), int(x1)) == want


def test_neg_log_is_monotone_in_k():
    rng = np.random.default_rng(4)
    for x0, x1 in rng.integers(0, 2**32, (5000, 2)):
        x0, x1 = int(x0), int(x1) & ~0xFFF
        k = (x0 << 20) | (x1 >> 12)
        if k + 1 >= 2**52:
            continue
        k2 = k + 1
        a = core.neg_log_uniform(x0, x1)
        b = core.neg_log_uniform(k2 >> 20, (k2 & 0xFFFFF) << 12)
        assert b <= a


@pytest.mark.parametrize("kind,mu,shift", [("exp", 1.0, 0.0), ("exp", 2.5, 0.0), ("shifted_exp", 2.0, 1.0)])
def test_delay_law(kind, mu, shift):
    """X = Delta + Exp(rate mu): mean Delta + 1/mu, variance 1/mu^2, KS against 1 - exp(-mu x)."""
    x = np.array([core.delay(kind, mu, shift, 11, r, w, s)
                  for r in range(40) for w in range(8) for s in range(400)])
    n = x.size
    assert x.min() >= shift
    assert abs(x.mean() - (shift + 1 / mu)) < 4 / mu / math.sqrt(n)
    assert abs(x.var() - 1 / mu**2) < 4 * math.sqrt(8.0 / n) / mu**2
    assert stats.kstest(x - shift, "expon", args=(0, 1 / mu)).pvalue > 1e-4
    if kind == "exp":   # the shift is ignored for the plain exponential
        assert core.delay("exp", mu, 123.0, 11, 0, 0, 0) == x[0]


def test_delay_streams_are_keyed_by_replica_worker_seq_seed():
    base = core.delay("exp", 1.0, 0.0, 5, 1, 2, 3)
    assert base == core.delay("exp", 1.0, 0.0, 5, 1, 2, 3)
    others = {core.delay("exp", 1.0, 0.0, *k) for k in [(6, 1, 2, 3), (5, 0, 2, 3), (5, 1, 3, 3),
                                                        (5, 1, 2, 4), (5 + 2**32, 1, 2, 3)]}
    assert base not in others and len(others) == 5
    # the delay is -ln(u)/mu of words 0,1 of the block with counter (tag 0 | chunk 0, seq, worker, replica)
    x = py_philox([5, 0], [0, 3, 2, 1])
    assert base == core.neg_log_uniform(x[0], x[1]) / 1.0


def test_minibatch_indices_formula_and_uniformity():
    n, m = 1000, 37
    idx = core.minibatch_indices(9, 4, 2, 6, n, m)
    want = []
    for q in range(m):
        x = py_philox([9, 0], [(1 << 24) | (q // 4), 6, 2, 4])
        want.append((x[q % 4] * n) >> 32)
    assert idx.tolist() == want
    big = np.concatenate([core.minibatch_indices(9, r, w, s, 64, 128)
                          for r in range(10) for w in range(4) for s in range(25)])
    assert big.min() >= 0 and big.max() < 64
    cnt = np.bincount(big, minlength=64)
    chi2 = ((cnt - cnt.mean()) ** 2 / cnt.mean()).sum()
    assert chi2 < stats.chi2.ppf(0.9999, 63)
    # a prefix property: the first m' draws of a task do not depend on m
    assert core.minibatch_indices(9, 4, 2, 6, n, 8).tolist() == want[:8]


def test_pareto_delay_law():
    """Pareto(shape 2, scale x_m): P(X > x) = (x_m / x)^2, median x_m sqrt(2); X = x_m / sqrt(u)."""
    xm = 1.5
    x = np.array([core.delay("pareto2", 2.0, xm, 21, r, w, s) for r in range(30) for w in range(8) for s in range(400)])
    assert x.min() >= xm
    assert stats.kstest(x / xm, "pareto", args=(2.0,)).pvalue > 1e-4
    assert abs(np.median(x) - xm * math.sqrt(2.0)) < 0.02 * xm
    w = py_philox([21, 0], [0, 3, 2, 1])
    k = (w[0] << 20) | (w[1] >> 12)
    assert core.delay("pareto2", 2.0, xm, 21, 1, 2, 3) == xm / math.sqrt((2 * k + 1) / 2.0**53)
