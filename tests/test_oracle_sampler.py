"""Pins for the oracle's samplers: the cumulative table against an independent
exact computation of the truncated discrete Gaussian, and the empirical
distribution of samples against the exact probabilities."""
from decimal import Decimal, getcontext

import numpy as np

from oracle import d2mhe_oracle as orc
from oracle import dgauss

from common import make_oracle, small_moduli

B = 19


def _pmf_decimal():
    """Pr[x] = rho(x)/Z, rho(x) = exp(-x^2/(2 sigma^2)), sigma = 3.2, |x| <= 19 (100 digits)."""
    getcontext().prec = 100
    two_sigma2 = Decimal("2") * Decimal("3.2") * Decimal("3.2")
    rho = [(-(Decimal(x * x)) / two_sigma2).exp() for x in range(-B, B + 1)]
    z = sum(rho)
    return [r / z for r in rho], z


def test_table_matches_independent_high_precision_computation():
    probs, z = _pmf_decimal()
    # the constants quoted for this distribution: Z and the centre / tail masses
    assert abs(z - Decimal("8.0212104712195")) < Decimal("1e-12")
    assert abs(probs[B] - Decimal("0.12466946274")) < Decimal("1e-10")
    assert abs(probs[0] - Decimal("2.7572212246e-9")) < Decimal("1e-18")
    table = dgauss.thresholds()
    assert len(table) == 2 * B
    acc = Decimal(0)
    for k in range(2 * B):
        acc += probs[k]
        assert table[k] == int((acc * (Decimal(2) ** 64)).to_integral_value(rounding="ROUND_FLOOR"))
    assert all(a < b for a, b in zip(table, table[1:]))
    # what is left above the last threshold is the mass of +B
    assert abs(Decimal(2**64 - table[-1]) / Decimal(2**64) - probs[-1]) < Decimal("1e-18")
    # symmetry of the pmf shows in the table: T[k] + T[2B-1-k] = 2^64 up to flooring
    for k in range(2 * B):
        assert abs(table[k] + table[2 * B - 1 - k] - 2**64) <= 1


def test_inversion_rule_on_boundaries():
    o = make_oracle(4, small_moduli(4, 30, 1), seed=1)
    table = dgauss.thresholds()
    assert o.gauss_from_r(0) == -B
    assert o.gauss_from_r(2**64 - 1) == B
    for k, thr in enumerate(table):
        assert o.gauss_from_r(thr) == -B + k + 1
        assert o.gauss_from_r(thr - 1) == -B + k
    # the centre value 0 is returned exactly on [T[18], T[19])
    assert o.gauss_from_r(2**63) == 0


def test_ternary_rule():
    assert orc.lib().orc_ternary_from_word(0) == -1
    assert orc.lib().orc_ternary_from_word(0x55555555) == -1
    assert orc.lib().orc_ternary_from_word(0x55555556) == 0
    assert orc.lib().orc_ternary_from_word(0xAAAAAAAA) == 0
    assert orc.lib().orc_ternary_from_word(0xAAAAAAAB) == 1
    assert orc.lib().orc_ternary_from_word(0xFFFFFFFF) == 1


def test_sample_streams_follow_the_counter_layout():
    """sample j of a stream = rule(Philox(key=seed, ctr=(j, idx, party | recipient << 16, tag)))."""
    seed = 0x0123456789ABCDEF
    o = make_oracle(6, small_moduli(6, 30, 2), seed=seed)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    s = o.sample_ternary(4, idx=9, party=3)
    e = o.sample_gauss(7, idx=5, party=2, recipient=6)
    for j in range(o.n):
        w = orc.philox4x32_10(key, [j, 9, 3, 4])
        assert s[j] == ((w[0] * 3) >> 32) - 1
        w = orc.philox4x32_10(key, [j, 5, 2 | (6 << 16), 7])
        assert e[j] == o.gauss_from_r((w[0] << 32) | w[1])
    assert np.array_equal(o.secret_share(3), o.sample_ternary(1, 0, 3))
    assert np.array_equal(o.pk_error(3), o.sample_gauss(2, 0, 3))


def test_uniform_p1_layout_and_range():
    seed = 5
    moduli = small_moduli(6, 30, 2)
    o = make_oracle(6, moduli, seed=seed)
    p1 = o.common_p1()
    key = [seed, 0]
    for l, q in enumerate(moduli):
        mask = (1 << int(q).bit_length()) - 1
        for j in range(o.n):
            attempt = 0
            while True:
                w = orc.philox4x32_10(key, [j, l, 0, 3 | (attempt << 8)])
                r = ((w[0] << 32) | w[1]) & mask
                if r < q:
                    break
                attempt += 1
            assert int(p1[l, j]) == r


def test_empirical_distributions():
    """2^18 samples each: chi-square against the exact pmf, mean and variance."""
    o = make_oracle(14, small_moduli(14, 36, 1), seed=11)
    g = np.concatenate([o.sample_gauss(5, idx=c, party=1).astype(np.int64) for c in range(16)])
    t = np.concatenate([o.sample_ternary(4, idx=c, party=1).astype(np.int64) for c in range(16)])
    n = g.size
    assert g.min() >= -B and g.max() <= B
    probs, _ = _pmf_decimal()
    probs = np.array([float(p) for p in probs])
    counts = np.bincount(g + B, minlength=2 * B + 1).astype(float)
    keep = probs * n >= 5  # pool the far tails
    chi2 = ((counts[keep] - probs[keep] * n) ** 2 / (probs[keep] * n)).sum()
    tail_expected = probs[~keep].sum() * n
    chi2 += (counts[~keep].sum() - tail_expected) ** 2 / max(tail_expected, 1e-9)
    dof = keep.sum()
    assert chi2 < dof + 6 * np.sqrt(2 * dof)
    assert abs(g.mean()) < 6 * 3.2 / np.sqrt(n)
    assert abs(g.var() - 3.2**2) < 0.1  # truncation at 6 sigma loses < 1e-7 of the variance
    tc = np.bincount(t + 1, minlength=3) / t.size
    assert np.all(np.abs(tc - 1 / 3) < 6 * np.sqrt(2 / 9 / t.size))
