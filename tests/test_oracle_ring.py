"""Pins for the oracle's ring arithmetic: the transform-based product against the
schoolbook definition (C and pure-Python big integers), transform identities."""
import numpy as np
import pytest

from oracle import d2mhe_oracle as orc
from oracle import definitions as defs
from paper_2207_04604_b200 import workloads as wl

from common import small_moduli


def _rand(n, p, rng):
    return rng.integers(0, p, size=n, dtype=np.uint64)


@pytest.mark.parametrize("log2_n", [1, 2, 3, 4, 5, 6])
@pytest.mark.parametrize("bits", [30, 36, 54, 60])
def test_product_equals_schoolbook_definition(log2_n, bits):
    rng = np.random.default_rng(100 * log2_n + bits)
    n = 1 << log2_n
    for p in wl.ntt_primes(bits, 1 << 17, 3):
        a, b = _rand(n, p, rng), _rand(n, p, rng)
        want = defs.negacyclic_mul([int(x) for x in a], [int(x) for x in b], p)
        assert [int(x) for x in orc.negacyclic_schoolbook(a, b, p)] == want
        assert [int(x) for x in orc.ring_mul(a, b, p)] == want


def test_wraparound_sign():
    """X^(N-1) * X = X^N = -1."""
    p = small_moduli(4, 30, 1)[0]
    n = 16
    a = np.zeros(n, dtype=np.uint64)
    b = np.zeros(n, dtype=np.uint64)
    a[n - 1] = 1
    b[1] = 1
    c = orc.ring_mul(a, b, p)
    assert int(c[0]) == p - 1 and not c[1:].any()


def test_transform_is_evaluation_at_odd_powers():
    rng = np.random.default_rng(3)
    for log2_n in (3, 5, 6):
        n = 1 << log2_n
        p = small_moduli(log2_n, 54, 1)[0]
        psi = orc.find_psi(p, log2_n)
        assert pow(psi, n, p) == p - 1
        a = _rand(n, p, rng)
        ev = orc.negacyclic_eval(a, psi, p)
        for j in range(n):
            assert int(ev[j]) == defs.horner([int(x) for x in a], pow(psi, 2 * j + 1, p), p)
            assert int(ev[j]) == orc.horner(a, pow(psi, 2 * j + 1, p), p)
        assert np.array_equal(orc.negacyclic_interp(ev, psi, p), a)


@pytest.mark.parametrize("log2_n,bits", [(12, 36), (13, 54), (14, 54), (16, 60)])
def test_full_size_round_trip_linearity_shift_and_spot_products(log2_n, bits):
    rng = np.random.default_rng(log2_n)
    n = 1 << log2_n
    p = wl.ntt_primes(bits, 2 * n, 1)[0]
    psi = orc.find_psi(p, log2_n)
    a, b = _rand(n, p, rng), _rand(n, p, rng)
    fa, fb = orc.negacyclic_eval(a, psi, p), orc.negacyclic_eval(b, psi, p)
    assert np.array_equal(orc.negacyclic_interp(fa, psi, p), a)
    # linearity
    s = ((a.astype(object) + b.astype(object)) % p).astype(np.uint64)
    fs = orc.negacyclic_eval(s, psi, p)
    assert np.array_equal(fs, ((fa.astype(object) + fb.astype(object)) % p).astype(np.uint64))
    # multiplying by X multiplies value j by psi^(2j+1)
    xa = np.empty_like(a)
    xa[1:] = a[:-1]
    xa[0] = (p - int(a[-1])) % p
    fxa = orc.negacyclic_eval(xa, psi, p)
    for j in (0, 1, n // 2, n - 1):
        assert int(fxa[j]) == int(fa[j]) * pow(psi, 2 * j + 1, p) % p
    # a handful of coefficients of the product straight from the definition
    c = orc.ring_mul(a, b, p)
    for k in (0, 1, n // 3, n - 1):
        assert int(c[k]) == orc.negacyclic_coeff(a, b, p, k)
        want = 0
        for i in range(n):
            j = (k - i) % n
            term = int(a[i]) * int(b[j])
            want += term if i + j == k else -term
        assert int(c[k]) == want % p


def test_muladd_definition():
    moduli = wl.sweep_moduli(60, 3)
    o = orc.Oracle(5, moduli, 65537, seed=1)
    a, b, c = (wl.random_polys(moduli, 5, 2, s) for s in (1, 2, 3))
    d = o.poly_muladd(a, b, c)
    for r in range(2):
        for l, q in enumerate(moduli):
            for j in range(32):
                assert int(d[r, l, j]) == (int(a[r, l, j]) * int(b[r, l, j]) + int(c[r, l, j])) % q


@pytest.mark.parametrize("log2_n,bits,L,batch", [(4, 30, 2, 2), (6, 54, 3, 3), (12, 36, 3, 2), (13, 54, 4, 2)])
def test_batched_transform_row_to_limb_mapping(log2_n, bits, L, batch):
    """Row (b, l) of a batch goes with limb l's prime and root (the ring isomorphism behind every
    product of Sec. 3.2): values by Horner evaluation in Python integers at psi_l^(2j+1), inverse by
    round trip and by the single-polynomial interpolation.  The limbs have different primes and
    different roots, and every row holds different data, so that a wrong limb-of-row mapping, a
    swapped root or a flipped direction switch fails."""
    n = 1 << log2_n
    moduli = wl.ntt_primes(bits, 2 * n, L)
    assert len(set(moduli)) == L
    o = orc.Oracle(log2_n, moduli, 65537, seed=1)
    psi = [orc.find_psi(p, log2_n) for p in moduli]
    # a second, different set of roots for the same primes: the wrapper must use the ones it is given
    psi_alt = [pow(r, 3, p) for r, p in zip(psi, moduli)]
    polys = wl.random_polys(moduli, log2_n, batch, seed=7)
    assert polys.shape == (batch, L, n)
    for roots in (psi, psi_alt):
        fwd = o.ntt(polys, np.array(roots, dtype=np.uint64))
        sample = range(n) if n <= 64 else (0, 1, 2, n // 2 - 1, n // 2, n - 2, n - 1)
        for b in range(batch):
            for l, p in enumerate(moduli):
                coeffs = [int(x) for x in polys[b, l]]
                for j in sample:
                    assert int(fwd[b, l, j]) == defs.horner(coeffs, pow(roots[l], 2 * j + 1, p), p)
        back = o.ntt(fwd, np.array(roots, dtype=np.uint64), inverse=True)
        assert np.array_equal(back, polys)
        # the inverse switch on its own: interpolation of one row through the single-polynomial routine
        b, l = batch - 1, L - 1
        assert np.array_equal(back[b, l], orc.negacyclic_interp(fwd[b, l], roots[l], moduli[l]))
        assert not np.array_equal(fwd[b, l], polys[b, l])
    # rows of different limbs really differ in modulus: the same coefficients under two limbs give different values
    same = np.broadcast_to(polys[0, 0] % np.uint64(min(moduli)), (1, L, n)).copy()
    f = o.ntt(same, np.array(psi, dtype=np.uint64))
    assert not np.array_equal(f[0, 0], f[0, 1])
