"""Pins for the oracle's protocol steps against what the paper fixes:
key form (Sec. 4.2 item 2), ciphertext form and decryption (Sec. 3.2 items 3, 5),
Convert's correctness derivation (Eq. 3), additivity (the neighbour-sum step of Algorithm 2), the
noise condition (Sec. 4.2 discussion), and the rounding as a rational number."""
import numpy as np
import pytest

from oracle import d2mhe_oracle as orc
from oracle import definitions as defs
from paper_2207_04604_b200 import workloads as wl

from common import T, from_big, make_oracle, psi_t_for, q_of, small_moduli, to_big


def _int_negacyclic(a, b):
    """Product in Z[X]/(X^N+1) with int64 numpy (small operands)."""
    n = len(a)
    full = np.convolve(a.astype(np.int64), b.astype(np.int64))
    out = full[:n].copy()
    out[: n - 1] -= full[n:]
    return out


def _centred_int(poly_limbs, moduli):
    q = q_of(moduli)
    return [defs.centred(x, q) for x in to_big(poly_limbs, moduli)]


# ----------------------------------------------------------------------------------
# tiny ring: every step against the big-integer definitions
# ----------------------------------------------------------------------------------


@pytest.mark.parametrize("log2_n,bits,L,K", [(4, 30, 2, 3), (5, 36, 3, 4), (6, 54, 2, 2)])
def test_every_step_equals_big_integer_definition(log2_n, bits, L, K):
    moduli = small_moduli(log2_n, bits, L)
    q = q_of(moduli)
    o = make_oracle(log2_n, moduli, seed=42 + log2_n)
    n = o.n
    parties = list(range(K))
    s = [o.secret_share(k).astype(int).tolist() for k in parties]
    e = [o.pk_error(k).astype(int).tolist() for k in parties]
    p1 = to_big(o.common_p1(), moduli)
    # MBFV.PubKeyGen
    p0 = [0] * n
    for k in parties:
        share = defs.pk_share(p1, s[k], e[k], q)
        assert to_big(o.pk_share(k), moduli) == share
        p0 = defs.poly_add(p0, share, q)
    pk = o.collective_pk(parties)
    assert to_big(pk[0], moduli) == p0 and to_big(pk[1], moduli) == p1
    # Lambda
    assert [int(x) for x in o.delta()] == [(q // T) % m for m in moduli]
    # encode
    rng = np.random.default_rng(1)
    values = rng.integers(-3000, 3001, size=(K, 2, n)).astype(np.int32)
    plain = o.encode(values)
    psi_t = psi_t_for(log2_n)
    for k in range(K):
        for c in range(2):
            assert defs.decode_slots([int(x) for x in plain[k, c]], psi_t, T) == values[k, c].tolist()
    assert np.array_equal(o.decode(plain), values)
    # BFV.Encrypt
    ct = o.encrypt(pk, parties, 5, plain)
    for k in range(K):
        for c in range(2):
            u = o.sample_ternary(4, 5 + c, k).astype(int).tolist()
            e0 = o.sample_gauss(5, 5 + c, k).astype(int).tolist()
            e1 = o.sample_gauss(6, 5 + c, k).astype(int).tolist()
            c0, c1 = defs.bfv_encrypt(p0, p1, [int(x) for x in plain[k, c]], u, e0, e1, q, T)
            assert to_big(ct[k, c, 0], moduli) == c0 and to_big(ct[k, c, 1], moduli) == c1
    # BFV.Add over lists
    offsets = np.array([0, 2, K], dtype=np.uint32)
    rows = np.array([0, K - 1] + list(range(K - (K - 2), K)), dtype=np.uint32)
    agg = o.aggregate(ct, offsets, rows)
    for i in range(2):
        lst = rows[offsets[i]:offsets[i + 1]]
        for c in range(2):
            for comp in range(2):
                want = [0] * n
                for r in lst:
                    want = defs.poly_add(want, to_big(ct[r, c, comp], moduli), q)
                assert to_big(agg[i, c, comp], moduli) == want
    # decryption shares and combine
    recipients = [1, 0]
    shares = o.partial_decrypt(agg, recipients, parties, 5)
    got = o.combine(agg, shares)
    s_sum = [sum(s[k][j] for k in parties) for j in range(n)]
    for i in range(2):
        for c in range(2):
            c1 = to_big(agg[i, c, 1], moduli)
            hs = []
            for k in parties:
                ek = o.sample_gauss(7, 5 + c, k, recipient=recipients[i]).astype(int).tolist()
                h = defs.decryption_share(c1, s[k], ek, q)
                assert to_big(shares[i, k, c], moduli) == h
                hs.append(h)
            x = defs.combine(to_big(agg[i, c, 0], moduli), hs, q, T)
            assert got[i, c].tolist() == x
            # Eq. 3: the same plaintext as BFV.Decrypt under s = sum_k s_k (noise far below q/2t)
            assert defs.bfv_decrypt(to_big(agg[i, c, 0], moduli), c1, s_sum, q, T) == x
            assert o.decrypt_single(agg[i, c], np.array(s_sum)).tolist() == x
    # additivity: decoded aggregate = sum of the listed users' values
    dec = o.decode(got)
    for i in range(2):
        lst = rows[offsets[i]:offsets[i + 1]]
        assert np.array_equal(dec[i], values[lst].sum(axis=0))


# ----------------------------------------------------------------------------------
# configuration-1 size: identities that hold over the integers
# ----------------------------------------------------------------------------------


@pytest.fixture(scope="module")
def cfg1():
    cfg = wl.round_config(1)
    o = make_oracle(cfg.log2_n, cfg.moduli, seed=1)
    parties = list(range(cfg.num_parties))
    pk = o.collective_pk(parties)
    s = np.stack([o.secret_share(k).astype(np.int64) for k in parties])
    e = np.stack([o.pk_error(k).astype(np.int64) for k in parties])
    return cfg, o, parties, pk, s, e


def test_collective_pk_has_the_standard_form(cfg1):
    """p0 + p1 * sum s_k = -sum e_k exactly (Sec. 4.2 item 2)."""
    cfg, o, parties, pk, s, e = cfg1
    s_sum = s.sum(axis=0)
    for l, p in enumerate(cfg.moduli):
        sl = np.array([int(x) % p for x in s_sum], dtype=np.uint64)
        lhs = (orc.ring_mul(pk[1, l], sl, p).astype(object) + pk[0, l].astype(object)) % p
        want = np.array([(-int(x)) % p for x in e.sum(axis=0)], dtype=object)
        assert np.array_equal(lhs, want)
    assert np.abs(e.sum(axis=0)).max() <= cfg.num_parties * 19


def test_fresh_ciphertext_noise_is_exactly_the_predicted_polynomial(cfg1):
    """c0 + c1 s - Lambda m = -u * sum e_k + e0 + e1 * s over the integers (Sec. 3.2 items 3, 5)."""
    cfg, o, parties, pk, s, e = cfg1
    values = wl.gradients(cfg, seed=1)
    plain = o.encode(values)
    ct = o.encrypt(pk, parties, 0, plain)
    s_sum, e_sum = s.sum(axis=0), e.sum(axis=0)
    bound = 19 * (2 * cfg.n * cfg.num_parties + 1)
    for k in (0, 3):
        for c in (0, 1):
            got_plain, noise = o.decrypt_single(ct[k, c], s_sum, want_noise=True)
            assert np.array_equal(got_plain, plain[k, c])  # Dec(Enc(m)) = m under s = sum s_k
            u = o.sample_ternary(4, c, k).astype(np.int64)
            e0 = o.sample_gauss(5, c, k).astype(np.int64)
            e1 = o.sample_gauss(6, c, k).astype(np.int64)
            want = -_int_negacyclic(u, e_sum) + e0 + _int_negacyclic(e1, s_sum)
            assert np.array_equal(noise, want)
            assert np.abs(noise).max() <= bound


def test_round_trip_single_party_key_and_extreme_plaintexts():
    cfg = wl.round_config(1)
    o = make_oracle(cfg.log2_n, cfg.moduli, seed=9)
    n = o.n
    half = (T - 1) // 2
    values = np.stack([np.zeros(n), np.full(n, half), np.full(n, -half),
                       np.random.default_rng(2).integers(-half, half + 1, size=n)]).astype(np.int32)
    for parties in ([2], [0, 1, 2, 3]):
        pk = o.collective_pk(parties)
        plain = o.encode(values[None].repeat(1, axis=0).reshape(1, 4, n))
        ct = o.encrypt(pk, [parties[0]], 0, plain)
        shares = o.partial_decrypt(ct, [0], parties, 0)
        out = o.decode(o.combine(ct, shares))
        assert np.array_equal(out[0], values)


def test_collective_decryption_equals_single_key_and_sums_are_exact(cfg1):
    """Whole configuration-1 round: Eq. 3 and the additive homomorphism on every output."""
    cfg, o, parties, pk, s, e = cfg1
    offsets, rows = wl.regular_graph(cfg.num_parties, cfg.degree, seed=1)
    values = wl.gradients(cfg, seed=1)
    ct = o.encrypt(pk, parties, 0, o.encode(values))
    agg = o.aggregate(ct, offsets, rows)
    shares = o.partial_decrypt(agg, parties, parties, 0)
    plain = o.combine(agg, shares)
    dec = o.decode(plain)
    s_sum = s.sum(axis=0)
    q = q_of(cfg.moduli)
    A = cfg.degree + 1
    bound = A * 19 * (2 * cfg.n * cfg.num_parties + 1)
    for i in parties:
        lst = rows[offsets[i]:offsets[i + 1]]
        want = values[lst].astype(np.int64).sum(axis=0)
        assert np.abs(want).max() <= (T - 1) // 2
        assert np.array_equal(dec[i], want)
        for c in range(cfg.num_cts):
            single, noise = o.decrypt_single(agg[i, c], s_sum, want_noise=True)
            assert np.array_equal(single, plain[i, c])
            assert np.abs(noise).max() <= bound
            # the shares add sum_k e_{i,k,c}; the total must stay below q/2t (Sec. 4.2 item 3)
            assert bound + cfg.num_parties * 19 < q // (2 * T) - T


def test_a_wrong_share_breaks_decryption(cfg1):
    """Dropping one party's share (or using the wrong recipient's noise stream only) must not
    go unnoticed: without all shares the result is not the plaintext."""
    cfg, o, parties, pk, s, e = cfg1
    values = wl.gradients(cfg, seed=3)[:, :1]
    ct = o.encrypt(pk, parties, 0, o.encode(values))
    shares = o.partial_decrypt(ct, parties, parties, 0)
    good = o.decode(o.combine(ct, shares))
    assert np.array_equal(good, values)
    bad = o.decode(o.combine(ct, shares[:, :-1]))
    assert not np.array_equal(bad, values)


# ----------------------------------------------------------------------------------
# rounding and composition
# ----------------------------------------------------------------------------------


def test_scale_and_round_exhaustive_on_toy_moduli():
    moduli, t = [97, 193], 17
    o = orc.Oracle(4, moduli, t, seed=0)
    q = 97 * 193
    from fractions import Fraction
    for v in range(q):
        want = round(Fraction(t * v, q)) % t  # no ties: q odd
        assert o.scale_round_residues([v % 97, v % 193]) == want
        assert want == ((2 * t * v + q) // (2 * q)) % t


def test_scale_and_round_and_crt_against_python_integers():
    rng = np.random.default_rng(5)
    for moduli in ([97, 193, 257], wl.round_config(1).moduli, wl.round_config(2).moduli,
                   wl.round_config(3).moduli, wl.sweep_moduli(60, 24)):
        t = 17 if moduli[0] == 97 else T
        o = orc.Oracle(4, moduli, t, seed=0)
        q = q_of(moduli)
        specials = [0, 1, q - 1, q // 2, q // 2 + 1, q // t, q // t - 1, (q // t) * (t - 1)]
        for i in range(300):
            v = specials[i] if i < len(specials) else int.from_bytes(rng.bytes(200), "little") % q
            res = [v % m for m in moduli]
            assert defs.crt(res, moduli) == v
            assert o.crt_int(res) == v
            assert o.scale_round_residues(res) == ((2 * t * v + q) // (2 * q)) % t


def test_rounding_is_indifferent_to_the_representative():
    """[c0+c1 s]_q in [0,q) or in (-q/2, q/2] gives the same plaintext mod t."""
    moduli = wl.round_config(1).moduli
    q = q_of(moduli)
    rng = np.random.default_rng(8)
    for _ in range(200):
        v = int.from_bytes(rng.bytes(32), "little") % q
        a = ((2 * T * v + q) // (2 * q)) % T
        vc = defs.centred(v, q)
        b = ((2 * T * vc + q) // (2 * q)) % T
        assert a == b


def test_encode_decode_properties():
    log2_n = 12
    o = make_oracle(log2_n, wl.round_config(1).moduli, seed=0)
    rng = np.random.default_rng(4)
    half = (T - 1) // 2
    v = rng.integers(-half // 2, half // 2, size=(2, o.n)).astype(np.int32)
    m = o.encode(v)
    assert np.array_equal(o.decode(m), v)
    msum = ((m[0].astype(np.int64) + m[1]) % T).astype(np.uint32)
    assert np.array_equal(o.decode(msum), v[0] + v[1])
    psi_t = psi_t_for(log2_n)
    assert psi_t == 6561
    for j in (0, 1, 77, o.n - 1):
        y = orc.horner(m[0].astype(np.uint64), pow(psi_t, 2 * j + 1, T), T)
        assert (y - T if y > half else y) == v[0, j]
    # a constant vector packs to a constant polynomial
    const = o.encode(np.full(o.n, 5, dtype=np.int32))
    assert const[0] == 5 and not const[1:].any()


def test_slot_roots_quoted_for_each_degree():
    assert [psi_t_for(b) for b in (12, 13, 14, 15)] == [6561, 81, 9, 3]
