"""Pins for the oracle's MBFV.Convert (Sec. 4.2 item 3): shares against the big-integer
definition of Eq. 2, the correctness derivation of Eq. 3 and its exact noise term
e_Covt = e_0 + sk_i e_1 + mu e_cl."""
import numpy as np
import pytest

from oracle import definitions as defs
from paper_2207_04604_b200 import workloads as wl

from common import T, make_oracle, q_of, small_moduli, to_big
from test_oracle_scheme import _int_negacyclic


@pytest.mark.parametrize("log2_n,bits,L,K", [(4, 30, 2, 3), (5, 54, 2, 2)])
def test_shares_and_user_keys_equal_big_integer_definitions(log2_n, bits, L, K):
    moduli = small_moduli(log2_n, bits, L)
    q = q_of(moduli)
    o = make_oracle(log2_n, moduli, seed=7)
    n = o.n
    parties = list(range(K))
    pk = o.collective_pk(parties)
    rng = np.random.default_rng(2)
    values = rng.integers(-2000, 2001, size=(K, 1, n)).astype(np.int32)
    ct = o.encrypt(pk, parties, 3, o.encode(values))
    recipients = [K - 1, 0]
    agg = o.aggregate(ct, np.array([0, K, K + 1], dtype=np.uint32), np.array(parties + [1], dtype=np.uint32))
    # user key pairs: pk_i = (-(sk_i p1_i + e_i), p1_i)
    pk_users = np.stack([o.user_pk(i) for i in recipients])
    for a, i in enumerate(recipients):
        sk = o.user_secret(i).astype(int).tolist()
        e = o.sample_gauss(9, 0, i).astype(int).tolist()
        p1 = to_big(pk_users[a, 1], moduli)
        assert to_big(pk_users[a, 0], moduli) == defs.pk_share(p1, sk, e, q)
        assert set(sk) <= {-1, 0, 1}
    shares = o.convert_share(agg, pk_users, recipients, parties, 3)
    for a, i in enumerate(recipients):
        c1 = to_big(agg[a, 0, 1], moduli)
        p0_i, p1_i = to_big(pk_users[a, 0], moduli), to_big(pk_users[a, 1], moduli)
        for k in parties:
            s_k = o.secret_share(k).astype(int).tolist()
            mu = o.sample_gauss(11, 3, k, recipient=i).astype(int).tolist()
            e0 = o.sample_gauss(12, 3, k, recipient=i).astype(int).tolist()
            e1 = o.sample_gauss(13, 3, k, recipient=i).astype(int).tolist()
            h0, h1 = defs.convert_share(c1, s_k, mu, e0, e1, p0_i, p1_i, q)
            assert to_big(shares[a, k, 0, 0], moduli) == h0
            assert to_big(shares[a, k, 0, 1], moduli) == h1
    conv = o.convert_combine(agg, shares)
    for a in range(2):
        want0 = to_big(agg[a, 0, 0], moduli)
        want1 = [0] * n
        for k in parties:
            want0 = defs.poly_add(want0, to_big(shares[a, k, 0, 0], moduli), q)
            want1 = defs.poly_add(want1, to_big(shares[a, k, 0, 1], moduli), q)
        assert to_big(conv[a, 0, 0], moduli) == want0 and to_big(conv[a, 0, 1], moduli) == want1
    # Eq. 3: the recipient decrypts with its own key
    secrets = np.stack([o.user_secret(i).astype(np.int32) for i in recipients])
    dec = o.decode(o.decrypt(conv, secrets))
    assert np.array_equal(dec[0, 0], values[:, 0].sum(axis=0))
    assert np.array_equal(dec[1, 0], values[1, 0])
    for a, i in enumerate(recipients):
        assert defs.bfv_decrypt(to_big(conv[a, 0, 0], moduli), to_big(conv[a, 0, 1], moduli),
                                secrets[a].tolist(), q, T) == o.decrypt(conv, secrets)[a, 0].tolist()


def test_conversion_noise_is_exactly_the_predicted_polynomial():
    """c0' + c1' sk_i - Lambda m = e_ct + e_0 + sk_i e_1 + mu e_cl over the integers (Eq. 3),
    with e_ct the noise under the collective key and e_cl = -e_i the error of pk_i."""
    cfg = wl.round_config(1)
    o = make_oracle(cfg.log2_n, cfg.moduli, seed=4)
    K = cfg.num_parties
    parties = list(range(K))
    pk = o.collective_pk(parties)
    offsets, rows = wl.regular_graph(K, cfg.degree, 4)
    values = wl.gradients(cfg, 4)[:, :1]
    ct = o.encrypt(pk, parties, 0, o.encode(values))
    agg = o.aggregate(ct, offsets, rows)
    recipients = [0, 2]
    pk_users = np.stack([o.user_pk(i) for i in recipients])
    shares = o.convert_share(agg[recipients], pk_users, recipients, parties, 0)
    conv = o.convert_combine(agg[recipients], shares)
    s_sum = np.stack([o.secret_share(k).astype(np.int64) for k in parties]).sum(axis=0)
    for a, i in enumerate(recipients):
        sk_i = o.user_secret(i).astype(np.int64)
        plain, e_ct = o.decrypt_single(agg[i, 0], s_sum, want_noise=True)       # under the collective key
        plain2, noise = o.decrypt_single(conv[a, 0], sk_i, want_noise=True)     # after conversion
        assert np.array_equal(plain, plain2)
        lst = rows[offsets[i]:offsets[i + 1]]
        assert np.array_equal(o.decode(plain2[None])[0], values[lst, 0].astype(np.int64).sum(axis=0))
        mu = sum(o.sample_gauss(11, 0, k, recipient=i).astype(np.int64) for k in parties)
        e0 = sum(o.sample_gauss(12, 0, k, recipient=i).astype(np.int64) for k in parties)
        e1 = sum(o.sample_gauss(13, 0, k, recipient=i).astype(np.int64) for k in parties)
        e_i = o.sample_gauss(9, 0, i).astype(np.int64)  # pk_i = (-(sk_i p1 + e_i), p1): p0 + sk_i p1 = -e_i
        want = e_ct + e0 + _int_negacyclic(sk_i, e1) - _int_negacyclic(mu, e_i)
        assert np.array_equal(noise, want)
        q = q_of(cfg.moduli)
        assert np.abs(noise).max() < q // (2 * T) - T  # the condition stated after Eq. 3
