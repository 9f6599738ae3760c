"""Pins for the oracle's MBFV.Bootstrap (Sec. 4.2 item 4, Eq. 4): shares and the refreshed
ciphertext against the big-integer definitions; the refreshed ciphertext decrypts to the same
plaintext with exactly the fresh noise sum_k e_{1,k} - (q mod t) kappa."""
import numpy as np
import pytest

from oracle import d2mhe_oracle as orc
from oracle import definitions as defs
from paper_2207_04604_b200 import workloads as wl

from common import T, make_oracle, q_of, small_moduli, to_big


@pytest.mark.parametrize("log2_n,bits,L,K", [(4, 30, 2, 3), (5, 54, 2, 2)])
def test_shares_and_refresh_equal_big_integer_definitions(log2_n, bits, L, K):
    moduli = small_moduli(log2_n, bits, L)
    q = q_of(moduli)
    o = make_oracle(log2_n, moduli, seed=21)
    n = o.n
    parties = list(range(K))
    pk = o.collective_pk(parties)
    values = np.random.default_rng(1).integers(-2000, 2001, size=(K, 1, n)).astype(np.int32)
    ct = o.encrypt(pk, parties, 2, o.encode(values))
    agg = o.aggregate(ct, np.array([0, K], dtype=np.uint32), np.array(parties, dtype=np.uint32))
    rec = [1]
    shares = o.boot_share(agg, rec, parties, 2)
    alpha = o.boot_alpha(1, 2)
    # alpha and the masks follow the documented streams
    key = [21, 0]
    for l, p in enumerate(moduli):
        mask = (1 << int(p).bit_length()) - 1
        for j in (0, n - 1):
            att = 0
            while True:
                w = orc.philox4x32_10(key, [j, 2, l | (1 << 16), 14 | (att << 8)])
                r = ((w[0] << 32) | w[1]) & mask
                if r < p:
                    break
                att += 1
            assert int(alpha[l, j]) == r
    mk0 = o.boot_mask(0, 1, 2)
    assert mk0.max() < T
    for j in (0, 3):
        att = 0
        while True:
            w = orc.philox4x32_10(key, [j, 2, 0 | (1 << 16), 15 | (att << 8)])
            r = ((w[0] << 32) | w[1]) & ((1 << 17) - 1)
            if r < T:
                break
            att += 1
        assert int(mk0[j]) == r
    c1 = to_big(agg[0, 0, 1], moduli)
    al = to_big(alpha, moduli)
    e0s, e1s = [], []
    for k in parties:
        s_k = o.secret_share(k).astype(int).tolist()
        m_k = o.boot_mask(k, 1, 2).astype(int).tolist()
        e0 = o.sample_gauss(16, 2, k, recipient=1).astype(int).tolist()
        e1 = o.sample_gauss(17, 2, k, recipient=1).astype(int).tolist()
        eta0, eta1 = defs.bootstrap_share(c1, al, s_k, m_k, e0, e1, q, T)
        assert to_big(shares[0, k, 0, 0], moduli) == eta0
        assert to_big(shares[0, k, 0, 1], moduli) == eta1
        e0s.append(eta0)
        e1s.append(eta1)
    fresh = o.boot_combine(agg, shares, rec, 2)
    c0n, c1n = defs.bootstrap_combine(to_big(agg[0, 0, 0], moduli), e0s, e1s, al, q, T)
    assert to_big(fresh[0, 0, 0], moduli) == c0n and to_big(fresh[0, 0, 1], moduli) == c1n
    s_sum = np.stack([o.secret_share(k).astype(np.int64) for k in parties]).sum(axis=0)
    assert np.array_equal(o.decode(o.decrypt_single(fresh[0, 0], s_sum)[None])[0], values[:, 0].sum(axis=0))


def test_refreshed_ciphertext_has_exactly_the_fresh_noise():
    cfg = wl.round_config(1)
    o = make_oracle(cfg.log2_n, cfg.moduli, seed=6)
    K = cfg.num_parties
    parties = list(range(K))
    pk = o.collective_pk(parties)
    offsets, rows = wl.regular_graph(K, cfg.degree, 6)
    values = wl.gradients(cfg, 6)[:, :1]
    agg = o.aggregate(o.encrypt(pk, parties, 0, o.encode(values)), offsets, rows)
    rec = [0, 3]
    shares = o.boot_share(agg[rec], rec, parties, 0)
    fresh = o.boot_combine(agg[rec], shares, rec, 0)
    s_sum = np.stack([o.secret_share(k).astype(np.int64) for k in parties]).sum(axis=0)
    q = q_of(cfg.moduli)
    for a, i in enumerate(rec):
        before, noise_before = o.decrypt_single(agg[i, 0], s_sum, want_noise=True)
        after, noise_after = o.decrypt_single(fresh[a, 0], s_sum, want_noise=True)
        assert np.array_equal(before, after)  # same plaintext
        assert np.array_equal(fresh[a, 0, 1], o.boot_alpha(i, 0))
        e0 = sum(o.sample_gauss(16, 0, k, recipient=i).astype(np.int64) for k in parties)
        e1 = sum(o.sample_gauss(17, 0, k, recipient=i).astype(np.int64) for k in parties)
        msum = sum(o.boot_mask(k, i, 0).astype(np.int64) for k in parties)
        # x = (m - sum M_k) mod t is what the rounding step sees; x + sum M_k = m + t kappa
        x = (before.astype(np.int64) - msum) % T
        kappa = (x + msum - before.astype(np.int64)) // T
        assert np.array_equal(x + msum - before.astype(np.int64), kappa * T)
        assert np.array_equal(noise_after, e1 - (q % T) * kappa)
        # independent of how much noise the input carried: only the fresh errors and the wrap term remain
        assert np.abs(noise_after).max() <= K * 19 + (q % T) * K
        assert np.abs(noise_before + e0).max() < q // (2 * T) - T
