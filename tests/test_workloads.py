"""The parameter presets and synthetic inputs: primes, graph regularity, quantiser, shards."""
import numpy as np

from paper_2207_04604_b200 import workloads as wl

from common import T, q_of


def test_prime_rule_and_preset_values():
    c1, c2, c3 = (wl.round_config(i) for i in (1, 2, 3))
    assert c1.moduli == [0xFFFFEE001, 0xFFFFC4001, 0xFFFFBE001]
    assert c2.moduli == [0x3FFFFFFFEF8001, 0x3FFFFFFFEB8001, 0x3FFFFFFFE7C001, 0x3FFFFFFFE64001]
    assert c3.moduli[-1] == 0x3FFFFFFFAF8001 and len(c3.moduli) == 8
    assert wl.round_config(4).moduli == c3.moduli
    assert [q_of(c.moduli) % T for c in (c1, c2, c3)] == [9225, 10950, 4529]
    for cfg in (c1, c2, c3):
        for p in cfg.moduli:
            assert wl.is_prime(p) and p % (2 * cfg.n) == 1 and p.bit_length() == cfg.prime_bits
        assert len(set(cfg.moduli)) == len(cfg.moduli)
    sweep = wl.sweep_moduli(60, 24)
    assert sweep[0] == 0xFFFFFFFFFFC0001 and all(p % (1 << 17) == 1 and p < 2**60 for p in sweep)
    assert wl.sweep_moduli(50, 2) == [0x3FFFFFFD20001, 0x3FFFFFFB80001]
    # nothing was skipped: no prime = 1 mod 2N lies between consecutive entries
    for a, b in zip(c2.moduli, c2.moduli[1:]):
        assert not any(wl.is_prime(x) for x in range(b + 2 * c2.n, a, 2 * c2.n))


def test_ciphertext_counts():
    assert [wl.round_config(i).num_cts for i in (1, 2, 3, 4)] == [2, 13, 66, 683]
    assert [wl.round_config(i).clip for i in (1, 2, 3, 4)] == [8192, 3276, 1638, 655]


def test_graphs_are_regular_symmetric_and_closed():
    for k, d in ((4, 2), (10, 4), (20, 6), (50, 8)):
        offsets, rows = wl.regular_graph(k, d, seed=1)
        assert offsets[-1] == k * (d + 1)
        adj = np.zeros((k, k), dtype=int)
        for i in range(k):
            lst = rows[offsets[i]:offsets[i + 1]]
            assert list(lst) == sorted(set(lst)) and i in lst and len(lst) == d + 1
            adj[i, lst] = 1
        assert np.array_equal(adj, adj.T)
    o4, r4 = wl.regular_graph(4, 2, seed=1)
    assert r4.tolist() == [0, 1, 3, 0, 1, 2, 1, 2, 3, 0, 2, 3]
    a = wl.regular_graph(10, 4, seed=1)
    b = wl.regular_graph(10, 4, seed=1)
    assert np.array_equal(a[1], b[1])


def test_gradients_are_sliceable_clipped_and_padded():
    cfg = wl.round_config(2)
    full = wl.gradients(cfg, seed=1)
    assert full.shape == (10, 13, 8192) and full.dtype == np.int32
    part = wl.gradients(cfg, seed=1, ct_first=4, n_cts=3)
    assert np.array_equal(part, full[:, 4:7])
    assert np.abs(full).max() <= cfg.clip
    tail = cfg.params - 12 * cfg.n
    assert not full[:, 12, tail:].any() and full[:, 12, :tail].any()
    # K-fold sums cannot wrap mod t
    assert cfg.num_parties * cfg.clip <= (T - 1) // 2
    # quantiser: round-half-even at scale 2^10
    g = np.array([0.5 / 1024, 1.5 / 1024, -2.5 / 1024, 10.0], dtype=np.float32)
    assert wl.quantise(g, 100).tolist() == [0, 2, -2, 100]
    c1 = wl.gradients(wl.round_config(1), seed=1)
    assert c1.min() >= -4096 and c1.max() <= 4096 and c1.shape == (4, 2, 4096)


def test_shards_partition_the_index_space():
    world, per = 4, 13
    seen = []
    for r in range(world):
        first, n = wl.shard_ct_range(r, world, per)
        seen.extend(range(first, first + n))
    assert seen == list(range(world * per))
