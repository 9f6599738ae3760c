"""GPU parity: every output of the CUDA library against the CPU oracle, bit for bit,
through the C ABI (via the thin ctypes binding)."""
import numpy as np
import pytest
import torch

from paper_2207_04604_b200 import workloads as wl

from common import T, make_oracle, psi_t_for, small_moduli

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def d2():
    from paper_2207_04604_b200 import build, d2mhe

    build.build()
    assert torch.cuda.is_available()
    return d2mhe


def _brv(n_bits):
    n = 1 << n_bits
    idx = np.arange(n)
    out = np.zeros(n, dtype=np.int64)
    for b in range(n_bits):
        out |= ((idx >> b) & 1) << (n_bits - 1 - b)
    return out


# ----------------------------------------------------------------------------------
# transforms and multiply-add
# ----------------------------------------------------------------------------------


@pytest.mark.parametrize("log2_n,bits,L,batch", [
    (3, 30, 1, 2), (4, 36, 2, 3), (5, 54, 3, 2), (6, 60, 2, 5), (7, 50, 2, 2), (8, 54, 1, 3),
    (9, 60, 2, 2), (10, 36, 3, 2), (11, 54, 2, 2), (12, 36, 3, 5), (12, 60, 4, 3),
    (13, 54, 4, 3), (13, 60, 1, 7), (14, 54, 8, 2), (14, 60, 3, 3),
    (15, 60, 2, 2), (15, 50, 3, 1), (16, 60, 3, 2), (16, 54, 1, 3),
])
def test_ntt_forward_inverse_against_oracle(d2, log2_n, bits, L, batch):
    moduli = wl.ntt_primes(bits, 1 << 17, L) if bits >= 50 else small_moduli(log2_n, bits, L)
    ctx = d2.Context(log2_n, moduli, 2, seed=1)
    o = make_oracle(log2_n, moduli, seed=1)
    a = wl.random_polys(moduli, log2_n, batch, seed=log2_n)
    # edge values
    a[0, :, 0] = 0
    a[0, :, 1] = np.array(moduli, dtype=np.uint64) - 1
    psi = [ctx.get_root(l) for l in range(L)]
    for l, p in enumerate(moduli):
        assert pow(psi[l], 1 << log2_n, p) == p - 1
    dev = d2.from_u64_numpy(a, ctx.device)
    ctx.ntt_forward(dev, batch)
    got = d2.to_u64_numpy(dev)
    want = o.ntt(a, psi)  # natural order: value j = a(psi^(2j+1))
    perm = _brv(log2_n)
    assert np.array_equal(got, want[..., perm])  # position p holds value brv(p)
    ctx.ntt_inverse(dev, batch)
    ctx.sync()
    assert np.array_equal(d2.to_u64_numpy(dev), a)
    # inverse alone, from the oracle's transform
    dev2 = d2.from_u64_numpy(np.ascontiguousarray(want[..., perm]), ctx.device)
    ctx.ntt_inverse(dev2, batch)
    assert np.array_equal(d2.to_u64_numpy(dev2), a)
    ctx.close()


@pytest.mark.parametrize("log2_n,bits,L,batch", [(4, 36, 2, 3), (12, 60, 4, 3), (13, 54, 3, 2), (16, 60, 2, 1)])
def test_poly_muladd_against_oracle(d2, log2_n, bits, L, batch):
    moduli = wl.ntt_primes(bits, 2 << log2_n, L)
    ctx = d2.Context(log2_n, moduli, 2, seed=1)
    o = make_oracle(log2_n, moduli, seed=1)
    a, b, c = (wl.random_polys(moduli, log2_n, batch, seed=s) for s in (1, 2, 3))
    a[0, :, :4] = np.array(moduli, dtype=np.uint64)[:, None] - 1
    b[0, :, :2] = np.array(moduli, dtype=np.uint64)[:, None] - 1
    c[0, :, 0] = np.array(moduli, dtype=np.uint64) - 1
    da, db, dc = (d2.from_u64_numpy(x, ctx.device) for x in (a, b, c))
    dd = torch.empty_like(da)
    ctx.poly_muladd(da, db, dc, dd, batch)
    ctx.sync()
    assert np.array_equal(d2.to_u64_numpy(dd), o.poly_muladd(a, b, c))
    ctx.poly_muladd(da, db, dc, da, batch)  # aliasing d = a
    assert np.array_equal(d2.to_u64_numpy(da), o.poly_muladd(a, b, c))
    ctx.close()


# ----------------------------------------------------------------------------------
# 32-bit-word transforms and multiply-add (every prime below 2^30)
# ----------------------------------------------------------------------------------


@pytest.mark.parametrize("log2_n,bits,L,batch", [
    (3, 20, 1, 2), (4, 24, 2, 3), (6, 30, 2, 5), (9, 28, 3, 1), (10, 30, 3, 4), (11, 30, 2, 7),
    (12, 30, 4, 5), (12, 25, 1, 2), (13, 30, 3, 3), (13, 30, 8, 2), (14, 30, 2, 3), (14, 29, 3, 2),
])
def test_ntt32_forward_inverse_against_oracle(d2, log2_n, bits, L, batch):
    """Same definition as the 64-bit transforms; odd batches leave one polynomial without a partner."""
    moduli = wl.ntt_primes(bits, 2 << log2_n, L)
    assert max(moduli) < 1 << 30
    ctx = d2.Context(log2_n, moduli, 2, seed=1)
    o = make_oracle(log2_n, moduli, seed=1)
    a = wl.random_polys(moduli, log2_n, batch, seed=100 + log2_n)
    a[0, :, 0] = 0
    a[0, :, 1] = np.array(moduli, dtype=np.uint64) - 1
    a[-1, :, -1] = np.array(moduli, dtype=np.uint64) - 1
    psi = [ctx.get_root(l) for l in range(L)]
    want = o.ntt(a, psi)
    perm = _brv(log2_n)
    dev = d2.from_u32_numpy(a.astype(np.uint32), ctx.device)
    ctx.ntt32_forward(dev, batch)
    got = d2.to_u32_numpy(dev).astype(np.uint64)
    assert np.array_equal(got, want[..., perm])
    ctx.ntt32_inverse(dev, batch)
    ctx.sync()
    assert np.array_equal(d2.to_u32_numpy(dev).astype(np.uint64), a)
    dev2 = d2.from_u32_numpy(np.ascontiguousarray(want[..., perm]).astype(np.uint32), ctx.device)
    ctx.ntt32_inverse(dev2, batch)
    assert np.array_equal(d2.to_u32_numpy(dev2).astype(np.uint64), a)
    # the 64-bit calls on the same context and data agree
    dev64 = d2.from_u64_numpy(a, ctx.device)
    ctx.ntt_forward(dev64, batch)
    assert np.array_equal(d2.to_u64_numpy(dev64), want[..., perm])
    ctx.close()


@pytest.mark.parametrize("log2_n,bits,L,batch", [(4, 24, 2, 3), (12, 30, 4, 3), (14, 30, 3, 2), (16, 30, 2, 1)])
def test_poly_muladd32_against_oracle(d2, log2_n, bits, L, batch):
    moduli = wl.ntt_primes(bits, 2 << log2_n, L)
    ctx = d2.Context(log2_n, moduli, 2, seed=1)
    o = make_oracle(log2_n, moduli, seed=1)
    a, b, c = (wl.random_polys(moduli, log2_n, batch, seed=s) for s in (4, 5, 6))
    a[0, :, :4] = np.array(moduli, dtype=np.uint64)[:, None] - 1
    b[0, :, :2] = np.array(moduli, dtype=np.uint64)[:, None] - 1
    c[0, :, 0] = np.array(moduli, dtype=np.uint64) - 1
    da, db, dc = (d2.from_u32_numpy(x.astype(np.uint32), ctx.device) for x in (a, b, c))
    dd = torch.empty_like(da)
    ctx.poly_muladd32(da, db, dc, dd, batch)
    ctx.sync()
    assert np.array_equal(d2.to_u32_numpy(dd).astype(np.uint64), o.poly_muladd(a, b, c))
    ctx.close()


def test_32_bit_calls_refuse_wide_primes_and_large_rings(d2):
    wide = d2.Context(12, wl.ntt_primes(36, 1 << 13, 2), 2, seed=1)
    x = wide.empty_u32(1, 2, 4096)
    for call in (lambda: wide.ntt32_forward(x, 1), lambda: wide.ntt32_inverse(x, 1),
                 lambda: wide.poly_muladd32(x, x, x, x, 1)):
        with pytest.raises(d2.D2mheError) as e:
            call()
        assert e.value.status == d2.ERR_UNSUPPORTED
    wide.close()
    big = d2.Context(15, wl.ntt_primes(30, 1 << 16, 2), 2, seed=1)
    y = big.empty_u32(1, 2, 1 << 15)
    with pytest.raises(d2.D2mheError) as e:
        big.ntt32_forward(y, 1)
    assert e.value.status == d2.ERR_UNSUPPORTED
    big.poly_muladd32(y, y, y, y, 1)  # the multiply-add has no size limit
    big.sync()
    big.close()


@pytest.mark.parametrize("log2_n", [12, 13, 14, 15, 16])
def test_sweep_shapes_against_oracle(d2, log2_n):
    """Kernel-sweep shapes: every L of the sweep at this N (60-bit primes), small batch."""
    for L in wl.SWEEP_LIMBS:
        moduli = wl.sweep_moduli(60, L)
        ctx = d2.Context(log2_n, moduli, 1, seed=1)
        o = make_oracle(log2_n, moduli, seed=1)
        a = wl.random_polys(moduli, log2_n, 2, seed=L)
        psi = [ctx.get_root(l) for l in range(L)]
        dev = d2.from_u64_numpy(a, ctx.device)
        ctx.ntt_forward(dev, 2)
        perm = _brv(log2_n)
        assert np.array_equal(d2.to_u64_numpy(dev), o.ntt(a, psi)[..., perm])
        ctx.ntt_inverse(dev, 2)
        assert np.array_equal(d2.to_u64_numpy(dev), a)
        b, c = wl.random_polys(moduli, log2_n, 2, seed=50 + L), wl.random_polys(moduli, log2_n, 2, seed=90 + L)
        db, dc = d2.from_u64_numpy(b, ctx.device), d2.from_u64_numpy(c, ctx.device)
        ctx.poly_muladd(dev, db, dc, dev, 2)
        assert np.array_equal(d2.to_u64_numpy(dev), o.poly_muladd(a, b, c))
        ctx.close()


def test_large_batch_transform_sampled_polynomials(d2):
    """Batch 1024 x L 4 at N = 16384 and batch 256 at N = 65536: sampled polynomials against the oracle."""
    for log2_n, batch in ((14, 1024), (16, 256)):
        moduli = wl.sweep_moduli(50, 4)
        ctx = d2.Context(log2_n, moduli, 1, seed=1)
        o = make_oracle(log2_n, moduli, seed=1)
        a = wl.random_polys(moduli, log2_n, batch, seed=3)
        psi = [ctx.get_root(l) for l in range(4)]
        dev = d2.from_u64_numpy(a, ctx.device)
        ctx.ntt_forward(dev, batch)
        got = d2.to_u64_numpy(dev)
        perm = _brv(log2_n)
        for r in (0, 1, batch // 3, batch - 1):
            assert np.array_equal(got[r], o.ntt(a[r:r + 1], psi)[0][..., perm])
        ctx.ntt_inverse(dev, batch)
        assert np.array_equal(d2.to_u64_numpy(dev), a)
        ctx.close()


def test_ring_product_through_transforms_equals_schoolbook(d2):
    """INTT(NTT(a) . NTT(b)) = a*b in Z_p[X]/(X^N+1) for tiny N (definition by brute force)."""
    from oracle import d2mhe_oracle as orc

    for log2_n in (3, 4, 5, 6):
        moduli = small_moduli(log2_n, 54, 2)
        ctx = d2.Context(log2_n, moduli, 2, seed=1)
        a, b = (wl.random_polys(moduli, log2_n, 1, seed=s) for s in (5, 6))
        da, db = d2.from_u64_numpy(a, ctx.device), d2.from_u64_numpy(b, ctx.device)
        zero = torch.zeros_like(da)
        ctx.ntt_forward(da, 1)
        ctx.ntt_forward(db, 1)
        ctx.poly_muladd(da, db, zero, da, 1)
        ctx.ntt_inverse(da, 1)
        got = d2.to_u64_numpy(da)
        for l, p in enumerate(moduli):
            assert np.array_equal(got[0, l], orc.negacyclic_schoolbook(a[0, l], b[0, l], p))
        ctx.close()


# ----------------------------------------------------------------------------------
# packing
# ----------------------------------------------------------------------------------


@pytest.mark.parametrize("log2_n", [4, 6, 9, 12, 13, 14, 15])
def test_encode_decode_against_oracle(d2, log2_n):
    moduli = wl.ntt_primes(54, 2 << log2_n, 1)
    ctx = d2.Context(log2_n, moduli, 2, seed=1)
    o = make_oracle(log2_n, moduli, seed=1)
    assert ctx.get_plain_root() == psi_t_for(log2_n)
    n = 1 << log2_n
    rng = np.random.default_rng(log2_n)
    half = (T - 1) // 2
    vals = rng.integers(-half, half + 1, size=(3, n)).astype(np.int32)
    vals[0, :3] = [half, -half, 0]
    dv = torch.from_numpy(vals).to(ctx.device)
    dp = ctx.empty_u32(3, n)
    ctx.encode(dv, 3, dp)
    ctx.sync()
    want = o.encode(vals)
    assert np.array_equal(d2.to_u32_numpy(dp), want)
    back = torch.empty_like(dv)
    ctx.decode(dp, 3, back)
    assert np.array_equal(back.cpu().numpy(), vals)
    # decode of arbitrary plaintext polynomials
    m = rng.integers(0, T, size=(2, n)).astype(np.uint32)
    dm = d2.from_u32_numpy(m, ctx.device)
    out = torch.empty((2, n), dtype=torch.int32, device=ctx.device)
    ctx.decode(dm, 2, out)
    assert np.array_equal(out.cpu().numpy(), o.decode(m))
    # in place
    ctx.encode(dv, 3, dv)
    assert np.array_equal(d2.to_u32_numpy(dv), want)
    ctx.close()


def test_encode_flags_out_of_range_values(d2):
    ctx = d2.Context(12, wl.round_config(1).moduli, 2, seed=1)
    vals = torch.zeros((1, 4096), dtype=torch.int32, device=ctx.device)
    vals[0, 17] = (T - 1) // 2 + 1
    out = ctx.empty_u32(1, 4096)
    ctx.encode(vals, 1, out)
    with pytest.raises(d2.D2mheError) as e:
        ctx.sync()
    assert e.value.status == d2.ERR_RANGE
    ctx.sync()  # flag cleared
    ctx.close()


# ----------------------------------------------------------------------------------
# the protocol, step by step
# ----------------------------------------------------------------------------------


def _run_round(d2, ctx, o, cfg_k, parties, offsets, rows, values, ct_first, keep=None):
    """Runs every step on the GPU and on the oracle and compares all messages
    (keep, if given, receives the oracle's messages)."""
    n_cts = values.shape[1]
    K = len(parties)
    L, n = o.num_limbs, o.n
    dev = ctx.device
    # keys
    ctx.keygen_share(parties)
    pk = ctx.empty_u64(2, L, n)
    pk_shares = ctx.empty_u64(K, L, n)
    ctx.collective_pk(parties, pk_shares, pk)
    ctx.sync()
    for k in parties:
        assert np.array_equal(ctx.debug_export_secret(k), o.secret_share(k))
    want_pk = o.collective_pk(parties)
    assert np.array_equal(d2.to_u64_numpy(pk), want_pk)
    got_shares = d2.to_u64_numpy(pk_shares)
    for a, k in enumerate(parties):
        assert np.array_equal(got_shares[a], o.pk_share(k, want_pk[1]))
    # encode + encrypt
    dv = torch.from_numpy(values).to(dev)
    plain = ctx.empty_u32(K, n_cts, n)
    ctx.encode(dv, K * n_cts, plain)
    want_plain = o.encode(values)
    assert np.array_equal(d2.to_u32_numpy(plain), want_plain)
    ct = ctx.empty_u64(K, n_cts, 2, L, n)
    ctx.encrypt(parties, ct_first, n_cts, plain, ct)
    want_ct = o.encrypt(want_pk, parties, ct_first, want_plain)
    assert np.array_equal(d2.to_u64_numpy(ct), want_ct)
    # aggregate
    n_out = len(offsets) - 1
    agg = ctx.empty_u64(n_out, n_cts, 2, L, n)
    ctx.aggregate(ct, K, n_cts, offsets, rows, agg)
    want_agg = o.aggregate(want_ct, offsets, rows)
    assert np.array_equal(d2.to_u64_numpy(agg), want_agg)
    # shares
    recipients = [i % K for i in range(n_out)]
    shares = ctx.empty_u64(n_out, K, n_cts, L, n)
    ctx.partial_decrypt(agg, recipients, parties, ct_first, n_cts, shares)
    want_shares = o.partial_decrypt(want_agg, recipients, parties, ct_first)
    assert np.array_equal(d2.to_u64_numpy(shares), want_shares)
    # combine + decode
    out_plain = ctx.empty_u32(n_out, n_cts, n)
    ctx.combine_decrypt(agg, shares, n_out, K, n_cts, out_plain)
    want_out = o.combine(want_agg, want_shares)
    assert np.array_equal(d2.to_u32_numpy(out_plain), want_out)
    sums = torch.empty((n_out, n_cts, n), dtype=torch.int32, device=dev)
    ctx.decode(out_plain, n_out * n_cts, sums)
    ctx.sync()
    got = sums.cpu().numpy()
    assert np.array_equal(got, o.decode(want_out))
    for i in range(n_out):
        lst = rows[offsets[i]:offsets[i + 1]]
        assert np.array_equal(got[i], values[lst].astype(np.int64).sum(axis=0))
    if keep is not None:
        keep.update(ct=want_ct, agg=want_agg, shares=want_shares, sums=got)
    return got


@pytest.mark.parametrize("log2_n,bits,L,K", [(3, 36, 2, 3), (4, 30, 2, 3), (5, 36, 3, 4), (6, 54, 2, 2), (8, 60, 3, 3), (10, 54, 5, 3), (6, 56, 2, 3), (7, 57, 2, 2)])
def test_small_rings_every_message(d2, log2_n, bits, L, K):
    moduli = small_moduli(log2_n, bits, L)
    seed = 77 + log2_n
    ctx = d2.Context(log2_n, moduli, K, seed=seed)
    o = make_oracle(log2_n, moduli, seed=seed)
    parties = list(range(K))
    rng = np.random.default_rng(log2_n)
    values = rng.integers(-3000, 3001, size=(K, 3, 1 << log2_n)).astype(np.int32)
    # irregular lists, one of them empty
    offsets = np.array([0, K, K, K + 1], dtype=np.uint32)
    rows = np.array(list(range(K)) + [K - 1], dtype=np.uint32)
    _run_round(d2, ctx, o, K, parties, offsets, rows, values, ct_first=11)
    ctx.close()


@pytest.mark.parametrize("log2_n,bits,L,K,ct_first", [
    (5, 54, 1, 1, 0),             # one party, one limb: plain BFV
    (6, 60, 24, 2, 5),            # the maximum number of limbs, 60-bit primes
    (12, 54, 6, 3, 2**32 - 2),    # cluster of 6 limbs; ciphertext indices up to 2^32 - 1
    (11, 36, 7, 2, 1),            # 7 limbs: a prime cluster size
])
def test_degenerate_and_extreme_parameter_sets(d2, log2_n, bits, L, K, ct_first):
    moduli = wl.ntt_primes(bits, 1 << 17, L) if bits >= 50 else small_moduli(log2_n, bits, L)
    ctx = d2.Context(log2_n, moduli, K, seed=99)
    o = make_oracle(log2_n, moduli, seed=99)
    n = 1 << log2_n
    half = (T - 1) // 2 // K
    values = np.random.default_rng(1).integers(-half, half + 1, size=(K, 2, n)).astype(np.int32)
    values[0, 0, :2] = [half, -half]  # extreme slot values
    offsets = np.array([0, K], dtype=np.uint32)
    rows = np.arange(K, dtype=np.uint32)
    _run_round(d2, ctx, o, K, list(range(K)), offsets, rows, values, ct_first)
    ctx.close()


def _check_whole_round_call(d2, ctx, cfg, offsets, rows, values, want):
    """The same round in the launch configuration the benchmark times: one whole-round call with a
    workspace for all C indices (configuration 2: sub-chunks of 7 + 6 indices on two streams).
    Each part of the workspace is [plain | ciphertexts | aggregates | shares] of its sub-chunk; all
    of it must be the oracle's messages (`want`, from the step-by-step comparison)."""
    K, L, n, C = cfg.num_parties, cfg.num_limbs, cfg.n, cfg.num_cts
    sizes, lanes = d2.round_plan(C, C)
    assert len(sizes) == lanes and sum(sizes) == C  # one pass: every sub-chunk is still held afterwards
    ws = torch.empty(ctx.round_workspace_bytes(C), dtype=torch.uint8, device=ctx.device)
    sums = torch.zeros((K, C, n), dtype=torch.int32, device=ctx.device)
    ctx.round_device(torch.from_numpy(values).to(ctx.device), 0, C, offsets, rows, sums, ws)
    ctx.sync()
    assert np.array_equal(sums.cpu().numpy(), want["sums"])
    held = ws.cpu().numpy()
    per_ct = ctx.round_workspace_bytes(1) - 256
    first = 0
    for cc in sizes:
        part = held[first * per_ct:(first + cc) * per_ct]
        words = part[4 * K * cc * n:].view(np.uint64)
        n_ct, n_sh = K * cc * 2 * L * n, K * K * cc * L * n
        sl = slice(first, first + cc)
        assert np.array_equal(words[:n_ct].reshape(K, cc, 2, L, n), want["ct"][:, sl])
        assert np.array_equal(words[n_ct:2 * n_ct].reshape(K, cc, 2, L, n), want["agg"][:, sl])
        assert np.array_equal(words[2 * n_ct:2 * n_ct + n_sh].reshape(K, K, cc, L, n), want["shares"][:, :, sl])
        first += cc


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_config1_every_message(d2, seed):
    cfg = wl.round_config(1)
    ctx = d2.Context(cfg.log2_n, cfg.moduli, cfg.num_parties, seed=seed)
    o = make_oracle(cfg.log2_n, cfg.moduli, seed=seed)
    offsets, rows = wl.regular_graph(cfg.num_parties, cfg.degree, seed)
    values = wl.gradients(cfg, seed)
    want = {}
    _run_round(d2, ctx, o, cfg.num_parties, list(range(cfg.num_parties)), offsets, rows, values, 0, keep=want)
    _check_whole_round_call(d2, ctx, cfg, offsets, rows, values, want)
    ctx.close()


def test_config2_every_message(d2):
    cfg = wl.round_config(2)
    seed = 1
    ctx = d2.Context(cfg.log2_n, cfg.moduli, cfg.num_parties, seed=seed)
    o = make_oracle(cfg.log2_n, cfg.moduli, seed=seed)
    offsets, rows = wl.regular_graph(cfg.num_parties, cfg.degree, seed)
    values = wl.gradients(cfg, seed)
    want = {}
    _run_round(d2, ctx, o, cfg.num_parties, list(range(cfg.num_parties)), offsets, rows, values, 0, keep=want)
    assert d2.round_plan(cfg.num_cts, cfg.num_cts) == ([7, 6], 2)
    _check_whole_round_call(d2, ctx, cfg, offsets, rows, values, want)
    ctx.close()


@pytest.mark.parametrize("index,sample", [(3, [0, 65]), (4, [341, 682])])
def test_large_configs_on_sampled_ciphertext_indices(d2, index, sample):
    """Configurations 3 and 4 at full K, N, L on two ciphertext indices each (the last one
    holds the ragged, zero-padded tail): every message is addressable by its counters."""
    cfg = wl.round_config(index)
    seed = 1
    ctx = d2.Context(cfg.log2_n, cfg.moduli, cfg.num_parties, seed=seed)
    o = make_oracle(cfg.log2_n, cfg.moduli, seed=seed)
    offsets, rows = wl.regular_graph(cfg.num_parties, cfg.degree, seed)
    parties = list(range(cfg.num_parties))
    ctx.keygen_share(parties)
    pk = ctx.empty_u64(2, cfg.num_limbs, cfg.n)
    ctx.collective_pk(parties, None, pk)
    want_pk = o.collective_pk(parties)
    assert np.array_equal(d2.to_u64_numpy(pk), want_pk)
    K, L, n = cfg.num_parties, cfg.num_limbs, cfg.n
    for c in sample:
        values = wl.gradients(cfg, seed, ct_first=c, n_cts=1)
        dv = torch.from_numpy(values).to(ctx.device)
        plain = ctx.empty_u32(K, 1, n)
        ctx.encode(dv, K, plain)
        ct = ctx.empty_u64(K, 1, 2, L, n)
        ctx.encrypt(parties, c, 1, plain, ct)
        agg = ctx.empty_u64(K, 1, 2, L, n)
        ctx.aggregate(ct, K, 1, offsets, rows, agg)
        # shares for three recipients only (each needs all K share holders)
        rec = [0, K // 2, K - 1]
        agg_sel = agg[rec].contiguous()
        shares = ctx.empty_u64(len(rec), K, 1, L, n)
        ctx.partial_decrypt(agg_sel, rec, parties, c, 1, shares)
        out_plain = ctx.empty_u32(len(rec), 1, n)
        ctx.combine_decrypt(agg_sel, shares, len(rec), K, 1, out_plain)
        sums = torch.empty((len(rec), 1, n), dtype=torch.int32, device=ctx.device)
        ctx.decode(out_plain, len(rec), sums)
        ctx.sync()
        want_plain = o.encode(values)
        want_ct = o.encrypt(want_pk, parties, c, want_plain)
        assert np.array_equal(d2.to_u64_numpy(ct), want_ct)
        want_agg = o.aggregate(want_ct, offsets, rows)
        assert np.array_equal(d2.to_u64_numpy(agg), want_agg)
        want_shares = o.partial_decrypt(want_agg[rec], rec, parties, c)
        assert np.array_equal(d2.to_u64_numpy(shares), want_shares)
        want_out = o.combine(want_agg[rec], want_shares)
        assert np.array_equal(d2.to_u32_numpy(out_plain), want_out)
        got = sums.cpu().numpy()
        for a, i in enumerate(rec):
            lst = rows[offsets[i]:offsets[i + 1]]
            assert np.array_equal(got[a], values[lst].astype(np.int64).sum(axis=0))
    ctx.close()


def test_config3_every_message_of_every_index(d2):
    """Configuration 3 (K = 20, N = 16384, L = 8) on all 66 ciphertext indices, three at a time:
    plaintexts, ciphertexts, neighbour sums, all K x K decryption shares, decrypted plaintexts and
    decoded sums against the oracle.  The slow test of the suite (the oracle needs about a minute
    and a half for this workload on 16 cores)."""
    cfg = wl.round_config(3)
    seed = 1
    K, L, n, C = cfg.num_parties, cfg.num_limbs, cfg.n, cfg.num_cts
    ctx = d2.Context(cfg.log2_n, cfg.moduli, K, seed=seed)
    o = make_oracle(cfg.log2_n, cfg.moduli, seed=seed)
    offsets, rows = wl.regular_graph(K, cfg.degree, seed)
    parties = list(range(K))
    ctx.keygen_share(parties)
    pk = ctx.empty_u64(2, L, n)
    ctx.collective_pk(parties, None, pk)
    want_pk = o.collective_pk(parties)
    assert np.array_equal(d2.to_u64_numpy(pk), want_pk)
    step = 3
    for first in range(0, C, step):
        cc = min(step, C - first)
        values = wl.gradients(cfg, seed, ct_first=first, n_cts=cc)
        dv = torch.from_numpy(values).to(ctx.device)
        plain = ctx.empty_u32(K, cc, n)
        ctx.encode(dv, K * cc, plain)
        ct = ctx.empty_u64(K, cc, 2, L, n)
        ctx.encrypt(parties, first, cc, plain, ct)
        agg = ctx.empty_u64(K, cc, 2, L, n)
        ctx.aggregate(ct, K, cc, offsets, rows, agg)
        shares = ctx.empty_u64(K, K, cc, L, n)
        ctx.partial_decrypt(agg, parties, parties, first, cc, shares)
        out_plain = ctx.empty_u32(K, cc, n)
        ctx.combine_decrypt(agg, shares, K, K, cc, out_plain)
        sums = torch.empty((K, cc, n), dtype=torch.int32, device=ctx.device)
        ctx.decode(out_plain, K * cc, sums)
        ctx.sync()
        want_plain = o.encode(values)
        assert np.array_equal(d2.to_u32_numpy(plain), want_plain)
        want_ct = o.encrypt(want_pk, parties, first, want_plain)
        assert np.array_equal(d2.to_u64_numpy(ct), want_ct)
        del ct
        want_agg = o.aggregate(want_ct, offsets, rows)
        del want_ct
        assert np.array_equal(d2.to_u64_numpy(agg), want_agg)
        want_shares = o.partial_decrypt(want_agg, parties, parties, first)
        assert np.array_equal(d2.to_u64_numpy(shares), want_shares)
        del shares
        want_out = o.combine(want_agg, want_shares)
        del want_shares, want_agg
        assert np.array_equal(d2.to_u32_numpy(out_plain), want_out)
        got = sums.cpu().numpy()
        assert np.array_equal(got, o.decode(want_out))
        for i in range(K):
            lst = rows[offsets[i]:offsets[i + 1]]
            assert np.array_equal(got[i], values[lst].astype(np.int64).sum(axis=0))
    ctx.close()


@pytest.mark.parametrize("index", [3, 4])
def test_whole_round_at_full_size_in_the_benchmark_configuration(d2, index):
    """Configurations 3 and 4 at full K, N, L and all C ciphertext indices through one whole-round call,
    cut as the benchmark cuts it (workspace sized from free memory, sub-chunks on two streams).
    Every index carries the workload's gradients.
    Every decrypted sum is checked against the plaintext neighbour sum; for the last ciphertext index
    (the ragged tail), whose sub-chunk is still in the workspace when the call returns, the
    ciphertexts, aggregates and the shares for three recipients are compared with the oracle."""
    cfg = wl.round_config(index)
    seed = 1
    K, L, n, C = cfg.num_parties, cfg.num_limbs, cfg.n, cfg.num_cts
    ctx = d2.Context(cfg.log2_n, cfg.moduli, K, seed=seed)
    dev = ctx.device
    parties = list(range(K))
    ctx.keygen_share(parties)
    ctx.collective_pk(parties)
    offsets, rows = wl.regular_graph(K, cfg.degree, seed)
    # inputs: the workload's gradients on every index (clipped Gaussian, zero-padded ragged tail)
    last = C - 1
    values = torch.from_numpy(wl.gradients(cfg, seed))
    tail = values[:, last:last + 1].numpy()
    dv = values.to(dev)
    free_b, _ = torch.cuda.mem_get_info(dev)
    per_ct = ctx.round_workspace_bytes(1) - 256
    cap = int(max(1, min(C, int(free_b * 0.35) // per_ct)))
    sizes, lanes = d2.round_plan(C, cap)
    assert lanes == 2 and sum(sizes) == C
    ws = torch.empty(ctx.round_workspace_bytes(cap), dtype=torch.uint8, device=dev)
    sums = torch.zeros((K, C, n), dtype=torch.int32, device=dev)
    ctx.round_device(dv, 0, C, offsets, rows, sums, ws)
    ctx.sync()
    for i in range(K):
        lst = torch.as_tensor(rows[offsets[i]:offsets[i + 1]].astype(np.int64), device=dev)
        assert torch.equal(sums[i], dv[lst].sum(dim=0, dtype=torch.int32))
    # where the last sub-chunk lives: stream (len - 1) mod lanes, whose part starts after the first
    # sub-chunks of the streams before it
    i_last = len(sizes) - 1
    lane, cc = i_last % lanes, sizes[i_last]
    base = sum(sizes[:lane]) * per_ct + 4 * K * cc * n
    n_ct, n_sh = K * cc * 2 * L * n, K * K * cc * L * n
    words = ws[base:base + 8 * (2 * n_ct + n_sh)].view(torch.int64)
    ct = words[:n_ct].view(K, cc, 2, L, n)[:, cc - 1]
    agg = words[n_ct:2 * n_ct].view(K, cc, 2, L, n)[:, cc - 1]
    rec = [0, K // 2, K - 1]
    shares = words[2 * n_ct:].view(K, K, cc, L, n)[rec][:, :, cc - 1]
    o = make_oracle(cfg.log2_n, cfg.moduli, seed=seed)
    want_pk = o.collective_pk(parties)
    want_ct = o.encrypt(want_pk, parties, last, o.encode(tail))
    assert np.array_equal(d2.to_u64_numpy(ct.contiguous()), want_ct[:, 0])
    want_agg = o.aggregate(want_ct, offsets, rows)
    assert np.array_equal(d2.to_u64_numpy(agg.contiguous()), want_agg[:, 0])
    want_shares = o.partial_decrypt(want_agg[rec], rec, parties, last)
    assert np.array_equal(d2.to_u64_numpy(shares.contiguous()), want_shares[:, :, 0])
    ctx.close()


# ----------------------------------------------------------------------------------
# conversion to the recipient's own key (MBFV.Convert) and decryption under it
# ----------------------------------------------------------------------------------


@pytest.mark.parametrize("log2_n,moduli_spec,K,n_cts", [
    (4, (30, 2), 3, 2), (6, (54, 3), 2, 1), (9, (60, 2), 3, 2), (12, None, 4, 2), (13, (54, 4), 3, 1), (14, (54, 5), 2, 1),
])
def test_convert_every_message(d2, log2_n, moduli_spec, K, n_cts):
    if moduli_spec is None:
        moduli = wl.round_config(1).moduli
    else:
        moduli = small_moduli(log2_n, *moduli_spec)
    seed = 31 + log2_n
    L, n = len(moduli), 1 << log2_n
    ctx = d2.Context(log2_n, moduli, K, seed=seed)
    o = make_oracle(log2_n, moduli, seed=seed)
    parties = list(range(K))
    ctx.keygen_share(parties)
    ctx.collective_pk(parties)
    pk = o.collective_pk(parties)
    rng = np.random.default_rng(seed)
    values = rng.integers(-4000, 4001, size=(K, n_cts, n)).astype(np.int32)
    offsets = np.array([0, K, K + 1], dtype=np.uint32)
    rows = np.array(parties + [0], dtype=np.uint32)
    want_ct = o.encrypt(pk, parties, 7, o.encode(values))
    want_agg = o.aggregate(want_ct, offsets, rows)
    agg = d2.from_u64_numpy(want_agg, ctx.device)
    recipients = [K - 1, 0]
    # own key pairs
    pk_users = ctx.empty_u64(2, 2, L, n)
    ctx.user_keygen(recipients, pk_users)
    ctx.sync()
    want_pk_users = np.stack([o.user_pk(i) for i in recipients])
    assert np.array_equal(d2.to_u64_numpy(pk_users), want_pk_users)
    for i in recipients:
        assert np.array_equal(ctx.debug_export_user_secret(i), o.user_secret(i))
    # shares
    shares = ctx.empty_u64(2, K, n_cts, 2, L, n)
    ctx.convert_share(agg, recipients, parties, 7, n_cts, shares)
    want_shares = o.convert_share(want_agg, want_pk_users, recipients, parties, 7)
    assert np.array_equal(d2.to_u64_numpy(shares), want_shares)
    # combination
    conv = ctx.empty_u64(2, n_cts, 2, L, n)
    ctx.convert_combine(agg, shares, 2, K, n_cts, conv)
    want_conv = o.convert_combine(want_agg, want_shares)
    assert np.array_equal(d2.to_u64_numpy(conv), want_conv)
    # decryption under the recipients' own keys
    scratch = ctx.empty_u64(2, n_cts, L, n)
    plain = ctx.empty_u32(2, n_cts, n)
    ctx.decrypt(recipients, conv, n_cts, scratch, plain)
    secrets = np.stack([o.user_secret(i).astype(np.int32) for i in recipients])
    want_plain = o.decrypt(want_conv, secrets)
    assert np.array_equal(d2.to_u32_numpy(plain), want_plain)
    sums = torch.empty((2, n_cts, n), dtype=torch.int32, device=ctx.device)
    ctx.decode(plain, 2 * n_cts, sums)
    ctx.sync()
    got = sums.cpu().numpy()
    assert np.array_equal(got[0], values.astype(np.int64).sum(axis=0))
    assert np.array_equal(got[1], values[0])
    # a recipient without an own key pair is refused
    if K > 2:
        with pytest.raises(d2.D2mheError) as e:
            ctx.convert_share(agg, [1, 0], parties, 7, n_cts, shares)
        assert e.value.status == d2.ERR_STATE
    ctx.close()


@pytest.mark.parametrize("log2_n,moduli_spec,K,n_cts", [
    (4, (30, 2), 3, 2), (7, (54, 3), 2, 1), (12, None, 4, 2), (13, (54, 4), 3, 1), (14, (60, 2), 2, 1),
])
def test_bootstrap_every_message(d2, log2_n, moduli_spec, K, n_cts):
    """MBFV.Bootstrap: shares, refreshed ciphertext, and that the refreshed ciphertext goes through
    the ordinary collective decryption to the same sums."""
    moduli = wl.round_config(1).moduli if moduli_spec is None else small_moduli(log2_n, *moduli_spec)
    seed = 51 + log2_n
    L, n = len(moduli), 1 << log2_n
    ctx = d2.Context(log2_n, moduli, K, seed=seed)
    o = make_oracle(log2_n, moduli, seed=seed)
    parties = list(range(K))
    ctx.keygen_share(parties)
    ctx.collective_pk(parties)
    pk = o.collective_pk(parties)
    values = np.random.default_rng(seed).integers(-4000, 4001, size=(K, n_cts, n)).astype(np.int32)
    offsets = np.array([0, K, K + 1], dtype=np.uint32)
    rows = np.array(parties + [K - 1], dtype=np.uint32)
    want_agg = o.aggregate(o.encrypt(pk, parties, 9, o.encode(values)), offsets, rows)
    agg = d2.from_u64_numpy(want_agg, ctx.device)
    recipients = [1, 0]
    shares = ctx.empty_u64(2, K, n_cts, 2, L, n)
    ctx.bootstrap_share(agg, recipients, parties, 9, n_cts, shares)
    want_shares = o.boot_share(want_agg, recipients, parties, 9)
    assert np.array_equal(d2.to_u64_numpy(shares), want_shares)
    fresh = ctx.empty_u64(2, n_cts, 2, L, n)
    scratch = ctx.empty_u32(2, n_cts, n)
    ctx.bootstrap_combine(agg, shares, recipients, K, 9, n_cts, scratch, fresh)
    want_fresh = o.boot_combine(want_agg, want_shares, recipients, 9)
    assert np.array_equal(d2.to_u64_numpy(fresh), want_fresh)
    # the refreshed ciphertexts decrypt collectively to the same sums
    dshares = ctx.empty_u64(2, K, n_cts, L, n)
    ctx.partial_decrypt(fresh, recipients, parties, 9, n_cts, dshares)
    plain = ctx.empty_u32(2, n_cts, n)
    ctx.combine_decrypt(fresh, dshares, 2, K, n_cts, plain)
    sums = torch.empty((2, n_cts, n), dtype=torch.int32, device=ctx.device)
    ctx.decode(plain, 2 * n_cts, sums)
    ctx.sync()
    got = sums.cpu().numpy()
    assert np.array_equal(got[0], values.astype(np.int64).sum(axis=0))
    assert np.array_equal(got[1], values[K - 1])
    ctx.close()


def test_private_dpsgd_equals_plaintext_dpsgd(d2):
    """Algorithm 2 on synthetic quadratic objectives L_i(W) = |W - a_i|^2 / 2: the encrypted loop gives
    bit for bit what plaintext D-PSGD gives on the same fixed-point values, and it converges."""
    from paper_2207_04604_b200 import dpsgd

    K, H, lr = 6, 10000, 0.5
    moduli = wl.round_config(1).moduli
    ctx = d2.Context(12, moduli, K, seed=8)
    parties = list(range(K))
    ctx.keygen_share(parties)
    ctx.collective_pk(parties)
    offsets, rows = wl.regular_graph(K, 2, 8)
    rng = np.random.default_rng(8)
    targets = rng.uniform(-1.0, 1.0, size=(K, H))
    w_enc = np.zeros((K, H))
    w_ref = np.zeros((K, H))
    loop = dpsgd.PrivateDPSGD(ctx, offsets, rows, H, chunk_cts=2)
    assert loop.C == 3
    losses = []
    for _ in range(6):
        w_enc = loop.step(w_enc, w_enc - targets, lr)
        w_ref = dpsgd.plaintext_mix(w_ref, offsets, rows, loop.clip) - lr * (w_ref - targets)
        assert np.array_equal(w_enc, w_ref)
        losses.append(float(((w_enc.mean(axis=0) - targets.mean(axis=0)) ** 2).mean()))
    assert losses[-1] < 0.05 * losses[0]
    ctx.close()


def test_per_neighbourhood_keys(d2):
    """The literal reading of Sec. 4.2 item 1: one collective key per closed neighbourhood U_i, shares
    only from U_i.  Expressed with the same calls by passing the neighbourhood as the party set."""
    cfg = wl.round_config(1)
    K, L, n = cfg.num_parties, cfg.num_limbs, cfg.n
    seed = 12
    ctx = d2.Context(cfg.log2_n, cfg.moduli, K, seed=seed)
    o = make_oracle(cfg.log2_n, cfg.moduli, seed=seed)
    offsets, rows = wl.regular_graph(K, cfg.degree, seed)
    values = wl.gradients(cfg, seed)[:, :1]
    ctx.keygen_share(list(range(K)))
    dv = torch.from_numpy(values).to(ctx.device)
    plain = ctx.empty_u32(K, 1, n)
    ctx.encode(dv, K, plain)
    for i in range(K):
        U = [int(x) for x in rows[offsets[i]:offsets[i + 1]]]
        S = len(U)
        pk = ctx.empty_u64(2, L, n)
        ctx.collective_pk(U, None, pk)  # key of this neighbourhood: s = sum_{k in U_i} s_k
        want_pk = o.collective_pk(U)
        assert np.array_equal(d2.to_u64_numpy(pk), want_pk)
        ct = ctx.empty_u64(S, 1, 2, L, n)
        ctx.encrypt(U, 0, 1, plain[U].contiguous(), ct)
        agg = ctx.empty_u64(1, 1, 2, L, n)
        ctx.aggregate(ct, S, 1, [0, S], list(range(S)), agg)
        shares = ctx.empty_u64(1, S, 1, L, n)
        ctx.partial_decrypt(agg, [i], U, 0, 1, shares)
        out = ctx.empty_u32(1, 1, n)
        ctx.combine_decrypt(agg, shares, 1, S, 1, out)
        sums = torch.empty((1, 1, n), dtype=torch.int32, device=ctx.device)
        ctx.decode(out, 1, sums)
        ctx.sync()
        assert np.array_equal(sums.cpu().numpy()[0, 0], values[U, 0].astype(np.int64).sum(axis=0))
        want_ct = o.encrypt(want_pk, U, 0, o.encode(values[U]))
        assert np.array_equal(d2.to_u64_numpy(ct), want_ct)
    ctx.close()


# ----------------------------------------------------------------------------------
# whole-round driver, chunking, determinism, error paths
# ----------------------------------------------------------------------------------


def test_round_driver_matches_stepwise_and_plain_sums(d2):
    cfg = wl.round_config(2)
    seed = 2
    K, n, C = cfg.num_parties, cfg.n, cfg.num_cts
    ctx = d2.Context(cfg.log2_n, cfg.moduli, K, seed=seed)
    parties = list(range(K))
    ctx.keygen_share(parties)
    ctx.collective_pk(parties)
    offsets, rows = wl.regular_graph(K, cfg.degree, seed)
    values = wl.gradients(cfg, seed)
    want = np.stack([values[rows[offsets[i]:offsets[i + 1]]].astype(np.int64).sum(axis=0) for i in range(K)])
    dv = torch.from_numpy(values).to(ctx.device)
    for chunk in (1, 2, 5, C, C + 3):
        ws = torch.empty(ctx.round_workspace_bytes(chunk), dtype=torch.uint8, device=ctx.device)
        sums = torch.zeros((K, C, n), dtype=torch.int32, device=ctx.device)
        ctx.round_device(dv, 0, C, offsets, rows, sums, ws)
        ctx.sync()
        assert np.array_equal(sums.cpu().numpy(), want)
    # The messages themselves, not only the sums: a workspace for three indices makes twelve
    # sub-chunks (2, 1, 1, ... indices) that alternate over two parts of it, the first two indices
    # wide, so that at the end the parts hold indices 11 (at offset 0) and 12 (at offset two), each as
    # [plain | ciphertexts | aggregates | shares | noise bytes].  They must be the messages the
    # step-by-step calls produce for those indices.
    L = cfg.num_limbs
    ws = torch.empty(ctx.round_workspace_bytes(3), dtype=torch.uint8, device=ctx.device)
    sums = torch.zeros((K, C, n), dtype=torch.int32, device=ctx.device)
    ctx.round_device(dv, 0, C, offsets, rows, sums, ws)
    ctx.sync()
    assert np.array_equal(sums.cpu().numpy(), want)
    per_ct = ctx.round_workspace_bytes(1) - 256
    ct_words, share_words = K * 2 * L * n, K * K * L * n
    assert per_ct == 4 * K * n + 8 * (2 * ct_words + share_words) + max(K * K, 3 * K) * n  # the last term: one byte per sample drawn ahead of a kernel
    held = ws.cpu().numpy()
    assert d2.round_plan(C, 3) == ([2] + [1] * 11, 2)
    for part, index in ((0, 11), (2, 12)):
        plain = ctx.empty_u32(K, 1, n)
        ct = ctx.empty_u64(K, 1, 2, L, n)
        agg = ctx.empty_u64(K, 1, 2, L, n)
        shares = ctx.empty_u64(K, K, 1, L, n)
        ctx.encode(dv[:, index:index + 1].contiguous(), K, plain)
        ctx.encrypt(parties, index, 1, plain, ct)
        ctx.aggregate(ct, K, 1, offsets, rows, agg)
        ctx.partial_decrypt(agg, parties, parties, index, 1, shares)
        ctx.sync()
        words = held[part * per_ct + 4 * K * n:(part + 1) * per_ct].view(np.uint64)
        assert np.array_equal(words[:ct_words], d2.to_u64_numpy(ct).ravel())
        assert np.array_equal(words[ct_words:2 * ct_words], d2.to_u64_numpy(agg).ravel())
        assert np.array_equal(words[2 * ct_words:2 * ct_words + share_words], d2.to_u64_numpy(shares).ravel())
    # host variant, pinned buffers
    hv = torch.from_numpy(values).pin_memory()
    hs = torch.zeros((K, C, n), dtype=torch.int32).pin_memory()
    ws = torch.empty(ctx.round_workspace_bytes(4), dtype=torch.uint8, device=ctx.device)
    ctx.round_host(hv, 0, C, offsets, rows, hs, ws)
    assert np.array_equal(hs.numpy(), want)
    # too small a workspace is refused
    tiny = torch.empty(1024, dtype=torch.uint8, device=ctx.device)
    with pytest.raises(d2.D2mheError) as e:
        ctx.round_device(dv, 0, C, offsets, rows, sums, tiny)
    assert e.value.status == d2.ERR_WORKSPACE
    ctx.close()


def test_round_calls_follow_changed_index_lists(d2):
    """The whole-round calls keep their index lists on the device between calls; a call with other
    neighbour lists, or after another collective key, must use the new ones."""
    cfg = wl.round_config(1)
    K, n = cfg.num_parties, cfg.n
    ctx = d2.Context(cfg.log2_n, cfg.moduli, K, seed=8)
    ctx.keygen_share(list(range(K)))
    ctx.collective_pk(list(range(K)))
    values = wl.gradients(cfg, 8, 0, 5)
    dv = torch.from_numpy(values).to(ctx.device)
    ws = torch.empty(ctx.round_workspace_bytes(5), dtype=torch.uint8, device=ctx.device)
    ring = wl.regular_graph(K, 2, 8)
    full = (np.arange(0, K * K + 1, K, dtype=np.uint32), np.tile(np.arange(K, dtype=np.uint32), K))
    lone = (np.arange(K + 1, dtype=np.uint32), np.arange(K, dtype=np.uint32))  # every user alone
    for offsets, rows in (ring, full, ring, lone, full):
        sums = torch.full((K, 5, n), -1, dtype=torch.int32, device=ctx.device)
        ctx.round_device(dv, 2, 5, offsets, rows, sums, ws)
        ctx.sync()
        want = np.stack([values[rows[offsets[i]:offsets[i + 1]]].astype(np.int64).sum(axis=0) for i in range(K)])
        assert np.array_equal(sums.cpu().numpy(), want)
    # a collective key over fewer parties: the list of share holders changes
    ctx.collective_pk([0, 2])
    sums = torch.zeros((K, 5, n), dtype=torch.int32, device=ctx.device)
    offsets, rows = ring
    ctx.round_device(dv, 2, 5, offsets, rows, sums, ws)
    ctx.sync()
    want = np.stack([values[rows[offsets[i]:offsets[i + 1]]].astype(np.int64).sum(axis=0) for i in range(K)])
    assert np.array_equal(sums.cpu().numpy(), want)
    ctx.close()


def test_ciphertext_index_shards_reproduce_the_whole(d2):
    """Index ranges are independent: two half-ranges equal the full range bit for bit
    (this is how several GPUs split a round without exchanging data)."""
    cfg = wl.round_config(1)
    K, L, n = cfg.num_parties, cfg.num_limbs, cfg.n
    ctx = d2.Context(cfg.log2_n, cfg.moduli, K, seed=5)
    parties = list(range(K))
    ctx.keygen_share(parties)
    ctx.collective_pk(parties)
    plain = d2.from_u32_numpy(np.random.default_rng(1).integers(0, T, size=(K, 4, n)).astype(np.uint32), ctx.device)
    whole = ctx.empty_u64(K, 4, 2, L, n)
    ctx.encrypt(parties, 0, 4, plain, whole)
    for first in (0, 2):
        first_r, cnt = wl.shard_ct_range(first // 2, 2, 2)
        part = ctx.empty_u64(K, 2, 2, L, n)
        ctx.encrypt(parties, first_r, cnt, plain[:, first_r:first_r + cnt].contiguous(), part)
        assert torch.equal(part, whole[:, first_r:first_r + cnt])
    again = ctx.empty_u64(K, 4, 2, L, n)
    ctx.encrypt(parties, 0, 4, plain, again)
    assert torch.equal(again, whole)  # deterministic
    ctx.close()


def test_sample_batches_of_one_call_reproduce_separate_calls(d2):
    """d2mhe_encrypt and d2mhe_partial_decrypt draw their samples into the context's 64 MiB scratch,
    as many (party, ciphertext) or (recipient, ciphertext) units per pair of launches as fit (rounded
    down to whole waves of thread blocks).  A call
    large enough to need several batches must produce, unit for unit, what one small call per slice
    of the index range produces (every sample is addressed by its counters, not by its batch)."""
    cfg = wl.round_config(1)
    K, n = cfg.num_parties, cfg.n
    moduli = cfg.moduli[:1]
    ctx = d2.Context(cfg.log2_n, moduli, K, seed=9)
    parties = list(range(K))
    ctx.keygen_share(parties)
    ctx.collective_pk(parties)
    scratch = ctx.sample_scratch_bytes()
    assert scratch >= 64 << 20
    cap_enc, cap_sh = scratch // (3 * n), scratch // (K * n)  # units that the scratch holds
    C = -(-(cap_enc + 600) // K)  # enough indices that both calls need more than one batch
    assert K * C > cap_enc > cap_sh
    gen = torch.Generator().manual_seed(3)
    plain = torch.randint(0, T, (K, C, n), dtype=torch.int32, generator=gen).to(ctx.device)
    whole = ctx.empty_u64(K, C, 2, 1, n)
    ctx.encrypt(parties, 7, C, plain, whole)
    shares = ctx.empty_u64(K, K, C, 1, n)
    ctx.partial_decrypt(whole, parties, parties, 7, C, shares)
    # Batches are cut to whole waves of thread blocks (592 resident blocks of this kernel on a 148-SM
    # device, one block per unit here).  The slices straddle the ends of the first batches under that
    # rule and the ones a cut at the scratch size would give.
    wave = 592
    edges = {cap_enc // wave * wave, cap_enc, cap_sh // wave * wave, cap_sh}
    firsts = sorted({0, C - 3} | {max(0, min(C - 5, e % C - 2)) for e in edges})
    for first, cnt in [(f, 3 if f in (0, C - 3) else 5) for f in firsts]:
        part = ctx.empty_u64(K, cnt, 2, 1, n)
        ctx.encrypt(parties, 7 + first, cnt, plain[:, first:first + cnt].contiguous(), part)
        assert torch.equal(part, whole[:, first:first + cnt])
        sh = ctx.empty_u64(K, K, cnt, 1, n)
        ctx.partial_decrypt(part, parties, parties, 7 + first, cnt, sh)
        assert torch.equal(sh, shares[:, :, first:first + cnt])
    ctx.close()


def test_error_statuses(d2):
    cfg = wl.round_config(1)
    K, L, n = cfg.num_parties, cfg.num_limbs, cfg.n
    ctx = d2.Context(cfg.log2_n, cfg.moduli, K, seed=1)
    plain = ctx.empty_u32(K, 1, n)
    ct = ctx.empty_u64(K, 1, 2, L, n)

    def status(fn, *a):
        with pytest.raises(d2.D2mheError) as e:
            fn(*a)
        return e.value.status

    assert status(ctx.encrypt, [0, 1, 2, 3], 0, 1, plain, ct) == d2.ERR_STATE  # no pk yet
    assert status(ctx.collective_pk, [0, 1]) == d2.ERR_STATE  # no key shares yet
    assert status(ctx.keygen_share, [0, K]) == d2.ERR_RANGE
    assert status(ctx.keygen_share, [0, 0]) == d2.ERR_INVALID_ARG
    ctx.keygen_share([0, 1, 2])
    assert status(ctx.collective_pk, [0, 1, 2, 3]) == d2.ERR_STATE  # party 3 has no share
    ctx.collective_pk([0, 1, 2])
    agg = ctx.empty_u64(1, 1, 2, L, n)
    assert status(ctx.aggregate, ct, K, 1, [0, 2], [0, K], agg) == d2.ERR_RANGE
    assert status(ctx.aggregate, ct, K, 1, [1, 2], [0, 1], agg) == d2.ERR_INVALID_ARG
    shares = ctx.empty_u64(1, 3, 1, L, n)
    assert status(ctx.partial_decrypt, agg, [0], [0, 1, 3], 0, 1, shares) == d2.ERR_STATE
    out = ctx.empty_u32(1, 1, n)
    assert status(ctx.combine_decrypt, agg, shares, 1, 2, 1, out) == d2.ERR_INVALID_ARG  # a share is missing
    misaligned = ctx.empty_u64(2 * L * n + 1)[1:]
    assert status(ctx.ntt_forward, misaligned, 1) == d2.ERR_INVALID_ARG
    ctx.sync()
    # the host-buffer round reports an out-of-range value itself (it returns after its own sync)
    offsets, rows = wl.regular_graph(K, cfg.degree, 1)
    ctx.keygen_share([3])
    ctx.collective_pk([0, 1, 2, 3])
    hv = torch.zeros((K, 1, n), dtype=torch.int32).pin_memory()
    hs = torch.zeros((K, 1, n), dtype=torch.int32).pin_memory()
    ws = torch.empty(ctx.round_workspace_bytes(1), dtype=torch.uint8, device=ctx.device)
    ctx.round_host(hv, 0, 1, offsets, rows, hs, ws)
    hv[1, 0, 5] = -(T - 1) // 2 - 1
    assert status(ctx.round_host, hv, 0, 1, offsets, rows, hs, ws) == d2.ERR_RANGE
    ctx.sync()  # the flag was cleared by the call that reported it
    hv[1, 0, 5] = 0
    ctx.round_host(hv, 0, 1, offsets, rows, hs, ws)
    assert not hs.any()
    # a run of more staged calls than the staging ring has slots keeps working (the fifth waits for the first)
    for _ in range(9):
        ctx.keygen_share([0])
    ctx.sync()
    big = d2.Context(15, wl.ntt_primes(54, 1 << 16, 1), 2, seed=1)
    assert status(big.keygen_share, [0]) == d2.ERR_UNSUPPORTED
    big.close()
    ctx.close()


# ----------------------------------------------------------------------------------
# the protocol calls on 32-bit words (every prime below 2^30)
# ----------------------------------------------------------------------------------


def _run_round32(d2, ctx, o, parties, offsets, rows, values, ct_first, also_64=True):
    """encrypt32 -> aggregate32 -> partial_decrypt32 -> combine_decrypt32 against the oracle, message
    by message, and against the 64-bit calls of the same context."""
    K, n_cts = len(parties), values.shape[1]
    L, n = o.num_limbs, o.n
    dev = ctx.device
    ctx.keygen_share(parties)
    ctx.collective_pk(parties)
    want_pk = o.collective_pk(parties)
    dv = torch.from_numpy(values).to(dev)
    plain = ctx.empty_u32(K, n_cts, n)
    ctx.encode(dv, K * n_cts, plain)
    want_plain = o.encode(values)
    ct = ctx.empty_u32(K, n_cts, 2, L, n)
    ctx.encrypt32(parties, ct_first, n_cts, plain, ct)
    want_ct = o.encrypt(want_pk, parties, ct_first, want_plain)
    assert np.array_equal(d2.to_u32_numpy(ct).astype(np.uint64), want_ct)
    n_out = len(offsets) - 1
    agg = ctx.empty_u32(n_out, n_cts, 2, L, n)
    ctx.aggregate32(ct, K, n_cts, offsets, rows, agg)
    want_agg = o.aggregate(want_ct, offsets, rows)
    assert np.array_equal(d2.to_u32_numpy(agg).astype(np.uint64), want_agg)
    recipients = [i % K for i in range(n_out)]
    shares = ctx.empty_u32(n_out, K, n_cts, L, n)
    ctx.partial_decrypt32(agg, recipients, parties, ct_first, n_cts, shares)
    want_shares = o.partial_decrypt(want_agg, recipients, parties, ct_first)
    assert np.array_equal(d2.to_u32_numpy(shares).astype(np.uint64), want_shares)
    out_plain = ctx.empty_u32(n_out, n_cts, n)
    ctx.combine_decrypt32(agg, shares, n_out, K, n_cts, out_plain)
    want_out = o.combine(want_agg, want_shares)
    assert np.array_equal(d2.to_u32_numpy(out_plain), want_out)
    sums = torch.empty((n_out, n_cts, n), dtype=torch.int32, device=dev)
    ctx.decode(out_plain, n_out * n_cts, sums)
    ctx.sync()
    got = sums.cpu().numpy()
    for i in range(n_out):
        lst = rows[offsets[i]:offsets[i + 1]]
        assert np.array_equal(got[i], values[lst].astype(np.int64).sum(axis=0))
    if also_64:
        ct64 = ctx.empty_u64(K, n_cts, 2, L, n)
        ctx.encrypt(parties, ct_first, n_cts, plain, ct64)
        assert np.array_equal(d2.to_u64_numpy(ct64), want_ct)
        sh64 = ctx.empty_u64(n_out, K, n_cts, L, n)
        ctx.partial_decrypt(d2.from_u64_numpy(want_agg, dev), recipients, parties, ct_first, n_cts, sh64)
        assert np.array_equal(d2.to_u64_numpy(sh64), want_shares)


@pytest.mark.parametrize("log2_n,bits,L,K,n_cts", [
    (4, 24, 2, 3, 1),    # odd numbers of units: the last thread block holds one
    (6, 30, 3, 2, 3),
    (10, 30, 5, 3, 2),
    (12, 29, 3, 4, 2),
    (13, 30, 2, 3, 1),
    (14, 30, 2, 2, 2),
])
def test_protocol_on_32_bit_words_every_message(d2, log2_n, bits, L, K, n_cts):
    moduli = wl.ntt_primes(bits, 2 << log2_n, L)
    seed = 200 + log2_n
    ctx = d2.Context(log2_n, moduli, K, seed=seed)
    o = make_oracle(log2_n, moduli, seed=seed)
    n = 1 << log2_n
    half = (T - 1) // 2 // K
    values = np.random.default_rng(log2_n).integers(-half, half + 1, size=(K, n_cts, n)).astype(np.int32)
    values[0, 0, :2] = [half, -half]
    offsets = np.array([0, K, K, K + 1], dtype=np.uint32)  # an empty list in the middle, three recipients
    rows = np.array(list(range(K)) + [K - 1], dtype=np.uint32)
    _run_round32(d2, ctx, o, list(range(K)), offsets, rows, values, ct_first=9)
    ctx.close()


def test_mnist_shaped_round_on_30_bit_limbs_every_message(d2):
    """The MNIST-shaped configuration with seven 30-bit limbs (log q = 210) through the 32-bit-word
    calls: every ciphertext, sum, share and plaintext of all 13 indices against the oracle."""
    cfg = wl.narrow_round_config()
    assert max(cfg.moduli) < 1 << 30 and len(cfg.moduli) == 7
    seed = 1
    ctx = d2.Context(cfg.log2_n, cfg.moduli, cfg.num_parties, seed=seed)
    o = make_oracle(cfg.log2_n, cfg.moduli, seed=seed)
    offsets, rows = wl.regular_graph(cfg.num_parties, cfg.degree, seed)
    values = wl.gradients(cfg, seed)
    _run_round32(d2, ctx, o, list(range(cfg.num_parties)), offsets, rows, values, 0, also_64=False)
    ctx.close()


def test_32_bit_calls_in_several_batches_reproduce_separate_calls(d2):
    """d2mhe_encrypt32 / d2mhe_partial_decrypt32 with more units than the sample scratch holds run as
    several batches (whole pairs of units, whole waves of thread blocks); an odd total leaves the last
    thread block with one unit.  Unit for unit they must equal small calls on slices of the index range."""
    log2_n, K = 12, 3
    n = 1 << log2_n
    moduli = wl.ntt_primes(30, 2 << log2_n, 1)
    ctx = d2.Context(log2_n, moduli, K, seed=11)
    parties = list(range(K))
    ctx.keygen_share(parties)
    ctx.collective_pk(parties)
    scratch = ctx.sample_scratch_bytes()
    cap_enc, cap_sh = scratch // (3 * n), scratch // (K * n)
    C = -(-(cap_sh + 700) // K) | 1  # odd, so that K * C is odd too: the last pair is a single unit
    assert K * C > max(cap_sh, cap_enc) and (K * C) % 2 == 1
    gen = torch.Generator().manual_seed(5)
    plain = torch.randint(0, T, (K, C, n), dtype=torch.int32, generator=gen).to(ctx.device)
    whole = ctx.empty_u32(K, C, 2, 1, n)
    ctx.encrypt32(parties, 3, C, plain, whole)
    shares = ctx.empty_u32(K, K, C, 1, n)
    ctx.partial_decrypt32(whole, parties, parties, 3, C, shares)
    wave = 592  # resident thread blocks of this kernel on a 148-SM device; one block per pair of units
    edges = {2 * (cap_enc // 2 // wave * wave), cap_enc, 2 * (cap_sh // 2 // wave * wave), cap_sh}
    firsts = sorted({0, C - 3} | {max(0, min(C - 5, e % C - 2)) for e in edges})
    for first in firsts:
        cnt = 3 if first in (0, C - 3) else 5
        part = ctx.empty_u32(K, cnt, 2, 1, n)
        ctx.encrypt32(parties, 3 + first, cnt, plain[:, first:first + cnt].contiguous(), part)
        assert torch.equal(part, whole[:, first:first + cnt])
        sh = ctx.empty_u32(K, K, cnt, 1, n)
        ctx.partial_decrypt32(part, parties, parties, 3 + first, cnt, sh)
        assert torch.equal(sh, shares[:, :, first:first + cnt])
    # and against the oracle on the last (single-unit) pair
    o = make_oracle(log2_n, moduli, seed=11)
    pk = o.collective_pk(parties)
    last = C - 1
    want_ct = o.encrypt(pk, parties, 3 + last, d2.to_u32_numpy(plain[:, last:last + 1].contiguous()))
    assert np.array_equal(d2.to_u32_numpy(whole[:, last:last + 1].contiguous()).astype(np.uint64), want_ct)
    want_sh = o.partial_decrypt(want_ct, parties, parties, 3 + last)
    assert np.array_equal(d2.to_u32_numpy(shares[:, :, last:last + 1].contiguous()).astype(np.uint64), want_sh)
    ctx.close()


def test_32_bit_protocol_calls_refuse_wide_primes(d2):
    cfg = wl.round_config(1)
    ctx = d2.Context(cfg.log2_n, cfg.moduli, 2, seed=1)
    ctx.keygen_share([0, 1])
    ctx.collective_pk([0, 1])
    plain = ctx.empty_u32(2, 1, cfg.n)
    ct = ctx.empty_u32(2, 1, 2, cfg.num_limbs, cfg.n)
    with pytest.raises(d2.D2mheError) as e:
        ctx.encrypt32([0, 1], 0, 1, plain, ct)
    assert e.value.status == d2.ERR_UNSUPPORTED
    with pytest.raises(d2.D2mheError) as e:
        ctx.partial_decrypt32(ct, [0], [0, 1], 0, 1, ct)
    assert e.value.status == d2.ERR_UNSUPPORTED
    ctx.close()


# ----------------------------------------------------------------------------------
# the checked kernel build (D2MHE_FLAG_DEVICE_CHECKS)
# ----------------------------------------------------------------------------------


def test_checked_build_gives_the_same_messages_and_reports_nothing(d2):
    """Every kernel of the checked build (index tests on coefficient, octet, shared-memory, twiddle and
    party indices) on a small ring, on configuration 1, on the conversion and refresh calls and on the
    stand-alone transforms: the same bit-exact messages, and no violation recorded."""
    log2_n, K = 6, 3
    moduli = small_moduli(log2_n, 54, 2)
    ctx = d2.Context(log2_n, moduli, K, seed=5, flags=d2.FLAG_DEVICE_CHECKS)
    o = make_oracle(log2_n, moduli, seed=5)
    values = np.random.default_rng(2).integers(-3000, 3001, size=(K, 2, 1 << log2_n)).astype(np.int32)
    offsets = np.array([0, K, K, K + 1], dtype=np.uint32)
    rows = np.array(list(range(K)) + [K - 1], dtype=np.uint32)
    _run_round(d2, ctx, o, K, list(range(K)), offsets, rows, values, ct_first=3)
    ctx.sync()
    ctx.close()

    cfg = wl.round_config(1)
    ctx = d2.Context(cfg.log2_n, cfg.moduli, cfg.num_parties, seed=2, flags=d2.FLAG_DEVICE_CHECKS)
    o = make_oracle(cfg.log2_n, cfg.moduli, seed=2)
    offsets, rows = wl.regular_graph(cfg.num_parties, cfg.degree, 2)
    values = wl.gradients(cfg, 2)
    want = {}
    parties = list(range(cfg.num_parties))
    _run_round(d2, ctx, o, cfg.num_parties, parties, offsets, rows, values, 0, keep=want)
    _check_whole_round_call(d2, ctx, cfg, offsets, rows, values, want)
    K, L, n = cfg.num_parties, cfg.num_limbs, cfg.n
    # conversion and refresh shares through the checked kernels
    agg = d2.from_u64_numpy(want["agg"][:2, :1].copy(), ctx.device)
    ctx.user_keygen([0, 1])
    sh = ctx.empty_u64(2, K, 1, 2, L, n)
    ctx.convert_share(agg, [0, 1], parties, 0, 1, sh)
    pk_users = np.stack([o.user_pk(i) for i in (0, 1)])
    assert np.array_equal(d2.to_u64_numpy(sh), o.convert_share(want["agg"][:2, :1], pk_users, [0, 1], parties, 0))
    ctx.bootstrap_share(agg, [0, 1], parties, 0, 1, sh)
    assert np.array_equal(d2.to_u64_numpy(sh), o.boot_share(want["agg"][:2, :1], [0, 1], parties, 0))
    # stand-alone transforms and multiply-add
    polys = wl.random_polys(cfg.moduli, cfg.log2_n, 3, seed=9)
    dp = d2.from_u64_numpy(polys, ctx.device)
    ctx.ntt_forward(dp, 3)
    ctx.ntt_inverse(dp, 3)
    assert np.array_equal(d2.to_u64_numpy(dp), polys)
    ctx.poly_muladd(dp, dp, dp, dp, 3)
    ctx.sync()  # D2MHE_ERR_DEVICE_CHECK would raise here
    ctx.close()
    # the two-pass transforms (N = 2^15) and the 32-bit-word calls
    big = d2.Context(15, wl.ntt_primes(54, 1 << 16, 2), 1, seed=1, flags=d2.FLAG_DEVICE_CHECKS)
    polys = wl.random_polys(big.moduli, 15, 2, seed=3)
    dp = d2.from_u64_numpy(polys, big.device)
    big.ntt_forward(dp, 2)
    big.ntt_inverse(dp, 2)
    assert np.array_equal(d2.to_u64_numpy(dp), polys)
    big.sync()
    big.close()
    # the protocol calls on 32-bit words
    n32_moduli = wl.ntt_primes(30, 2 << 10, 3)
    n32 = d2.Context(10, n32_moduli, 3, seed=6, flags=d2.FLAG_DEVICE_CHECKS)
    vals = np.random.default_rng(4).integers(-2000, 2001, size=(3, 3, 1 << 10)).astype(np.int32)
    _run_round32(d2, n32, make_oracle(10, n32_moduli, seed=6), [0, 1, 2], np.array([0, 3, 3, 4], dtype=np.uint32),
                 np.array([0, 1, 2, 2], dtype=np.uint32), vals, ct_first=1, also_64=False)
    n32.sync()
    n32.close()
    narrow = d2.Context(12, small_moduli(12, 30, 2), 1, seed=1, flags=d2.FLAG_DEVICE_CHECKS)
    p32 = wl.random_polys(narrow.moduli, 12, 3, seed=4).astype(np.uint32)
    d32 = d2.from_u32_numpy(p32, narrow.device)
    narrow.ntt32_forward(d32, 3)
    narrow.ntt32_inverse(d32, 3)
    assert np.array_equal(d2.to_u32_numpy(d32), p32)
    narrow.sync()
    narrow.close()


def test_checked_build_reports_a_violation_without_losing_the_context(d2):
    """The self-test hook runs the index test on an index equal to its limit (no memory is touched):
    the next sync reports it once, with its site, index and limit, and the context keeps working.
    Without the flag the same hook does nothing."""
    cfg = wl.round_config(1)
    ctx = d2.Context(cfg.log2_n, cfg.moduli, 2, seed=1, flags=d2.FLAG_DEVICE_CHECKS)
    ctx.sync()
    ctx.debug_check_selftest()
    with pytest.raises(d2.D2mheError) as e:
        ctx.sync()
    assert e.value.status == d2.ERR_DEVICE_CHECK
    assert ctx.debug_last_device_check() == [15, 1, 1, 0]
    ctx.sync()  # reported once, then cleared
    polys = wl.random_polys(cfg.moduli, cfg.log2_n, 2, seed=1)
    dp = d2.from_u64_numpy(polys, ctx.device)
    ctx.ntt_forward(dp, 2)
    ctx.ntt_inverse(dp, 2)
    assert np.array_equal(d2.to_u64_numpy(dp), polys)
    ctx.sync()
    ctx.close()
    plain = d2.Context(cfg.log2_n, cfg.moduli, 2, seed=1)
    plain.debug_check_selftest()
    plain.sync()
    assert plain.debug_last_device_check() == [0, 0, 0, 0]
    plain.close()
