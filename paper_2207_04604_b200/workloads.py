"""Seeded synthetic inputs and parameter presets for the D2-MHE hot path.

This module holds no ring arithmetic, no sampling rule of the scheme and no
transform: it only chooses parameters (ring degree, RNS primes, graph) and
draws the *inputs* (integer gradients, random residue polynomials) that are
handed unchanged to whatever implementation is under test.

Presets follow the benchmark configurations: synthetic gradients shaped like
an MNIST MLP, a CIFAR-10 CNN and a ResNet-18 stand in for the datasets the
paper trains on (Sec. 6); only their length and value distribution matter to
the cryptographic path.
"""
from dataclasses import dataclass, field
from typing import List

import os

import numpy as np

PLAIN_MODULUS = 65537


# ---------------------------------------------------------------------------
# RNS primes: the `count` largest primes below 2^bits that are 1 mod 2N.
# ---------------------------------------------------------------------------

_MR_BASES = (2, 3, 5, 7, 11, 13, 17, 19, 23, 29, 31, 37)


def is_prime(n: int) -> bool:
    """Deterministic Miller-Rabin for n < 2^64."""
    if n < 2:
        return False
    for p in _MR_BASES:
        if n % p == 0:
            return n == p
    d, r = n - 1, 0
    while d % 2 == 0:
        d //= 2
        r += 1
    for a in _MR_BASES:
        x = pow(a, d, n)
        if x in (1, n - 1):
            continue
        for _ in range(r - 1):
            x = x * x % n
            if x == n - 1:
                break
        else:
            return False
    return True


def ntt_primes(bits: int, two_n: int, count: int) -> List[int]:
    """Largest `count` primes p < 2^bits with p = 1 (mod two_n), descending."""
    out = []
    p = ((1 << bits) - 1) // two_n * two_n + 1
    while len(out) < count and p > two_n:
        if p < (1 << bits) and is_prime(p):
            out.append(p)
        p -= two_n
    if len(out) < count:
        raise ValueError("not enough primes")
    return out


# ---------------------------------------------------------------------------
# Presets
# ---------------------------------------------------------------------------


@dataclass
class RoundConfig:
    name: str
    num_parties: int          # K users
    degree: int               # graph degree (neighbours per user)
    log2_n: int               # ring degree N = 2^log2_n
    prime_bits: int
    num_limbs: int
    params: int               # gradient length per user
    grad_sigma: float         # std of the fp32 gradients (0: integer inputs)
    int_range: int = 0        # config 1 draws integers uniform in [-int_range, int_range]
    moduli: List[int] = field(default_factory=list)

    def __post_init__(self):
        if not self.moduli:
            self.moduli = ntt_primes(self.prime_bits, 2 << self.log2_n, self.num_limbs)

    @property
    def n(self) -> int:
        return 1 << self.log2_n

    @property
    def num_cts(self) -> int:
        """Ciphertexts per user: ceil(params / N) (one value per slot)."""
        return -(-self.params // self.n)

    @property
    def clip(self) -> int:
        """Largest |value| such that a K-fold sum stays inside (-t/2, t/2)."""
        return ((PLAIN_MODULUS - 1) // 2) // self.num_parties


def round_config(index: int) -> RoundConfig:
    if index == 1:
        return RoundConfig("tiny-ring-K4", 4, 2, 12, 36, 3, 8192, 0.0, int_range=4096)
    if index == 2:
        return RoundConfig("mnist-mlp-784-128-10-K10", 10, 4, 13, 54, 4, 101770, 1e-2)
    if index == 3:
        return RoundConfig("cifar10-cnn-K20", 20, 6, 14, 54, 8, 1070794, 1e-2)
    if index == 4:
        return RoundConfig("resnet18-K50", 50, 8, 14, 54, 8, 11173962, 1e-3)
    raise ValueError("round configs are 1..4")


def narrow_round_config() -> RoundConfig:
    """The MNIST-shaped configuration on 30-bit limbs (for the 32-bit-word protocol calls): same K,
    graph, N, gradient and plaintext modulus; seven primes below 2^30 give log q = 210 against the 216
    of four 54-bit primes."""
    return RoundConfig("mnist-mlp-784-128-10-K10-30bit-limbs", 10, 4, 13, 30, 7, 101770, 1e-2)


SWEEP_LOG2_N = (12, 13, 14, 15, 16)
SWEEP_LIMBS = (1, 4, 8, 16, 24)
SWEEP_BATCH = (1, 64, 1024, 4096)


def sweep_moduli(prime_bits: int, num_limbs: int) -> List[int]:
    """Kernel-sweep primes: 1 mod 2^17 so that one list serves every N <= 65536."""
    return ntt_primes(prime_bits, 1 << 17, num_limbs)


# ---------------------------------------------------------------------------
# Graph: random d-regular, returned as closed neighbourhoods in CSR form.
# ---------------------------------------------------------------------------


def regular_graph(num_parties: int, degree: int, seed: int):
    """Closed neighbourhood lists {i} + nbr(i), ascending, as (offsets, rows) uint32.

    Starts from the circulant graph i ~ i +- 1..d/2 and applies 10*K*d attempted
    double-edge swaps (numpy Generator), rejecting loops and multi-edges.  With
    degree 2 and no swaps requested this is the plain ring.
    """
    k, d = num_parties, degree
    assert d % 2 == 0 and d < k
    edges = set()
    for i in range(k):
        for h in range(1, d // 2 + 1):
            a, b = i, (i + h) % k
            edges.add((min(a, b), max(a, b)))
    edge_list = sorted(edges)
    if d > 2:
        rng = np.random.default_rng(seed)
        for _ in range(10 * k * d):
            i1, i2 = rng.integers(0, len(edge_list), size=2)
            if i1 == i2:
                continue
            (a, b), (c, e) = edge_list[i1], edge_list[i2]
            if rng.integers(0, 2):
                c, e = e, c
            n1, n2 = (min(a, c), max(a, c)), (min(b, e), max(b, e))
            if a == c or b == e or n1 in edges or n2 in edges or n1 == n2:
                continue
            edges.discard(edge_list[i1])
            edges.discard(edge_list[i2])
            edges.add(n1)
            edges.add(n2)
            edge_list[i1], edge_list[i2] = n1, n2
    nbr = [[i] for i in range(k)]
    for a, b in edges:
        nbr[a].append(b)
        nbr[b].append(a)
    offsets = [0]
    rows = []
    for i in range(k):
        lst = sorted(nbr[i])
        assert len(lst) == d + 1
        rows.extend(lst)
        offsets.append(len(rows))
    return np.asarray(offsets, dtype=np.uint32), np.asarray(rows, dtype=np.uint32)


# ---------------------------------------------------------------------------
# Gradients: fp32 -> fixed point (scale 2^10) -> clip -> zero-pad to C*N slots.
# ---------------------------------------------------------------------------

FIXED_POINT_SCALE = 1024.0


def quantise(grad_f32: np.ndarray, clip: int) -> np.ndarray:
    """Fixed-point conversion (Sec. 6 cites a 2^-d fixed-point representation)."""
    scaled = np.rint(grad_f32.astype(np.float32) * np.float32(FIXED_POINT_SCALE))
    return np.clip(scaled, -clip, clip).astype(np.int32)


def gradients(cfg: RoundConfig, seed: int, ct_first: int = 0, n_cts: int = None, threads: int = 0) -> np.ndarray:
    """int32 [K, n_cts, N] slot values for ciphertext indices ct_first .. ct_first+n_cts-1.

    Each (party, ciphertext index) block has its own generator, so any slice of
    the gradient can be produced without materialising the whole of it, and the
    blocks can be filled by `threads` host threads (0: one per core, at most 16)
    with the same result.
    """
    n_cts = cfg.num_cts if n_cts is None else n_cts
    out = np.zeros((cfg.num_parties, n_cts, cfg.n), dtype=np.int32)

    def fill(c):
        idx = ct_first + c
        first = idx * cfg.n
        valid = max(0, min(cfg.n, cfg.params - first))
        for k in range(cfg.num_parties):
            rng = np.random.default_rng([1000 + seed, k, idx])
            if cfg.int_range:
                block = rng.integers(-cfg.int_range, cfg.int_range + 1, size=cfg.n).astype(np.int32)
            else:
                g = rng.normal(0.0, cfg.grad_sigma, size=cfg.n).astype(np.float32)
                block = quantise(g, cfg.clip)
            block[valid:] = 0
            out[k, c] = block

    if threads <= 0:
        threads = min(16, os.cpu_count() or 1)
    if threads == 1 or n_cts * cfg.num_parties < 64:
        for c in range(n_cts):
            fill(c)
    else:
        from concurrent.futures import ThreadPoolExecutor

        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(fill, range(n_cts)))
    return out


def random_polys(moduli, log2_n: int, batch: int, seed: int) -> np.ndarray:
    """uint64 [batch, L, N], residues uniform in [0, q_l)."""
    rng = np.random.default_rng(seed)
    n = 1 << log2_n
    out = np.empty((batch, len(moduli), n), dtype=np.uint64)
    for l, q in enumerate(moduli):
        out[:, l, :] = rng.integers(0, q, size=(batch, n), dtype=np.uint64)
    return out


def shard_ct_range(rank: int, world_size: int, cts_per_rank: int):
    """Ciphertext indices owned by `rank`: every index is independent through the
    whole round, so ranks take disjoint contiguous index ranges and never exchange data."""
    assert 0 <= rank < world_size
    return rank * cts_per_rank, cts_per_rank
