"""Helpers shared by the tests (no scheme arithmetic beyond parameter derivation)."""
import numpy as np

from oracle import d2mhe_oracle as orc
from paper_2207_04604_b200 import workloads as wl

T = wl.PLAIN_MODULUS


def psi_t_for(log2_n, t=T, generator=3):
    """psi_t = g^((t-1)/2N) mod t; 3 is a primitive root of 65537."""
    two_n = 2 << log2_n
    assert (t - 1) % two_n == 0
    return pow(generator, (t - 1) // two_n, t)


def small_moduli(log2_n, bits, count):
    return wl.ntt_primes(bits, 2 << log2_n, count)


def make_oracle(log2_n, moduli, seed, t=T):
    two_n = 2 << log2_n
    psi = psi_t_for(log2_n, t) if (t - 1) % two_n == 0 else None
    return orc.Oracle(log2_n, moduli, t, seed, psi_t=psi)


def oracle_for_config(cfg, seed):
    return make_oracle(cfg.log2_n, cfg.moduli, seed)


def q_of(moduli):
    q = 1
    for m in moduli:
        q *= int(m)
    return q


def to_big(poly_limbs, moduli):
    """[L, N] residues -> list of N Python integers in [0, q) (CRT in Python integers)."""
    from oracle.definitions import crt
    L, n = poly_limbs.shape
    return [crt([int(poly_limbs[l, j]) for l in range(L)], moduli) for j in range(n)]


def from_big(poly_big, moduli):
    return np.array([[x % m for x in poly_big] for m in moduli], dtype=np.uint64)
