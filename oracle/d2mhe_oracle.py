"""ctypes front end of the C oracle (d2mhe_oracle.c).

TEST INFRASTRUCTURE.  Only tests, the smoke check and the CPU-baseline leg of
the benchmark may import this module; the CUDA library never does.  The two
share no code.  Arrays are numpy, row-major, limb-major polynomials
``[..., L, N]`` of uint64 residues in [0, q_l) in the coefficient domain.
"""
import ctypes
import os
import subprocess

import numpy as np

from . import dgauss

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "d2mhe_oracle.c")
_LIB = os.path.join(_HERE, "_build", "libd2mhe_oracle.so")

MAX_LIMBS = 24
CDT_LEN = 38


def build(force=False):
    """Compile the C oracle with gcc (plain -O2, OpenMP over independent units)."""
    os.makedirs(os.path.dirname(_LIB), exist_ok=True)
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", tmp, _SRC]
        )
        os.replace(tmp, _LIB)
    return _LIB


class _Params(ctypes.Structure):
    _fields_ = [
        ("log2_n", ctypes.c_uint32),
        ("num_limbs", ctypes.c_uint32),
        ("moduli", ctypes.c_uint64 * MAX_LIMBS),
        ("plain_modulus", ctypes.c_uint64),
        ("psi_t", ctypes.c_uint64),
        ("seed", ctypes.c_uint64),
        ("cdt", ctypes.c_uint64 * CDT_LEN),
        ("gauss_bound", ctypes.c_int32),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_mulmod.restype = ctypes.c_uint64
        _lib.orc_mulmod.argtypes = [ctypes.c_uint64] * 3
        _lib.orc_powmod.restype = ctypes.c_uint64
        _lib.orc_powmod.argtypes = [ctypes.c_uint64] * 3
        _lib.orc_find_psi.restype = ctypes.c_uint64
        _lib.orc_find_psi.argtypes = [ctypes.c_uint64, ctypes.c_uint32]
        _lib.orc_negacyclic_coeff.restype = ctypes.c_uint64
        _lib.orc_horner.restype = ctypes.c_uint64
        _lib.orc_scale_round_residues.restype = ctypes.c_uint32
        _lib.orc_gauss_from_r.restype = ctypes.c_int32
        _lib.orc_gauss_from_r.argtypes = [ctypes.c_void_p, ctypes.c_uint64]
        _lib.orc_ternary_from_word.restype = ctypes.c_int32
        _lib.orc_ternary_from_word.argtypes = [ctypes.c_uint32]
        _lib.orc_decrypt_single.restype = ctypes.c_int
        _lib.orc_threads.restype = ctypes.c_int
    return _lib


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def _u64(a):
    return np.ascontiguousarray(a, dtype=np.uint64)


def _u32(a):
    return np.ascontiguousarray(a, dtype=np.uint32)


def threads():
    return int(lib().orc_threads())


def set_threads(n):
    os.environ["OMP_NUM_THREADS"] = str(n)


# ---- stand-alone arithmetic helpers -------------------------------------------------


def mulmod(a, b, p):
    return int(lib().orc_mulmod(a, b, p))


def find_psi(p, log2_n):
    return int(lib().orc_find_psi(p, log2_n))


def negacyclic_schoolbook(a, b, p):
    a, b = _u64(a), _u64(b)
    c = np.empty_like(a)
    lib().orc_negacyclic_schoolbook(_p(a), _p(b), _p(c), ctypes.c_uint32(a.size), ctypes.c_uint64(p))
    return c


def negacyclic_coeff(a, b, p, k):
    a, b = _u64(a), _u64(b)
    return int(
        lib().orc_negacyclic_coeff(_p(a), _p(b), ctypes.c_uint32(a.size), ctypes.c_uint64(p), ctypes.c_uint32(k))
    )


def ring_mul(a, b, p):
    a, b = _u64(a), _u64(b)
    c = np.empty_like(a)
    log2_n = int(a.size).bit_length() - 1
    lib().orc_ring_mul(_p(a), _p(b), _p(c), ctypes.c_uint32(log2_n), ctypes.c_uint64(p))
    return c


def negacyclic_eval(a, psi, p):
    a = _u64(a)
    out = np.empty_like(a)
    log2_n = int(a.size).bit_length() - 1
    lib().orc_negacyclic_eval(_p(a), _p(out), ctypes.c_uint32(log2_n), ctypes.c_uint64(psi), ctypes.c_uint64(p))
    return out


def negacyclic_interp(vals, psi, p):
    vals = _u64(vals)
    out = np.empty_like(vals)
    log2_n = int(vals.size).bit_length() - 1
    lib().orc_negacyclic_interp(_p(vals), _p(out), ctypes.c_uint32(log2_n), ctypes.c_uint64(psi), ctypes.c_uint64(p))
    return out


def horner(a, x, p):
    a = _u64(a)
    return int(lib().orc_horner(_p(a), ctypes.c_uint32(a.size), ctypes.c_uint64(x), ctypes.c_uint64(p)))


def philox4x32_10(key, ctr):
    k = _u32(key)
    c = _u32(ctr)
    out = np.empty(4, dtype=np.uint32)
    lib().orc_philox4x32_10(_p(k), _p(c), _p(out))
    return [int(x) for x in out]


# ---- the scheme ---------------------------------------------------------------------


class Oracle:
    """One parameter set (N, q_l, t, seed); methods mirror the protocol calls."""

    def __init__(self, log2_n, moduli, plain_modulus, seed, psi_t=None, gauss_bound=19):
        self.log2_n = int(log2_n)
        self.n = 1 << self.log2_n
        self.moduli = [int(m) for m in moduli]
        self.num_limbs = len(self.moduli)
        self.t = int(plain_modulus)
        self.seed = int(seed)
        self.P = _Params()
        self.P.log2_n = self.log2_n
        self.P.num_limbs = self.num_limbs
        for i, m in enumerate(self.moduli):
            self.P.moduli[i] = m
        self.P.plain_modulus = self.t
        self.P.psi_t = int(psi_t) if psi_t is not None else 0
        self.P.seed = self.seed
        self.P.gauss_bound = gauss_bound
        self.cdt = dgauss.thresholds(gauss_bound)
        for i, v in enumerate(self.cdt):
            self.P.cdt[i] = v
        self._ref = ctypes.byref(self.P)
        lib()

    # samplers (streams are documented in d2mhe_oracle.c)
    def sample_ternary(self, tag, idx, party, recipient=0):
        out = np.empty(self.n, dtype=np.int8)
        lib().orc_sample_ternary(self._ref, ctypes.c_uint32(tag), ctypes.c_uint32(idx), ctypes.c_uint32(party),
                                 ctypes.c_uint32(recipient), _p(out))
        return out

    def sample_gauss(self, tag, idx, party, recipient=0):
        out = np.empty(self.n, dtype=np.int8)
        lib().orc_sample_gauss(self._ref, ctypes.c_uint32(tag), ctypes.c_uint32(idx), ctypes.c_uint32(party),
                               ctypes.c_uint32(recipient), _p(out))
        return out

    def gauss_from_r(self, r):
        return int(lib().orc_gauss_from_r(ctypes.addressof(self.P), ctypes.c_uint64(r)))

    # keys
    def secret_share(self, party):
        out = np.empty(self.n, dtype=np.int8)
        lib().orc_secret_share(self._ref, ctypes.c_uint32(party), _p(out))
        return out

    def pk_error(self, party):
        out = np.empty(self.n, dtype=np.int8)
        lib().orc_pk_error(self._ref, ctypes.c_uint32(party), _p(out))
        return out

    def common_p1(self):
        out = np.empty((self.num_limbs, self.n), dtype=np.uint64)
        lib().orc_common_p1(self._ref, _p(out))
        return out

    def pk_share(self, party, p1=None):
        p1 = self.common_p1() if p1 is None else _u64(p1)
        out = np.empty((self.num_limbs, self.n), dtype=np.uint64)
        lib().orc_pk_share(self._ref, ctypes.c_uint32(party), _p(p1), _p(out))
        return out

    def collective_pk(self, parties):
        parties = _u32(parties)
        out = np.empty((2, self.num_limbs, self.n), dtype=np.uint64)
        lib().orc_collective_pk(self._ref, _p(parties), ctypes.c_uint32(parties.size), _p(out))
        return out

    def delta(self):
        out = np.zeros(self.num_limbs, dtype=np.uint64)
        lib().orc_delta(self._ref, _p(out))
        return out

    # packing
    def encode(self, values):
        v = np.ascontiguousarray(values, dtype=np.int32).reshape(-1, self.n)
        out = np.empty(v.shape, dtype=np.uint32)
        lib().orc_encode_batch(self._ref, _p(v), ctypes.c_uint32(v.shape[0]), _p(out))
        return out.reshape(np.shape(values))

    def decode(self, plain):
        m = _u32(plain).reshape(-1, self.n)
        out = np.empty(m.shape, dtype=np.int32)
        lib().orc_decode_batch(self._ref, _p(m), ctypes.c_uint32(m.shape[0]), _p(out))
        return out.reshape(np.shape(plain))

    # round
    def encrypt(self, pk, parties, ct_first, plain):
        """plain [n_parties, n_cts, N] -> ct [n_parties, n_cts, 2, L, N]."""
        pk = _u64(pk)
        parties = _u32(parties)
        plain = _u32(plain)
        n_parties, n_cts = plain.shape[0], plain.shape[1]
        assert parties.size == n_parties
        ct = np.empty((n_parties, n_cts, 2, self.num_limbs, self.n), dtype=np.uint64)
        lib().orc_encrypt_batch(self._ref, _p(pk), _p(parties), ctypes.c_uint32(n_parties), ctypes.c_uint32(ct_first),
                                ctypes.c_uint32(n_cts), _p(plain), _p(ct))
        return ct

    def aggregate(self, ct, offsets, rows):
        """ct [n_rows, n_cts, 2, L, N], CSR (offsets, rows) -> [n_out, n_cts, 2, L, N]."""
        ct = _u64(ct)
        offsets, rows = _u32(offsets), _u32(rows)
        n_out = offsets.size - 1
        agg = np.empty((n_out,) + ct.shape[1:], dtype=np.uint64)
        lib().orc_aggregate_batch(self._ref, _p(ct), ctypes.c_uint32(ct.shape[0]), ctypes.c_uint32(ct.shape[1]),
                                  _p(offsets), _p(rows), ctypes.c_uint32(n_out), _p(agg))
        return agg

    def partial_decrypt(self, agg, recipients, parties, ct_first):
        """agg [n_rec, n_cts, 2, L, N] -> shares [n_rec, n_parties, n_cts, L, N]."""
        agg = _u64(agg)
        recipients, parties = _u32(recipients), _u32(parties)
        n_rec, n_cts = agg.shape[0], agg.shape[1]
        shares = np.empty((n_rec, parties.size, n_cts, self.num_limbs, self.n), dtype=np.uint64)
        lib().orc_partial_decrypt_batch(self._ref, _p(agg), _p(recipients), ctypes.c_uint32(n_rec), _p(parties),
                                        ctypes.c_uint32(parties.size), ctypes.c_uint32(ct_first),
                                        ctypes.c_uint32(n_cts), _p(shares))
        return shares

    def combine(self, agg, shares):
        """agg [n_rec, n_cts, 2, L, N], shares [n_rec, S, n_cts, L, N] -> plain [n_rec, n_cts, N]."""
        agg, shares = _u64(agg), _u64(shares)
        n_rec, n_cts = agg.shape[0], agg.shape[1]
        plain = np.empty((n_rec, n_cts, self.n), dtype=np.uint32)
        lib().orc_combine_batch(self._ref, _p(agg), _p(shares), ctypes.c_uint32(n_rec),
                                ctypes.c_uint32(shares.shape[1]), ctypes.c_uint32(n_cts), _p(plain))
        return plain

    # MBFV.Convert to a recipient's own key (Sec. 4.2 item 3)
    def user_secret(self, user):
        out = np.empty(self.n, dtype=np.int8)
        lib().orc_user_secret(self._ref, ctypes.c_uint32(user), _p(out))
        return out

    def user_pk(self, user):
        out = np.empty((2, self.num_limbs, self.n), dtype=np.uint64)
        lib().orc_user_pk(self._ref, ctypes.c_uint32(user), _p(out))
        return out

    def convert_share(self, agg, pk_users, recipients, parties, ct_first):
        """agg [n_rec, n_cts, 2, L, N], pk_users [n_rec, 2, L, N] -> [n_rec, n_parties, n_cts, 2, L, N]."""
        agg, pk_users = _u64(agg), _u64(pk_users)
        recipients, parties = _u32(recipients), _u32(parties)
        n_rec, n_cts = agg.shape[0], agg.shape[1]
        shares = np.empty((n_rec, parties.size, n_cts, 2, self.num_limbs, self.n), dtype=np.uint64)
        lib().orc_convert_share_batch(self._ref, _p(agg), _p(pk_users), _p(recipients), ctypes.c_uint32(n_rec),
                                      _p(parties), ctypes.c_uint32(parties.size), ctypes.c_uint32(ct_first),
                                      ctypes.c_uint32(n_cts), _p(shares))
        return shares

    def convert_combine(self, agg, shares):
        agg, shares = _u64(agg), _u64(shares)
        out = np.empty_like(agg)
        lib().orc_convert_combine_batch(self._ref, _p(agg), _p(shares), ctypes.c_uint32(agg.shape[0]),
                                        ctypes.c_uint32(shares.shape[1]), ctypes.c_uint32(agg.shape[1]), _p(out))
        return out

    def decrypt(self, ct, secrets):
        """ct [n, n_cts, 2, L, N], secrets int [n, N] -> plain [n, n_cts, N]."""
        ct = _u64(ct)
        secrets = np.ascontiguousarray(secrets, dtype=np.int32)
        plain = np.empty((ct.shape[0], ct.shape[1], self.n), dtype=np.uint32)
        lib().orc_decrypt_batch(self._ref, _p(ct), _p(secrets), ctypes.c_uint32(ct.shape[0]),
                                ctypes.c_uint32(ct.shape[1]), _p(plain))
        return plain

    # MBFV.Bootstrap (Sec. 4.2 item 4)
    def boot_alpha(self, recipient, ct_index):
        out = np.empty((self.num_limbs, self.n), dtype=np.uint64)
        lib().orc_boot_alpha(self._ref, ctypes.c_uint32(recipient), ctypes.c_uint32(ct_index), _p(out))
        return out

    def boot_mask(self, party, recipient, ct_index):
        out = np.empty(self.n, dtype=np.uint32)
        lib().orc_boot_mask(self._ref, ctypes.c_uint32(party), ctypes.c_uint32(recipient), ctypes.c_uint32(ct_index), _p(out))
        return out

    def boot_share(self, agg, recipients, parties, ct_first):
        agg = _u64(agg)
        recipients, parties = _u32(recipients), _u32(parties)
        n_rec, n_cts = agg.shape[0], agg.shape[1]
        shares = np.empty((n_rec, parties.size, n_cts, 2, self.num_limbs, self.n), dtype=np.uint64)
        lib().orc_boot_share_batch(self._ref, _p(agg), _p(recipients), ctypes.c_uint32(n_rec), _p(parties),
                                   ctypes.c_uint32(parties.size), ctypes.c_uint32(ct_first), ctypes.c_uint32(n_cts),
                                   _p(shares))
        return shares

    def boot_combine(self, agg, shares, recipients, ct_first):
        agg, shares = _u64(agg), _u64(shares)
        recipients = _u32(recipients)
        out = np.empty_like(agg)
        lib().orc_boot_combine_batch(self._ref, _p(agg), _p(shares), _p(recipients), ctypes.c_uint32(agg.shape[0]),
                                     ctypes.c_uint32(shares.shape[1]), ctypes.c_uint32(ct_first),
                                     ctypes.c_uint32(agg.shape[1]), _p(out))
        return out

    def decrypt_single(self, ct, s, want_noise=False):
        """BFV.Decrypt of one ciphertext [2, L, N] under an explicit integer secret s[N]."""
        ct = _u64(ct)
        s = np.ascontiguousarray(s, dtype=np.int32)
        plain = np.empty(self.n, dtype=np.uint32)
        noise = np.empty(self.n, dtype=np.int64) if want_noise else None
        rc = lib().orc_decrypt_single(self._ref, _p(ct), _p(s), _p(plain), _p(noise) if want_noise else None)
        if want_noise:
            if rc != 0:
                raise ValueError("noise does not fit in 63 bits")
            return plain, noise
        return plain

    def scale_round_residues(self, residues):
        r = _u64(residues)
        return int(lib().orc_scale_round_residues(self._ref, _p(r)))

    def crt_int(self, residues):
        r = _u64(residues)
        words = np.zeros(64, dtype=np.uint32)
        lib().orc_crt_words(self._ref, _p(r), _p(words))
        return sum(int(w) << (32 * i) for i, w in enumerate(words))

    def ntt(self, polys, psi, inverse=False):
        """Batch [batch, L, N]: values at psi_l^(2j+1) in natural order (or back)."""
        polys = _u64(polys)
        psi = _u64(psi)
        out = np.empty_like(polys)
        batch = polys.size // (self.num_limbs * self.n)
        lib().orc_ntt_batch(self._ref, _p(psi), _p(polys), _p(out), ctypes.c_uint32(batch),
                            ctypes.c_int(1 if inverse else 0))
        return out

    def poly_muladd(self, a, b, c):
        a, b, c = _u64(a), _u64(b), _u64(c)
        d = np.empty_like(a)
        batch = a.size // (self.num_limbs * self.n)
        lib().orc_poly_muladd(self._ref, _p(a), _p(b), _p(c), _p(d), ctypes.c_uint32(batch))
        return d
