"""Python binding of libd2mhe.so: argument marshalling only.

Every function has the name and meaning of the C entry point in include/d2mhe.h;
tensors are torch CUDA tensors used purely as device memory, and the current
torch stream is handed to the library.  There is no fallback: if the shared
library cannot be loaded, importing a context fails.
"""
import ctypes
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libd2mhe.so")

OK = 0
ERR_INVALID_ARG = -1
ERR_BAD_PARAMS = -2
ERR_STATE = -3
ERR_WORKSPACE = -4
ERR_CUDA = -5
ERR_RANGE = -6
ERR_UNSUPPORTED = -7
ERR_DEVICE_CHECK = -8
FLAG_DEVICE_CHECKS = 1

EXPORTS = [
    "d2mhe_create", "d2mhe_destroy", "d2mhe_set_stream", "d2mhe_sync", "d2mhe_strerror",
    "d2mhe_keygen_share", "d2mhe_collective_pk", "d2mhe_encode", "d2mhe_decode", "d2mhe_encrypt",
    "d2mhe_aggregate", "d2mhe_partial_decrypt", "d2mhe_combine_decrypt", "d2mhe_ntt_forward",
    "d2mhe_ntt_inverse", "d2mhe_poly_muladd", "d2mhe_ntt32_forward", "d2mhe_ntt32_inverse",
    "d2mhe_poly_muladd32", "d2mhe_encrypt32", "d2mhe_aggregate32", "d2mhe_partial_decrypt32",
    "d2mhe_combine_decrypt32", "d2mhe_round_workspace_bytes", "d2mhe_round_plan", "d2mhe_round_device",
    "d2mhe_round_host", "d2mhe_round_device_static", "d2mhe_user_keygen", "d2mhe_convert_share",
    "d2mhe_convert_combine", "d2mhe_decrypt", "d2mhe_bootstrap_share", "d2mhe_bootstrap_combine", "d2mhe_debug_export_user_secret", "d2mhe_debug_export_secret", "d2mhe_debug_int_throughput", "d2mhe_debug_last_device_check",
    "d2mhe_debug_check_selftest", "d2mhe_get_root", "d2mhe_get_plain_root",
    "d2mhe_launch_count", "d2mhe_sample_scratch_bytes",
]


class Params(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("log2_n", ctypes.c_uint32),
        ("num_limbs", ctypes.c_uint32),
        ("num_parties", ctypes.c_uint32),
        ("moduli", ctypes.POINTER(ctypes.c_uint64)),
        ("plain_modulus", ctypes.c_uint64),
        ("seed", ctypes.c_uint64),
        ("gauss_bound", ctypes.c_uint32),
        ("flags", ctypes.c_uint32),
        ("device", ctypes.c_int32),
    ]


class D2mheError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        super().__init__("%s: %s (status %d)" % (what, strerror(status), status))


_lib = None


def load():
    """Loads the shared library (raises if it is missing: there is no other path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                "libd2mhe.so is not built; run `python -m paper_2207_04604_b200.build` "
                "(or __graft_entry__.build())")
        lib = ctypes.CDLL(LIB_PATH)
        vp, u32, u64, sz = ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_size_t
        lib.d2mhe_create.argtypes = [ctypes.POINTER(Params), ctypes.POINTER(vp)]
        lib.d2mhe_destroy.argtypes = [vp]
        lib.d2mhe_destroy.restype = None
        lib.d2mhe_set_stream.argtypes = [vp, vp]
        lib.d2mhe_sync.argtypes = [vp]
        lib.d2mhe_strerror.argtypes = [ctypes.c_int32]
        lib.d2mhe_strerror.restype = ctypes.c_char_p
        lib.d2mhe_keygen_share.argtypes = [vp, vp, u32]
        lib.d2mhe_collective_pk.argtypes = [vp, vp, u32, vp, vp]
        lib.d2mhe_encode.argtypes = [vp, vp, u32, vp]
        lib.d2mhe_decode.argtypes = [vp, vp, u32, vp]
        lib.d2mhe_encrypt.argtypes = [vp, vp, u32, u32, u32, vp, vp]
        lib.d2mhe_aggregate.argtypes = [vp, vp, u32, u32, vp, vp, u32, vp]
        lib.d2mhe_partial_decrypt.argtypes = [vp, vp, vp, u32, vp, u32, u32, u32, vp]
        lib.d2mhe_combine_decrypt.argtypes = [vp, vp, vp, u32, u32, u32, vp]
        lib.d2mhe_ntt_forward.argtypes = [vp, vp, u32]
        lib.d2mhe_ntt_inverse.argtypes = [vp, vp, u32]
        lib.d2mhe_poly_muladd.argtypes = [vp, vp, vp, vp, vp, u32]
        lib.d2mhe_ntt32_forward.argtypes = [vp, vp, u32]
        lib.d2mhe_ntt32_inverse.argtypes = [vp, vp, u32]
        lib.d2mhe_poly_muladd32.argtypes = [vp, vp, vp, vp, vp, u32]
        lib.d2mhe_encrypt32.argtypes = [vp, vp, u32, u32, u32, vp, vp]
        lib.d2mhe_aggregate32.argtypes = [vp, vp, u32, u32, vp, vp, u32, vp]
        lib.d2mhe_partial_decrypt32.argtypes = [vp, vp, vp, u32, vp, u32, u32, u32, vp]
        lib.d2mhe_combine_decrypt32.argtypes = [vp, vp, vp, u32, u32, u32, vp]
        lib.d2mhe_round_plan.argtypes = [u32, ctypes.c_uint64, vp, u32, vp]
        lib.d2mhe_round_plan.restype = ctypes.c_uint32
        lib.d2mhe_round_workspace_bytes.argtypes = [vp, u32]
        lib.d2mhe_round_workspace_bytes.restype = sz
        lib.d2mhe_round_device.argtypes = [vp, vp, u32, u32, vp, vp, vp, vp, sz]
        lib.d2mhe_round_host.argtypes = [vp, vp, u32, u32, vp, vp, vp, vp, sz]
        lib.d2mhe_round_device_static.argtypes = [vp, vp, u32, u32, vp, vp, vp]
        lib.d2mhe_debug_export_secret.argtypes = [vp, u32, vp]
        lib.d2mhe_debug_export_user_secret.argtypes = [vp, u32, vp]
        lib.d2mhe_user_keygen.argtypes = [vp, vp, u32, vp]
        lib.d2mhe_convert_share.argtypes = [vp, vp, vp, u32, vp, u32, u32, u32, vp]
        lib.d2mhe_convert_combine.argtypes = [vp, vp, vp, u32, u32, u32, vp]
        lib.d2mhe_decrypt.argtypes = [vp, vp, u32, vp, u32, vp, vp]
        lib.d2mhe_bootstrap_share.argtypes = [vp, vp, vp, u32, vp, u32, u32, u32, vp]
        lib.d2mhe_bootstrap_combine.argtypes = [vp, vp, vp, vp, u32, u32, u32, u32, vp, vp]
        lib.d2mhe_debug_int_throughput.argtypes = [vp, u32, u32, ctypes.POINTER(ctypes.c_double)]
        lib.d2mhe_debug_last_device_check.argtypes = [vp, vp]
        lib.d2mhe_debug_check_selftest.argtypes = [vp]
        lib.d2mhe_get_root.argtypes = [vp, u32, ctypes.POINTER(u64)]
        lib.d2mhe_get_plain_root.argtypes = [vp, ctypes.POINTER(u64)]
        lib.d2mhe_launch_count.argtypes = [vp]
        lib.d2mhe_launch_count.restype = u64
        lib.d2mhe_sample_scratch_bytes.argtypes = [vp]
        lib.d2mhe_sample_scratch_bytes.restype = sz
        for name in EXPORTS:
            fn = getattr(lib, name)
            if fn.restype is ctypes.c_int:  # default: every remaining entry returns d2mhe_status
                fn.restype = ctypes.c_int32
        _lib = lib
    return _lib


def round_plan(n_cts, cap_cts):
    """(sub-chunk sizes, internal streams used) of a whole-round call: d2mhe_round_plan."""
    lib = load()
    lanes = ctypes.c_uint32(0)
    n_sub = int(lib.d2mhe_round_plan(n_cts, cap_cts, None, 0, ctypes.byref(lanes)))
    sizes = (ctypes.c_uint32 * max(n_sub, 1))()
    lib.d2mhe_round_plan(n_cts, cap_cts, sizes, n_sub, ctypes.byref(lanes))
    return [int(x) for x in sizes[:n_sub]], int(lanes.value)


def strerror(status):
    return load().d2mhe_strerror(int(status)).decode()


def _host_u32(a):
    arr = np.ascontiguousarray(a, dtype=np.uint32)
    return arr, arr.ctypes.data_as(ctypes.c_void_p)


def _dev(t, dtype=None):
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous()):
        raise TypeError("expected a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError("expected dtype %s, got %s" % (dtype, t.dtype))
    return ctypes.c_void_p(t.data_ptr())


# uint32 / uint64 device arrays are carried as int32 / int64 torch tensors (same bits).
U32 = torch.int32
U64 = torch.int64


class Context:
    """d2mhe_ctx.  Methods are the C calls with the same names (without the prefix)."""

    def __init__(self, log2_n, moduli, num_parties, seed, plain_modulus=65537, device=0, gauss_bound=19, flags=0):
        lib = load()
        self.log2_n, self.n = int(log2_n), 1 << int(log2_n)
        self.moduli = [int(m) for m in moduli]
        self.num_limbs, self.num_parties = len(self.moduli), int(num_parties)
        self.t = int(plain_modulus)
        self.device = torch.device("cuda", device)
        self._moduli_arr = (ctypes.c_uint64 * len(self.moduli))(*self.moduli)
        p = Params()
        p.struct_size = ctypes.sizeof(Params)
        p.log2_n, p.num_limbs, p.num_parties = self.log2_n, self.num_limbs, self.num_parties
        p.moduli = ctypes.cast(self._moduli_arr, ctypes.POINTER(ctypes.c_uint64))
        p.plain_modulus, p.seed = self.t, int(seed)
        p.gauss_bound, p.flags, p.device = gauss_bound, flags, device
        self._params = p
        self._h = ctypes.c_void_p()
        st = lib.d2mhe_create(ctypes.byref(p), ctypes.byref(self._h))
        if st != OK:
            self._h = None
            raise D2mheError(st, "d2mhe_create")
        self.use_current_stream()

    def close(self):
        if getattr(self, "_h", None):
            load().d2mhe_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st, what):
        if st != OK:
            raise D2mheError(st, what)

    def use_current_stream(self):
        s = torch.cuda.current_stream(self.device).cuda_stream
        self._check(load().d2mhe_set_stream(self._h, ctypes.c_void_p(s)), "d2mhe_set_stream")

    def sync(self):
        self._check(load().d2mhe_sync(self._h), "d2mhe_sync")

    def launch_count(self):
        return int(load().d2mhe_launch_count(self._h))

    def sample_scratch_bytes(self):
        return int(load().d2mhe_sample_scratch_bytes(self._h))

    # ---- allocation helpers (torch is the allocator) ----
    def empty_u64(self, *shape):
        return torch.empty(shape, dtype=U64, device=self.device)

    def empty_u32(self, *shape):
        return torch.empty(shape, dtype=U32, device=self.device)

    # ---- protocol calls ----
    def keygen_share(self, parties):
        arr, ptr = _host_u32(parties)
        self._check(load().d2mhe_keygen_share(self._h, ptr, arr.size), "d2mhe_keygen_share")

    def collective_pk(self, parties, pk_shares=None, pk=None):
        arr, ptr = _host_u32(parties)
        self._check(load().d2mhe_collective_pk(self._h, ptr, arr.size, _dev(pk_shares, U64), _dev(pk, U64)),
                    "d2mhe_collective_pk")

    def encode(self, values, n_cts, plain):
        self._check(load().d2mhe_encode(self._h, _dev(values, torch.int32), n_cts, _dev(plain, U32)), "d2mhe_encode")

    def decode(self, plain, n_cts, values):
        self._check(load().d2mhe_decode(self._h, _dev(plain, U32), n_cts, _dev(values, torch.int32)), "d2mhe_decode")

    def encrypt(self, parties, ct_first, n_cts, plain, ct):
        arr, ptr = _host_u32(parties)
        self._check(load().d2mhe_encrypt(self._h, ptr, arr.size, ct_first, n_cts, _dev(plain, U32), _dev(ct, U64)),
                    "d2mhe_encrypt")

    def aggregate(self, ct, n_rows, n_cts, nbr_offsets, nbr_rows, agg):
        off, offp = _host_u32(nbr_offsets)
        rows, rowsp = _host_u32(nbr_rows)
        self._check(load().d2mhe_aggregate(self._h, _dev(ct, U64), n_rows, n_cts, offp, rowsp, off.size - 1,
                                           _dev(agg, U64)), "d2mhe_aggregate")

    def partial_decrypt(self, agg, recipients, parties, ct_first, n_cts, shares):
        rec, recp = _host_u32(recipients)
        par, parp = _host_u32(parties)
        self._check(load().d2mhe_partial_decrypt(self._h, _dev(agg, U64), recp, rec.size, parp, par.size, ct_first,
                                                 n_cts, _dev(shares, U64)), "d2mhe_partial_decrypt")

    def combine_decrypt(self, agg, shares, n_rec, n_shares, n_cts, plain):
        self._check(load().d2mhe_combine_decrypt(self._h, _dev(agg, U64), _dev(shares, U64), n_rec, n_shares, n_cts,
                                                 _dev(plain, U32)), "d2mhe_combine_decrypt")

    def ntt_forward(self, polys, batch):
        self._check(load().d2mhe_ntt_forward(self._h, _dev(polys, U64), batch), "d2mhe_ntt_forward")

    def ntt_inverse(self, polys, batch):
        self._check(load().d2mhe_ntt_inverse(self._h, _dev(polys, U64), batch), "d2mhe_ntt_inverse")

    def poly_muladd(self, a, b, c, d, batch):
        self._check(load().d2mhe_poly_muladd(self._h, _dev(a, U64), _dev(b, U64), _dev(c, U64), _dev(d, U64), batch),
                    "d2mhe_poly_muladd")

    def ntt32_forward(self, polys, batch):
        self._check(load().d2mhe_ntt32_forward(self._h, _dev(polys, U32), batch), "d2mhe_ntt32_forward")

    def ntt32_inverse(self, polys, batch):
        self._check(load().d2mhe_ntt32_inverse(self._h, _dev(polys, U32), batch), "d2mhe_ntt32_inverse")

    def poly_muladd32(self, a, b, c, d, batch):
        self._check(load().d2mhe_poly_muladd32(self._h, _dev(a, U32), _dev(b, U32), _dev(c, U32), _dev(d, U32), batch),
                    "d2mhe_poly_muladd32")

    # ---- the protocol calls on 32-bit words ----
    def encrypt32(self, parties, ct_first, n_cts, plain, ct):
        arr, ptr = _host_u32(parties)
        self._check(load().d2mhe_encrypt32(self._h, ptr, arr.size, ct_first, n_cts, _dev(plain, U32), _dev(ct, U32)),
                    "d2mhe_encrypt32")

    def aggregate32(self, ct, n_rows, n_cts, nbr_offsets, nbr_rows, agg):
        off, offp = _host_u32(nbr_offsets)
        rows, rowsp = _host_u32(nbr_rows)
        self._check(load().d2mhe_aggregate32(self._h, _dev(ct, U32), n_rows, n_cts, offp, rowsp, off.size - 1,
                                             _dev(agg, U32)), "d2mhe_aggregate32")

    def partial_decrypt32(self, agg, recipients, parties, ct_first, n_cts, shares):
        rec, recp = _host_u32(recipients)
        par, parp = _host_u32(parties)
        self._check(load().d2mhe_partial_decrypt32(self._h, _dev(agg, U32), recp, rec.size, parp, par.size, ct_first,
                                                   n_cts, _dev(shares, U32)), "d2mhe_partial_decrypt32")

    def combine_decrypt32(self, agg, shares, n_rec, n_shares, n_cts, plain):
        self._check(load().d2mhe_combine_decrypt32(self._h, _dev(agg, U32), _dev(shares, U32), n_rec, n_shares, n_cts,
                                                   _dev(plain, U32)), "d2mhe_combine_decrypt32")

    def round_workspace_bytes(self, chunk_cts):
        return int(load().d2mhe_round_workspace_bytes(self._h, chunk_cts))

    def round_device(self, values, ct_first, n_cts, nbr_offsets, nbr_rows, sums, workspace):
        off, offp = _host_u32(nbr_offsets)
        rows, rowsp = _host_u32(nbr_rows)
        self._check(load().d2mhe_round_device(self._h, _dev(values, torch.int32), ct_first, n_cts, offp, rowsp,
                                              _dev(sums, torch.int32), _dev(workspace),
                                              workspace.numel() * workspace.element_size()), "d2mhe_round_device")

    def round_device_static(self, values, ct_first, n_cts, nbr_offsets, nbr_rows, sums):
        """d2mhe_round_device with the library's built-in 64 MiB scratch: nothing is allocated."""
        off, offp = _host_u32(nbr_offsets)
        rows, rowsp = _host_u32(nbr_rows)
        self._check(load().d2mhe_round_device_static(self._h, _dev(values, torch.int32), ct_first, n_cts, offp, rowsp,
                                                     _dev(sums, torch.int32)), "d2mhe_round_device_static")

    def round_host(self, values_host, ct_first, n_cts, nbr_offsets, nbr_rows, sums_host, workspace):
        """values_host / sums_host: CPU int32 tensors (pinned recommended)."""
        off, offp = _host_u32(nbr_offsets)
        rows, rowsp = _host_u32(nbr_rows)
        for t in (values_host, sums_host):
            if t.is_cuda or t.dtype != torch.int32 or not t.is_contiguous():
                raise TypeError("expected contiguous CPU int32 tensors")
        self._check(load().d2mhe_round_host(self._h, ctypes.c_void_p(values_host.data_ptr()), ct_first, n_cts, offp,
                                            rowsp, ctypes.c_void_p(sums_host.data_ptr()), _dev(workspace),
                                            workspace.numel() * workspace.element_size()), "d2mhe_round_host")

    # ---- conversion to the recipient's own key ----
    def user_keygen(self, users, pk_out=None):
        arr, ptr = _host_u32(users)
        self._check(load().d2mhe_user_keygen(self._h, ptr, arr.size, _dev(pk_out, U64)), "d2mhe_user_keygen")

    def convert_share(self, agg, recipients, parties, ct_first, n_cts, shares):
        rec, recp = _host_u32(recipients)
        par, parp = _host_u32(parties)
        self._check(load().d2mhe_convert_share(self._h, _dev(agg, U64), recp, rec.size, parp, par.size, ct_first,
                                               n_cts, _dev(shares, U64)), "d2mhe_convert_share")

    def convert_combine(self, agg, shares, n_rec, n_shares, n_cts, ct_out):
        self._check(load().d2mhe_convert_combine(self._h, _dev(agg, U64), _dev(shares, U64), n_rec, n_shares, n_cts,
                                                 _dev(ct_out, U64)), "d2mhe_convert_combine")

    def decrypt(self, users, ct, n_cts, scratch, plain):
        arr, ptr = _host_u32(users)
        self._check(load().d2mhe_decrypt(self._h, ptr, arr.size, _dev(ct, U64), n_cts, _dev(scratch, U64),
                                         _dev(plain, U32)), "d2mhe_decrypt")

    # ---- collective noise refresh ----
    def bootstrap_share(self, agg, recipients, parties, ct_first, n_cts, shares):
        rec, recp = _host_u32(recipients)
        par, parp = _host_u32(parties)
        self._check(load().d2mhe_bootstrap_share(self._h, _dev(agg, U64), recp, rec.size, parp, par.size, ct_first,
                                                 n_cts, _dev(shares, U64)), "d2mhe_bootstrap_share")

    def bootstrap_combine(self, agg, shares, recipients, n_shares, ct_first, n_cts, plain_scratch, ct_out):
        rec, recp = _host_u32(recipients)
        self._check(load().d2mhe_bootstrap_combine(self._h, _dev(agg, U64), _dev(shares, U64), recp, rec.size,
                                                   n_shares, ct_first, n_cts, _dev(plain_scratch, U32),
                                                   _dev(ct_out, U64)), "d2mhe_bootstrap_combine")

    def debug_export_user_secret(self, user):
        out = np.empty(self.n, dtype=np.int8)
        self._check(load().d2mhe_debug_export_user_secret(self._h, user, out.ctypes.data_as(ctypes.c_void_p)),
                    "d2mhe_debug_export_user_secret")
        return out

    # ---- test hooks ----
    def debug_export_secret(self, party):
        out = np.empty(self.n, dtype=np.int8)
        self._check(load().d2mhe_debug_export_secret(self._h, party, out.ctypes.data_as(ctypes.c_void_p)),
                    "d2mhe_debug_export_secret")
        return out

    def debug_int_throughput(self, kind, iters):
        """Lane operations per second of a register-only integer loop: d2mhe_debug_int_throughput."""
        v = ctypes.c_double()
        self._check(load().d2mhe_debug_int_throughput(self._h, kind, iters, ctypes.byref(v)),
                    "d2mhe_debug_int_throughput")
        return float(v.value)

    def debug_last_device_check(self):
        out = (ctypes.c_uint32 * 4)()
        self._check(load().d2mhe_debug_last_device_check(self._h, out), "d2mhe_debug_last_device_check")
        return [int(x) for x in out]

    def debug_check_selftest(self):
        self._check(load().d2mhe_debug_check_selftest(self._h), "d2mhe_debug_check_selftest")

    def get_root(self, limb):
        v = ctypes.c_uint64()
        self._check(load().d2mhe_get_root(self._h, limb, ctypes.byref(v)), "d2mhe_get_root")
        return int(v.value)

    def get_plain_root(self):
        v = ctypes.c_uint64()
        self._check(load().d2mhe_get_plain_root(self._h, ctypes.byref(v)), "d2mhe_get_plain_root")
        return int(v.value)


def to_u64_numpy(t):
    """int64 CUDA tensor holding uint64 bits -> numpy uint64."""
    return t.cpu().numpy().view(np.uint64)


def to_u32_numpy(t):
    return t.cpu().numpy().view(np.uint32)


def from_u64_numpy(a, device):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint64).view(np.int64)).to(device)


def from_u32_numpy(a, device):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint32).view(np.int32)).to(device)
