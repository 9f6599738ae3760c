"""No GPU needed: the shared library loads and exports every symbol the header declares."""
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "d2mhe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(d2mhe_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported():
    from paper_2207_04604_b200 import build, d2mhe

    build.build()
    lib = d2mhe.load()
    names = _declared_symbols()
    assert len(names) >= 20
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(d2mhe.EXPORTS) == names


def test_strerror_needs_no_device():
    from paper_2207_04604_b200 import d2mhe

    assert d2mhe.strerror(0) == "success"
    assert "range" in d2mhe.strerror(d2mhe.ERR_RANGE)
    assert d2mhe.strerror(-99) == "unknown status"


def test_create_rejects_bad_arguments_before_touching_the_device():
    import ctypes

    from paper_2207_04604_b200 import d2mhe

    lib = d2mhe.load()
    h = ctypes.c_void_p()
    assert lib.d2mhe_create(None, ctypes.byref(h)) == d2mhe.ERR_INVALID_ARG
    p = d2mhe.Params()
    p.struct_size = 4
    assert lib.d2mhe_create(ctypes.byref(p), ctypes.byref(h)) == d2mhe.ERR_INVALID_ARG
    mods = (ctypes.c_uint64 * 2)(0xFFFFEE001, 0xFFFFEE001)
    p.struct_size = ctypes.sizeof(d2mhe.Params)
    p.log2_n, p.num_limbs, p.num_parties = 12, 2, 4
    p.moduli = ctypes.cast(mods, ctypes.POINTER(ctypes.c_uint64))
    p.plain_modulus, p.seed, p.gauss_bound, p.flags, p.device = 65537, 1, 19, 0, 0
    assert lib.d2mhe_create(ctypes.byref(p), ctypes.byref(h)) == d2mhe.ERR_BAD_PARAMS  # repeated prime
    mods[1] = 0xFFFFEE003  # not 1 mod 2N
    assert lib.d2mhe_create(ctypes.byref(p), ctypes.byref(h)) == d2mhe.ERR_BAD_PARAMS
    mods[1] = 0xFFFFC4001
    p.gauss_bound = 20
    assert lib.d2mhe_create(ctypes.byref(p), ctypes.byref(h)) == d2mhe.ERR_BAD_PARAMS
    p.gauss_bound = 19
    p.plain_modulus = 65536
    assert lib.d2mhe_create(ctypes.byref(p), ctypes.byref(h)) == d2mhe.ERR_BAD_PARAMS
    assert not h.value
    # flags: bit 0 (device-side index checks) is accepted, every other bit is refused
    p.plain_modulus = 65537
    p.flags = 2
    assert lib.d2mhe_create(ctypes.byref(p), ctypes.byref(h)) == d2mhe.ERR_BAD_PARAMS
    p.flags = d2mhe.FLAG_DEVICE_CHECKS | 4
    assert lib.d2mhe_create(ctypes.byref(p), ctypes.byref(h)) == d2mhe.ERR_BAD_PARAMS
    p.flags = d2mhe.FLAG_DEVICE_CHECKS
    st = lib.d2mhe_create(ctypes.byref(p), ctypes.byref(h))
    import torch

    if torch.cuda.is_available():
        assert st == d2mhe.OK
        lib.d2mhe_destroy(h)
    else:
        assert st == d2mhe.ERR_CUDA and not h.value  # the parameters passed validation; there is no device here


def test_round_plan_invariants():
    """How a whole-round call cuts its index range (host logic, no device): every index once, sizes
    within one of each other and non-increasing, whole passes over the streams unless every sub-chunk
    is a single index, and the sub-chunks in flight at the start (the largest) fit the workspace."""
    from paper_2207_04604_b200 import d2mhe

    assert d2mhe.round_plan(0, 5) == ([], 0)
    assert d2mhe.round_plan(5, 0) == ([], 0)
    for n_cts in list(range(1, 40)) + [66, 683, 1000]:
        for cap in list(range(1, 12)) + [13, 23, 66, 100, 5000]:
            sizes, lanes = d2mhe.round_plan(n_cts, cap)
            assert lanes == min(2 if n_cts >= 4 else 1, cap, n_cts)  # fewer than four indices: one stream
            assert sum(sizes) == n_cts and min(sizes) >= 1
            assert max(sizes) - min(sizes) <= 1
            assert sizes == sorted(sizes, reverse=True)
            assert len(sizes) % lanes == 0 or len(sizes) == n_cts
            assert sum(sizes[:lanes]) <= cap
            # no coarser cut with whole passes would have fitted
            fewer = len(sizes) - lanes
            if fewer >= lanes and len(sizes) % lanes == 0:
                small, big = divmod(n_cts, fewer)
                first = sum(small + (1 if l < big else 0) for l in range(lanes))
                assert first > cap
    # the benchmark configurations: 13 indices in a workspace for 13 -> 7 + 6 on two streams
    assert d2mhe.round_plan(13, 13) == ([7, 6], 2)
    assert d2mhe.round_plan(13, 3) == ([2] + [1] * 11, 2)
    assert d2mhe.round_plan(13, 1) == ([1] * 13, 1)
    assert d2mhe.round_plan(2, 100) == ([2], 1)
    assert d2mhe.round_plan(3, 2) == ([2, 1], 1)
    assert d2mhe.round_plan(4, 100) == ([2, 2], 2)
