"""Pins for the oracle's Philox4x32-10: published known answers, an independent
Python transcription, and ATen's open-source host engine."""
import os
import subprocess
import sys

import numpy as np
import pytest

from oracle import d2mhe_oracle as orc
from oracle import definitions as defs


def _kat(golden_dir):
    rows = []
    with open(os.path.join(golden_dir, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            v = [int(x, 16) for x in line.split()]
            rows.append((v[0:4], v[4:6], v[6:10]))
    return rows


def test_known_answers(golden_dir):
    rows = _kat(golden_dir)
    assert len(rows) == 3
    for ctr, key, out in rows:
        assert orc.philox4x32_10(key, ctr) == out
        assert defs.philox4x32_10(key, ctr) == out


def test_c_and_python_agree_on_random_counters():
    rng = np.random.default_rng(7)
    for _ in range(200):
        key = [int(x) for x in rng.integers(0, 2**32, size=2)]
        ctr = [int(x) for x in rng.integers(0, 2**32, size=4)]
        assert orc.philox4x32_10(key, ctr) == defs.philox4x32_10(key, ctr)


def test_distinct_counters_give_distinct_blocks():
    seen = set()
    for j in range(64):
        for tag in range(1, 8):
            seen.add(tuple(orc.philox4x32_10([1, 0], [j, 0, 0, tag])))
    assert len(seen) == 64 * 7


_ATEN_SRC = r"""
#include <ATen/core/PhiloxRNGEngine.h>
#include <cstdio>
#include <cstdlib>
int main(int argc, char** argv) {
  unsigned long long seed = strtoull(argv[1], 0, 0), sub = strtoull(argv[2], 0, 0), off = strtoull(argv[3], 0, 0);
  at::philox_engine e(seed, sub, off);
  for (int i = 0; i < 4; ++i) printf("%u\n", e());
  return 0;
}
"""


def test_against_aten_host_engine(tmp_path):
    import torch

    inc = os.path.join(os.path.dirname(torch.__file__), "include")
    if not os.path.exists(os.path.join(inc, "ATen", "core", "PhiloxRNGEngine.h")):
        pytest.skip("ATen Philox header not shipped")
    src = tmp_path / "aten_philox.cpp"
    src.write_text(_ATEN_SRC)
    exe = tmp_path / "aten_philox"
    r = subprocess.run(["g++", "-std=c++17", "-O1", "-I", inc, str(src), "-o", str(exe)], capture_output=True, text=True)
    if r.returncode != 0:
        pytest.skip("ATen header does not compile stand-alone: " + r.stderr[-300:])
    # engine(seed, subsequence, offset): key = seed words, counter = (offset lo, hi, subsequence lo, hi)
    for seed, sub, off in [(0, 0, 0), (0x123456789ABCDEF, 77, 5), (2**64 - 1, 2**40 + 3, 2**33 + 9)]:
        out = subprocess.run([str(exe), str(seed), str(sub), str(off)], capture_output=True, text=True, check=True)
        got = [int(x) for x in out.stdout.split()]
        key = [seed & 0xFFFFFFFF, seed >> 32]
        ctr = [off & 0xFFFFFFFF, off >> 32, sub & 0xFFFFFFFF, sub >> 32]
        assert orc.philox4x32_10(key, ctr) == got
