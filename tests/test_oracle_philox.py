"""Pins for the oracle's Philox4x32-10 and its 16-bit field mapping (CPU only)."""
import os
import subprocess
import sys

import numpy as np
import pytest

from oracle import ref

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def _kat():
    rows = []
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        rows.append((w[:4], w[4:6], w[6:]))
    return rows


def test_known_answers():
    rows = _kat()
    assert len(rows) == 3
    for ctr, key, out in rows:
        assert list(ref.philox4x32_10(ctr, key)) == out


def _philox_bigint(ctr, key):
    """Philox4x32-10 written over Python integers from the published round function."""
    c = list(ctr)
    k = list(key)
    for _ in range(10):
        p0 = 0xD2511F53 * c[0]
        p1 = 0xCD9E8D57 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & 0xFFFFFFFF, (p0 >> 32) ^ c[3] ^ k[1], p0 & 0xFFFFFFFF]
        k = [(k[0] + 0x9E3779B9) & 0xFFFFFFFF, (k[1] + 0xBB67AE85) & 0xFFFFFFFF]
    return c


def test_against_bigint_restatement():
    rng = np.random.default_rng(1)
    for _ in range(200):
        ctr = [int(x) for x in rng.integers(0, 2**32, 4)]
        key = [int(x) for x in rng.integers(0, 2**32, 2)]
        assert list(ref.philox4x32_10(ctr, key)) == _philox_bigint(ctr, key)


_PROBE = r"""
#include <ATen/core/PhiloxRNGEngine.h>
#include <cstdio>
#include <cstdlib>
int main(int argc, char** argv) {
  unsigned long long seed = strtoull(argv[1], 0, 0), sub = strtoull(argv[2], 0, 0), off = strtoull(argv[3], 0, 0);
  int blocks = atoi(argv[4]);
  at::philox_engine e(seed, sub, off);
  for (int i = 0; i < 4 * blocks; ++i) printf("%u\n", e());
  return 0;
}
"""


@pytest.fixture(scope="module")
def aten_probe(tmp_path_factory):
    import torch
    inc = os.path.join(os.path.dirname(torch.__file__), "include")
    if not os.path.exists(os.path.join(inc, "ATen", "core", "PhiloxRNGEngine.h")):
        pytest.skip("torch's Philox header is not installed")
    d = tmp_path_factory.mktemp("philox")
    src, exe = d / "probe.cpp", d / "probe"
    src.write_text(_PROBE)
    r = subprocess.run(["g++", "-std=c++17", "-O1", "-I", inc, str(src), "-o", str(exe)],
                       capture_output=True, text=True)
    if r.returncode != 0:
        pytest.skip("cannot compile against torch's Philox header: " + r.stderr[-300:])
    return str(exe)


def test_against_library_philox(aten_probe):
    """Black-box comparison with torch's header-only Philox4x32-10 engine, whose documented
    mapping is key = seed, counter = (offset, subsequence)."""
    cases = [(0, 0, 0), (1234567890123456789, 7, 3), (2**64 - 1, 2**40 + 5, 2**33 + 11)]
    for seed, sub, off in cases:
        blocks = 5
        out = subprocess.run([aten_probe, str(seed), str(sub), str(off), str(blocks)],
                             capture_output=True, text=True, check=True).stdout.split()
        lib = [int(x) for x in out]
        mine = []
        for b in range(blocks):
            o = off + b
            mine += list(ref.philox4x32_10(
                [o & 0xFFFFFFFF, o >> 32, sub & 0xFFFFFFFF, sub >> 32],
                [seed & 0xFFFFFFFF, seed >> 32]))
        assert mine == lib


def test_rand16_field_mapping():
    seed, it = 0x0123456789ABCDEF, 0x1122334455667788
    for blk in (0, 1, 2**32 + 3):
        words = ref.philox4x32_10([blk & 0xFFFFFFFF, blk >> 32, it & 0xFFFFFFFF, it >> 32],
                                  [seed & 0xFFFFFFFF, seed >> 32])
        for e in range(8):
            want = (int(words[e >> 1]) >> (16 * (e & 1))) & 0xFFFF
            assert ref.rand16(seed, it, 8 * blk + e) == want


def test_rand16_uniform_and_stream_separation():
    n = 1 << 16
    a = np.array([ref.rand16(5, 0, i) for i in range(n)])
    b = np.array([ref.rand16(5, 1, i) for i in range(n)])
    assert (a != b).mean() > 0.99                      # another iter, another stream
    hist = np.bincount(a >> 8, minlength=256)          # chi-square on the top byte
    chi2 = ((hist - n / 256) ** 2 / (n / 256)).sum()
    assert chi2 < 400                                  # 255 dof: mean 255, sd ~22.6
    assert abs(a.mean() - 32767.5) < 4 * 65536 / np.sqrt(12 * n)
