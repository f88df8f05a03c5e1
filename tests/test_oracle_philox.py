"""Pins for the oracle's Philox4x32-10 stream and stratum uniforms."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch
from scipy import stats

from conftest import ROOT, golden_lines


def test_known_answers(oracle_mod):
    # Published known-answer vectors (tests/golden/philox4x32_10_kat.txt).
    for row in golden_lines("philox4x32_10_kat.txt"):
        w = [int(t, 16) for t in row]
        out = oracle_mod.philox4x32_10(w[0:4], w[4:6])
        assert [int(x) for x in out] == w[6:10]


@pytest.fixture(scope="module")
def aten_probe(tmp_path_factory):
    inc = os.path.join(os.path.dirname(torch.__file__), "include")
    exe = str(tmp_path_factory.mktemp("aten") / "aten_philox_probe")
    subprocess.check_call(["g++", "-O1", "-std=c++17", "-I", inc, "-o", exe,
                           os.path.join(ROOT, "tests", "aten_philox_probe.cpp")])
    return exe


def test_against_aten_engine(oracle_mod, aten_probe):
    # An independently written Philox4x32-10: key = seed, counter = (offset, subsequence).
    rng = np.random.default_rng(7)
    triples = [(0, 0, 0), (1, 0, 0), (0, 1, 0), (0, 0, 1), (2**64 - 1, 2**64 - 1, 2**64 - 1)]
    triples += [tuple(int(v) for v in rng.integers(0, 2**63, size=3)) for _ in range(2000)]
    text = "\n".join("%d %d %d" % t for t in triples) + "\n"
    out = subprocess.run([aten_probe], input=text, capture_output=True, text=True, check=True).stdout.split("\n")
    for (seed, sub, off), line in zip(triples, out):
        want = [int(t, 16) for t in line.split()]
        ctr = [off & 0xFFFFFFFF, off >> 32, sub & 0xFFFFFFFF, sub >> 32]
        key = [seed & 0xFFFFFFFF, seed >> 32]
        assert [int(x) for x in oracle_mod.philox4x32_10(ctr, key)] == want


def test_stratum_uniform_layout(oracle_mod, aten_probe):
    # u_k of (seed, call, k) is word 0 of the block at subsequence = call, offset = k.
    cases = [(0, 0, 0), (0, 5, 31), (123456789012345, 2**40 + 3, 65535), (2**64 - 1, 99, 7)]
    text = "\n".join("%d %d %d" % (s, c, k) for s, c, k in cases) + "\n"
    out = subprocess.run([aten_probe], input=text, capture_output=True, text=True, check=True).stdout.split("\n")
    for (s, c, k), line in zip(cases, out):
        w0 = int(line.split()[0], 16)
        u = oracle_mod.stratum_uniform(s, c, k)
        assert u == w0 / 2.0**32
        assert 0.0 <= u < 1.0


def test_distinct_counters_distinct_blocks(oracle_mod):
    # The round function is a bijection of the counter for a fixed key.
    seen = set()
    for k in range(4096):
        seen.add(tuple(int(x) for x in oracle_mod.philox4x32_10([k, 0, 3, 0], [11, 0])))
    assert len(seen) == 4096


def test_uniformity_chi_square(oracle_mod):
    n, bins = 200_000, 64
    u = np.array([oracle_mod.stratum_uniform(42, call, k) for call in range(n // 1000) for k in range(1000)])
    counts = np.bincount((u * bins).astype(np.int64), minlength=bins)
    chi2 = ((counts - n / bins) ** 2 / (n / bins)).sum()
    assert stats.chi2.sf(chi2, bins - 1) > 1e-4
    assert abs(u.mean() - 0.5) < 0.005
