"""Pins for the oracle's random numbers and sampling key (no GPU).

Philox4x32-10 is pinned to an independent implementation reachable through a
public API on the box (Triton's `tl.philox`, run by Triton's CPU interpreter),
the unit exponential to -log1p(-v) in FP64, and the race key to its definition.
"""
import json
import math
import os
import subprocess
import sys

import numpy as np

import oracle

_TRITON_SNIPPET = r"""
import json, sys
import torch, triton, triton.language as tl

@triton.jit
def k(out, seed, c0, c1, c2, c3):
    z = tl.full((1,), 0, tl.uint32)
    a, b, c, d = tl.philox(seed, z + c0, z + c1, z + c2, z + c3, 10)
    o = tl.arange(0, 1)
    tl.store(out + o, a.to(tl.int64))
    tl.store(out + 1 + o, b.to(tl.int64))
    tl.store(out + 2 + o, c.to(tl.int64))
    tl.store(out + 3 + o, d.to(tl.int64))

cases = json.loads(sys.argv[1])
res = []
for seed, ctr in cases:
    out = torch.zeros(4, dtype=torch.int64)
    k[(1,)](out, seed, ctr[0], ctr[1], ctr[2], ctr[3])
    res.append([int(v) & 0xFFFFFFFF for v in out])
print("RESULT" + json.dumps(res))
"""


def _triton_philox(cases):
    env = dict(os.environ, TRITON_INTERPRET="1", CUDA_VISIBLE_DEVICES="")
    p = subprocess.run([sys.executable, "-c", _TRITON_SNIPPET, json.dumps(cases)], env=env,
                       capture_output=True, text=True, timeout=600)
    # no skip: without this independent implementation the oracle's Philox would silently lose its pin
    assert p.returncode == 0, "Triton's CPU interpreter (the independent Philox4x32-10) did not run: " + p.stderr[-600:]
    line = [ln for ln in p.stdout.splitlines() if ln.startswith("RESULT")][-1]
    return json.loads(line[len("RESULT"):])


def test_philox_matches_independent_implementation():
    # seeds below 2^31 so that the interpreter passes them as plain integers; counters likewise
    cases = [(0, [0, 0, 0, 0]), (1, [0, 0, 0, 0]), (0, [1, 0, 0, 0]), (12345, [7, 3, 0, 0]),
             (2**31 - 1, [2**31 - 1, 2**31 - 5, 17, 0]), (987654321, [250000, 4999, 0, 0])]
    theirs = _triton_philox(cases)
    for (seed, ctr), want in zip(cases, theirs):
        got = oracle.philox4x32_10(ctr, [seed & 0xFFFFFFFF, seed >> 32])
        assert got == want, (seed, ctr, got, want)


def test_draw_word_mapping():
    # coefficient j uses word j mod 4 of the block with counter (j // 4, t_lo, t_hi, 0), key = seed
    seed, t = (0xDEADBEEF << 32) | 0x12345678, (3 << 32) | 77
    for j in (0, 1, 2, 3, 4, 5, 1023, 9_999_999):
        blk = oracle.philox4x32_10([j >> 2, t & 0xFFFFFFFF, t >> 32, 0], [seed & 0xFFFFFFFF, seed >> 32])
        assert oracle.draw_word(seed, t, j) == blk[j & 3]


def test_words_are_uniform():
    # chi-square on the top byte and on the low byte of 2^16 consecutive draws
    n = 1 << 16
    w = np.array([oracle.draw_word(0, 5, j) for j in range(n)], dtype=np.uint64)
    for shift in (24, 0):
        counts = np.bincount(((w >> shift) & 0xFF).astype(np.int64), minlength=256)
        chi2 = ((counts - n / 256) ** 2 / (n / 256)).sum()
        assert chi2 < 360.0, chi2      # 255 dof: mean 255, sd 22.6; 360 is > 4.6 sd
    # different rounds and different seeds give different streams
    w2 = np.array([oracle.draw_word(0, 6, j) for j in range(1024)], dtype=np.uint64)
    w3 = np.array([oracle.draw_word(1, 5, j) for j in range(1024)], dtype=np.uint64)
    assert (w2 != w[:1024]).mean() > 0.99 and (w3 != w[:1024]).mean() > 0.99


def test_unit_exponential_against_log1p():
    rng = np.random.default_rng(0)
    xs = list(rng.integers(0, 2**32, size=20000, dtype=np.uint64))
    xs += [0, 1, 2, 3, 2**24 - 1, 2**24, 2**24 + 1, 2**31 - 1, 2**31, 2**31 + 128, 2**31 + 129,
           2**32 - 1, 2**32 - 2, 2**32 - 300]
    xs += [int(v) for v in (2.0**32 * (1 - 2.0 ** -np.arange(1, 24)))]       # q near powers of two
    xs += [int(v) for v in (2.0**32 * (1 - math.sqrt(0.5) * 2.0 ** -np.arange(0, 23)))]  # m near sqrt(2)
    worst = 0.0
    for x in xs:
        x = int(x)
        # v as FP32 arithmetic defines it (the fma is exact or rounds once; emulate in FP64 then round)
        v = float(np.float32(float(np.float32(x)) * 2.0**-32 + 2.0**-33))
        v = min(v, 1.0 - 2.0**-24)
        want = -math.log1p(-v)
        got = oracle.unit_exponential(x)
        assert got > 0.0
        worst = max(worst, abs(got / want - 1.0))
    assert worst < 1e-6, worst


def test_unit_exponential_is_monotone_in_the_small_tail():
    # the winners of the race are the smallest E: distinct small words must stay ordered
    prev = 0.0
    for x in range(0, 4096):
        e = oracle.unit_exponential(x)
        assert e > prev
        prev = e


def test_unit_exponential_distribution():
    # mean 1, variance 1, P(E > 1) = 1/e for a unit exponential
    rng = np.random.default_rng(1)
    xs = rng.integers(0, 2**32, size=200000, dtype=np.uint64)
    e = np.array([oracle.unit_exponential(int(x)) for x in xs])
    n = len(e)
    assert abs(e.mean() - 1.0) < 5 / math.sqrt(n)
    assert abs(e.var() - 1.0) < 5 * math.sqrt(8.0 / n)
    assert abs((e > 1.0).mean() - math.exp(-1)) < 5 * math.sqrt(0.25 / n)


def test_race_key_definition():
    # T = E / (delta^2 + eta), all in FP32
    rng = np.random.default_rng(2)
    for _ in range(2000):
        x = int(rng.integers(0, 2**32))
        d = np.float32(10.0 ** rng.uniform(-6, 4))
        eta = np.float32(10.0 ** rng.uniform(-8, -3))
        w = np.float32(float(d) * float(d) + float(eta))          # fma = one rounding of the exact value
        want = np.float32(np.float32(oracle.unit_exponential(x)) / w)
        assert np.float32(oracle.race_key(d, eta, x)) == want
    # never-updated coefficients (delta = C) race ~1e14 times faster than settled ones (delta = 0)
    assert oracle.race_key(1e4, 1e-6, 123456) * 1e13 < oracle.race_key(0.0, 1e-6, 123456)
