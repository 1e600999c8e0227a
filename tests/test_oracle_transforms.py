"""Pins for the oracle's distribution transforms: closed forms, library
quantile / log / sin / cos in fp64, moments and goodness of fit."""
import math

import numpy as np
import pytest
import scipy.stats
import torch

import oracle
from test_oracle_philox import py_philox, MASK


def words(seed, stream, n):
    """Philox words for elements 0..n-1 from the big-integer restatement."""
    out = []
    key = (seed & MASK, seed >> 32)
    for j in range((n + 3) // 4):
        out.extend(py_philox((j & MASK, j >> 32, stream & MASK, stream >> 32), key))
    return np.array(out[:n], dtype=np.uint64)


def test_uniform_closed_form_and_range():
    w = words(5, 0, 4096)
    x = oracle.gen(5, 0, oracle.UNIFORM_PM1, 4096)
    want = ((w >> 8).astype(np.float64) * 2.0 ** -23 - 1.0)
    assert np.array_equal(x.astype(np.float64), want)        # exact
    big = oracle.gen(6, 0, oracle.UNIFORM_PM1, 1 << 20)
    assert big.min() >= -1.0 and big.max() < 1.0
    assert abs(big.mean()) < 4 * (1 / math.sqrt(3)) / math.sqrt(big.size)
    assert abs(big.std() - 1 / math.sqrt(3)) < 2e-3
    assert oracle.uniform_pm1(0) == -1.0
    assert oracle.uniform_pm1(0xFFFFFFFF) == 1.0 - 2.0 ** -23


def test_student_t2_is_the_quantile_function():
    w = words(7, 0, 20000)
    x = oracle.gen(7, 0, oracle.STUDENT_T2, 20000).astype(np.float64)
    u = (2.0 * (w >> 9).astype(np.float64) + 1.0) * 2.0 ** -24
    want = scipy.stats.t.ppf(u, 2)
    assert np.all(np.abs(x - want) <= 1e-6 * np.abs(want) + 1e-12)
    # extremes: symmetric, finite, heavy tails reach the hundreds
    lo, hi = oracle.student_t2(0), oracle.student_t2(0xFFFFFFFF)
    assert lo == -hi and 2000 < hi < 3000
    big = oracle.gen(8, 0, oracle.STUDENT_T2, 1 << 20)
    assert np.isfinite(big).all() and np.abs(big).max() > 100
    # quartiles of t(2): +- 1/sqrt(2) * ... = ppf(0.75, 2)
    assert abs(np.quantile(big, 0.75) - scipy.stats.t.ppf(0.75, 2)) < 1e-2


def test_log_exhaustive_against_fp64():
    worst = 0.0
    chunk = 1 << 22
    for first in range(1, (1 << 24) + 1, chunk):
        cnt = min(chunk, (1 << 24) + 1 - first)
        got = oracle.log_unit_range(first, cnt).astype(np.float64)
        k = np.arange(first, first + cnt, dtype=np.float64)
        want = np.log(k * 2.0 ** -24)
        assert np.all(got <= 0.0)                             # sqrt(-2 log u) is always real
        err = np.abs(got - want) / np.maximum(np.abs(want), 1e-300)
        err[want == 0.0] = np.abs(got[want == 0.0])
        worst = max(worst, float(err.max()))
    assert worst < 4e-7, worst
    assert oracle.log_unit(1 << 24) == 0.0


def test_sincos_exhaustive_against_fp64():
    worst = 0.0
    chunk = 1 << 22
    for first in range(0, 1 << 24, chunk):
        s, c = oracle.sincos_turn_range(first, chunk)
        a = np.arange(first, first + chunk, dtype=np.float64) * (2.0 * math.pi / 2 ** 24)
        worst = max(worst, float(np.abs(s - np.sin(a)).max()), float(np.abs(c - np.cos(a)).max()))
        assert np.all(np.abs(s.astype(np.float64) ** 2 + c.astype(np.float64) ** 2 - 1.0) < 5e-7)
    assert worst < 1.5e-7, worst
    # exact values on the axes and the octant signs
    assert oracle.sincos_turn(0) == (0.0, 1.0)
    assert oracle.sincos_turn(1 << 22) == (1.0, pytest.approx(0.0, abs=1e-7))
    assert oracle.sincos_turn(1 << 23)[1] == -1.0
    assert oracle.sincos_turn(3 << 22)[0] == -1.0


def test_box_muller_pairs_against_fp64():
    n = 40000
    w = words(9, 0, n)
    z = oracle.gen(9, 0, oracle.NORMAL, n).astype(np.float64)
    w = w.reshape(-1, 4)
    for a, b, off in [(0, 1, 0), (2, 3, 2)]:
        u1 = ((w[:, a] >> 8).astype(np.float64) + 1.0) * 2.0 ** -24
        u2 = (w[:, b] >> 8).astype(np.float64) * 2.0 ** -24
        rad = np.sqrt(-2.0 * np.log(u1))
        ze, zo = rad * np.cos(2 * math.pi * u2), rad * np.sin(2 * math.pi * u2)
        got_e, got_o = z[off::4], z[off + 1::4]
        assert np.all(np.abs(got_e - ze) < 2e-6)
        assert np.all(np.abs(got_o - zo) < 2e-6)


def test_normal_moments_and_fit():
    z = oracle.gen(10, 0, oracle.NORMAL, 1 << 21).astype(np.float64)
    n = z.size
    assert np.isfinite(z).all()
    assert abs(z.mean()) < 4.5 / math.sqrt(n)
    assert abs(z.var() - 1.0) < 4.5 * math.sqrt(2.0 / n)
    assert abs(scipy.stats.kurtosis(z, fisher=False) - 3.0) < 0.03
    assert abs(scipy.stats.skew(z)) < 0.01
    assert np.abs(z).max() < 5.8                            # sqrt(-2 log 2^-24) = 5.77
    assert scipy.stats.kstest(z[:400000], "norm").pvalue > 1e-3
    # even / odd lanes are uncorrelated
    assert abs(np.corrcoef(z[0::2], z[1::2])[0, 1]) < 5.0 / math.sqrt(n / 2)


def test_large_magnitude_is_exactly_scaled():
    z = oracle.gen(12, 0, oracle.NORMAL, 10000)
    zz = oracle.gen(12, 0, oracle.NORMAL_1E4, 10000)
    assert np.array_equal((z * np.float32(1e4)).view(np.uint32), zz.view(np.uint32))
    assert 9e3 < zz.std() < 1.1e4


def test_sparse_mask_comes_from_the_next_stream():
    n = 1 << 16
    for seed, stream in [(13, 0), (13, 2), (4, (3 << 32) | 0)]:
        z = oracle.gen(seed, stream, oracle.NORMAL, n)
        sp = oracle.gen(seed, stream, oracle.SPARSE90, n)
        m = words(seed, stream + 1, n)
        zero = m < 0xE6666666
        assert np.array_equal(sp[~zero].view(np.uint32), z[~zero].view(np.uint32))
        assert np.all(sp[zero].view(np.uint32) == 0)         # +0.0 exactly
    big = oracle.gen(14, 0, oracle.SPARSE90, 1 << 21)
    frac = float((big == 0).mean())
    assert abs(frac - 0.9) < 4 * math.sqrt(0.09 / big.size) + 1e-6


def test_bf16_is_round_to_nearest_even():
    for dist in oracle.DISTS:
        f = oracle.gen(15, 0, dist, 50000)
        b = oracle.gen(15, 0, dist, 50000, dtype=oracle.BF16)
        want = torch.from_numpy(f).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        assert np.array_equal(b, want)
    # ties go to even, halves round up past odd
    assert oracle.bf16_rne(np.float32(1.0 + 2.0 ** -8)) == 0x3F80      # tie -> even (down)
    assert oracle.bf16_rne(np.float32(1.0 + 3 * 2.0 ** -8)) == 0x3F82  # tie -> even (up)
    assert oracle.bf16_rne(np.float32(-0.0)) == 0x8000


def test_distributions_differ_by_seed_and_stream():
    a = oracle.gen(1, 0, oracle.NORMAL, 1024)
    assert not np.array_equal(a, oracle.gen(2, 0, oracle.NORMAL, 1024))
    assert not np.array_equal(a, oracle.gen(1, 2, oracle.NORMAL, 1024))
    assert np.array_equal(a, oracle.gen(1, 0, oracle.NORMAL, 1024))
