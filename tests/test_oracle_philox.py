"""Pins for the oracle's Philox4x32-10 and its counter/stream layout.

Nothing here re-types the oracle's own code path: the pins are (1) ATen's
host-side Philox engine, compiled from the installed torch headers and run as a
separate program; (2) a big-integer restatement of the published round function
written in a different style; (3) the inverse of the round function (the
bijection property of Philox); (4) avalanche statistics.
"""
import os
import random
import subprocess
import sys

import numpy as np
import pytest

import oracle

M0, M1 = 0xD2511F53, 0xCD9E8D57
W0, W1 = 0x9E3779B9, 0xBB67AE85
MASK = 0xFFFFFFFF


def py_philox(ctr, key, rounds=10):
    """Published definition, with Python integers and divmod."""
    c = list(ctr)
    k = list(key)
    for r in range(rounds):
        hi0, lo0 = divmod(M0 * c[0], 1 << 32)
        hi1, lo1 = divmod(M1 * c[2], 1 << 32)
        c = [hi1 ^ c[1] ^ k[0], lo1, hi0 ^ c[3] ^ k[1], lo0]
        k = [(k[0] + W0) & MASK, (k[1] + W1) & MASK]
    return tuple(c)


def py_philox_inverse(out, key, rounds=10):
    """Undo the rounds: the multipliers are odd, hence invertible mod 2^32."""
    inv0, inv1 = pow(M0, -1, 1 << 32), pow(M1, -1, 1 << 32)
    keys = [((key[0] + r * W0) & MASK, (key[1] + r * W1) & MASK) for r in range(rounds)]
    n = list(out)
    for r in reversed(range(rounds)):
        k0, k1 = keys[r]
        c0 = (n[3] * inv0) & MASK
        c2 = (n[1] * inv1) & MASK
        hi0 = (M0 * c0) >> 32
        hi1 = (M1 * c2) >> 32
        n = [c0, n[0] ^ hi1 ^ k0, c2, n[2] ^ hi0 ^ k1]
    return tuple(n)


@pytest.fixture(scope="module")
def aten_pin(tmp_path_factory):
    import torch
    inc = os.path.join(os.path.dirname(torch.__file__), "include")
    hdr = os.path.join(inc, "ATen", "core", "PhiloxRNGEngine.h")
    assert os.path.exists(hdr), "torch's PhiloxRNGEngine.h is the independent Philox pin"
    src = os.path.join(os.path.dirname(__file__), "helpers", "aten_philox_pin.cpp")
    exe = str(tmp_path_factory.mktemp("pin") / "aten_philox_pin")
    subprocess.check_call(["g++", "-O1", "-std=c++17", f"-I{inc}", "-o", exe, src])
    return exe


def test_matches_aten_engine(aten_pin):
    rnd = random.Random(1234)
    triples = [(0, 0, 0), (1, 0, 0), (0, 1, 0), (0, 0, 1), (2**64 - 1,) * 3,
               (0, 0, 2**32 - 1), (0, 0, 2**32), (0, 2**32, 0), (2**32, 0, 0)]
    for _ in range(12000):
        triples.append((rnd.getrandbits(64), rnd.getrandbits(64), rnd.getrandbits(64)))
    text = "".join(f"{s} {q} {o}\n" for s, q, o in triples)
    out = subprocess.run([aten_pin], input=text, capture_output=True, text=True, check=True)
    lines = out.stdout.strip().split("\n")
    assert len(lines) == len(triples)
    for (seed, subseq, off), line in zip(triples, lines):
        want = tuple(int(x) for x in line.split())
        ctr = (off & MASK, off >> 32, subseq & MASK, subseq >> 32)
        key = (seed & MASK, seed >> 32)
        assert oracle.philox4x32_10(ctr, key) == want


def test_matches_bigint_restatement():
    rnd = random.Random(99)
    for _ in range(3000):
        ctr = [rnd.getrandbits(32) for _ in range(4)]
        key = [rnd.getrandbits(32) for _ in range(2)]
        assert oracle.philox4x32_10(ctr, key) == py_philox(ctr, key)


def test_rounds_invert():
    rnd = random.Random(7)
    for _ in range(2000):
        ctr = tuple(rnd.getrandbits(32) for _ in range(4))
        key = tuple(rnd.getrandbits(32) for _ in range(2))
        assert py_philox_inverse(oracle.philox4x32_10(ctr, key), key) == ctr


def test_avalanche():
    rnd = random.Random(5)
    flips = []
    for _ in range(400):
        ctr = [rnd.getrandbits(32) for _ in range(4)]
        key = [rnd.getrandbits(32) for _ in range(2)]
        a = oracle.philox4x32_10(ctr, key)
        bit = rnd.randrange(128)
        ctr2 = list(ctr)
        ctr2[bit // 32] ^= 1 << (bit % 32)
        b = oracle.philox4x32_10(ctr2, key)
        flips.append(sum(bin(x ^ y).count("1") for x, y in zip(a, b)))
    m = np.mean(flips)
    assert 60.0 < m < 68.0            # 64 +- a few standard errors (sd ~ 5.7/sqrt(400))
    assert min(flips) > 30


def test_counter_and_lane_layout():
    """Element i uses word i & 3 of block i >> 2; key = seed; counter words 2,3 =
    stream id.  Checked through the exactly invertible uniform transform."""
    for seed, stream in [(0, 0), (1, 2), (0xDEADBEEFCAFEF00D, (5 << 32) | 17)]:
        first = 4 * 1000
        x = oracle.gen(seed, stream, oracle.UNIFORM_PM1, 64, first_elem=first)
        key = (seed & MASK, seed >> 32)
        for q in range(64):
            i = first + q
            j = i >> 2
            w = py_philox((j & MASK, j >> 32, stream & MASK, stream >> 32), key)[i & 3]
            want = np.float32((w >> 8) * 2.0 ** -23 - 1.0)   # exact in fp64 and fp32
            assert x[q] == want


def test_block_index_crosses_32_bits():
    first = (1 << 34) - 8                                     # j crosses 2^32
    x = oracle.gen(3, 0, oracle.UNIFORM_PM1, 16, first_elem=first)
    for q in range(16):
        i = first + q
        j = i >> 2
        w = py_philox((j & MASK, j >> 32, 0, 0), (3, 0))[i & 3]
        assert x[q] == np.float32((w >> 8) * 2.0 ** -23 - 1.0)


def test_first_elem_is_a_window():
    for dist in oracle.DISTS:
        full = oracle.gen(11, 4, dist, 4096)
        for first, n in [(0, 7), (1, 5), (2, 9), (3, 64), (1021, 300), (4095, 1)]:
            part = oracle.gen(11, 4, dist, n, first_elem=first)
            assert np.array_equal(part.view(np.uint32), full[first:first + n].view(np.uint32))
