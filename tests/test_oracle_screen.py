"""Pins for the oracle's task-soundness screens (App. A.1, the filtering criteria).

The oracle is compared with numpy restatements written in another style (whole-array
reductions instead of loops), with closed forms, and with special cases whose answer is
known without computing anything.
"""
import math
import os

import numpy as np
import pytest

import oracle

F32 = np.float32


def paper_facts():
    out = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "paper_facts.txt")) as fh:
        for line in fh:
            line = line.split("#", 1)[0].strip()
            if "=" in line:
                k, v = line.split("=", 1)
                out[k.strip()] = v.strip()
    return out


LIM = float(paper_facts()["soundness_threshold"])


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even), returned as uint16 bit patterns."""
    b = a.astype(F32).view(np.uint32).astype(np.uint64)
    b = (b + 0x7FFF + ((b >> 16) & 1)) >> 16
    return b.astype(np.uint16)


def bf16_values(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(F32)


def numpy_screen(outs, range_lim=LIM, std_lim=LIM, spread_lim=LIM):
    """Whole-array restatement (fp32 inputs)."""
    x = np.stack(outs)                                  # [S, rows, cols]
    S, rows, cols = x.shape
    fin = np.isfinite(x)
    v = x[fin].astype(np.float64)
    res = {"n_values": x.size, "n_nonfinite": int((~fin).sum())}
    res["vmin"] = F32(v.min()) if v.size else F32(np.inf)
    res["vmax"] = F32(v.max()) if v.size else F32(-np.inf)
    res["mean"] = float(v.mean()) if v.size else 0.0
    res["std"] = float(v.std()) if v.size else 0.0
    ok = fin.all(axis=0).reshape(-1)
    if S >= 2 and ok.any():
        flat = x.reshape(S, -1)
        spread = np.where(ok, flat.max(axis=0) - flat.min(axis=0), F32(-1)).astype(F32)
        res["max_seed_spread"] = F32(spread.max())
        res["argmax_seed_spread"] = int(np.argmax(spread))
    else:
        res["max_seed_spread"] = F32(-1)
        res["argmax_seed_spread"] = oracle.NO_INDEX
    bits = x.view(np.uint32)
    f = 0
    if v.size and res["vmin"] >= -F32(range_lim) and res["vmax"] <= F32(range_lim):
        f |= oracle.SCREEN_NARROW_RANGE
    if v.size and res["std"] < std_lim:
        f |= oracle.SCREEN_LOW_STD
    if S >= 2 and ok.any() and res["max_seed_spread"] < F32(spread_lim):
        f |= oracle.SCREEN_LOW_SEED_VARIATION
    if rows >= 2 and (bits == bits[:, :1, :]).all():
        f |= oracle.SCREEN_UNIFORM_AXIS0
    if cols >= 2 and (bits == bits[:, :, :1]).all():
        f |= oracle.SCREEN_UNIFORM_AXIS1
    if res["n_nonfinite"]:
        f |= oracle.SCREEN_NONFINITE
    res["flags"] = f
    return res


def assert_same(got: dict, want: dict, where=""):
    for k in ("flags", "n_values", "n_nonfinite", "argmax_seed_spread"):
        assert int(got[k]) == int(want[k]), f"{where}: {k}: {got[k]} != {want[k]}"
    for k in ("vmin", "vmax", "max_seed_spread"):
        assert F32(got[k]).tobytes() == F32(want[k]).tobytes(), f"{where}: {k}: {got[k]} != {want[k]}"
    for k in ("mean", "std"):
        assert got[k] == pytest.approx(want[k], rel=1e-12, abs=1e-15), f"{where}: {k}"


@pytest.mark.parametrize("seed", range(12))
def test_against_whole_array_numpy_on_small_random_cases(seed):
    rng = np.random.default_rng(seed)
    S = int(rng.integers(1, 6))
    rows, cols = int(rng.integers(1, 9)), int(rng.integers(1, 12))
    scale = float(rng.choice([1e-3, 5e-3, 1e-2, 1.0, 1e4]))
    base = rng.standard_normal((rows, cols)) * scale
    outs = [(base + rng.standard_normal((rows, cols)) * scale * float(rng.choice([0, 1e-3, 1]))).astype(F32)
            for _ in range(S)]
    if seed % 3 == 0:                                    # plant non-finite values
        outs[0].reshape(-1)[int(rng.integers(0, rows * cols))] = np.nan
        outs[-1].reshape(-1)[int(rng.integers(0, rows * cols))] = np.inf
    assert_same(oracle.screen(outs), numpy_screen(outs), f"seed {seed}")


def test_closed_form_of_an_arithmetic_ramp():
    # x_i = a + b*i, i < N: mean a + b(N-1)/2, population std |b| sqrt((N^2-1)/12)
    N, a, b = 4096, 0.25, 2.0 ** -10
    x = (a + b * np.arange(N)).astype(F32).reshape(64, 64)       # exact in fp32
    r = oracle.screen([x])
    assert r["mean"] == pytest.approx(a + b * (N - 1) / 2, rel=1e-14)
    assert r["std"] == pytest.approx(b * math.sqrt((N * N - 1) / 12), rel=1e-13)
    assert r["vmin"] == F32(a) and r["vmax"] == F32(a + b * (N - 1))
    assert r["flags"] == 0 and r["max_seed_spread"] == -1.0 and r["argmax_seed_spread"] == oracle.NO_INDEX


def test_a_large_offset_does_not_cost_the_standard_deviation_its_digits():
    # values 1e4 +- 2^-7: the spread is exactly representable, the std is 2^-7
    x = np.full((32, 32), 1e4, dtype=F32)
    x[:, ::2] += F32(2.0 ** -7)
    x[:, 1::2] -= F32(2.0 ** -7)
    r = oracle.screen([x])
    assert r["std"] == pytest.approx(2.0 ** -7, rel=1e-12)
    assert r["flags"] == oracle.SCREEN_LOW_STD | oracle.SCREEN_UNIFORM_AXIS0


def test_each_criterion_alone():
    rng = np.random.default_rng(5)
    big = [rng.standard_normal((16, 24)).astype(F32) for _ in range(3)]
    assert oracle.screen(big)["flags"] == 0
    # (1) narrow range: everything within +-0.01, but varying and seed dependent
    small = [np.clip(b * F32(0.004), -0.01, 0.01).astype(F32) for b in big]
    f = oracle.screen(small, std_lim=0.0, spread_lim=0.0)["flags"]
    assert f == oracle.SCREEN_NARROW_RANGE
    # (2) low standard deviation around a large mean
    near = [(5.0 + b * F32(0.001)).astype(F32) for b in big]
    assert oracle.screen(near, spread_lim=0.0)["flags"] == oracle.SCREEN_LOW_STD
    # (3) uniform along one axis only
    col_pattern = [np.tile(b[:1, :], (16, 1)) for b in big]          # every column constant
    assert oracle.screen(col_pattern)["flags"] == oracle.SCREEN_UNIFORM_AXIS0
    row_pattern = [np.tile(b[:, :1], (1, 24)) for b in big]          # every row constant
    assert oracle.screen(row_pattern)["flags"] == oracle.SCREEN_UNIFORM_AXIS1
    # (4) the same output whatever the seed
    same = [big[0].copy() for _ in range(3)]
    r = oracle.screen(same)
    assert r["flags"] == oracle.SCREEN_LOW_SEED_VARIATION and r["max_seed_spread"] == 0.0
    assert r["argmax_seed_spread"] == 0
    # one element that moves by 0.02 between seeds is enough variation
    same[2][7, 5] += F32(0.02)
    r = oracle.screen(same)
    assert r["flags"] == 0 and r["argmax_seed_spread"] == 7 * 24 + 5


def test_a_constant_output_trips_everything():
    c = [np.full((8, 8), 0.5 * math.tanh(1.0), dtype=F32) for _ in range(2)]
    want = (oracle.SCREEN_LOW_STD | oracle.SCREEN_LOW_SEED_VARIATION | oracle.SCREEN_UNIFORM_AXIS0 |
            oracle.SCREEN_UNIFORM_AXIS1)
    r = oracle.screen(c)
    assert r["flags"] == want and r["std"] == 0.0 and r["vmin"] == r["vmax"]
    z = [np.zeros((8, 8), dtype=F32) for _ in range(2)]
    assert oracle.screen(z)["flags"] == want | oracle.SCREEN_NARROW_RANGE


def test_threshold_edges():
    lim = F32(LIM)
    up = np.nextafter(lim, F32(1))
    x = np.zeros((4, 4), dtype=F32)
    x[1, 2], x[3, 0] = lim, -lim
    assert oracle.screen([x], std_lim=0.0)["flags"] == oracle.SCREEN_NARROW_RANGE        # the range is closed
    x[1, 2] = up
    assert oracle.screen([x], std_lim=0.0)["flags"] == 0
    # spread exactly at the limit is enough variation (strictly below is not)
    a = np.arange(16, dtype=F32).reshape(4, 4)
    b = a.copy(); b[2, 2] += F32(0.5)
    assert oracle.screen([a, b], spread_lim=0.5)["flags"] == 0
    assert oracle.screen([a, b], spread_lim=float(np.nextafter(F32(0.5), F32(1))))["flags"] == \
        oracle.SCREEN_LOW_SEED_VARIATION
    # std exactly at the limit is not low
    two = np.array([[1.0, -1.0]], dtype=F32)
    assert oracle.screen([two], std_lim=1.0)["flags"] == 0
    assert oracle.screen([two], std_lim=1.0000001)["flags"] == oracle.SCREEN_LOW_STD


def test_nonfinite_values_are_counted_and_left_out():
    x = np.arange(12, dtype=F32).reshape(3, 4)
    y = x + F32(1)
    y[0, 1] = np.nan
    x[2, 3] = -np.inf
    r = oracle.screen([x, y])
    assert r["n_nonfinite"] == 2 and r["flags"] & oracle.SCREEN_NONFINITE
    assert r["vmin"] == 0.0 and r["vmax"] == 12.0
    assert r["max_seed_spread"] == 1.0 and r["argmax_seed_spread"] == 0
    allnan = np.full((2, 2), np.nan, dtype=F32)
    r = oracle.screen([allnan, allnan])
    assert r["n_nonfinite"] == 8 and r["vmin"] == np.inf and r["vmax"] == -np.inf
    assert r["max_seed_spread"] == -1.0 and r["argmax_seed_spread"] == oracle.NO_INDEX
    assert not (r["flags"] & (oracle.SCREEN_NARROW_RANGE | oracle.SCREEN_LOW_STD | oracle.SCREEN_LOW_SEED_VARIATION))


def test_signed_zeros_differ_bit_for_bit():
    x = np.zeros((2, 3), dtype=F32)
    assert oracle.screen([x])["flags"] & oracle.SCREEN_UNIFORM_AXIS0
    x[1, 1] = -0.0
    f = oracle.screen([x])["flags"]
    assert not (f & oracle.SCREEN_UNIFORM_AXIS0) and not (f & oracle.SCREEN_UNIFORM_AXIS1)


def test_bf16_outputs_are_their_exact_upcasts():
    rng = np.random.default_rng(9)
    vals = [rng.standard_normal((6, 10)).astype(F32) * F32(0.02) for _ in range(3)]
    bits = [bf16_bits(v) for v in vals]
    got = oracle.screen(bits)
    want = numpy_screen([bf16_values(b) for b in bits])
    assert_same(got, want, "bf16")


def test_single_row_single_column_and_single_seed():
    x = np.full((1, 5), 2.0, dtype=F32)
    f = oracle.screen([x])["flags"]
    assert f & oracle.SCREEN_UNIFORM_AXIS1 and not (f & oracle.SCREEN_UNIFORM_AXIS0)      # one row: no axis 0
    y = np.full((5, 1), 2.0, dtype=F32)
    f = oracle.screen([y])["flags"]
    assert f & oracle.SCREEN_UNIFORM_AXIS0 and not (f & oracle.SCREEN_UNIFORM_AXIS1)
    assert not (f & oracle.SCREEN_LOW_SEED_VARIATION)                                    # one seed: no (4)


def test_bad_arguments():
    with pytest.raises(ValueError):
        oracle.screen([np.zeros((2, 2), dtype=F32), np.zeros((2, 3), dtype=F32)])
    with pytest.raises(TypeError):
        oracle.screen([np.zeros((2, 2), dtype=np.float64)])
