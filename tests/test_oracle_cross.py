"""Pins of the oracle's cross-seed variation check and copy-of-any-input check (Sec. 3, the
loophole list; App. A.1, criterion 4 read on a candidate).  Each is held against a whole-array
numpy restatement on random cases and against planted cases whose answer is known."""
import numpy as np
import pytest

import oracle
from oracle import CROSS_IDENTICAL, CROSS_LOW_SPREAD, CROSS_NONFINITE, CROSS_WITHIN_TOL, NO_INDEX


def _numpy_cross(outs, atol, rtol, lim):
    a = np.stack([o.astype(np.float32) for o in outs])                     # exact widening for fp16
    bits = np.stack([o.view(np.uint16) if o.dtype == np.float16 else o.view(np.uint32) for o in outs])
    S = len(outs)
    fin = np.isfinite(a)
    allfin = fin.all(axis=0)
    ident = bool((bits == bits[0]).all())
    x0 = a[0]
    with np.errstate(invalid="ignore", over="ignore"):
        thr = np.float32(atol) + (np.float32(rtol) * np.abs(x0)).astype(np.float32)
        close = np.abs((a - x0).astype(np.float32)) <= thr
        close = np.where(fin & fin[0], close, np.isinf(a) & (a == x0))
        spread = (a.max(axis=0) - a.min(axis=0)).astype(np.float32)
    within = bool(close[1:].all()) if S > 1 else False
    sp = np.where(allfin, spread, np.float32(-2))
    flags = 0
    if S >= 2 and allfin.any():
        ms = float(sp.max()); arg = int(np.argmax(sp))
    else:
        ms, arg = -1.0, NO_INDEX
    if S >= 2 and ident: flags |= CROSS_IDENTICAL
    if S >= 2 and within: flags |= CROSS_WITHIN_TOL
    if S >= 2 and 0 <= ms < lim: flags |= CROSS_LOW_SPREAD
    if (~allfin).any(): flags |= CROSS_NONFINITE
    return {"flags": flags, "n_nonfinite": int((~allfin).sum()), "argmax_spread": arg, "max_spread": ms}


@pytest.mark.parametrize("seed", range(12))
def test_cross_seed_against_whole_array_numpy(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.choice([1, 2, 17, 1000, 4099]))
    S = int(rng.choice([1, 2, 3, 8]))
    dt = [np.float32, np.float16][seed % 2]
    base = rng.standard_normal(n).astype(np.float32)
    scale = [0.0, 1e-7, 1e-3, 1.0][seed % 4]
    outs = [(base + scale * rng.standard_normal(n)).astype(dt) for _ in range(S)]
    if seed % 3 == 0 and n > 2:
        outs[-1][1] = np.nan
        outs[0][2] = np.inf
        if S > 1:
            outs[1][2] = np.inf
    got = oracle.cross_seed(outs, 1e-5, 1e-5, 0.01)
    want = _numpy_cross(outs, 1e-5, 1e-5, 0.01)
    assert got["flags"] == want["flags"] and got["n_nonfinite"] == want["n_nonfinite"]
    assert got["argmax_spread"] == want["argmax_spread"]
    assert np.float32(got["max_spread"]) == np.float32(want["max_spread"])


def test_a_candidate_that_ignores_its_input_is_identical_across_seeds():
    x = np.full(1000, np.float32(np.tanh(1.0) * 2.0))            # one hard-coded value everywhere
    r = oracle.cross_seed([x, x.copy(), x.copy()], 1e-5, 1e-5)
    assert r["flags"] == CROSS_IDENTICAL | CROSS_WITHIN_TOL | CROSS_LOW_SPREAD
    assert r["max_spread"] == 0.0 and r["argmax_spread"] == 0


def test_a_single_differing_element_is_located_and_clears_the_identical_flag():
    rng = np.random.default_rng(1)
    x = rng.standard_normal(5000).astype(np.float32)
    y = x.copy(); y[3210] += np.float32(0.5)
    z = x.copy(); z[77] += np.float32(0.5)                       # an equal spread at a smaller index: it wins
    r = oracle.cross_seed([x, y], 1e-5, 1e-5, 0.01)
    assert r["flags"] == 0 and r["argmax_spread"] == 3210
    assert np.float32(r["max_spread"]) == np.float32(y[3210]) - np.float32(x[3210])
    r = oracle.cross_seed([x, y, z], 1e-5, 1e-5, 0.01)
    assert r["argmax_spread"] in (77, 3210)
    d77 = np.float32(z[77]) - np.float32(x[77]); d3210 = np.float32(y[3210]) - np.float32(x[3210])
    assert r["argmax_spread"] == (77 if d77 >= d3210 else 3210)
    # within tolerance but not identical: a difference of one ulp
    w = x.copy(); w[5] = np.nextafter(w[5], np.float32(10))
    r = oracle.cross_seed([x, w], 1e-5, 1e-5, 0.01)
    assert r["flags"] == CROSS_WITHIN_TOL | CROSS_LOW_SPREAD


def test_signed_zeros_differ_in_bits_but_not_in_value():
    a = np.zeros(8, dtype=np.float32)
    b = -a
    r = oracle.cross_seed([a, b], 0.0, 0.0, 0.01)
    assert r["flags"] == CROSS_WITHIN_TOL | CROSS_LOW_SPREAD and r["max_spread"] == 0.0


def test_the_tolerance_is_taken_on_seed_zero():
    a = np.array([1.0, 100.0], dtype=np.float32)
    b = np.array([1.0, 100.5], dtype=np.float32)
    assert oracle.cross_seed([a, b], 0.0, 5.0e-3)["flags"] & CROSS_WITHIN_TOL          # 0.5 <= 5e-3 * 100
    assert oracle.cross_seed([b, a], 0.0, 4.99e-3)["flags"] & CROSS_WITHIN_TOL         # 0.5 <= 4.99e-3 * 100.5
    assert oracle.cross_seed([a, b], 0.0, 4.99e-3)["flags"] & CROSS_WITHIN_TOL == 0    # 0.5 >  4.99e-3 * 100
    # threshold edges of the spread limit: strict
    assert oracle.cross_seed([a, b], 0.0, 0.0, 0.5)["flags"] & CROSS_LOW_SPREAD == 0
    assert oracle.cross_seed([a, b], 0.0, 0.0, 0.5000001)["flags"] & CROSS_LOW_SPREAD


def test_nonfinite_elements_are_left_out_of_the_spread():
    a = np.array([1.0, np.nan, np.inf, 4.0], dtype=np.float32)
    b = np.array([1.5, 2.0, np.inf, 4.0], dtype=np.float32)
    r = oracle.cross_seed([a, b], 1.0, 0.0, 0.01)
    assert r["n_nonfinite"] == 2 and r["argmax_spread"] == 0 and r["max_spread"] == 0.5
    assert r["flags"] == CROSS_NONFINITE                        # NaN is never close
    a[1] = 2.0
    assert oracle.cross_seed([a, b], 1.0, 0.0, 0.01)["flags"] == CROSS_NONFINITE | CROSS_WITHIN_TOL   # equal infinities are
    allnan = np.full(4, np.nan, dtype=np.float32)
    r = oracle.cross_seed([allnan, allnan], 1.0, 0.0)
    assert r["max_spread"] == -1.0 and r["argmax_spread"] == NO_INDEX and r["flags"] == CROSS_NONFINITE | CROSS_IDENTICAL


def test_copy_of_any_input():
    rng = np.random.default_rng(3)
    n = 3000
    x, w, g = (rng.standard_normal(n).astype(np.float32) for _ in range(3))
    assert oracle.copy_of_inputs([x, w, g], w.copy()) == 0b010
    assert oracle.copy_of_inputs([x, w, g], g.copy()) == 0b100
    assert oracle.copy_of_inputs([x, w, g], (x + w).astype(np.float32)) == 0
    assert oracle.copy_of_inputs([x, x.copy(), g], x.copy()) == 0b011        # two equal inputs: both bits
    y = x.copy(); y[n - 1] = np.nextafter(y[n - 1], np.float32(9))
    assert oracle.copy_of_inputs([x], y) == 0                                 # one element, one ulp
    z = np.zeros(4, np.float32)
    assert oracle.copy_of_inputs([z], -z) == 0                                # a copy is a byte copy: -0 != +0
    h = rng.standard_normal(100).astype(np.float16)
    assert oracle.copy_of_inputs([h[::-1].copy(), h], h.copy()) == 0b10
    for seed in range(5):                                                     # against numpy on random masks
        r2 = np.random.default_rng(seed)
        ins = [r2.integers(0, 3, 50).astype(np.float32) for _ in range(4)]
        c = ins[int(r2.integers(0, 4))].copy() if seed % 2 else r2.integers(0, 3, 50).astype(np.float32)
        want = sum(1 << m for m, a in enumerate(ins) if np.array_equal(a.view(np.uint32), c.view(np.uint32)))
        assert oracle.copy_of_inputs(ins, c) == want
