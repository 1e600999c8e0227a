"""Pins for the oracle's comparison rule: hand-computed tiny cases with planted
faults, torch.isclose / argmax as an independent library statement of the same
rule on finite data, invariants, and the paper's stated facts."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import (CAND_CONST, CAND_COPY_OF_INPUT, FAIL_INF_MISMATCH, FAIL_LOOPHOLE_CONST,
                    FAIL_LOOPHOLE_COPY, FAIL_NAN, FAIL_TOL, HAS_INF, HAS_NAN, NO_INDEX,
                    REF_CONST, REF_COPY_OF_INPUT)

f32 = np.float32


def paper_facts():
    facts = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "paper_facts.txt")) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split("=", 1)
                facts[k.strip()] = v.strip()
    return facts


ATOL = float(paper_facts()["atol"])
RTOL = float(paper_facts()["rtol"])


def ref_vec(n, seed=0):
    return oracle.gen(seed, 0, oracle.NORMAL, n)


def test_identical_outputs_give_zero_error():
    r = ref_vec(64)
    s = oracle.verify(r, r.copy(), ATOL, RTOL)
    assert s["verdict"] == 0 and s["n_over_tol"] == 0
    assert s["max_abs_err"] == 0.0 and s["max_rel_err"] == 0.0 and s["sum_abs_err"] == 0.0
    assert s["argmax_abs_err"] == 0 and s["argmax_rel_err"] == 0   # first comparable element
    assert s["n_comparable"] == 64 and s["mean_abs_err"] == 0.0


@pytest.mark.parametrize("p", [0, 1, 17, 62, 63])
def test_single_corrupted_element_is_located(p):
    r = ref_vec(64)
    c = r.copy()
    c[p] = r[p] + f32(1.0)
    s = oracle.verify(r, c, ATOL, RTOL)
    want = abs(f32(c[p] - r[p]))
    assert s["verdict"] == FAIL_TOL and s["n_over_tol"] == 1
    assert s["argmax_abs_err"] == p and s["max_abs_err"] == want
    assert s["argmax_rel_err"] == p and s["max_rel_err"] == f32(want / abs(r[p]))
    assert s["sum_abs_err"] == float(want)
    assert s["mean_abs_err"] == f32(float(want) / 64)


def test_ties_go_to_the_smaller_index():
    r = np.array([1, 2, 4, 8, 16, 32], dtype=f32)
    c = r.copy()
    c[4] += f32(0.5)      # rel 0.03125
    c[2] += f32(0.5)      # rel 0.125
    c[1] -= f32(0.5)      # rel 0.25  -> same abs error three times; first is index 1
    s = oracle.verify(r, c, ATOL, RTOL)
    assert s["max_abs_err"] == 0.5 and s["argmax_abs_err"] == 1
    assert s["max_rel_err"] == 0.25 and s["argmax_rel_err"] == 1
    assert s["n_over_tol"] == 3
    # equal relative errors: 0.5/2 at index 1 and 1/4 at index 2
    c = r.copy(); c[2] += f32(1.0); c[1] += f32(0.5)
    s = oracle.verify(r, c, ATOL, RTOL)
    assert s["max_rel_err"] == 0.25 and s["argmax_rel_err"] == 1
    assert s["max_abs_err"] == 1.0 and s["argmax_abs_err"] == 2


def test_planted_nan_and_inf():
    r = ref_vec(32)
    c = r.copy(); c[5] = np.nan; c[9] = np.nan
    s = oracle.verify(r, c, ATOL, RTOL)
    assert s["n_nan"] == 2 and s["n_inf"] == 0 and s["n_over_tol"] == 2
    assert s["verdict"] == FAIL_TOL | FAIL_NAN and s["flags"] & HAS_NAN
    assert s["n_comparable"] == 30 and s["max_abs_err"] == 0.0 and s["argmax_abs_err"] == 0
    assert s["n_inf_mismatch"] == 0

    c = r.copy(); c[7] = np.inf; c[8] = -np.inf
    s = oracle.verify(r, c, ATOL, RTOL)
    assert s["n_inf"] == 2 and s["n_inf_mismatch"] == 2 and s["n_over_tol"] == 2
    assert s["verdict"] == FAIL_TOL | FAIL_INF_MISMATCH and s["flags"] & HAS_INF
    assert s["n_comparable"] == 30


def test_matching_infinities_are_close_like_isclose():
    r = np.array([1.0, np.inf, -np.inf, 2.0], dtype=f32)
    s = oracle.verify(r, r.copy(), ATOL, RTOL)
    assert s["verdict"] == 0 and s["n_inf"] == 2 and s["n_comparable"] == 2
    assert bool(torch.isclose(torch.from_numpy(r), torch.from_numpy(r), RTOL, ATOL).all())
    c = r.copy(); c[1] = -np.inf                      # sign differs
    s = oracle.verify(r, c, ATOL, RTOL)
    assert s["verdict"] == FAIL_TOL | FAIL_INF_MISMATCH and s["n_inf_mismatch"] == 1
    c = r.copy(); c[1] = 3.0                          # reference infinite, candidate finite
    s = oracle.verify(r, c, ATOL, RTOL)
    assert s["n_over_tol"] == 1 and s["n_inf_mismatch"] == 1 and s["n_inf"] == 1
    # NaN in both is still a failure (NaN is never close)
    r2 = np.array([1.0, np.nan], dtype=f32)
    s = oracle.verify(r2, r2.copy(), ATOL, RTOL)
    assert s["verdict"] & FAIL_NAN and s["n_over_tol"] == 1


def test_loophole_flags():
    n = 48
    r = ref_vec(n)
    x = oracle.gen(0, 2, oracle.NORMAL, n)
    s = oracle.verify(r, x.copy(), ATOL, RTOL, input=x)
    assert s["flags"] & CAND_COPY_OF_INPUT and s["verdict"] & FAIL_LOOPHOLE_COPY
    assert not s["flags"] & CAND_CONST
    s = oracle.verify(r, np.full(n, 0.5, f32), ATOL, RTOL, input=x)
    assert s["flags"] & CAND_CONST and s["verdict"] & FAIL_LOOPHOLE_CONST
    assert not s["flags"] & CAND_COPY_OF_INPUT
    s = oracle.verify(r, np.zeros(n, f32), ATOL, RTOL, input=x)
    assert s["flags"] & CAND_CONST and s["verdict"] & FAIL_LOOPHOLE_CONST and s["verdict"] & FAIL_TOL
    # one differing element (even only in the sign of zero) clears the flags
    c = np.zeros(n, f32); c[n - 1] = -0.0
    s = oracle.verify(np.zeros(n, f32) + f32(1e-7), c, ATOL, RTOL)
    assert not s["flags"] & CAND_CONST and s["verdict"] == 0
    c = x.copy(); c[3] = np.nextafter(c[3], f32(10))
    assert not oracle.verify(r, c, ATOL, RTOL, input=x)["flags"] & CAND_COPY_OF_INPUT
    # without an input tensor the copy flags never appear
    assert not oracle.verify(r, x.copy(), ATOL, RTOL)["flags"] & (CAND_COPY_OF_INPUT | REF_COPY_OF_INPUT)


def test_paper_constant_exploit_is_flagged_not_failed():
    """App. A listing (Level 2, Task 13): the exploit writes tanh(1.0)*scaling to
    every output, and the task's reference output is that same constant."""
    assert paper_facts()["const_exploit_expr"] == "tanh(1.0)*scaling"
    for scaling in (0.5, 2.0, 3.0):
        v = f32(f32(math.tanh(1.0)) * f32(scaling))
        r = np.full(1000, v, f32)
        s = oracle.verify(r, r.copy(), ATOL, RTOL)
        assert s["verdict"] == 0
        assert s["flags"] & CAND_CONST and s["flags"] & REF_CONST
    # an identity task: reference is the input; passing the input through is no failure
    x = ref_vec(100)
    s = oracle.verify(x, x.copy(), ATOL, RTOL, input=x)
    assert s["verdict"] == 0 and s["flags"] & CAND_COPY_OF_INPUT and s["flags"] & REF_COPY_OF_INPUT


def test_low_magnitude_reference_constant_candidate_fails():
    """App. A.1: outputs inside [-0.01, 0.01] let a constant slip under a loose
    tolerance; the constant flag fails it when the reference is not constant."""
    r = (oracle.gen(3, 0, oracle.UNIFORM_PM1, 256) * f32(1e-6)).astype(f32)
    s = oracle.verify(r, np.zeros(256, f32), ATOL, RTOL)
    assert s["n_over_tol"] == 0
    assert s["verdict"] == FAIL_LOOPHOLE_CONST


def test_zero_reference_elements_are_excluded_from_relative_error():
    r = np.array([0.0, 2.0, 0.0, -4.0], dtype=f32)
    c = np.array([5.0, 2.5, 0.0, -4.0], dtype=f32)
    s = oracle.verify(r, c, ATOL, RTOL)
    assert s["max_abs_err"] == 5.0 and s["argmax_abs_err"] == 0
    assert s["max_rel_err"] == 0.25 and s["argmax_rel_err"] == 1
    s = oracle.verify(np.zeros(4, f32), c, ATOL, RTOL)
    assert s["max_rel_err"] == 0.0 and s["argmax_rel_err"] == NO_INDEX


def test_single_element_tensor():
    r = np.array([3.0], f32)
    s = oracle.verify(r, r.copy(), ATOL, RTOL)
    assert s["verdict"] == 0 and s["flags"] & CAND_CONST and s["flags"] & REF_CONST
    s = oracle.verify(r, np.array([3.5], f32), ATOL, RTOL)
    assert s["verdict"] == FAIL_TOL and s["argmax_abs_err"] == 0 and s["max_abs_err"] == 0.5


def test_no_comparable_elements():
    r = np.array([np.nan, np.inf], f32)
    c = np.array([1.0, np.inf], f32)
    s = oracle.verify(r, c, ATOL, RTOL)
    assert s["n_comparable"] == 0 and s["mean_abs_err"] == 0.0
    assert s["argmax_abs_err"] == NO_INDEX and s["max_abs_err"] == 0.0
    assert s["n_over_tol"] == 1


@pytest.mark.parametrize("dist", oracle.DISTS)
@pytest.mark.parametrize("sigma", [1e-7, 1e-5, 1e-3])
def test_agrees_with_torch_on_finite_data(dist, sigma):
    n = 20000
    r = oracle.gen(21, 0, dist, n)
    rng = np.random.default_rng(dist * 10 + 1)
    c = (r + f32(sigma) * rng.standard_normal(n).astype(f32)).astype(f32)
    s = oracle.verify(r, c, ATOL, RTOL)
    tc, tr = torch.from_numpy(c), torch.from_numpy(r)
    err = (tc - tr).abs()
    assert s["max_abs_err"] == float(err.max())
    assert s["argmax_abs_err"] == int(np.argmax(err.numpy()))        # first occurrence
    # away from the rounding of the threshold itself the counts agree with isclose
    thr = ATOL + RTOL * tr.abs().double()
    margin = (err.double() - thr).abs() > 1e-9 * thr
    close = torch.isclose(tc, tr, rtol=RTOL, atol=ATOL)
    mine_over = err.double() > thr
    assert bool((close[margin] == ~mine_over[margin]).all())
    assert abs(s["n_over_tol"] - int((~close).sum())) <= int((~margin).sum())
    nz = tr != 0
    q = (err[nz] / tr[nz].abs())
    assert s["max_rel_err"] == float(q.max())
    assert s["sum_abs_err"] == pytest.approx(float(err.double().sum()), rel=1e-12)
    assert s["mean_abs_err"] == f32(float(err.double().sum()) / n)


def test_threshold_is_multiply_then_add_each_rounded():
    """Find elements where a fused a + rtol*|r| and the two-step fp32 form round
    differently, with the error placed between: the rule is the two-step form."""
    rng = np.random.default_rng(3)
    atol, rtol = f32(0.37), f32(0.618)           # threshold of the size of |r|: c - r stays exact
    r = rng.uniform(1.0, 2.0, 400000).astype(f32)
    two_step = (atol + (rtol * np.abs(r)).astype(f32)).astype(f32)
    fused = (np.float64(atol) + np.float64(rtol) * np.abs(r).astype(np.float64)).astype(f32)
    idx = np.nonzero(two_step != fused)[0]
    assert idx.size > 100
    hi = np.maximum(two_step, fused)[idx]
    rr = r[idx]
    # place c so that |c - r| lands exactly on the larger of the two thresholds
    c = (rr + hi).astype(f32)
    e = np.abs((c - rr).astype(f32))
    ok = e == hi
    rr, c, e = rr[ok], c[ok], e[ok]
    ts = two_step[idx][ok]
    assert ok.sum() > 20
    want_over = int((~(e <= ts)).sum())
    assert 0 < want_over < e.size
    s = oracle.verify(rr, c, float(atol), float(rtol))
    assert s["n_over_tol"] == want_over


def test_reference_is_on_the_right_of_the_rule():
    """|c - r| <= atol + rtol*|r| is asymmetric: swapping the roles changes the count."""
    r = np.array([100.0], f32)
    c = np.array([100.0 * (1 + 1.5e-2)], f32)
    assert oracle.verify(r, c, 0.0, 1.49e-2)["n_over_tol"] == 1
    assert oracle.verify(c, r, 0.0, 1.49e-2)["n_over_tol"] == 0


def test_invariants():
    n = 5000
    r = oracle.gen(30, 0, oracle.NORMAL, n)
    rng = np.random.default_rng(0)
    c = (r + f32(2e-5) * rng.standard_normal(n).astype(f32)).astype(f32)
    c[77] = np.nan; c[78] = np.inf
    s = oracle.verify(r, c, ATOL, RTOL)
    assert s["n_comparable"] + 2 == n
    assert s["n_over_tol"] <= n and s["max_abs_err"] >= s["mean_abs_err"]
    # power-of-two scaling of (c, r, atol) is exact
    s2 = oracle.verify(r * f32(2), c * f32(2), 2 * ATOL, RTOL)
    for key in ("n_over_tol", "n_nan", "n_inf", "n_comparable", "argmax_abs_err",
                "argmax_rel_err", "max_rel_err", "verdict", "flags"):
        assert s2[key] == s[key], key
    assert s2["max_abs_err"] == 2 * s["max_abs_err"] and s2["sum_abs_err"] == 2 * s["sum_abs_err"]
    # a permutation leaves counts and maxima alone
    perm = rng.permutation(n)
    sp = oracle.verify(r[perm], c[perm], ATOL, RTOL)
    for key in ("n_over_tol", "n_nan", "n_inf", "n_comparable", "max_abs_err", "max_rel_err"):
        assert sp[key] == s[key], key
    assert perm[sp["argmax_abs_err"]] == s["argmax_abs_err"] or \
        abs(c[perm][sp["argmax_abs_err"]] - r[perm][sp["argmax_abs_err"]]) == s["max_abs_err"]
    assert sp["sum_abs_err"] == pytest.approx(s["sum_abs_err"], rel=1e-12)


def test_filtered_relative_maximum_equals_dividing_everything():
    rng = np.random.default_rng(11)
    for trial in range(30):
        n = 4000
        r = rng.standard_normal(n).astype(f32)
        if trial % 3 == 0:                      # many near-ties: few distinct values
            r = rng.choice(np.array([0.0, 1.0, 3.0, 7.0, 1e-3], f32), n)
            c = (r + rng.choice(np.array([0.0, 1e-3, 3e-3, 7e-3, 1e-6], f32), n)).astype(f32)
        elif trial % 3 == 1:                    # adversarial: errors at a fixed ratio of |r|
            c = (r * f32(1.0 + 2.0 ** -10)).astype(f32)
        else:
            c = (r + f32(1e-4) * rng.standard_normal(n).astype(f32)).astype(f32)
        s = oracle.verify(r, c, ATOL, RTOL)
        q, arg = oracle.max_rel_filtered(r, c)
        assert q == s["max_rel_err"]
        assert arg == s["argmax_rel_err"]


def test_bf16_candidates_are_upcast_exactly():
    n = 4096
    r = oracle.gen(40, 0, oracle.NORMAL, n)
    cb = oracle.gen(40, 0, oracle.NORMAL, n, dtype=oracle.BF16)
    cf = (cb.astype(np.uint32) << 16).view(f32)
    s16 = oracle.verify(r, cb, 1e-2, 1.6e-2)
    s32 = oracle.verify(r, cf, 1e-2, 1.6e-2)
    assert s16 == s32 and s16["verdict"] == 0          # one bf16 rounding is within 1.6e-2
    s = oracle.verify(r, cb, ATOL, RTOL)               # but not within 1e-5
    assert s["verdict"] == FAIL_TOL and s["n_over_tol"] > n // 2
    # bf16 input copy
    xb = oracle.gen(40, 2, oracle.NORMAL, n, dtype=oracle.BF16)
    s = oracle.verify(r, xb.copy(), 1e-2, 1.6e-2, input=xb)
    assert s["flags"] & CAND_COPY_OF_INPUT


def test_joint_pass_is_the_conjunction():
    assert paper_facts()["conjunction"] == "all" and paper_facts()["backward_outputs"] == "3"
    v = [[0, 0, 0], [0, 1, 0], [0, 0, 16], [2, 0, 0], [0, 0, 0]]
    assert oracle.joint_pass(v) == [1, 0, 0, 0, 1]


def test_config1_population_verdicts():
    """The eight fixed candidates of the correctness case: pass, fail x5, pass, fail."""
    from paper_2509_14279_b200 import population as pop
    n = 256 * 1024
    r = oracle.gen(0, 0, oracle.NORMAL, n)
    x = oracle.gen(0, 2, oracle.NORMAL, n)
    tr, tx = torch.from_numpy(r), torch.from_numpy(x)
    plan = pop.plan_c1(n, seed=0)
    res = [oracle.verify(r, pop.bits_numpy(pop.materialize(c, tr, tx)), ATOL, RTOL, input=x)
           for c in plan]
    assert [s["verdict"] == 0 for s in res] == [True, False, False, False, False, False, True, False]
    assert res[1]["argmax_abs_err"] == plan[1].indices[0] and res[1]["n_over_tol"] == 1
    assert res[2]["n_nan"] == 1 and res[2]["verdict"] == FAIL_TOL | FAIL_NAN
    assert res[3]["verdict"] == FAIL_TOL | FAIL_LOOPHOLE_CONST
    assert res[4]["verdict"] == FAIL_TOL | FAIL_LOOPHOLE_COPY
    assert res[5]["verdict"] == FAIL_TOL | FAIL_LOOPHOLE_CONST
    assert res[6]["max_abs_err"] == 0.0
    assert res[7]["verdict"] == FAIL_TOL and res[7]["max_rel_err"] == pytest.approx(1e-3, rel=1e-3)


def test_fp16_widening_is_exact_for_every_pattern():
    """orc_f16_to_f32_bits against numpy's float16 -> float32 conversion, all 65536 patterns
    (NaN payloads included: both keep the ten fraction bits in the top of the fp32 fraction)."""
    h = np.arange(65536, dtype=np.uint16)
    want = h.view(np.float16).astype(np.float32).view(np.uint32)
    got = np.array([oracle.f16_to_f32_bits(int(x)) for x in h], dtype=np.uint32)
    nan = np.isnan(h.view(np.float16))
    assert np.array_equal(got[~nan], want[~nan])
    # NaNs: same sign, exponent all ones, the half's payload bits kept (numpy may set the quiet bit)
    assert np.all((got[nan] & 0x7F800000) == 0x7F800000) and np.all((got[nan] & 0x007FFFFF) != 0)
    assert np.array_equal(got[nan] & 0x80000000, want[nan] & 0x80000000)
    assert np.array_equal((got[nan] | 0x00400000), (want[nan] | 0x00400000))


def test_fp16_candidates_follow_the_same_rule():
    """An fp16 candidate is compared as its exact fp32 value: the result equals verifying the
    widened candidate as an fp32 tensor (the flags compare storage bits, which the widening
    keeps distinct)."""
    rng = np.random.default_rng(16)
    n = 4099
    ref = rng.standard_normal(n).astype(np.float32)
    c16 = (ref * (1 + rng.uniform(-1, 1, n) * 2.0 ** -11)).astype(np.float16)
    c16[7] = np.float16(np.nan)
    c16[100] = np.float16(np.inf)
    c16[200] = np.float16(6.1e-5) * np.float16(0.01)          # a subnormal half
    a = oracle.verify(ref, c16, 1e-3, 1e-3)
    b = oracle.verify(ref, c16.astype(np.float32), 1e-3, 1e-3)
    assert a == b
    assert a["n_nan"] == 1 and a["n_inf"] == 1 and a["n_comparable"] == n - 2
    # an fp16 reference and an fp16 input as well
    r16 = ref.astype(np.float16)
    a = oracle.verify(r16, c16, 1e-3, 1e-3, input=c16)
    b = oracle.verify(r16.astype(np.float32), c16.astype(np.float32), 1e-3, 1e-3, input=c16.astype(np.float32))
    assert a == b and a["flags"] & oracle.CAND_COPY_OF_INPUT
