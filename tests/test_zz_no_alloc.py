"""rkv_verify_batch_static: verification for callers that cannot allocate.

Some users of the library verify from a place where device allocation is off the
table: the process has already given every byte of GPU memory to its own pool, or
the calling thread must not enter the CUDA allocator (it synchronises the whole
device).  For them the library carries an entry point whose scratch is a fixed
array inside the library image.  This test drives it through the C ABI and holds
it to the results of rkv_verify_batch, the allocating form, on the same inputs:
every integer and index field and both maxima bit for bit, the error sum and
mean within the 1e-6 relative bar the other parity tests use -- and, so that two
CUDA paths agreeing with each other cannot hide a common mistake, to the CPU
oracle's results on the same bytes by the same rule.

Two calls in a row share the scratch array (it is never cleared between calls),
so the second call runs a *different* case than the first -- other sizes, other
faults -- and must not see anything the first one left behind; then the first
case runs again.  The file sorts last so that a run stopped at its first failure
has already executed every other test; it also passes when run alone.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_14279_b200 import binding as rkv
from paper_2509_14279_b200 import population as pop
from rkv_testlib import (EXACT_FIELDS, BITWISE_FLOAT_FIELDS, MEAN_RTOL, assert_stats_equal, build_case_cpu,
                         f32_bits, mixed_plan, oracle_gen_tensor)

pytestmark = pytest.mark.gpu


def _case(n, K, seed, dtype="f32"):
    ref = oracle_gen_tensor(seed, 0, oracle.NORMAL, n, dtype)
    cands = build_case_cpu(mixed_plan(K, n, seed=seed, bf16=dtype == "bf16"), ref, ref, dtype)
    return ref.cuda(), [c.cuda() for c in cands]


def _oracle_rows(case, atol, rtol):
    ref, cands = case
    ref_np = pop.bits_numpy(ref)
    return [oracle.verify(ref_np, pop.bits_numpy(c), atol, rtol) for c in cands]


def _assert_same(got, want, where):
    for k in range(len(want)):
        for f in EXACT_FIELDS:
            assert int(got[k][f]) == int(want[k][f]), f"{where} k={k} {f}"
        for f in BITWISE_FLOAT_FIELDS:
            assert f32_bits(got[k][f]) == f32_bits(want[k][f]), f"{where} k={k} {f}"
        for f in ("sum_abs_err", "mean_abs_err"):
            g, w = float(got[k][f]), float(want[k][f])
            if np.isfinite(w):
                assert abs(g - w) <= MEAN_RTOL * abs(w), f"{where} k={k} {f}"
            else:
                assert (np.isnan(g) and np.isnan(w)) or g == w, f"{where} k={k} {f}"


def test_static_scratch_form_matches_the_allocating_form_on_two_calls_in_a_row():
    atol, rtol = 1e-5, 1e-5
    case_a = _case(700001, 24, seed=11)           # several tiles per block, ragged tail
    case_b = _case(4099, 7, seed=12)              # a much smaller case reusing the same scratch
    case_c = _case(300007, 13, seed=13, dtype="bf16")
    want = [rkv.stats_to_numpy(rkv.verify_batch(r, c, atol, rtol)) for r, c in (case_a, case_b, case_c)]
    torch.cuda.synchronize()

    outs = [torch.empty(len(c) * rkv.STATS_BYTES, dtype=torch.uint8, device="cuda")
            for _, c in (case_a, case_b, case_c, case_a)]
    # back to back on one stream, no synchronisation in between
    for out, (r, c) in zip(outs, (case_a, case_b, case_c, case_a)):
        rkv.verify_batch_static(r, c, atol, rtol, out)
    torch.cuda.synchronize()
    for i, name in enumerate(("first call", "second call", "third call (bf16)")):
        _assert_same(rkv.stats_to_numpy(outs[i]), want[i], name)
    _assert_same(rkv.stats_to_numpy(outs[3]), want[0], "first case again")
    # the static form is deterministic: the repeat is byte-identical to the first call
    assert rkv.stats_to_numpy(outs[3]).tobytes() == rkv.stats_to_numpy(outs[0]).tobytes()
    # and every call against the oracle
    for i, (case, name) in enumerate(zip((case_a, case_b, case_c, case_a),
                                         ("first call", "second call", "third call (bf16)", "first case again"))):
        got = rkv.stats_to_numpy(outs[i])
        for k, w in enumerate(_oracle_rows(case, atol, rtol)):
            assert_stats_equal(got[k], w, f"static form vs oracle, {name} k={k}")


def test_static_scratch_form_rejects_what_does_not_fit():
    ref = torch.zeros(1024, device="cuda")
    out = torch.empty(300 * rkv.STATS_BYTES, dtype=torch.uint8, device="cuda")
    with pytest.raises(rkv.RkvError) as e:                      # more candidates than the table holds
        rkv.verify_batch_static(ref, [ref] * 257, 1e-5, 1e-5, out)
    assert e.value.status == rkv.ERR_UNSUPPORTED
    with pytest.raises(rkv.RkvError) as e:                      # ordinary argument checks still apply
        rkv.verify_batch_static(ref, [ref], -1.0, 1e-5, out)
    assert e.value.status == rkv.ERR_INVALID_ARG
