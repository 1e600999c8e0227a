"""GPU parity of the two reference-free loophole checks (cross-seed variation, copy of any
input) against the oracle, through the C ABI: every field bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_14279_b200 import binding as rkv
from paper_2509_14279_b200 import population as pop
from rkv_testlib import f32_bits, oracle_gen_tensor

pytestmark = pytest.mark.gpu

TD = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}


def _candidate_outputs(kind, n, S, dtype, seed):
    """The outputs of one candidate kernel for S input seeds (CPU tensors)."""
    refs = [oracle_gen_tensor(seed, 100 + s, oracle.NORMAL, n, "f32") for s in range(S)]
    if kind == "honest":                      # depends on the input: a different output per seed
        outs = refs
    elif kind == "hardcoded":                 # one constant, whatever the input
        outs = [torch.full((n,), float(np.tanh(1.0) * 2.0)) for _ in range(S)]
    elif kind == "ignores_input":             # a fixed tensor, the same for every seed
        outs = [refs[0].clone() for _ in range(S)]
    elif kind == "nearly_fixed":              # the same up to rounding noise
        outs = [refs[0] * (1.0 + 1e-7 * s) for s in range(S)]
    elif kind == "one_element":               # identical but for a single element of one seed
        outs = [refs[0].clone() for _ in range(S)]
        outs[-1][n // 3] += 0.75
    elif kind == "low_magnitude":             # varies, but by less than the spread limit
        outs = [r * 1e-3 for r in refs]
    elif kind == "nonfinite":
        outs = [r.clone() for r in refs]
        outs[0][n // 2] = float("nan")
        outs[-1][n - 1] = float("inf")
    else:
        raise ValueError(kind)
    return [o.to(TD[dtype]).contiguous() for o in outs]


KINDS = ["honest", "hardcoded", "ignores_input", "nearly_fixed", "one_element", "low_magnitude", "nonfinite"]


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("n,S", [(1, 2), (5, 3), (1000, 1), (4099, 2), (65537, 4), (70001, 6), (200003, 8), (300001, 9),
                                 (1 << 20, 16)])
def test_cross_seed_matches_the_oracle(dtype, n, S):
    outs = [_candidate_outputs(k, n, S, dtype, seed=7 + i) for i, k in enumerate(KINDS)]
    atol, rtol = (1e-5, 1e-5) if dtype == "f32" else (1e-2, 1.6e-2)
    stats, _ = rkv.cross_seed([[t.cuda() for t in row] for row in outs], atol, rtol, 0.01)
    got = rkv.cross_to_numpy(stats)
    for k, row in enumerate(outs):
        want = oracle.cross_seed([pop.bits_numpy(t) for t in row], atol, rtol, 0.01)
        where = f"{KINDS[k]} {dtype} n={n} S={S}"
        assert int(got[k]["flags"]) == want["flags"], where
        assert int(got[k]["n_nonfinite"]) == want["n_nonfinite"], where
        assert int(got[k]["argmax_spread"]) == want["argmax_spread"], where
        assert f32_bits(got[k]["max_spread"]) == f32_bits(want["max_spread"]), where
    if S >= 2 and n >= 1000:
        flags = {KINDS[k]: int(got[k]["flags"]) for k in range(len(KINDS))}
        assert flags["honest"] == 0
        assert flags["hardcoded"] & rkv.CROSS_IDENTICAL and flags["ignores_input"] & rkv.CROSS_IDENTICAL
        assert flags["nearly_fixed"] & rkv.CROSS_WITHIN_TOL
        if dtype == "f32":                    # (16-bit rounding swallows the 1e-7 differences)
            assert not flags["nearly_fixed"] & rkv.CROSS_IDENTICAL
        assert flags["one_element"] == 0 and int(got[KINDS.index("one_element")]["argmax_spread"]) == n // 3
        assert flags["low_magnitude"] & rkv.CROSS_LOW_SPREAD
        assert flags["nonfinite"] & rkv.CROSS_NONFINITE


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("S", [2, 4, 7, 11])
def test_cross_seed_zeros_of_both_signs_and_subnormals(dtype, S):
    """Outputs that differ across seeds only in the sign of a zero, and outputs of subnormal size:
    the spread is a zero of the oracle's sign, the outputs are not identical but within tolerance;
    minimum and maximum of 16-bit values are taken on pairs of values, which must not show."""
    n = 4099
    g = torch.Generator().manual_seed(5)
    signs = [torch.where(torch.rand(n, generator=g) < 0.5, 0.0, -0.0) for _ in range(S)]
    tiny = {"f32": 1e-41, "bf16": 1e-39, "f16": 3e-7}[dtype]
    small = [(torch.randint(-3, 4, (n,), generator=g).double() * tiny).to(TD[dtype]) for _ in range(S)]
    mixed = [torch.where(torch.rand(n, generator=g) < 0.3, sg.to(TD[dtype]), sm) for sg, sm in zip(signs, small)]
    outs = [[t.to(TD[dtype]).contiguous() for t in signs], small, mixed]
    stats, _ = rkv.cross_seed([[t.cuda() for t in row] for row in outs], 1e-5, 1e-5, 0.01)
    got = rkv.cross_to_numpy(stats)
    for k, row in enumerate(outs):
        want = oracle.cross_seed([pop.bits_numpy(t) for t in row], 1e-5, 1e-5, 0.01)
        assert int(got[k]["flags"]) == want["flags"], (k, dtype, S)
        assert int(got[k]["n_nonfinite"]) == want["n_nonfinite"] == 0
        assert int(got[k]["argmax_spread"]) == want["argmax_spread"], (k, dtype, S)
        assert f32_bits(got[k]["max_spread"]) == f32_bits(want["max_spread"]), (k, dtype, S)
    assert f32_bits(got[0]["max_spread"]) == 0 and int(got[0]["argmax_spread"]) == 0
    assert int(got[0]["flags"]) & rkv.CROSS_WITHIN_TOL and not int(got[0]["flags"]) & rkv.CROSS_IDENTICAL


def test_cross_seed_is_deterministic_and_validates():
    outs = [[t.cuda() for t in _candidate_outputs("honest", 123457, 5, "f32", seed=3)] for _ in range(3)]
    a, ws = rkv.cross_seed(outs, 1e-5, 1e-5)
    b, _ = rkv.cross_seed(outs, 1e-5, 1e-5, workspace=ws)
    assert rkv.cross_to_numpy(a).tobytes() == rkv.cross_to_numpy(b).tobytes()
    with pytest.raises(rkv.RkvError) as e:
        rkv.cross_seed([[outs[0][0]] * 17], 1e-5, 1e-5)
    assert e.value.status == rkv.ERR_UNSUPPORTED
    with pytest.raises(rkv.RkvError) as e:
        rkv.cross_seed(outs, -1.0, 1e-5)
    assert e.value.status == rkv.ERR_INVALID_ARG
    with pytest.raises(rkv.RkvError) as e:
        rkv.cross_seed(outs, 1e-5, 1e-5, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.status == rkv.ERR_WORKSPACE


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("n", [1, 3, 9, 4096, 100003, (1 << 21) + 5])
def test_copy_of_any_input_matches_the_oracle(dtype, n):
    """Three operands as in a linear layer's backward pass (activations, weights, the incoming
    gradient), flattened to one size; candidates that copy one of them, differ in the last
    element only, differ in the sign of a zero, or are honest."""
    ops = [oracle_gen_tensor(11, 200 + m, oracle.NORMAL, n, "f32").to(TD[dtype]) for m in range(3)]
    ops.append(ops[1].clone())                                   # a fourth operand equal to the second
    cands = [ops[0].clone(), ops[2].clone(), ops[1].clone(), (ops[0] + ops[1]).to(TD[dtype])]
    c = ops[2].clone(); c.view(torch.int16 if dtype != "f32" else torch.int32)[n - 1] ^= 1      # last element, one bit
    cands.append(c)
    z = torch.zeros(n, dtype=TD[dtype]); cands.append(z)
    if n > 1:
        c = ops[0].clone(); c[n // 2] = ops[0][n // 2] * 0 - 0.0 if float(ops[0][n // 2]) == 0 else -ops[0][n // 2]
        cands.append(c)
    mask, _ = rkv.copy_of_inputs([t.cuda() for t in ops], [t.cuda() for t in cands])
    got = mask.cpu().tolist()
    want = [oracle.copy_of_inputs([pop.bits_numpy(t) for t in ops], pop.bits_numpy(t)) for t in cands]
    assert got == want, (dtype, n)
    assert got[0] == 0b0001 and got[1] == 0b0100 and got[2] == 0b1010 and got[4] == 0
    if n > 1:
        assert got[3] == 0
