"""Parity of rkv_screen_outputs (task-soundness screens, App. A.1) with the oracle.

Exact fields (flags, counts, the argmax index, the spread as a bit pattern, the range as
numbers) must agree exactly.  mean and std are fp64 sums taken in another order and about
a pivot: mean within 1e-12 of the largest magnitude, std within 1e-9 relative (fp64 rounding
of a few hundred terms per thread plus the merge tree, amplified by at most
1 + (pivot - mean)^2 / variance).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_14279_b200 import binding as rkv
from paper_2509_14279_b200 import population as pop
from rkv_testlib import oracle_gen_tensor

pytestmark = pytest.mark.gpu

LIM = 0.01


def run_both(outs_cpu, **lims):
    outs = [o.cuda() for o in outs_cpu]
    stats, _ = rkv.screen_outputs(outs, **lims)
    got = rkv.screen_to_numpy(stats)[0]
    want = oracle.screen([pop.bits_numpy(o.reshape(-1)).reshape(o.shape) for o in outs_cpu], **lims)
    return got, want


def check(outs_cpu, where="", **lims):
    got, want = run_both(outs_cpu, **lims)
    for k in ("flags", "n_values", "n_nonfinite", "argmax_seed_spread"):
        assert int(got[k]) == int(want[k]), f"{where}: {k}: gpu {int(got[k])} oracle {int(want[k])}"
    assert np.float32(got["max_seed_spread"]).tobytes() == np.float32(want["max_seed_spread"]).tobytes(), \
        f"{where}: max_seed_spread: gpu {got['max_seed_spread']} oracle {want['max_seed_spread']}"
    for k in ("vmin", "vmax"):
        assert float(got[k]) == float(want[k]), f"{where}: {k}: gpu {got[k]} oracle {want[k]}"
    scale = max(abs(float(want["vmin"])), abs(float(want["vmax"]))) if want["n_values"] > want["n_nonfinite"] else 1.0
    assert abs(float(got["mean"]) - want["mean"]) <= 1e-12 * max(scale, 1e-300), f"{where}: mean"
    assert abs(float(got["std"]) - want["std"]) <= 1e-9 * want["std"] + 1e-300, \
        f"{where}: std: gpu {float(got['std'])!r} oracle {want['std']!r}"
    return got, want


def gen(seed, stream, dist, shape, dtype="f32"):
    n = shape[0] * shape[1]
    return oracle_gen_tensor(seed, stream, dist, n, dtype).reshape(shape)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", [(1, 1), (1, 7), (7, 1), (3, 5), (16, 24), (33, 100), (257, 1000), (64, 4096),
                                   (1000, 1001), (2048, 2048)])
def test_shapes_and_seed_counts(shape, dtype):
    for S in (1, 2, 5):
        outs = [gen(100 + s, 0, oracle.NORMAL, shape, dtype) for s in range(S)]
        got, _ = check(outs, f"{dtype} {shape} S={S}")
        if shape[0] * shape[1] > 1000:
            assert int(got["flags"]) == 0


@pytest.mark.parametrize("dist", oracle.DISTS)
def test_every_distribution_and_sixteen_seeds(dist):
    outs = [gen(7, s, dist, (512, 1024)) for s in range(16)]
    check(outs, f"dist {dist}")
    with pytest.raises(rkv.RkvError):
        rkv.screen_outputs([o.cuda() for o in outs] + [outs[0].cuda()])


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_each_criterion_alone(dtype):
    td = torch.float32 if dtype == "f32" else torch.bfloat16
    big = [gen(3, s, oracle.NORMAL, (96, 256), dtype) for s in range(3)]
    got, _ = check(big, "sound")
    assert int(got["flags"]) == 0
    small = [(b.float() * 0.004).clamp(-0.0099, 0.0099).to(td) for b in big]     # (bf16(0.01) > 0.01)
    got, _ = check(small, "narrow", std_lim=0.0, spread_lim=0.0)
    assert int(got["flags"]) == rkv.SCREEN_NARROW_RANGE
    near = [(5.0 + b.float() * 0.001).to(td) for b in big]
    got, _ = check(near, "low std", spread_lim=0.0)
    assert int(got["flags"]) & rkv.SCREEN_LOW_STD
    cols = [b[:1, :].repeat(96, 1).contiguous() for b in big]
    got, _ = check(cols, "axis 0")
    assert int(got["flags"]) == rkv.SCREEN_UNIFORM_AXIS0
    rows = [b[:, :1].repeat(1, 256).contiguous() for b in big]
    got, _ = check(rows, "axis 1")
    assert int(got["flags"]) == rkv.SCREEN_UNIFORM_AXIS1
    same = [big[0].clone() for _ in range(3)]
    got, _ = check(same, "same for every seed")
    assert int(got["flags"]) == rkv.SCREEN_LOW_SEED_VARIATION and int(got["argmax_seed_spread"]) == 0
    same[2][50, 77] += 0.5
    got, _ = check(same, "one element moves")
    assert int(got["flags"]) == 0 and int(got["argmax_seed_spread"]) == 50 * 256 + 77
    const = [torch.full((96, 256), 0.380797, dtype=td) for _ in range(2)]
    got, _ = check(const, "constant")
    assert int(got["flags"]) == (rkv.SCREEN_LOW_STD | rkv.SCREEN_LOW_SEED_VARIATION | rkv.SCREEN_UNIFORM_AXIS0 |
                                 rkv.SCREEN_UNIFORM_AXIS1)


def test_a_late_break_of_uniformity_is_seen():
    # uniform along both axes except for the very last element / one element mid tensor
    for pos in [(299, 511), (150, 3), (1, 0), (0, 511)]:
        x = torch.full((300, 512), 1.25)
        x[pos] = 1.2500001
        got, _ = check([x, x.clone()], f"break at {pos}")
        assert not int(got["flags"]) & (rkv.SCREEN_UNIFORM_AXIS0 | rkv.SCREEN_UNIFORM_AXIS1)
    # a column pattern broken in one place: axis 0 no longer uniform, axis 1 never was
    base = gen(4, 0, oracle.NORMAL, (1, 512)).repeat(300, 1).contiguous()
    got, _ = check([base], "column pattern")
    assert int(got["flags"]) == rkv.SCREEN_UNIFORM_AXIS0
    base[299, 100] = -base[299, 100]
    got, _ = check([base], "column pattern broken")
    assert int(got["flags"]) == 0
    z = torch.zeros(64, 64)
    z[63, 63] = -0.0
    got, _ = check([z], "signed zero", std_lim=0.0, range_lim=0.0)
    assert int(got["flags"]) == 0 or int(got["flags"]) == rkv.SCREEN_NARROW_RANGE


def test_nonfinite_values():
    outs = [gen(9, s, oracle.NORMAL, (128, 384)) for s in range(4)]
    outs[0][0, 0] = float("nan")
    outs[1][5, 5] = float("inf")
    outs[3][127, 383] = float("-inf")
    outs[2][64, :] = float("nan")
    got, want = check(outs, "nonfinite")
    assert int(got["n_nonfinite"]) == 3 + 384 and int(got["flags"]) & rkv.SCREEN_NONFINITE
    # three and two outputs take the kernel that loads two positions at a time
    got, _ = check(outs[:3], "nonfinite, three outputs")
    assert int(got["n_nonfinite"]) == 2 + 384
    got, _ = check(outs[1:3], "nonfinite, two outputs")
    assert int(got["n_nonfinite"]) == 1 + 384
    allnan = [torch.full((8, 8), float("nan")) for _ in range(2)]
    got, _ = check(allnan, "all nan")
    assert int(got["argmax_seed_spread"]) == oracle.NO_INDEX and float(got["max_seed_spread"]) == -1.0


def test_large_offset_and_heavy_tail_keep_the_standard_deviation():
    # an offset of 1e4 with deviations of 1e-2; the pivot takes the offset out
    x = [(1e4 + gen(11, s, oracle.UNIFORM_PM1, (256, 512)) * 0.01) for s in range(2)]
    check(x, "offset")
    # a first element far from the mean
    y = [gen(12, s, oracle.STUDENT_T2, (256, 512)) for s in range(2)]
    y[0][0, :8] = 1e6
    check(y, "outliers in the pivot sample")


def test_threshold_edges_and_limits_as_arguments():
    a = torch.arange(64 * 64, dtype=torch.float32).reshape(64, 64)
    b = a.clone(); b[10, 10] += 0.5
    got, _ = check([a, b], "spread at the limit", spread_lim=0.5)
    assert int(got["flags"]) == 0
    got, _ = check([a, b], "spread below the limit", spread_lim=0.5000001)
    assert int(got["flags"]) == rkv.SCREEN_LOW_SEED_VARIATION
    x = torch.zeros(32, 32); x[3, 4] = 0.01; x[9, 9] = -0.01
    got, _ = check([x], "closed range", std_lim=0.0)
    assert int(got["flags"]) == rkv.SCREEN_NARROW_RANGE


def test_full_size_like_the_benchmark():
    shape = (4096, 4096)
    outs = [rkv.gen_inputs_ex(21, s, rkv.DIST_NORMAL, shape[0] * shape[1]).reshape(shape) for s in range(8)]
    stats, ws = rkv.screen_outputs(outs)
    got = rkv.screen_to_numpy(stats)[0]
    assert int(got["flags"]) == 0 and int(got["n_values"]) == 8 * 4096 * 4096 and int(got["n_nonfinite"]) == 0
    assert abs(float(got["mean"])) < 1e-3 and abs(float(got["std"]) - 1.0) < 1e-3
    # sampled element: the spread reported at argmax is the spread of that element, and no
    # sampled element has a larger one
    i = int(got["argmax_seed_spread"])
    col = torch.stack([o.reshape(-1)[i] for o in outs]).cpu().numpy()
    assert np.float32(col.max() - col.min()) == np.float32(got["max_seed_spread"])
    idx = torch.randint(0, 4096 * 4096, (100000,), device="cuda")
    vals = torch.stack([o.reshape(-1)[idx] for o in outs])
    assert float((vals.max(0).values - vals.min(0).values).max()) <= float(got["max_seed_spread"])
    # run to run determinism, reusing the workspace
    stats2, _ = rkv.screen_outputs(outs, workspace=ws)
    assert stats2.cpu().numpy().tobytes() == stats.cpu().numpy().tobytes()
    # the oracle on one seed pair of the same data (slow path kept small)
    sub = [o[:512].contiguous().cpu() for o in outs[:2]]
    check(sub, "oracle on a slice")


def test_error_codes():
    x = torch.zeros(4, 4, device="cuda")
    with pytest.raises(rkv.RkvError):
        rkv.screen_outputs([x], range_lim=-1.0)
    with pytest.raises(rkv.RkvError):
        rkv.screen_outputs([x], workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    with pytest.raises(ValueError):
        rkv.screen_outputs([x, torch.zeros(4, 5, device="cuda")])
