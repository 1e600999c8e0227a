"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The whole population of a workload is verified in one rkv_verify_multi call (as the
benchmark does); a seeded sample of candidates -- every faulty kind present plus a few
benign ones -- is then copied back and checked against the oracle field by field, and
properties that hold at any size are checked for all K candidates.
"""
import numpy as np
import pytest
import torch

import bench
import oracle
from paper_2509_14279_b200 import binding as rkv
from paper_2509_14279_b200 import population as pop
from rkv_testlib import assert_stats_equal

pytestmark = pytest.mark.gpu

DIST_OF = {"c2": 2, "c3": 0, "c4": 3, "c5": 1}       # index into the workload's distribution list


def _sample(plan, rng, n_benign=2):
    """One candidate of every kind in the plan, plus a few more benign ones."""
    by_kind = {}
    for k, c in enumerate(plan):
        by_kind.setdefault(c.kind, []).append(k)
    picks = sorted({ks[int(rng.integers(0, len(ks)))] for ks in by_kind.values()})
    benign = [k for k, c in enumerate(plan) if c.kind not in pop.FAULT_KINDS and k not in picks]
    picks += [benign[int(i)] for i in rng.choice(len(benign), size=min(n_benign, len(benign)), replace=False)]
    return sorted(set(picks))


@pytest.mark.parametrize("name", ["c2", "c3", "c4", "c5"])
def test_full_size_workload_matches_the_oracle_on_sampled_candidates(name):
    free, _ = torch.cuda.mem_get_info()
    if free < 40 << 30:
        pytest.skip("needs 40 GB of free device memory")
    W0 = pop.WORKLOADS[name]
    di = DIST_OF[name] % len(W0.dists)
    # build only the chosen distribution: temporarily narrow the workload's list
    import dataclasses
    pop.WORKLOADS[name] = dataclasses.replace(W0, dists=(W0.dists[di],))
    try:
        W, cases = bench.build_workload(name, rank=0)
    finally:
        pop.WORKLOADS[name] = W0
    case = cases[0]
    descs, K, T = case["descs"], case["K"], len(case["descs"])
    dist = pop.DIST_IDS[case["dist"]]
    stats, joint, ws = rkv.verify_multi(descs, K)
    assert rkv.device_status(ws) == rkv.OK
    got = rkv.stats_to_numpy(stats).reshape(K, T)
    joint = joint.cpu().numpy()

    # ---- properties for every candidate -------------------------------------------------
    for t, d in enumerate(descs):
        g = got[:, t]
        assert np.all(g["n_comparable"] <= d.n) and np.all(g["n_over_tol"] <= d.n)
        assert np.all(g["max_abs_err"] >= g["mean_abs_err"] * (1 - 1e-6))
        assert np.all((g["verdict"] == 0) == ((g["n_over_tol"] == 0) & (g["n_nan"] == 0) &
                                              (g["n_inf_mismatch"] == 0) & ((g["verdict"] & 24) == 0)))
        ok_idx = g["argmax_abs_err"][g["n_comparable"] > 0]
        assert np.all(ok_idx < d.n)
    assert np.array_equal(joint, np.all(got["verdict"] == 0, axis=1).astype(joint.dtype))

    # ---- a sample of candidates against the oracle ---------------------------------------
    rng = np.random.default_rng(123)
    plan = case["plan_last"]
    picks = _sample(plan, rng)
    seed0 = W.seeds[0]
    for t, d in enumerate(descs):
        if d.n < 1 << 20:
            cand_picks = range(K)                # small tensors: every candidate
        elif t == T - 1:
            cand_picks = picks                   # the tensor whose plan is known
        else:
            cand_picks = picks[:3]
        cand_picks = list(cand_picks)[:8] if d.n >= 1 << 20 else list(cand_picks)
        if d.ref is not None:
            ref_np = pop.bits_numpy(d.ref.reshape(-1))
            inp_np = pop.bits_numpy(d.input.reshape(-1))
        else:                                    # fused: the oracle regenerates both tensors itself
            ref_np = oracle.gen(d.ref_gen[0], d.ref_gen[1], d.ref_gen[2], d.n)
            bf = d.cands[0].dtype == torch.bfloat16
            inp_np = oracle.gen(d.input_gen[0], d.input_gen[1], d.input_gen[2], d.n,
                                dtype=oracle.BF16 if bf else oracle.F32)
        for k in cand_picks:
            want = oracle.verify(ref_np, pop.bits_numpy(d.cands[k]), d.atol, d.rtol, input=inp_np)
            assert_stats_equal(got[k, t], want, f"{name} t={t} k={k}")
    # every planted fault of the known plan fails
    for k, c in enumerate(plan):
        if c.kind in pop.FAULT_KINDS:
            assert joint[k] == 0, (k, c.kind)
    del cases, descs
    torch.cuda.empty_cache()
