"""rkv_verify_sweep: many test cases of one task in one launch.

The paper calls a kernel correct iff it passes for ALL input sizes x initialisation
settings x seeds (App. "Kernel Evaluation Environment"), the cases being expanded from the
single_/multi_ config lists of a task (listing "Linear config").  The shapes below are the
small ones of those listings (batch 16 / 64 / 4, features 128 / 4096 / 10, a scalar loss),
as forward outputs (one tensor) and backward outputs (three gradient tensors), in the
three storage types.  Every (case, candidate, tensor) result is compared with the oracle,
the per-case verdict with the oracle's AND over tensors, the overall verdict with the AND
over cases.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_14279_b200 import binding as rkv
from paper_2509_14279_b200 import population as pop
from rkv_testlib import assert_stats_equal, build_case_cpu, mixed_plan, oracle_gen_tensor

pytestmark = pytest.mark.gpu

TD = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}


def _case_list(K, seed):
    """[(tensors of the case: [(n, cand_dtype, ref_dtype, atol, rtol)])]"""
    shapes = [(16, 128), (64, 128), (4, 128), (16, 4096), (64, 4096), (4, 10), (64, 10), (1,)]
    cases = []
    rng = np.random.default_rng(seed)
    for i, shp in enumerate(shapes):
        n = int(np.prod(shp))
        kind = ["f32", "bf16", "f16"][i % 3]
        tol = (1e-5, 1e-5) if kind == "f32" else (1e-2, 1.6e-2) if kind == "bf16" else (1e-3, 2e-3)
        cases.append([(n, kind, "f32", *tol)])                                   # a forward output
        if len(shp) == 2:                                                        # a backward triple
            b, f = shp
            cases.append([(b * f, "f32", "f32", 1e-5, 1e-5), (f * 10, "f32", "f32", 1e-5, 1e-5),
                          (10, "f32", "f32", 1e-4, 1e-5)])
    return cases


def _build(K, seed):
    spec = _case_list(K, seed)
    cases_gpu, cases_cpu = [], []
    for c, tensors in enumerate(spec):
        g, h = [], []
        for t, (n, cdt, rdt, atol, rtol) in enumerate(tensors):
            s = seed + 100 * c + t
            ref = oracle_gen_tensor(s, 0, oracle.DISTS[(c + t) % 5], n, "f32").to(TD[rdt])
            inp = oracle_gen_tensor(s, 2, oracle.DISTS[(c + t) % 5], n, "f32").to(TD[cdt])
            # the same candidate kernels in every case: kind by candidate index, faults hit only some cases
            plan = mixed_plan(K, n, seed=s, bf16=cdt != "f32")
            for k in range(K):
                if plan[k].is_fault and (c + k) % 3 != 0:
                    plan[k] = pop.Candidate(pop.REF_EXACT)
            cands = build_case_cpu(plan, ref, inp, cdt)
            h.append((ref, inp, cands, atol, rtol))
            g.append(rkv.TensorDesc(n=n, cands=[x.cuda() for x in cands], atol=atol, rtol=rtol,
                                    ref=ref.cuda(), input=inp.cuda()))
        cases_gpu.append(g)
        cases_cpu.append(h)
    return cases_gpu, cases_cpu


@pytest.mark.parametrize("K", [1, 8, 70])
def test_sweep_matches_the_oracle_case_by_case(K):
    cases_gpu, cases_cpu = _build(K, seed=500 + K)
    stats, case_pass, all_pass, ws = rkv.verify_sweep(cases_gpu, K)
    assert rkv.device_status(ws) == rkv.OK
    got = rkv.stats_to_numpy(stats)
    case_pass = case_pass.cpu().numpy()
    all_pass = all_pass.cpu().numpy()
    at = 0
    want_all = np.ones(K, dtype=np.int64)
    for c, tensors in enumerate(cases_cpu):
        T = len(tensors)
        verdicts = [[0] * T for _ in range(K)]
        for t, (ref, inp, cands, atol, rtol) in enumerate(tensors):
            for k in range(K):
                w = oracle.verify(pop.bits_numpy(ref), pop.bits_numpy(cands[k]), atol, rtol, input=pop.bits_numpy(inp))
                assert_stats_equal(got[at + k * T + t], w, f"case {c} k={k} t={t}")
                verdicts[k][t] = w["verdict"]
        want_case = oracle.joint_pass(verdicts)
        assert case_pass[c].tolist() == want_case, f"case {c}"
        want_all &= np.array(want_case)
        at += K * T
    assert all_pass.tolist() == want_all.tolist()
    if K >= 8:
        assert 0 < int(all_pass.sum()) < K


def test_sweep_equals_one_call_per_case():
    K = 9
    cases_gpu, _ = _build(K, seed=77)
    stats, case_pass, all_pass, _ = rkv.verify_sweep(cases_gpu, K)
    got = rkv.stats_to_numpy(stats)
    at = 0
    for c, tensors in enumerate(cases_gpu):
        s1, j1, _ = rkv.verify_multi(tensors, K)
        one = rkv.stats_to_numpy(s1)
        assert got[at:at + K * len(tensors)].tobytes() == one.tobytes(), f"case {c}"
        assert case_pass[c].cpu().tolist() == j1.cpu().tolist()
        at += K * len(tensors)


def test_sweep_with_regenerated_references_and_a_large_case_among_small_ones():
    """One case large enough for all three item groups next to tiny ones; references and
    inputs regenerated on the device."""
    K = 6
    spec = [(3584 * 2200 + 3, "f32", oracle.NORMAL), (10, "f32", oracle.UNIFORM_PM1), (7168 * 3 + 1, "bf16", oracle.SPARSE90),
            (1, "f32", oracle.NORMAL)]
    cases_gpu, cpu = [], []
    for c, (n, cdt, dist) in enumerate(spec):
        ref = oracle_gen_tensor(900 + c, 0, dist, n, "f32")
        inp = oracle_gen_tensor(900 + c, 2, dist, n, cdt)
        cands = build_case_cpu(mixed_plan(K, n, seed=900 + c, bf16=cdt != "f32"), ref, inp, cdt)
        tol = (1e-5, 1e-5) if cdt == "f32" else (1e-2, 1.6e-2)
        cpu.append((ref, inp, cands, tol))
        cases_gpu.append([rkv.TensorDesc(n=n, cands=[x.cuda() for x in cands], atol=tol[0], rtol=tol[1],
                                         ref_gen=(900 + c, 0, dist), input_gen=(900 + c, 2, dist))])
    stats, case_pass, all_pass, ws = rkv.verify_sweep(cases_gpu, K)
    assert rkv.device_status(ws) == rkv.OK
    got = rkv.stats_to_numpy(stats)
    for c, (ref, inp, cands, tol) in enumerate(cpu):
        for k in range(K):
            w = oracle.verify(pop.bits_numpy(ref), pop.bits_numpy(cands[k]), tol[0], tol[1], input=pop.bits_numpy(inp))
            assert_stats_equal(got[c * K + k], w, f"case {c} k={k}")
            assert int(case_pass[c, k]) == int(w["verdict"] == 0)


def test_sweep_of_short_tensors_with_warm_up_and_split_main_groups():
    """Three tensors of 30 to 151 tiles among forty of one tile: more tiles than the first wave of
    blocks holds, so every tensor has a warm-up group of its own (the square root of its tiles), and fewer
    main-group tiles than blocks, so the main group splits the candidates into parts.  Stored and
    regenerated references, the three storage types, faults in every group; a copy of a regenerated
    input goes through the copy check of a short tensor."""
    K = 10
    spec = [(3584 * 150 + 17, "f32", oracle.NORMAL, True), (7168 * 90 + 5, "bf16", oracle.STUDENT_T2, False),
            (7168 * 29 + 7000, "f16", oracle.UNIFORM_PM1, False), (3584 * 40 + 1, "bf16", oracle.NORMAL_1E4, True)]
    spec += [(1 + 97 * i, "f32" if i % 2 else "bf16", oracle.DISTS[i % 5], i % 4 == 0) for i in range(40)]
    cases_gpu, cpu = [], []
    for c, (n, cdt, dist, regenerated) in enumerate(spec):
        rdt = "f32"
        ref = oracle_gen_tensor(1300 + c, 0, dist, n, rdt)
        inp = oracle_gen_tensor(1300 + c, 2, dist, n, "bf16" if cdt == "bf16" else "f32").to(TD[cdt])
        cands = build_case_cpu(mixed_plan(K, n, seed=1300 + c, bf16=cdt != "f32"), ref, inp, cdt)
        tol = (1e-5, 1e-5) if cdt == "f32" else (1e-2, 1.6e-2)
        cpu.append((ref, inp, cands, tol))
        if regenerated and cdt != "f16":
            cases_gpu.append([rkv.TensorDesc(n=n, cands=[x.cuda() for x in cands], atol=tol[0], rtol=tol[1],
                                             ref_gen=(1300 + c, 0, dist), input_gen=(1300 + c, 2, dist))])
        else:
            cases_gpu.append([rkv.TensorDesc(n=n, cands=[x.cuda() for x in cands], atol=tol[0], rtol=tol[1],
                                             ref=ref.cuda(), input=inp.cuda())])
    stats, case_pass, all_pass, ws = rkv.verify_sweep(cases_gpu, K)
    assert rkv.device_status(ws) == rkv.OK
    got = rkv.stats_to_numpy(stats)
    seen_fail = 0
    for c, (ref, inp, cands, tol) in enumerate(cpu):
        for k in range(K):
            w = oracle.verify(pop.bits_numpy(ref), pop.bits_numpy(cands[k]), tol[0], tol[1], input=pop.bits_numpy(inp))
            assert_stats_equal(got[c * K + k], w, f"case {c} k={k}")
            assert int(case_pass[c, k]) == int(w["verdict"] == 0)
            seen_fail += int(w["verdict"] != 0)
    assert seen_fail > 0
    # the same launch twice: byte for byte
    stats2, _, _, _ = rkv.verify_sweep(cases_gpu, K)
    assert rkv.stats_to_numpy(stats2).tobytes() == got.tobytes()
