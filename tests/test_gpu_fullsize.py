"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

Every (distribution, seed) pair of a workload is built exactly as the benchmark builds it
and verified in one rkv_verify_multi call.  The oracle then gets the same candidate bytes
(copied back one candidate at a time) and ITS OWN reference and input tensors, generated
on the host cores from the same (seed, stream, distribution) -- where the GPU read those
tensors from memory, the resident copies are first checked bit for bit against the
oracle's.  Which candidates meet the oracle:

  c2   all five distributions, all 64 candidates
  c3   all 64 candidates
  c4   all three distributions; the large tensor: every faulty candidate and 16 benign
       ones; the two small tensors: all 128 candidates
  c5   all 20 (distribution, seed) pairs, seeds 10..13; per tensor every faulty candidate
       and 16 benign ones; the pair (normal, 10) with all 2 x 128 candidates

Properties that hold at any size are checked for every candidate of every case.  The
oracle calls run on the host cores in parallel (ctypes releases the interpreter lock).
"""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

import bench
import oracle
from paper_2509_14279_b200 import binding as rkv
from paper_2509_14279_b200 import population as pop
from rkv_testlib import assert_stats_equal

pytestmark = pytest.mark.gpu

THREADS = max(1, min(os.cpu_count() or 1, 32))
N_BENIGN = 16


def _oracle_tensor(seed, stream, dist, n, bf16, pool):
    """The oracle's tensor (seed, stream, dist), generated in chunks on the pool."""
    chunk = (-(-n // THREADS) + 3) // 4 * 4
    spans = [(s, min(chunk, n - s)) for s in range(0, n, chunk)]
    parts = list(pool.map(lambda sp: oracle.gen(seed, stream, dist, sp[1], dtype=oracle.BF16 if bf16 else oracle.F32,
                                                first_elem=sp[0]), spans))
    return np.concatenate(parts)


def _picks(plan, all_k, rng):
    if all_k:
        return list(range(len(plan)))
    faulty = [k for k, c in enumerate(plan) if c.is_fault]
    benign = [k for k, c in enumerate(plan) if not c.is_fault]
    take = rng.choice(len(benign), size=min(N_BENIGN, len(benign)), replace=False)
    return sorted(faulty + [benign[int(i)] for i in take])


def _check_case(W, case, all_k, pool, where):
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
        assert np.all(g["argmax_abs_err"][g["n_comparable"] > 0] < d.n)
    assert np.array_equal(joint, np.all(got["verdict"] == 0, axis=1).astype(joint.dtype))
    for t, plan in enumerate(case["plans"]):
        for k, c in enumerate(plan):
            if c.kind in pop.SCALE_FREE_FAULT_KINDS:
                assert got[k, t]["verdict"] != 0 and joint[k] == 0, (where, t, k, c.kind)

    # ---- candidates against the oracle, on the oracle's own reference and input -----------
    rng = np.random.default_rng([123, dist, case["seed"]])
    checked = 0
    for t, d in enumerate(descs):
        bf = d.cands[0].dtype == torch.bfloat16
        if d.ref is not None:
            seed, ref_stream, inp_stream = case["gens"][2 * t][0], case["gens"][2 * t][1], case["gens"][2 * t + 1][1]
        else:
            seed, ref_stream, inp_stream = d.ref_gen[0], d.ref_gen[1], d.input_gen[1]
        ref_np = _oracle_tensor(seed, ref_stream, dist, d.n, False, pool)
        inp_np = _oracle_tensor(seed, inp_stream, dist, d.n, bf, pool)
        if d.ref is not None:          # the tensors the GPU read are the oracle's, bit for bit
            assert np.array_equal(pop.bits_numpy(d.ref).view(np.uint32), ref_np.view(np.uint32)), (where, t, "ref")
            assert np.array_equal(pop.bits_numpy(d.input).view(inp_np.dtype if bf else np.uint32),
                                  inp_np if bf else inp_np.view(np.uint32)), (where, t, "input")
        ks = _picks(case["plans"][t], all_k or d.n < (1 << 20), rng)
        for lo in range(0, len(ks), THREADS):
            batch = ks[lo:lo + THREADS]
            hosts = [pop.bits_numpy(d.cands[k]) for k in batch]
            wants = list(pool.map(lambda c: oracle.verify(ref_np, c, d.atol, d.rtol, input=inp_np), hosts))
            for k, want in zip(batch, wants):
                assert_stats_equal(got[k, t], want, f"{where} t={t} k={k} ({case['plans'][t][k].kind})")
            checked += len(batch)
    return checked


def _run(name, all_k_pairs=None, all_k=False):
    free, _ = torch.cuda.mem_get_info()
    if free < 40 << 30:
        pytest.skip("needs 40 GB of free device memory")
    W = pop.WORKLOADS[name]
    pairs = [(d, s) for s in W.seeds for d in W.dists]
    total = 0
    with ThreadPoolExecutor(max_workers=THREADS) as pool:
        for (d, s) in pairs:
            case = bench.build_case(W, d, s)
            every = all_k or (all_k_pairs is not None and (d, s) in all_k_pairs)
            total += _check_case(W, case, every, pool, f"{name} {d} seed {s}")
            del case
            torch.cuda.empty_cache()
    return total, len(pairs)


def test_c2_every_distribution_every_candidate():
    total, pairs = _run("c2", all_k=True)
    assert pairs == 5 and total == 5 * 64


def test_c3_every_candidate():
    total, pairs = _run("c3", all_k=True)
    assert pairs == 1 and total == 64


def test_c4_every_distribution_every_fault_and_sixteen_benign_per_tensor():
    total, pairs = _run("c4")
    assert pairs == 3 and total >= 3 * (16 + 128 + 128)


def test_c5_every_distribution_and_seed():
    total, pairs = _run("c5", all_k_pairs={("normal", 10)})
    assert pairs == 20 and total >= 19 * 2 * 16 + 256
