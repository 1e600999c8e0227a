"""GPU parity: the verification path through the C ABI against the oracle.

Bit-exact on verdicts, flags, counts, maxima and their indices; 1e-6 relative
on the error sum and mean (see rkv_testlib.MEAN_RTOL).  The reference / input
tensors handed to the oracle come from the oracle's own generator; the GPU
either reads the same bytes or regenerates them with its own generator.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_14279_b200 import binding as rkv
from paper_2509_14279_b200 import population as pop
from rkv_testlib import (assert_stats_equal, build_case_cpu, mixed_plan, oracle_case,
                         oracle_gen_tensor)

pytestmark = pytest.mark.gpu

ATOL = RTOL = 1e-5


def run_gpu(ref_cpu, cands_cpu, atol, rtol, inp_cpu=None, gen_ref=None, gen_inp=None, ref_dtype=None):
    dev = "cuda"
    cands = [c.to(dev) for c in cands_cpu]
    desc = rkv.TensorDesc(
        n=cands[0].numel(), cands=cands, atol=atol, rtol=rtol,
        ref=None if gen_ref else ref_cpu.to(dev),
        input=None if (gen_inp or inp_cpu is None) else inp_cpu.to(dev),
        ref_gen=gen_ref, input_gen=gen_inp, ref_dtype=ref_dtype)
    stats, joint, ws = rkv.verify_multi([desc], len(cands))
    assert rkv.device_status(ws) == rkv.OK
    return rkv.stats_to_numpy(stats), joint.cpu().numpy()


def check_case(ref_cpu, cands_cpu, atol, rtol, inp_cpu=None, where="", **kw):
    got, joint = run_gpu(ref_cpu, cands_cpu, atol, rtol, inp_cpu, **kw)
    want = oracle_case(pop.bits_numpy(ref_cpu), [pop.bits_numpy(c) for c in cands_cpu], atol, rtol,
                       None if inp_cpu is None else pop.bits_numpy(inp_cpu))
    for k, w in enumerate(want):
        assert_stats_equal(got[k], w, f"{where} k={k}")
        assert int(joint[k]) == int(w["verdict"] == 0)
    return got, want


def test_config1_population():
    n = 256 * 1024
    ref = oracle_gen_tensor(0, 0, oracle.NORMAL, n, "f32")
    inp = oracle_gen_tensor(0, 2, oracle.NORMAL, n, "f32")
    plan = pop.plan_c1(n, seed=0)
    cands = build_case_cpu(plan, ref, inp, "f32")
    got, want = check_case(ref, cands, ATOL, RTOL, inp, where="c1")
    assert [int(g["verdict"]) == 0 for g in got] == [True, False, False, False, False, False, True, False]
    assert int(got[1]["argmax_abs_err"]) == plan[1].indices[0]
    # same case with the reference and the input regenerated on the device
    got2, _ = run_gpu(ref, cands, ATOL, RTOL, gen_ref=(0, 0, rkv.DIST_NORMAL), gen_inp=(0, 2, rkv.DIST_NORMAL))
    assert got2.tobytes() == got.tobytes()


@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 31, 32, 33, 127, 128, 129, 4095, 4096, 4097, 50001])
def test_small_and_ragged_sizes_fp32(n):
    ref = oracle_gen_tensor(20 + n, 0, oracle.NORMAL, n, "f32")
    inp = oracle_gen_tensor(20 + n, 2, oracle.NORMAL, n, "f32")
    for K in (1, 2, 7, 9, 12):
        cands = build_case_cpu(mixed_plan(K, n, seed=n + K), ref, inp, "f32")
        check_case(ref, cands, ATOL, RTOL, inp, where=f"n={n} K={K}")
    cands = build_case_cpu(mixed_plan(5, n, seed=n), ref, inp, "f32")
    check_case(ref, cands, ATOL, RTOL, None, where=f"n={n} no input")


@pytest.mark.parametrize("K", [33, 65, 300])
def test_many_candidates_cross_the_merge_chunk_and_hint_limits(K):
    n = 30011
    ref = oracle_gen_tensor(3, 0, oracle.STUDENT_T2, n, "f32")
    inp = oracle_gen_tensor(3, 2, oracle.STUDENT_T2, n, "f32")
    cands = build_case_cpu(mixed_plan(K, n, seed=K), ref, inp, "f32")
    check_case(ref, cands, ATOL, RTOL, inp, where=f"K={K}")


@pytest.mark.parametrize("cand_dtype", ["f32", "bf16"])
def test_several_tiles_per_block_in_one_part(cand_dtype):
    """More tiles than resident blocks: a block meets the same candidates tile after tile,
    carries its running maxima over, and uses the maxima other blocks have published."""
    n = 4096 * 296 * 2 + 4096 * 40 + 1234
    ref = oracle_gen_tensor(77, 0, oracle.NORMAL, n, "f32")
    inp = oracle_gen_tensor(77, 2, oracle.NORMAL, n, cand_dtype)
    plan = mixed_plan(12, n, seed=77, bf16=cand_dtype == "bf16")
    # equal maxima far apart: the first index must win across blocks and tiles
    plan.append(pop.Candidate(pop.CORRUPT, delta=1.0, indices=(n - 5, n // 2, 4096 * 300 + 17)))
    cands = build_case_cpu(plan, ref, inp, cand_dtype)
    tol = (1e-5, 1e-5) if cand_dtype == "f32" else (1e-2, 1.6e-2)
    check_case(ref, cands, tol[0], tol[1], inp, where=f"multi-tile {cand_dtype}")


@pytest.mark.parametrize("cand_dtype", ["f32", "bf16"])
def test_large_tensor_with_a_warm_up_group(cand_dtype):
    """A tensor large enough to be cut into a leading group of tiles (verified first, by all
    blocks), the bulk, and a tail group of short items (its last tiles, verified last): results
    must not depend on which group an element falls in."""
    tile = 8192               # the larger of the two tile sizes: both dtypes get a second group
    n = tile * 2100 + 77
    ref = oracle_gen_tensor(88, 0, oracle.STUDENT_T2, n, "f32")
    inp = oracle_gen_tensor(88, 2, oracle.STUDENT_T2, n, cand_dtype)
    bf16 = cand_dtype == "bf16"
    plan = [
        pop.Candidate(pop.BF16_ULP if bf16 else pop.NOISE, sigma=1e-7, noise_seed=1),
        # equal errors in the leading group and far behind it: the first index wins
        pop.Candidate(pop.CORRUPT, delta=1.0, indices=(tile * 5 + 3, tile * 18 + 1, n - 2)),
        # the only error lies behind the leading group
        pop.Candidate(pop.CORRUPT, delta=1.0, indices=(tile * 1000 + 11,)),
        pop.Candidate(pop.NAN_AT, indices=(tile * 17 + 4095,)),
        pop.Candidate(pop.INF_AT, indices=(n - 1,)),
        pop.Candidate(pop.INPUT_COPY),
        pop.Candidate(pop.CONST, value=0.5),
        pop.Candidate(pop.REF_EXACT),
        pop.Candidate(pop.SCALE, factor=1.001),
    ]
    cands = build_case_cpu(plan, ref, inp, cand_dtype)
    tol = (1e-5, 1e-5) if not bf16 else (1e-2, 1.6e-2)
    got, want = check_case(ref, cands, tol[0], tol[1], inp, where=f"warm-up {cand_dtype}")
    if not bf16:      # (bf16 rounding of the heavy tail outweighs the planted +1.0)
        assert int(got[1]["argmax_abs_err"]) in (tile * 5 + 3, tile * 18 + 1, n - 2)
    # and with the reference regenerated on the device
    got2, _ = run_gpu(ref, cands, tol[0], tol[1], gen_ref=(88, 0, rkv.DIST_STUDENT_T2),
                      gen_inp=(88, 2, rkv.DIST_STUDENT_T2))
    assert got2.tobytes() == got.tobytes()


@pytest.mark.parametrize("dist", oracle.DISTS)
def test_every_distribution_several_tiles_per_block(dist):
    n = 296 * 128 * 3 + 77            # several tiles, ragged tail
    ref = oracle_gen_tensor(7, 0, dist, n, "f32")
    inp = oracle_gen_tensor(7, 2, dist, n, "f32")
    cands = build_case_cpu(mixed_plan(12, n, seed=dist), ref, inp, "f32")
    check_case(ref, cands, ATOL, RTOL, inp, where=f"dist={dist}")
    # fused: reference and input regenerated on the device
    got_a, _ = run_gpu(ref, cands, ATOL, RTOL, inp)
    got_b, _ = run_gpu(ref, cands, ATOL, RTOL, gen_ref=(7, 0, dist), gen_inp=(7, 2, dist))
    assert got_a.tobytes() == got_b.tobytes()


@pytest.mark.parametrize("cand_dtype,ref_dtype", [("bf16", "f32"), ("bf16", "bf16"), ("f32", "bf16")])
@pytest.mark.parametrize("n", [1, 7, 8, 9, 1000, 4099, 120001])
def test_bf16_combinations(cand_dtype, ref_dtype, n):
    ref = oracle_gen_tensor(31, 0, oracle.NORMAL, n, ref_dtype)
    inp = oracle_gen_tensor(31, 2, oracle.NORMAL, n, cand_dtype)
    cands = build_case_cpu(mixed_plan(12, n, seed=n, bf16=True), ref, inp, cand_dtype)
    check_case(ref, cands, 1e-2, 1.6e-2, inp, where=f"{cand_dtype}/{ref_dtype} n={n}")
    check_case(ref, cands[:5], 1e-2, 1.6e-2, None, where=f"{cand_dtype}/{ref_dtype} n={n} no input")
    # generated reference rounded to ref_dtype, generated input in the candidates' dtype
    got_a, _ = run_gpu(ref, cands, 1e-2, 1.6e-2, inp)
    got_b, _ = run_gpu(ref, cands, 1e-2, 1.6e-2, gen_ref=(31, 0, rkv.DIST_NORMAL),
                       gen_inp=(31, 2, rkv.DIST_NORMAL),
                       ref_dtype=rkv.F32 if ref_dtype == "f32" else rkv.BF16)
    assert got_a.tobytes() == got_b.tobytes()


@pytest.mark.parametrize("atol,rtol", [(1e-2, 1.6e-2), (0.0, 1.6e-2), (1e-2, 0.0), (0.0, 0.0)])
def test_bf16_candidates_at_the_edges_of_the_skip_tests(atol, rtol):
    """Errors proportional to |r| around rtol, reference zeros with errors around atol,
    values so small that e - t*|r| underflows, exact copies, equal quotients in every
    tile, quotients that overflow: everything the bf16 path decides from a sign test."""
    n = 8192 * 5 + 100
    bf = torch.bfloat16
    ref = oracle_gen_tensor(77, 0, oracle.NORMAL, n, "f32")
    inp = oracle_gen_tensor(77, 2, oracle.NORMAL, n, "bf16")
    cands = [ref.to(bf)]
    for k in (0.5, 0.99, 1.0, 1.01, 1.5):
        cands.append((ref * (1.0 + 1.6e-2 * k)).to(bf))
    c = ref.to(bf).clone(); c[30000] = (ref[30000] * 1.05).to(bf); cands.append(c)   # one element, late tile
    c = ref.to(bf).clone(); c[17] = (ref[17] * 1.05).to(bf); cands.append(c)         # one element, first tile
    check_case(ref, cands, atol, rtol, inp, where="proportional")

    # reference zeros: errors just below, at and above atol there; elsewhere rounding only
    sp = oracle_gen_tensor(78, 0, oracle.SPARSE90, n, "f32")
    zi = torch.nonzero(sp == 0).flatten()
    cands = [sp.to(bf)]
    for v in (0.99e-2, 1e-2, 1.01e-2, 1e-30, 1.0):
        c = sp.to(bf).clone(); c[zi[::97]] = torch.tensor(v).to(bf); cands.append(c)
    c = sp.to(bf).clone(); c[zi[-1]] = 0.5; cands.append(c)
    check_case(sp, cands, atol, rtol, inp, where="zeros")

    # tiny magnitudes: products and differences in and below the subnormal range
    for scale in (1e-30, 1e-36, 1e-38, 3e-41):
        tiny = (ref * scale).contiguous()
        cands = [tiny.to(bf), (tiny * 1.01).to(bf), (tiny * 1.02).to(bf), torch.zeros(n, dtype=bf)]
        c = tiny.to(bf).clone(); c[20000] = 1e-20; cands.append(c)                    # quotient overflows
        check_case(tiny, cands, atol, rtol, inp, where=f"tiny {scale}")

    # a reference that bf16 holds exactly: exact copies, and the same quotient everywhere
    rb = ref.to(bf).to(torch.float32)
    cands = [rb.to(bf), (rb * 2.0).to(bf), (rb * 1.5).to(bf), (rb * 1.0078125).to(bf)]
    c = rb.to(bf).clone(); c[n - 1] = (rb[n - 1] * 2.0).to(bf); cands.append(c)
    c = rb.to(bf).clone(); c[0] = (rb[0] * 2.0).to(bf); cands.append(c)
    check_case(rb, cands, atol, rtol, inp, where="exact")
    check_case(rb.to(bf), cands, atol, rtol, inp, where="exact, bf16 reference", ref_dtype=None)


def test_nonfinite_everywhere():
    n = 40000
    ref = oracle_gen_tensor(41, 0, oracle.NORMAL, n, "f32")
    inp = oracle_gen_tensor(41, 2, oracle.NORMAL, n, "f32")
    r2 = ref.clone()
    r2[5] = float("inf"); r2[6] = float("-inf"); r2[7] = float("nan"); r2[30000] = float("inf")
    big = ref.clone(); big[100] = 3e38
    cands = []
    c = r2.clone(); cands.append(c)                                   # matches, NaN vs NaN fails
    c = r2.clone(); c[5] = float("-inf"); cands.append(c)             # sign mismatch
    c = ref.clone(); c[5] = 1.0; cands.append(c)                      # finite vs infinite ref
    c = ref.clone(); c[100] = -3e38; cands.append(c)                  # finite difference overflows
    c = ref.clone(); c[n - 1] = float("nan"); c[0] = float("inf"); cands.append(c)
    c = torch.full((n,), float("nan")); cands.append(c)
    c = torch.full((n,), float("inf")); cands.append(c)
    check_case(r2, cands, ATOL, RTOL, inp, where="nonfinite ref")
    check_case(big, cands, ATOL, RTOL, inp, where="huge ref")
    check_case(ref, cands, ATOL, RTOL, None, where="finite ref")


def test_ties_resolve_to_the_first_index():
    n = 296 * 128 * 2 + 5
    ref = torch.full((n,), 2.0)
    ref[::3] = 4.0
    ref[1::7] = 0.0
    inp = oracle_gen_tensor(1, 2, oracle.UNIFORM_PM1, n, "f32")
    cands = []
    c = ref.clone(); c += 0.5; cands.append(c)                        # same error everywhere
    c = ref.clone(); c[n // 2:] += 0.5; cands.append(c)               # first hit mid-tensor
    c = ref.clone(); c[n - 1] += 0.5; c[n - 3] += 0.5; cands.append(c)
    c = ref.clone(); c[40000] -= 1.0; c[123] += 1.0; c[124] += 1.0; cands.append(c)
    c = ref * 1.5; cands.append(c)                                    # equal relative error
    got, want = check_case(ref, cands, ATOL, RTOL, inp, where="ties")
    assert int(got[0]["argmax_abs_err"]) == 0
    assert int(got[1]["argmax_abs_err"]) == n // 2


def test_multi_tensor_joint_verdict():
    shapes = [70001, 4096, 4096]
    tols = [(1e-5, 1e-5), (1e-5, 1e-5), (1e-4, 1e-5)]
    K = 10
    plans = pop.plan_multi(K, tuple(shapes), seed=3, fault_rate=0.4)
    refs, inps, cands = [], [], []
    for t, n in enumerate(shapes):
        refs.append(oracle_gen_tensor(3, (t << 32) | 0, oracle.NORMAL, n, "f32"))
        inps.append(oracle_gen_tensor(3, (t << 32) | 2, oracle.NORMAL, n, "f32"))
        cands.append([pop.materialize(plans[k][t], refs[t], inps[t], "f32") for k in range(K)])
    descs = [rkv.TensorDesc(n=n, cands=[c.cuda() for c in cands[t]], atol=tols[t][0], rtol=tols[t][1],
                            ref=refs[t].cuda(), input=inps[t].cuda()) for t, n in enumerate(shapes)]
    stats, joint, ws = rkv.verify_multi(descs, K)
    got = rkv.stats_to_numpy(stats).reshape(K, len(shapes))
    verdicts = []
    for k in range(K):
        row = []
        for t in range(len(shapes)):
            w = oracle.verify(pop.bits_numpy(refs[t]), pop.bits_numpy(cands[t][k]), tols[t][0], tols[t][1],
                              input=pop.bits_numpy(inps[t]))
            assert_stats_equal(got[k, t], w, f"k={k} t={t}")
            row.append(w["verdict"])
        verdicts.append(row)
    assert joint.cpu().tolist() == oracle.joint_pass(verdicts)
    assert 0 < sum(joint.cpu().tolist()) < K
    # fused variant: references and inputs regenerated per tensor stream
    descs_f = [rkv.TensorDesc(n=n, cands=descs[t].cands, atol=tols[t][0], rtol=tols[t][1],
                              ref_gen=(3, (t << 32) | 0, rkv.DIST_NORMAL),
                              input_gen=(3, (t << 32) | 2, rkv.DIST_NORMAL)) for t, n in enumerate(shapes)]
    stats_f, joint_f, _ = rkv.verify_multi(descs_f, K)
    assert rkv.stats_to_numpy(stats_f).tobytes() == rkv.stats_to_numpy(stats).tobytes()
    assert torch.equal(joint, joint_f)


def test_mixed_dtype_pair_like_the_large_sweep():
    """Two tensors per candidate pair: an fp32 and a bf16 output of one reference."""
    n, K = 90000, 6
    ref = oracle_gen_tensor(10, 0, oracle.SPARSE90, n, "f32")
    inp32 = oracle_gen_tensor(10, 2, oracle.SPARSE90, n, "f32")
    inp16 = oracle_gen_tensor(10, 2, oracle.SPARSE90, n, "bf16")
    c32 = build_case_cpu(mixed_plan(K, n, seed=1), ref, inp32, "f32")
    c16 = build_case_cpu(mixed_plan(K, n, seed=2, bf16=True), ref, inp16, "bf16")
    descs = [
        rkv.TensorDesc(n=n, cands=[c.cuda() for c in c32], atol=1e-5, rtol=1e-5,
                       ref_gen=(10, 0, rkv.DIST_SPARSE90), input_gen=(10, 2, rkv.DIST_SPARSE90)),
        rkv.TensorDesc(n=n, cands=[c.cuda() for c in c16], atol=1e-2, rtol=1.6e-2,
                       ref_gen=(10, 0, rkv.DIST_SPARSE90), input_gen=(10, 2, rkv.DIST_SPARSE90)),
    ]
    stats, joint, _ = rkv.verify_multi(descs, K)
    got = rkv.stats_to_numpy(stats).reshape(K, 2)
    for k in range(K):
        assert_stats_equal(got[k, 0], oracle.verify(pop.bits_numpy(ref), pop.bits_numpy(c32[k]), 1e-5, 1e-5,
                                                     input=pop.bits_numpy(inp32)), f"f32 k={k}")
        assert_stats_equal(got[k, 1], oracle.verify(pop.bits_numpy(ref), pop.bits_numpy(c16[k]), 1e-2, 1.6e-2,
                                                     input=pop.bits_numpy(inp16)), f"bf16 k={k}")


def test_runs_are_deterministic():
    n, K = 200003, 9
    ref = oracle_gen_tensor(5, 0, oracle.NORMAL, n, "f32")
    inp = oracle_gen_tensor(5, 2, oracle.NORMAL, n, "f32")
    cands = build_case_cpu(mixed_plan(K, n, seed=5), ref, inp, "f32")
    a, _ = run_gpu(ref, cands, ATOL, RTOL, inp)
    for _ in range(3):
        b, _ = run_gpu(ref, cands, ATOL, RTOL, inp)
        assert a.tobytes() == b.tobytes()


def test_plain_two_call_form():
    shape = (256, 1024)
    ref = rkv.gen_inputs(0, rkv.DIST_NORMAL, shape)
    n = ref.numel()
    ref_cpu = oracle_gen_tensor(0, 0, oracle.NORMAL, n, "f32")
    cands_cpu = build_case_cpu(mixed_plan(8, n, seed=0), ref_cpu, ref_cpu, "f32")
    stats = rkv.verify_batch(ref, [c.cuda() for c in cands_cpu], ATOL, RTOL)
    got = rkv.stats_to_numpy(stats)
    want = oracle_case(pop.bits_numpy(ref_cpu), [pop.bits_numpy(c) for c in cands_cpu], ATOL, RTOL)
    for k in range(8):
        assert_stats_equal(got[k], want[k], f"k={k}")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_host_buffer_form(dtype):
    n, K = 150001, 37
    ref = oracle_gen_tensor(6, 0, oracle.NORMAL, n, dtype)
    cands = build_case_cpu(mixed_plan(K, n, seed=6, bf16=dtype == "bf16"), ref, ref, dtype)
    got = rkv.verify_batch_host(ref, cands, 1e-2, 1.6e-2)
    want = oracle_case(pop.bits_numpy(ref), [pop.bits_numpy(c) for c in cands], 1e-2, 1.6e-2)
    for k in range(K):
        assert_stats_equal(got[k], want[k], f"host k={k}")


def test_host_buffer_form_on_a_tensor_with_all_three_item_groups():
    """Chunks of candidates (16, then the rest) over a tensor long enough for the warm-up
    and the tail group; a ragged last tile."""
    n, K = 4096 * 2100 + 5, 20
    ref = oracle_gen_tensor(8, 0, oracle.UNIFORM_PM1, n, "f32")
    plan = mixed_plan(K, n, seed=8)
    plan[17] = pop.Candidate(pop.CORRUPT, delta=1.0, indices=(n - 1,))
    plan[3] = pop.Candidate(pop.NAN_AT, indices=(4096 * 2050 + 7,))
    cands = build_case_cpu(plan, ref, ref, "f32")
    got = rkv.verify_batch_host(ref, cands, ATOL, RTOL)
    want = oracle_case(pop.bits_numpy(ref), [pop.bits_numpy(c) for c in cands], ATOL, RTOL)
    for k in range(K):
        assert_stats_equal(got[k], want[k], f"host, large k={k}")
    assert int(got[17]["argmax_abs_err"]) == n - 1


def test_host_buffer_form_of_the_general_case():
    """rkv_verify_multi_host: an fp32 tensor read from host memory (reference and input) next to
    a bf16 tensor whose reference and input are regenerated on the device; more candidates than
    one chunk holds, so the partial results carry over between the chunk launches."""
    n32, n16, K = 4096 * 40 + 3, 8192 * 33 + 5, 37
    ref32 = oracle_gen_tensor(21, 0, oracle.NORMAL, n32, "f32")
    inp32 = oracle_gen_tensor(21, 2, oracle.NORMAL, n32, "f32")
    ref16 = oracle_gen_tensor(21, 1 << 32, oracle.UNIFORM_PM1, n16, "f32")
    inp16 = oracle_gen_tensor(21, (1 << 32) | 2, oracle.UNIFORM_PM1, n16, "bf16")
    c32 = build_case_cpu(mixed_plan(K, n32, seed=31), ref32, inp32, "f32")
    c16 = build_case_cpu(mixed_plan(K, n16, seed=32, bf16=True), ref16, inp16, "bf16")
    c16 = c16[12:] + c16[:12]               # another order than the fp32 tensor, same kinds per position
    descs = [
        rkv.TensorDesc(n=n32, cands=c32, atol=1e-5, rtol=1e-5, ref=ref32, input=inp32),
        rkv.TensorDesc(n=n16, cands=c16, atol=1e-2, rtol=1.6e-2,
                       ref_gen=(21, 1 << 32, rkv.DIST_UNIFORM_PM1), input_gen=(21, (1 << 32) | 2, rkv.DIST_UNIFORM_PM1)),
    ]
    got, joint = rkv.verify_multi_host(descs, K)
    verdicts = []
    for k in range(K):
        w0 = oracle.verify(pop.bits_numpy(ref32), pop.bits_numpy(c32[k]), 1e-5, 1e-5, input=pop.bits_numpy(inp32))
        w1 = oracle.verify(pop.bits_numpy(ref16), pop.bits_numpy(c16[k]), 1e-2, 1.6e-2, input=pop.bits_numpy(inp16))
        assert_stats_equal(got[k, 0], w0, f"host multi f32 k={k}")
        assert_stats_equal(got[k, 1], w1, f"host multi bf16 k={k}")
        verdicts.append([w0["verdict"], w1["verdict"]])
    assert joint.tolist() == oracle.joint_pass(verdicts)
    assert 0 < int(joint.sum()) < K


def test_error_codes_on_device():
    n = 1024
    ref = torch.zeros(n + 4, device="cuda")
    cand = torch.zeros(n, device="cuda")
    d = rkv.TensorDesc(n=n, cands=[cand], atol=1e-5, rtol=1e-5, ref=ref[1:n + 1])
    with pytest.raises(rkv.RkvError) as e:
        rkv.verify_multi([d], 1)
    assert e.value.status == rkv.ERR_ALIGNMENT
    d = rkv.TensorDesc(n=n, cands=[cand], atol=1e-5, rtol=1e-5, ref=ref[:n])
    with pytest.raises(rkv.RkvError) as e:
        rkv.verify_multi([d], 1, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == rkv.ERR_WORKSPACE
    d = rkv.TensorDesc(n=n, cands=[cand], atol=-1.0, rtol=1e-5, ref=ref[:n])
    with pytest.raises(rkv.RkvError) as e:
        rkv.verify_multi([d], 1)
    assert e.value.status == rkv.ERR_INVALID_ARG


def test_a_capturing_stream_is_refused_and_nothing_is_recorded():
    """The descriptor tables travel from host memory that dies with the call, so a call on a
    stream under capture must return UNSUPPORTED without enqueueing anything.  The capture is
    ended without ever being replayed."""
    n = 4096
    ref = torch.zeros(n, device="cuda")
    cands = [torch.zeros(n, device="cuda")]
    d = rkv.TensorDesc(n=n, cands=cands, atol=1e-5, rtol=1e-5, ref=ref)
    stats, joint, ws = rkv.verify_multi([d], 1)                       # buffers allocated outside the capture
    rkv.verify_batch(ref, cands, 1e-5, 1e-5, stats_out=stats)         # grows the library's own scratch now
    rkv.verify_batch_static(ref, cands, 1e-5, 1e-5, stats)            # first static call outside capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    seen = []
    with torch.cuda.stream(side):
        graph.capture_begin(capture_error_mode="thread_local")
        try:
            for call in (lambda: rkv.verify_multi([d], 1, workspace=ws, stats_out=stats, joint_pass=joint),
                         lambda: rkv.verify_batch(ref, cands, 1e-5, 1e-5, stats_out=stats),
                         lambda: rkv.verify_batch_static(ref, cands, 1e-5, 1e-5, stats)):
                try:
                    call()
                    seen.append(rkv.OK)
                except rkv.RkvError as e:
                    seen.append(e.status)
        finally:
            graph.capture_end()
    del graph
    assert seen == [rkv.ERR_UNSUPPORTED] * 3
    # the same calls work again once the capture has ended
    rkv.verify_multi([d], 1, workspace=ws, stats_out=stats, joint_pass=joint)
    assert rkv.device_status(ws) == rkv.OK
    assert int(rkv.stats_to_numpy(stats)[0]["verdict"]) == 0


@pytest.mark.parametrize("case", range(24))
def test_seeded_random_cases_match_the_oracle(case):
    """Sizes, candidate counts, dtypes, distributions and tolerances drawn from a seeded
    generator: every statistic of every candidate against the oracle."""
    rng = np.random.default_rng([2509, case])
    n = int(rng.choice([1, 2, 7, 33, 1000, 3583, 3584, 3585, 4096, 7168, 7169, 8193, 20000, 65537, 200003, 1048577]))
    if case % 6 == 5:
        n = int(rng.integers(1, 300000))
    K = int(rng.choice([1, 2, 3, 12, 13, 31, 64, 65, 70]))
    cand_dtype, ref_dtype = [("f32", "f32"), ("bf16", "f32"), ("bf16", "bf16"), ("f32", "bf16")][case % 4]
    dist = int(rng.choice(oracle.DISTS))
    atol, rtol = [(1e-5, 1e-5), (1e-2, 1.6e-2), (0.0, 1e-3), (1e-3, 0.0), (0.0, 0.0), (1.0, 1.0)][int(rng.integers(0, 6))]
    with_input = bool(rng.integers(0, 2))
    ref = oracle_gen_tensor(300 + case, 0, dist, n, ref_dtype)
    inp = oracle_gen_tensor(300 + case, 2, dist, n, cand_dtype)
    cands = build_case_cpu(mixed_plan(K, n, seed=case, bf16=(cand_dtype == "bf16")), ref, inp, cand_dtype)
    where = f"case {case}: n={n} K={K} {cand_dtype}/{ref_dtype} dist={dist} tol=({atol},{rtol}) input={with_input}"
    got, _ = check_case(ref, cands, atol, rtol, inp if with_input else None, where=where)
    # the same bytes with reference (and input) regenerated on the device
    got2, _ = run_gpu(ref, cands, atol, rtol, gen_ref=(300 + case, 0, dist),
                      gen_inp=(300 + case, 2, dist) if with_input else None,
                      ref_dtype=rkv.F32 if ref_dtype == "f32" else rkv.BF16)
    assert got2.tobytes() == got.tobytes(), where


@pytest.mark.parametrize("cand_dtype,ref_dtype", [("f16", "f32"), ("f16", "f16"), ("f32", "f16"), ("bf16", "f16")])
@pytest.mark.parametrize("n", [1, 9, 7168, 7169, 100003])
def test_fp16_storage(cand_dtype, ref_dtype, n):
    """Half-precision candidates and references (the paper's kernels dispatch half too): widened
    exactly, compared by the same rule; flags compare storage bits."""
    K = 13
    ref = oracle_gen_tensor(40, 0, oracle.NORMAL, n, "f32").to(torch_dtype_of(ref_dtype))
    inp = oracle_gen_tensor(40, 2, oracle.NORMAL, n, "f32").to(torch_dtype_of(cand_dtype))
    plan = mixed_plan(K, n, seed=40 + n % 7, bf16=cand_dtype != "f32")
    cands = build_case_cpu(plan, ref, inp, cand_dtype)
    tol = (1e-2, 1.6e-2) if cand_dtype == "bf16" else (1e-3, 2e-3)
    got, want = check_case(ref, cands, tol[0], tol[1], inp, where=f"fp16 {cand_dtype}/{ref_dtype} n={n}")
    if n > 1:
        assert any(int(g["verdict"]) == 0 for g in got) and any(int(g["verdict"]) != 0 for g in got)


def torch_dtype_of(code):
    return {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[code]


def test_fp16_cannot_be_regenerated():
    n = 1024
    c = [torch.zeros(n, dtype=torch.float16, device="cuda")]
    d = rkv.TensorDesc(n=n, cands=c, atol=1e-3, rtol=1e-3, ref=torch.zeros(n, device="cuda"), input_gen=(0, 2, 0))
    with pytest.raises(rkv.RkvError) as e:
        rkv.verify_multi([d], 1)
    assert e.value.status == rkv.ERR_UNSUPPORTED
    d = rkv.TensorDesc(n=n, cands=c, atol=1e-3, rtol=1e-3, ref_gen=(0, 0, 0), ref_dtype=rkv.F16)
    with pytest.raises(rkv.RkvError) as e:
        rkv.verify_multi([d], 1)
    assert e.value.status == rkv.ERR_UNSUPPORTED


def test_error_sum_bits_do_not_depend_on_which_block_took_which_tile():
    """A tensor of thousands of tiles (blocks draw tickets: which block verifies which tile
    differs from run to run) with heavy-tailed errors spanning many binades.  The sum is stored
    per tile and added in tile order, so every run gives the same bits; a second workspace and
    the host-buffer form (other launches, other candidate chunks) give them too."""
    n, K = 3584 * 2500 + 11, 5
    ref = oracle_gen_tensor(50, 0, oracle.NORMAL, n, "f32")
    noise = oracle_gen_tensor(50, 4, oracle.STUDENT_T2, n, "f32")
    cands = [ref + noise * s for s in (1e-9, 1e-4, 1.0, 1e4, 1e-12)]
    runs = [run_gpu(ref, cands, ATOL, RTOL)[0] for _ in range(4)]
    for r in runs[1:]:
        assert r.tobytes() == runs[0].tobytes()
    host = rkv.verify_batch_host(ref, cands, ATOL, RTOL)
    assert host.tobytes() == runs[0].tobytes()
    want = oracle_case(pop.bits_numpy(ref), [pop.bits_numpy(c) for c in cands], ATOL, RTOL)
    for k in range(K):
        assert_stats_equal(runs[0][k], want[k], f"k={k}")


def test_a_bounded_wait_that_runs_out_is_reported_and_the_workspace_stays_usable():
    """Fault drill: block 0 skips its third copy -- the ring stage is neither armed nor filled,
    so nothing is in flight because of it and nothing faults -- and every wait of that launch
    gives up after about a millisecond.  The kernel must return, the status word must say TIMEOUT, and the next
    ordinary call on the same workspace must match the oracle."""
    n, K = 3584 * 700 + 5, 6
    ref = oracle_gen_tensor(60, 0, oracle.NORMAL, n, "f32")
    cands_cpu = build_case_cpu(mixed_plan(K, n, seed=60), ref, ref, "f32")
    cands = [c.cuda() for c in cands_cpu]
    d = rkv.TensorDesc(n=n, cands=cands, atol=ATOL, rtol=RTOL, ref=ref.cuda())
    stats, joint, ws = rkv.verify_multi([d], K)
    assert rkv.device_status(ws) == rkv.OK
    rkv.debug_fault_drill(3, 2_000_000)
    rkv.verify_multi([d], K, workspace=ws, stats_out=stats, joint_pass=joint)
    assert rkv.device_status(ws) == rkv.ERR_TIMEOUT
    # the drill applied to that one call only
    rkv.verify_multi([d], K, workspace=ws, stats_out=stats, joint_pass=joint)
    assert rkv.device_status(ws) == rkv.OK
    got = rkv.stats_to_numpy(stats)
    want = oracle_case(pop.bits_numpy(ref), [pop.bits_numpy(c) for c in cands_cpu], ATOL, RTOL)
    for k in range(K):
        assert_stats_equal(got[k], want[k], f"after the drill k={k}")


@pytest.mark.parametrize("dtype,tile", [("f32", 3584), ("bf16", 7168)])
def test_copy_of_a_regenerated_input_on_a_tensor_with_a_warm_up_group(dtype, tile):
    """Reference and input regenerated on the device, a tensor long enough to have a warm-up
    group: the candidates are compared with the input on the warm-up tiles only, and whoever is
    still bit-equal to it afterwards is compared over the whole tensor by the copy-check kernel.
    A true copy must be flagged; copies that differ in one element (inside the warm-up tiles,
    right behind them, in the middle, at the very end) must not."""
    n = tile * 2048 + (1234 if dtype == "f32" else 77)
    odt = "f32" if dtype == "f32" else "bf16"
    ref = oracle_gen_tensor(5, 0, oracle.UNIFORM_PM1, n, "f32")
    inp = oracle_gen_tensor(5, 2, oracle.UNIFORM_PM1, n, odt)
    def copy_but(i):
        c = inp.clone()
        c[i] = 0.25 if float(c[i]) != 0.25 else 0.5
        return c
    cands = [inp.clone(), copy_but(3 * tile + 1), copy_but(18 * tile + 5), copy_but(n // 2 + 3), copy_but(n - 1),
             pop.materialize(pop.Candidate(pop.REF_EXACT), ref, inp, dtype),
             pop.materialize(pop.Candidate(pop.BF16_ULP if dtype == "bf16" else pop.NOISE, sigma=1e-7, noise_seed=9),
                             ref, inp, dtype),
             inp.clone()]
    tol = (1e-5, 1e-5) if dtype == "f32" else (1e-2, 1.6e-2)
    got, joint = run_gpu(ref, cands, tol[0], tol[1], gen_ref=(5, 0, rkv.DIST_UNIFORM_PM1),
                         gen_inp=(5, 2, rkv.DIST_UNIFORM_PM1))
    want = oracle_case(pop.bits_numpy(ref), [pop.bits_numpy(c) for c in cands], tol[0], tol[1], pop.bits_numpy(inp))
    for k, w in enumerate(want):
        assert_stats_equal(got[k], w, f"copy check {dtype} k={k}")
    copy_flag = [bool(int(g["flags"]) & rkv.FLAG_CAND_COPY_OF_INPUT) for g in got]
    assert copy_flag == [True, False, False, False, False, False, False, True]


@pytest.mark.parametrize("dtype", ["bf16", "f16"])
def test_two_candidates_per_step_fall_back_late_in_a_long_tensor(dtype):
    """16-bit candidates of a tensor with a warm-up group are taken two per step once the
    published maxima make the common case common.  Planted far behind the warm-up tiles: a new
    largest error, a NaN, an infinity and a lone element over tolerance, each in another
    candidate of a pair (and in both of one pair), so that the step has to give both candidates
    to the one-by-one code, which reads their pieces again from global memory."""
    tile = 7168
    n = tile * 2100 + 13
    ref = oracle_gen_tensor(8, 0, oracle.UNIFORM_PM1, n, "f32")
    td = torch.bfloat16 if dtype == "bf16" else torch.float16
    base = ref.to(td)
    def planted(edits):
        c = base.clone()
        for i, v in edits:
            c[i] = v
        return c
    late = tile * 2000
    cands = [base.clone(), planted([(n - 5, 3.0)]),
             planted([(late + 3, float("nan"))]), planted([(late + tile + 9, float("inf"))]),
             planted([(late + 5 * tile + 1, 0.75), (late + 5 * tile + 2, -0.75)]), base.clone(),
             planted([(late + 77, float(base[late + 77]) + 0.125)])]
    atol, rtol = 1e-2, 1.6e-2
    got, joint = run_gpu(ref, cands, atol, rtol)
    want = oracle_case(pop.bits_numpy(ref), [pop.bits_numpy(c) for c in cands], atol, rtol)
    for k, w in enumerate(want):
        assert_stats_equal(got[k], w, f"late fallback {dtype} k={k}")
        assert int(joint[k]) == int(w["verdict"] == 0)
    assert int(got[1]["argmax_abs_err"]) == n - 5
    assert [int(j) for j in joint] == [1, 0, 0, 0, 0, 1, 0]
