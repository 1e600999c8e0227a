"""Helpers shared by the GPU parity tests: run a case through the C ABI and
through the oracle, compare field by field."""
from __future__ import annotations

import math

import numpy as np
import torch

import oracle
from paper_2509_14279_b200 import population as pop

EXACT_FIELDS = ("verdict", "flags", "n_over_tol", "n_nan", "n_inf", "n_inf_mismatch",
                "n_comparable", "argmax_abs_err", "argmax_rel_err")
BITWISE_FLOAT_FIELDS = ("max_abs_err", "max_rel_err")
# mean-error statistics: the oracle sums every element in fp64.  The GPU sums a thread's 16
# (fp32 candidates) or 32 (16-bit candidates) errors of a tile in a balanced fp32 tree (4 or 5
# levels), the 32 threads of a warp in 5 more fp32 levels, and everything above that in fp64.
# All terms are non-negative, so the relative error is at most 9 or 10 roundings of 2^-24,
# about 6e-7; the bar is 1e-6.
MEAN_RTOL = 1e-6


def f32_bits(x) -> int:
    return int(np.float32(x).view(np.uint32))


def assert_stats_equal(gpu_row, orc: dict, where: str = "") -> None:
    for f in EXACT_FIELDS:
        assert int(gpu_row[f]) == int(orc[f]), f"{where}: {f}: gpu {int(gpu_row[f])} oracle {int(orc[f])}"
    for f in BITWISE_FLOAT_FIELDS:
        assert f32_bits(gpu_row[f]) == f32_bits(orc[f]), \
            f"{where}: {f}: gpu {float(gpu_row[f])!r} oracle {float(orc[f])!r}"
    for f in ("sum_abs_err", "mean_abs_err"):
        g, o = float(gpu_row[f]), float(orc[f])
        if math.isinf(o) or math.isnan(o):
            assert (math.isinf(g) and math.isinf(o) and g == o) or (math.isnan(g) and math.isnan(o)), \
                f"{where}: {f}: gpu {g} oracle {o}"
        else:
            assert abs(g - o) <= MEAN_RTOL * abs(o), f"{where}: {f}: gpu {g!r} oracle {o!r}"


def oracle_case(ref_np, cands_np, atol, rtol, input_np=None) -> list:
    return [oracle.verify(ref_np, c, atol, rtol, input=input_np) for c in cands_np]


def torch_dtype(code: str):
    return {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[code]


def oracle_gen_tensor(seed, stream, dist, n, dtype: str) -> torch.Tensor:
    """CPU torch tensor of the oracle's generated tensor."""
    a = oracle.gen(seed, stream, dist, n, dtype=oracle.F32 if dtype == "f32" else oracle.BF16)
    return pop.from_bits(a)


def build_case_cpu(plan, ref_cpu: torch.Tensor, inp_cpu, cand_dtype: str) -> list:
    """Materialise a candidate plan on the CPU (the same bytes go to both sides)."""
    return [pop.materialize(c, ref_cpu, inp_cpu, cand_dtype) for c in plan]


def mixed_plan(K: int, n: int, seed: int, bf16: bool = False) -> list:
    """A small plan that exercises every kind at least once when K allows."""
    rng = np.random.default_rng([seed, K, n])
    kinds = [
        pop.Candidate(pop.REF_EXACT),
        pop.Candidate(pop.BF16_ULP if bf16 else pop.NOISE, sigma=1e-7, noise_seed=seed + 1),
        pop.Candidate(pop.CORRUPT, delta=1.0, indices=(int(rng.integers(0, n)),)),
        pop.Candidate(pop.NAN_AT, indices=(int(rng.integers(0, n)),)),
        pop.Candidate(pop.INPUT_COPY),
        pop.Candidate(pop.CONST, value=0.5),
        pop.Candidate(pop.INF_AT, indices=(int(rng.integers(0, n)),)),
        pop.Candidate(pop.ZEROS),
        pop.Candidate(pop.SCALE, factor=1.001),
        pop.Candidate(pop.NOISE, sigma=1e-3, noise_seed=seed + 2),
        pop.Candidate(pop.CORRUPT, delta=0.25,
                      indices=tuple(sorted(set(int(x) for x in rng.integers(0, n, size=min(n, 9)))))),
        pop.Candidate(pop.NOISE, sigma=1e-5, noise_seed=seed + 3),
    ]
    out = []
    for k in range(K):
        c = kinds[k % len(kinds)]
        if k >= len(kinds) and c.kind == pop.NOISE:
            c = pop.Candidate(pop.NOISE, sigma=c.sigma, noise_seed=seed + 100 + k)
        out.append(c)
    return out
