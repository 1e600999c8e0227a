"""Seeded synthetic candidate populations (inputs *to* the verification path).

This module holds none of the method's arithmetic: it neither generates the
reference / input tensors (the Philox generator does) nor compares anything.
Given a reference and an input tensor it builds the K candidate tensors a
verification call receives, from a seeded plan.  It is the one module that both
the CPU oracle's tests and the CUDA path's tests and benchmark use, so both
sides see the same bytes.  Random draws here come from numpy's PCG64 and
torch's generators, never from the method's Philox streams.

The candidate kinds model behaviours of the candidate kernels printed in the
paper's appendix (arxiv 2509.14279): reordered summation and atomics (small
Gaussian noise), fast-math (relative noise), outputs allocated uninitialised or
only partly written (single / multi element corruption), sentinels leaking
(Inf), NaN, and the loopholes of Sec. 3 / App. A.1: a constant written
everywhere, the input passed through, all zeros.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

# candidate kinds
REF_EXACT = "ref_exact"
NOISE = "noise"            # c = r + sigma * z
SCALE = "scale"            # c = r * factor
CORRUPT = "corrupt"        # m seeded elements get += delta
NAN_AT = "nan_at"          # one seeded element is NaN
INF_AT = "inf_at"          # one seeded element is +Inf
ZEROS = "zeros"
CONST = "const"            # every element = value
INPUT_COPY = "input_copy"
BF16_ULP = "bf16_ulp"      # c = r * (1 + 2^-8 u), u uniform in [-1,1): about one bf16 ulp

FAULT_KINDS = (CORRUPT, NAN_AT, INF_AT, CONST, INPUT_COPY, ZEROS)
# Faults that fail whatever the scale of the data.  A CORRUPT element (+delta) is within
# tolerance where rtol * |r| exceeds delta, as on the 1e4-scaled distribution under the
# bf16 tolerances.
SCALE_FREE_FAULT_KINDS = (NAN_AT, INF_AT, CONST, INPUT_COPY, ZEROS)


@dataclass
class Candidate:
    kind: str
    sigma: float = 0.0
    factor: float = 1.0
    value: float = 0.0
    delta: float = 1.0
    indices: tuple = ()
    noise_seed: int = 0
    # which tensor of a multi-tensor case carries the fault (others get `base`)
    fault_tensor: int = 0
    base: "Candidate | None" = None

    @property
    def is_fault(self) -> bool:
        return self.kind in FAULT_KINDS or (self.kind == NOISE and self.sigma >= 1e-4) \
            or self.kind == SCALE


@dataclass
class Workload:
    """One verification case: shapes, dtypes, tolerances, generator settings."""
    name: str
    K: int
    shapes: tuple               # one shape per tensor of the case
    cand_dtype: str = "f32"     # "f32" | "bf16"
    ref_dtype: str = "f32"
    tols: tuple = ((1e-5, 1e-5),)   # (atol, rtol) per tensor
    dists: tuple = ("normal",)
    seeds: tuple = (0,)
    fault_rate: float = 0.0
    fused: bool = False
    notes: str = ""
    extra: dict = field(default_factory=dict)

    @property
    def numels(self) -> tuple:
        return tuple(int(np.prod(s)) for s in self.shapes)


# The five configurations the benchmark metric is quoted on.  "c5" holds two
# tensors per candidate pair: an fp32 and a bf16 output of the same reference
# (128 + 128 = 256 candidate tensors, 12 GiB streamed).
WORKLOADS = {
    "c1": Workload("c1", 8, ((256, 1024),), seeds=(0,), dists=("normal",),
                   notes="fixed eight candidates, correctness case"),
    "c2": Workload("c2", 64, ((4096, 4096),), seeds=(1,),
                   dists=("normal", "uniform_pm1", "student_t2", "sparse90", "normal_1e4"),
                   fault_rate=0.4, notes="main fp32 throughput case"),
    "c3": Workload("c3", 64, ((8192, 4096),), cand_dtype="bf16", ref_dtype="f32",
                   tols=((1e-2, 1.6e-2),), seeds=(2,), dists=("normal",), fault_rate=0.01,
                   notes="bf16 outputs, fp32 reference"),
    "c4": Workload("c4", 128, ((8192, 4096), (4096,), (4096,)),
                   tols=((1e-5, 1e-5), (1e-5, 1e-5), (1e-4, 1e-5)), seeds=(3,),
                   dists=("normal", "student_t2", "sparse90"), fault_rate=0.1,
                   notes="three gradient tensors per candidate, joint verdict"),
    "c5": Workload("c5", 128, ((4096, 4096), (4096, 4096)), cand_dtype="mixed",
                   tols=((1e-5, 1e-5), (1e-2, 1.6e-2)), seeds=(10, 11, 12, 13),
                   dists=("normal", "uniform_pm1", "student_t2", "sparse90", "normal_1e4"),
                   fault_rate=0.05, fused=True,
                   notes="128 fp32 + 128 bf16 candidate tensors, reference regenerated on device"),
}

DIST_IDS = {"normal": 0, "uniform_pm1": 1, "student_t2": 2, "sparse90": 3, "normal_1e4": 4}


def _seeded_indices(rng: np.random.Generator, n: int, m: int) -> tuple:
    m = min(m, n)
    if m == 1:
        return (int(rng.integers(0, n)),)
    return tuple(int(x) for x in np.sort(rng.choice(n, size=m, replace=False)))


def _random_fault(rng: np.random.Generator, n: int) -> Candidate:
    kind = rng.choice([CORRUPT, CORRUPT, NAN_AT, INF_AT, INPUT_COPY, CONST, ZEROS])
    if kind == CORRUPT:
        m = 1 if rng.random() < 0.5 else int(rng.integers(2, 1025))
        return Candidate(CORRUPT, delta=1.0, indices=_seeded_indices(rng, n, m))
    if kind in (NAN_AT, INF_AT):
        return Candidate(str(kind), indices=_seeded_indices(rng, n, 1))
    if kind == CONST:
        return Candidate(CONST, value=0.5)
    return Candidate(str(kind))


def plan_c1(n: int, seed: int = 0) -> list:
    """The eight fixed candidates of the correctness case, in their stated order."""
    rng = np.random.default_rng([seed, 8])
    return [
        Candidate(NOISE, sigma=1e-7, noise_seed=seed * 1000 + 1),
        Candidate(CORRUPT, delta=1.0, indices=_seeded_indices(rng, n, 1)),
        Candidate(NAN_AT, indices=_seeded_indices(rng, n, 1)),
        Candidate(ZEROS),
        Candidate(INPUT_COPY),
        Candidate(CONST, value=0.5),
        Candidate(REF_EXACT),
        Candidate(SCALE, factor=1.001),
    ]


def plan_mixed(K: int, n: int, seed: int, fault_rate: float, bf16: bool = False,
               force_one_fault: bool = True) -> list:
    """K candidates: benign noise with probability 1 - fault_rate, else a fault
    of a seeded kind.  fp32 noise is Gaussian with sigma drawn from
    {1e-7 .. 1e-3}; bf16 noise is relative, about one bf16 ulp."""
    rng = np.random.default_rng([seed, 8, K])
    out = []
    for k in range(K):
        nseed = seed * 100003 + k
        if bf16:
            benign = Candidate(BF16_ULP, noise_seed=nseed)
        else:
            sigma = float(rng.choice([1e-7, 1e-6, 1e-5, 1e-4, 1e-3],
                                     p=[0.4, 0.3, 0.2, 0.05, 0.05]))
            benign = Candidate(NOISE, sigma=sigma, noise_seed=nseed)
        if rng.random() < fault_rate:
            f = _random_fault(rng, n)
            f.noise_seed = nseed
            out.append(f)
        else:
            out.append(benign)
    if force_one_fault and not any(c.kind in FAULT_KINDS for c in out):
        k = int(rng.integers(0, K))
        f = _random_fault(rng, n)
        f.noise_seed = seed * 100003 + k
        out[k] = f
    return out


def plan_multi(K: int, numels: tuple, seed: int, fault_rate: float) -> list:
    """Per candidate one plan entry per tensor; a faulty candidate carries its
    fault in one seeded tensor and benign noise in the others."""
    rng = np.random.default_rng([seed, 8, K, len(numels)])
    plans = []
    for k in range(K):
        row = []
        faulty = rng.random() < fault_rate
        t_fault = int(rng.integers(0, len(numels)))
        for t, n in enumerate(numels):
            nseed = (seed * 100003 + k) * 7 + t
            sigma = float(rng.choice([1e-7, 1e-6], p=[0.6, 0.4]))
            if faulty and t == t_fault:
                f = _random_fault(rng, n)
                f.noise_seed = nseed
                f.fault_tensor = t
                row.append(f)
            else:
                row.append(Candidate(NOISE, sigma=sigma, noise_seed=nseed))
        plans.append(row)
    return plans


def _torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[name]


def materialize(cand: Candidate, ref: torch.Tensor, inp: torch.Tensor | None,
                dtype: str = "f32") -> torch.Tensor:
    """Build one candidate tensor (flat, contiguous, on ref's device).

    ``ref`` is fp32 (or bf16, upcast here); ``inp`` has the candidate's dtype.
    """
    dev = ref.device
    n = ref.numel()
    td = _torch_dtype(dtype)
    r = ref.reshape(-1).to(torch.float32)
    g = torch.Generator(device=dev)
    g.manual_seed(int(cand.noise_seed) & 0x7FFFFFFFFFFFFFFF)
    k = cand.kind
    if k == REF_EXACT:
        c = r.clone()
    elif k == NOISE:
        c = torch.randn(n, generator=g, device=dev, dtype=torch.float32)
        c.mul_(cand.sigma).add_(r)
    elif k == BF16_ULP:
        c = torch.rand(n, generator=g, device=dev, dtype=torch.float32)
        c.mul_(2.0).sub_(1.0).mul_(2.0 ** -8).add_(1.0).mul_(r)
    elif k == SCALE:
        c = r * cand.factor
    elif k == CORRUPT:
        c = r.clone()
        idx = torch.tensor(cand.indices, dtype=torch.long, device=dev)
        c[idx] += cand.delta
    elif k == NAN_AT:
        c = r.clone()
        c[cand.indices[0]] = float("nan")
    elif k == INF_AT:
        c = r.clone()
        c[cand.indices[0]] = float("inf")
    elif k == ZEROS:
        c = torch.zeros(n, device=dev, dtype=torch.float32)
    elif k == CONST:
        c = torch.full((n,), cand.value, device=dev, dtype=torch.float32)
    elif k == INPUT_COPY:
        if inp is None:
            raise ValueError("input_copy candidate needs the input tensor")
        return inp.reshape(-1).to(td).clone()
    else:
        raise ValueError(f"unknown candidate kind {k!r}")
    return c.to(td).contiguous()


def bits_numpy(t: torch.Tensor) -> np.ndarray:
    """A CPU tensor as the numpy array the oracle takes (bf16 -> uint16 bits, fp16 -> float16)."""
    t = t.detach().cpu().contiguous().reshape(-1)
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def from_bits(a: np.ndarray, device="cpu") -> torch.Tensor:
    """Inverse of :func:`bits_numpy`."""
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).to(device)
    return torch.from_numpy(a.copy()).to(device)
