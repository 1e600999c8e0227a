"""CPU oracle for the verification path -- TEST INFRASTRUCTURE ONLY.

A ctypes front for ``rkv_oracle.c`` (plain C, fp32 arithmetic as the method
fixes it, fp64 for the error sum).  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this package; the CUDA library and its
Python binding never do, and this package never imports them.

The functions take and return numpy arrays.  bf16 tensors are ``uint16``
arrays holding the raw storage bits.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rkv_oracle.c")
_HDR = os.path.join(_HERE, "rkv_oracle.h")
_LIB = os.path.join(_HERE, "liboracle.so")

F32, BF16, F16 = 0, 1, 2
NORMAL, UNIFORM_PM1, STUDENT_T2, SPARSE90, NORMAL_1E4 = range(5)
DISTS = (NORMAL, UNIFORM_PM1, STUDENT_T2, SPARSE90, NORMAL_1E4)

FAIL_TOL, FAIL_NAN, FAIL_INF_MISMATCH, FAIL_LOOPHOLE_CONST, FAIL_LOOPHOLE_COPY = (
    1, 2, 4, 8, 16)
CAND_CONST, CAND_COPY_OF_INPUT, REF_CONST, REF_COPY_OF_INPUT, HAS_NAN, HAS_INF = (
    1, 2, 4, 8, 16, 32)
NO_INDEX = 2**64 - 1

CFLAGS = ["-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared"]


class Result(ctypes.Structure):
    _fields_ = [
        ("verdict", ctypes.c_uint32),
        ("flags", ctypes.c_uint32),
        ("n_over_tol", ctypes.c_uint64),
        ("n_nan", ctypes.c_uint64),
        ("n_inf", ctypes.c_uint64),
        ("n_inf_mismatch", ctypes.c_uint64),
        ("n_comparable", ctypes.c_uint64),
        ("argmax_abs_err", ctypes.c_uint64),
        ("argmax_rel_err", ctypes.c_uint64),
        ("sum_abs_err", ctypes.c_double),
        ("max_abs_err", ctypes.c_float),
        ("max_rel_err", ctypes.c_float),
        ("mean_abs_err", ctypes.c_float),
        ("pad", ctypes.c_uint32),
    ]

    def as_dict(self) -> dict:
        return {name: getattr(self, name) for name, _ in self._fields_ if name != "pad"}


class ScreenResult(ctypes.Structure):
    _fields_ = [
        ("flags", ctypes.c_uint32),
        ("pad", ctypes.c_uint32),
        ("n_values", ctypes.c_uint64),
        ("n_nonfinite", ctypes.c_uint64),
        ("argmax_seed_spread", ctypes.c_uint64),
        ("mean", ctypes.c_double),
        ("std", ctypes.c_double),
        ("vmin", ctypes.c_float),
        ("vmax", ctypes.c_float),
        ("max_seed_spread", ctypes.c_float),
        ("pad2", ctypes.c_uint32),
    ]

    def as_dict(self) -> dict:
        return {name: getattr(self, name) for name, _ in self._fields_ if not name.startswith("pad")}


class CrossResult(ctypes.Structure):
    _fields_ = [
        ("flags", ctypes.c_uint32),
        ("pad", ctypes.c_uint32),
        ("n_nonfinite", ctypes.c_uint64),
        ("argmax_spread", ctypes.c_uint64),
        ("max_spread", ctypes.c_float),
        ("pad2", ctypes.c_uint32),
    ]

    def as_dict(self) -> dict:
        return {name: getattr(self, name) for name, _ in self._fields_ if not name.startswith("pad")}


CROSS_IDENTICAL, CROSS_WITHIN_TOL, CROSS_LOW_SPREAD, CROSS_NONFINITE = 1, 2, 4, 8
SCREEN_NARROW_RANGE, SCREEN_LOW_STD, SCREEN_LOW_SEED_VARIATION = 1, 2, 4
SCREEN_UNIFORM_AXIS0, SCREEN_UNIFORM_AXIS1, SCREEN_NONFINITE = 8, 16, 32


def build(force: bool = False) -> str:
    """Compile ``liboracle.so`` next to the source with gcc; return its path."""
    stale = (not os.path.exists(_LIB)
             or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR)))
    if force or stale:
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", *CFLAGS, "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        u32p = ctypes.POINTER(ctypes.c_uint32)
        f32p = ctypes.POINTER(ctypes.c_float)
        L.orc_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.orc_philox4x32_10.restype = None
        L.orc_log_unit.argtypes = [ctypes.c_uint32]
        L.orc_log_unit.restype = ctypes.c_float
        L.orc_sincos_turn.argtypes = [ctypes.c_uint32, f32p, f32p]
        L.orc_sincos_turn.restype = None
        L.orc_log_unit_range.argtypes = [ctypes.c_uint32, ctypes.c_uint32, ctypes.c_void_p]
        L.orc_log_unit_range.restype = None
        L.orc_sincos_turn_range.argtypes = [ctypes.c_uint32, ctypes.c_uint32, ctypes.c_void_p,
                                            ctypes.c_void_p]
        L.orc_sincos_turn_range.restype = None
        L.orc_box_muller.argtypes = [ctypes.c_uint32, ctypes.c_uint32, f32p, f32p]
        L.orc_box_muller.restype = None
        L.orc_uniform_pm1.argtypes = [ctypes.c_uint32]
        L.orc_uniform_pm1.restype = ctypes.c_float
        L.orc_student_t2.argtypes = [ctypes.c_uint32]
        L.orc_student_t2.restype = ctypes.c_float
        L.orc_bf16_rne.argtypes = [ctypes.c_float]
        L.orc_bf16_rne.restype = ctypes.c_uint16
        L.orc_f16_to_f32_bits.argtypes = [ctypes.c_uint16]
        L.orc_f16_to_f32_bits.restype = ctypes.c_uint32
        L.orc_gen_value.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int, ctypes.c_uint64]
        L.orc_gen_value.restype = ctypes.c_float
        L.orc_gen.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int, ctypes.c_uint64,
                              ctypes.c_uint64, ctypes.c_int, ctypes.c_void_p]
        L.orc_gen.restype = ctypes.c_int
        L.orc_verify.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_int,
                                 ctypes.c_void_p, ctypes.c_int, ctypes.c_uint64,
                                 ctypes.c_float, ctypes.c_float, ctypes.POINTER(Result)]
        L.orc_verify.restype = ctypes.c_int
        L.orc_max_rel_filtered.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_uint64,
                                           ctypes.POINTER(ctypes.c_uint64)]
        L.orc_max_rel_filtered.restype = ctypes.c_float
        L.orc_joint_pass.argtypes = [ctypes.POINTER(Result), ctypes.c_int, ctypes.c_int, u32p]
        L.orc_joint_pass.restype = None
        L.orc_screen.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.c_int, ctypes.c_uint64,
                                 ctypes.c_uint64, ctypes.c_int, ctypes.c_float, ctypes.c_double,
                                 ctypes.c_float, ctypes.POINTER(ScreenResult)]
        L.orc_screen.restype = ctypes.c_int
        L.orc_cross_seed.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.c_int, ctypes.c_uint64, ctypes.c_int,
                                     ctypes.c_float, ctypes.c_float, ctypes.c_float, ctypes.POINTER(CrossResult)]
        L.orc_cross_seed.restype = ctypes.c_int
        L.orc_copy_of_inputs.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.c_int, ctypes.c_void_p,
                                         ctypes.c_uint64, ctypes.c_int, ctypes.POINTER(ctypes.c_uint32)]
        L.orc_copy_of_inputs.restype = ctypes.c_int
        _lib = L
    return _lib


def _dtype_of(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    if a.dtype == np.float16:
        return F16
    raise TypeError(f"oracle tensors are float32, float16 or uint16 (bf16 bits), got {a.dtype}")


def philox4x32_10(ctr, key) -> tuple:
    c = (ctypes.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in ctr])
    k = (ctypes.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    o = (ctypes.c_uint32 * 4)()
    lib().orc_philox4x32_10(c, k, o)
    return tuple(int(x) for x in o)


def log_unit(k24: int) -> float:
    return float(lib().orc_log_unit(int(k24)))


def sincos_turn(k24: int) -> tuple:
    s, c = ctypes.c_float(), ctypes.c_float()
    lib().orc_sincos_turn(int(k24), ctypes.byref(s), ctypes.byref(c))
    return float(s.value), float(c.value)


def log_unit_range(k_first: int, count: int) -> np.ndarray:
    out = np.empty(count, dtype=np.float32)
    lib().orc_log_unit_range(int(k_first), int(count), out.ctypes.data_as(ctypes.c_void_p))
    return out


def sincos_turn_range(k_first: int, count: int) -> tuple:
    s = np.empty(count, dtype=np.float32)
    c = np.empty(count, dtype=np.float32)
    lib().orc_sincos_turn_range(int(k_first), int(count), s.ctypes.data_as(ctypes.c_void_p),
                                c.ctypes.data_as(ctypes.c_void_p))
    return s, c


def box_muller(w0: int, w1: int) -> tuple:
    a, b = ctypes.c_float(), ctypes.c_float()
    lib().orc_box_muller(int(w0), int(w1), ctypes.byref(a), ctypes.byref(b))
    return float(a.value), float(b.value)


def uniform_pm1(w: int) -> float:
    return float(lib().orc_uniform_pm1(int(w)))


def student_t2(w: int) -> float:
    return float(lib().orc_student_t2(int(w)))


def bf16_rne(x: float) -> int:
    return int(lib().orc_bf16_rne(ctypes.c_float(x)))


def f16_to_f32_bits(h: int) -> int:
    return int(lib().orc_f16_to_f32_bits(int(h) & 0xFFFF))


def gen(seed: int, stream_id: int, dist: int, n: int, dtype: int = F32,
        first_elem: int = 0) -> np.ndarray:
    """Elements ``first_elem .. first_elem+n-1`` of the tensor (seed, stream_id, dist)."""
    out = np.empty(int(n), dtype=np.float32 if dtype == F32 else np.uint16)
    rc = lib().orc_gen(int(seed), int(stream_id), int(dist), int(n), int(first_elem),
                       int(dtype), out.ctypes.data_as(ctypes.c_void_p))
    if rc != 0:
        raise ValueError("orc_gen: bad argument")
    return out


def verify(ref: np.ndarray, cand: np.ndarray, atol: float, rtol: float,
           input: np.ndarray | None = None) -> dict:
    """Verify one candidate against the reference; returns the result fields."""
    ref = np.ascontiguousarray(ref).reshape(-1)
    cand = np.ascontiguousarray(cand).reshape(-1)
    if ref.size != cand.size:
        raise ValueError("ref and cand differ in size")
    ip, it = None, 0
    if input is not None:
        input = np.ascontiguousarray(input).reshape(-1)
        if input.size != ref.size:
            raise ValueError("input and ref differ in size")
        ip, it = input.ctypes.data_as(ctypes.c_void_p), _dtype_of(input)
    r = Result()
    rc = lib().orc_verify(ref.ctypes.data_as(ctypes.c_void_p), _dtype_of(ref), ip, it,
                          cand.ctypes.data_as(ctypes.c_void_p), _dtype_of(cand),
                          ref.size, float(atol), float(rtol), ctypes.byref(r))
    if rc != 0:
        raise ValueError("orc_verify: bad argument")
    return r.as_dict()


def max_rel_filtered(ref: np.ndarray, cand: np.ndarray) -> tuple:
    ref = np.ascontiguousarray(ref, dtype=np.float32).reshape(-1)
    cand = np.ascontiguousarray(cand, dtype=np.float32).reshape(-1)
    arg = ctypes.c_uint64()
    v = lib().orc_max_rel_filtered(ref.ctypes.data_as(ctypes.c_void_p),
                                   cand.ctypes.data_as(ctypes.c_void_p), ref.size,
                                   ctypes.byref(arg))
    return float(v), int(arg.value)


def joint_pass(verdicts) -> list:
    """``verdicts[k][t]`` -> list of K 0/1 values: pass on every tensor."""
    K, T = len(verdicts), len(verdicts[0])
    arr = (Result * (K * T))()
    for k in range(K):
        for t in range(T):
            arr[k * T + t].verdict = int(verdicts[k][t])
    out = (ctypes.c_uint32 * K)()
    lib().orc_joint_pass(arr, K, T, out)
    return [int(x) for x in out]


def screen(outs, range_lim: float = 0.01, std_lim: float = 0.01, spread_lim: float = 0.01) -> dict:
    """Task-soundness screens over the reference outputs of S seeds (2-D arrays of one shape)."""
    arrs = [np.ascontiguousarray(a) for a in outs]
    rows, cols = arrs[0].shape
    for a in arrs:
        if a.shape != (rows, cols) or a.dtype != arrs[0].dtype:
            raise ValueError("outputs differ in shape or dtype")
    ptrs = (ctypes.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])
    r = ScreenResult()
    rc = lib().orc_screen(ptrs, len(arrs), rows, cols, _dtype_of(arrs[0].reshape(-1)), float(range_lim),
                          float(std_lim), float(spread_lim), ctypes.byref(r))
    if rc != 0:
        raise ValueError("orc_screen: bad argument")
    return r.as_dict()


def cross_seed(outs, atol: float, rtol: float, spread_lim: float = 0.01) -> dict:
    """Cross-seed variation of one candidate: outs[s] is its output for input seed s."""
    arrs = [np.ascontiguousarray(a).reshape(-1) for a in outs]
    for a in arrs:
        if a.size != arrs[0].size or a.dtype != arrs[0].dtype:
            raise ValueError("outputs differ in size or dtype")
    ptrs = (ctypes.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])
    r = CrossResult()
    rc = lib().orc_cross_seed(ptrs, len(arrs), arrs[0].size, _dtype_of(arrs[0]), float(atol), float(rtol),
                              float(spread_lim), ctypes.byref(r))
    if rc != 0:
        raise ValueError("orc_cross_seed: bad argument")
    return r.as_dict()


def copy_of_inputs(inputs, cand) -> int:
    """Bit m set iff cand is a bit copy of inputs[m]."""
    arrs = [np.ascontiguousarray(a).reshape(-1) for a in inputs]
    c = np.ascontiguousarray(cand).reshape(-1)
    for a in arrs:
        if a.size != c.size or a.dtype != c.dtype:
            raise ValueError("inputs and candidate differ in size or dtype")
    ptrs = (ctypes.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])
    m = ctypes.c_uint32()
    rc = lib().orc_copy_of_inputs(ptrs, len(arrs), c.ctypes.data_as(ctypes.c_void_p), c.size, _dtype_of(c),
                                  ctypes.byref(m))
    if rc != 0:
        raise ValueError("orc_copy_of_inputs: bad argument")
    return int(m.value)
