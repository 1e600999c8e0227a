"""ctypes binding of ``librkv.so`` (declared in ``include/rkv.h``).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  torch is used for device memory (``tensor.data_ptr()``) and for the
current stream.  There is no fallback: if the library is missing, loading
raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass, field

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# RKV_LIB selects another build of the same library (the range-checked debug build,
# `python -m paper_2509_14279_b200.build --debug-bounds`, writes librkv_dbg.so)
LIB_PATH = os.environ.get("RKV_LIB") or os.path.join(_PKG, "librkv.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_BOUNDS = (
    0, -1, -2, -3, -4, -5, -6, -7)
F32, BF16, F16 = 0, 1, 2
DIST_NORMAL, DIST_UNIFORM_PM1, DIST_STUDENT_T2, DIST_SPARSE90, DIST_NORMAL_1E4 = range(5)
SRC_NONE, SRC_POINTER, SRC_GENERATED = 0, 1, 2
FAIL_TOL, FAIL_NAN, FAIL_INF_MISMATCH, FAIL_LOOPHOLE_CONST, FAIL_LOOPHOLE_COPY = 1, 2, 4, 8, 16
(FLAG_CAND_CONST, FLAG_CAND_COPY_OF_INPUT, FLAG_REF_CONST, FLAG_REF_COPY_OF_INPUT,
 FLAG_HAS_NAN, FLAG_HAS_INF) = 1, 2, 4, 8, 16, 32
NO_INDEX = 2**64 - 1

STATS_DTYPE = np.dtype([
    ("verdict", "<u4"), ("flags", "<u4"), ("n_over_tol", "<u8"), ("n_nan", "<u8"),
    ("n_inf", "<u8"), ("n_inf_mismatch", "<u8"), ("n_comparable", "<u8"),
    ("argmax_abs_err", "<u8"), ("argmax_rel_err", "<u8"), ("sum_abs_err", "<f8"),
    ("max_abs_err", "<f4"), ("max_rel_err", "<f4"), ("mean_abs_err", "<f4"), ("reserved", "<u4"),
])
STATS_BYTES = STATS_DTYPE.itemsize

SCREEN_DTYPE = np.dtype([
    ("flags", "<u4"), ("reserved", "<u4"), ("n_values", "<u8"), ("n_nonfinite", "<u8"),
    ("argmax_seed_spread", "<u8"), ("mean", "<f8"), ("std", "<f8"), ("vmin", "<f4"), ("vmax", "<f4"),
    ("max_seed_spread", "<f4"), ("reserved2", "<u4")])
SCREEN_BYTES = SCREEN_DTYPE.itemsize
CROSS_DTYPE = np.dtype([("flags", "<u4"), ("reserved", "<u4"), ("n_nonfinite", "<u8"), ("argmax_spread", "<u8"),
                        ("max_spread", "<f4"), ("reserved2", "<u4")])
CROSS_BYTES = CROSS_DTYPE.itemsize
CROSS_IDENTICAL, CROSS_WITHIN_TOL, CROSS_LOW_SPREAD, CROSS_NONFINITE = 1, 2, 4, 8
SCREEN_NARROW_RANGE, SCREEN_LOW_STD, SCREEN_LOW_SEED_VARIATION = 1, 2, 4
SCREEN_UNIFORM_AXIS0, SCREEN_UNIFORM_AXIS1, SCREEN_NONFINITE = 8, 16, 32
assert STATS_BYTES == 88


class RkvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


class GenSpec(ctypes.Structure):
    _fields_ = [("seed", ctypes.c_uint64), ("stream_id", ctypes.c_uint64),
                ("dist", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class TensorDescC(ctypes.Structure):
    _fields_ = [
        ("n", ctypes.c_uint64),
        ("ref", ctypes.c_void_p),
        ("input", ctypes.c_void_p),
        ("cands", ctypes.POINTER(ctypes.c_void_p)),
        ("ref_gen", GenSpec),
        ("input_gen", GenSpec),
        ("cand_dtype", ctypes.c_int32),
        ("ref_dtype", ctypes.c_int32),
        ("ref_src", ctypes.c_int32),
        ("input_src", ctypes.c_int32),
        ("atol", ctypes.c_float),
        ("rtol", ctypes.c_float),
    ]


class CaseDescC(ctypes.Structure):
    _fields_ = [("tensors", ctypes.POINTER(TensorDescC)), ("T", ctypes.c_int32), ("reserved", ctypes.c_int32)]


_lib = None


def lib() -> ctypes.CDLL:
    """Load the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2509_14279_b200.build` "
                "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, u64, i32, f32 = ctypes.c_void_p, ctypes.c_uint64, ctypes.c_int, ctypes.c_float
        L.rkv_version.restype = i32
        L.rkv_version.argtypes = []
        L.rkv_status_string.restype = ctypes.c_char_p
        L.rkv_status_string.argtypes = [i32]
        L.rkv_set_stream.restype = i32
        L.rkv_set_stream.argtypes = [vp]
        L.rkv_gen_inputs.restype = i32
        L.rkv_gen_inputs.argtypes = [u64, i32, ctypes.POINTER(ctypes.c_int64), i32, i32, vp]
        L.rkv_gen_inputs_ex.restype = i32
        L.rkv_gen_inputs_ex.argtypes = [u64, u64, i32, u64, u64, i32, vp, vp]
        L.rkv_verify_batch.restype = i32
        L.rkv_verify_batch.argtypes = [vp, ctypes.POINTER(vp), i32, u64, i32, f32, f32, vp]
        L.rkv_verify_multi.restype = i32
        L.rkv_verify_multi.argtypes = [ctypes.POINTER(TensorDescC), i32, i32, vp, vp, vp,
                                       ctypes.c_size_t, vp]
        L.rkv_workspace_bytes.restype = ctypes.c_size_t
        L.rkv_workspace_bytes.argtypes = [ctypes.POINTER(TensorDescC), i32, i32]
        L.rkv_device_status.restype = i32
        L.rkv_device_status.argtypes = [vp, vp]
        L.rkv_verify_batch_host.restype = i32
        L.rkv_verify_batch_host.argtypes = [vp, ctypes.POINTER(vp), i32, u64, i32, f32, f32, vp]
        L.rkv_verify_multi_host.restype = i32
        L.rkv_verify_multi_host.argtypes = [ctypes.POINTER(TensorDescC), i32, i32, vp, vp]
        L.rkv_verify_sweep.restype = i32
        L.rkv_verify_sweep.argtypes = [ctypes.POINTER(CaseDescC), i32, i32, vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.rkv_sweep_workspace_bytes.restype = ctypes.c_size_t
        L.rkv_sweep_workspace_bytes.argtypes = [ctypes.POINTER(CaseDescC), i32, i32]
        L.rkv_debug_fault_drill.restype = i32
        L.rkv_debug_fault_drill.argtypes = [ctypes.c_uint, ctypes.c_ulonglong]
        L.rkv_debug_bounds_build.restype = i32
        L.rkv_debug_bounds_build.argtypes = []
        L.rkv_cross_workspace_bytes.restype = ctypes.c_size_t
        L.rkv_cross_workspace_bytes.argtypes = [i32, i32]
        L.rkv_cross_seed.restype = i32
        L.rkv_cross_seed.argtypes = [ctypes.POINTER(vp), i32, i32, u64, i32, f32, f32, f32, vp, vp, ctypes.c_size_t, vp]
        L.rkv_copy_workspace_bytes.restype = ctypes.c_size_t
        L.rkv_copy_workspace_bytes.argtypes = [i32, i32]
        L.rkv_copy_of_inputs.restype = i32
        L.rkv_copy_of_inputs.argtypes = [ctypes.POINTER(vp), i32, ctypes.POINTER(vp), i32, u64, i32, vp, vp,
                                         ctypes.c_size_t, vp]
        L.rkv_verify_batch_static.restype = i32
        L.rkv_verify_batch_static.argtypes = [vp, ctypes.POINTER(vp), i32, u64, i32, f32, f32, vp, vp]
        u32p = ctypes.POINTER(ctypes.c_uint32)
        L.rkv_plan_items.restype = i32
        L.rkv_plan_items.argtypes = [u64, i32, i32, i32, u32p, u32p, u32p, u32p, u32p, u32p, u32p]
        L.rkv_release_cached.restype = i32
        L.rkv_release_cached.argtypes = []
        L.rkv_screen_workspace_bytes.restype = ctypes.c_size_t
        L.rkv_screen_workspace_bytes.argtypes = []
        L.rkv_screen_outputs.restype = i32
        L.rkv_screen_outputs.argtypes = [ctypes.POINTER(vp), i32, u64, u64, i32, f32, ctypes.c_double, f32,
                                         vp, vp, ctypes.c_size_t, vp]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().rkv_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise RkvError(status, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float16:
        return F16
    raise TypeError(f"rkv tensors are float32, bfloat16 or float16, got {t.dtype}")


def _require(t, what: str, device=None, dtype=None, numel=None, min_bytes=None) -> None:
    """Check a tensor before its raw pointer crosses the C ABI (the library sees no sizes).

    The candidates come from machine-written kernels, so a tensor of the wrong shape, dtype
    or device is an ordinary failure here: it must raise on the host, not become a read
    past the end of a buffer on the device."""
    if not isinstance(t, torch.Tensor):
        raise TypeError(f"{what}: expected a torch.Tensor, got {type(t).__name__}")
    if device is not None:
        if t.device.type != device.type or (device.type == "cuda" and device.index is not None
                                            and t.device.index != device.index):
            raise ValueError(f"{what}: on {t.device}, expected {device}")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{what}: dtype {t.dtype}, expected {dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{what}: not contiguous")
    if numel is not None and t.numel() != numel:
        raise ValueError(f"{what}: {t.numel()} elements, expected {numel}")
    if min_bytes is not None and t.numel() * t.element_size() < min_bytes:
        raise ValueError(f"{what}: {t.numel() * t.element_size()} bytes, needs at least {min_bytes}")


def _require_case(ref, cands, what: str, stats_out=None, device_type: str = "cuda"):
    """ref and every candidate: same device, same dtype, contiguous, n elements each."""
    if len(cands) < 1:
        raise ValueError(f"{what}: no candidates")
    _require(ref, f"{what}: ref")
    if ref.device.type != device_type:
        raise ValueError(f"{what}: ref is on {ref.device}, expected a {device_type} tensor")
    _dtype_code(ref)
    for k, c in enumerate(cands):
        _require(c, f"{what}: candidate {k}", device=ref.device, dtype=ref.dtype, numel=ref.numel())
    if stats_out is not None:
        _require(stats_out, f"{what}: stats_out", device=ref.device, dtype=torch.uint8,
                 min_bytes=len(cands) * STATS_BYTES)


def _stream_ptr(stream=None) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return int(s.cuda_stream)


def version() -> int:
    return int(lib().rkv_version())


def set_stream(stream=None) -> None:
    _check(lib().rkv_set_stream(ctypes.c_void_p(_stream_ptr(stream))), "rkv_set_stream")


def plan_items(n: int, K: int, num_sms: int, cand_dtype: int = F32) -> tuple:
    """Host-only: (tile_elems, n_tiles, warm_tiles, parts_warm, parts_main, tail_tiles, parts_tail)
    for a tensor of n elements and K candidates."""
    v = [ctypes.c_uint32() for _ in range(7)]
    _check(lib().rkv_plan_items(int(n), int(cand_dtype), int(K), int(num_sms), *[ctypes.byref(x) for x in v]),
           "rkv_plan_items")
    return tuple(int(x.value) for x in v)


def gen_inputs(seed: int, dist: int, shape, dtype: torch.dtype = torch.float32,
               out: torch.Tensor | None = None) -> torch.Tensor:
    """rkv_gen_inputs: the tensor (seed, stream 0, dist) on the current device and stream."""
    shape = tuple(int(s) for s in shape)
    if out is None:
        out = torch.empty(shape, dtype=dtype, device="cuda")
    else:
        _require(out, "gen_inputs: out", device=torch.device("cuda"), numel=int(np.prod(shape)))
    set_stream()
    arr = (ctypes.c_int64 * len(shape))(*shape)
    _check(lib().rkv_gen_inputs(int(seed), int(dist), arr, len(shape), _dtype_code(out),
                                ctypes.c_void_p(out.data_ptr())), "rkv_gen_inputs")
    return out


def gen_inputs_ex(seed: int, stream_id: int, dist: int, n: int, first_elem: int = 0,
                  dtype: torch.dtype = torch.float32, out: torch.Tensor | None = None,
                  stream=None) -> torch.Tensor:
    if out is None:
        out = torch.empty(int(n), dtype=dtype, device="cuda")
    else:
        _require(out, "gen_inputs_ex: out", device=torch.device("cuda"), min_bytes=int(n) * out.element_size())
    _check(lib().rkv_gen_inputs_ex(int(seed), int(stream_id), int(dist), int(n), int(first_elem),
                                   _dtype_code(out), ctypes.c_void_p(out.data_ptr()),
                                   ctypes.c_void_p(_stream_ptr(stream))), "rkv_gen_inputs_ex")
    return out


def stats_to_numpy(stats: torch.Tensor) -> np.ndarray:
    """Device (or host) stats buffer -> structured numpy array (synchronises)."""
    return stats.detach().cpu().numpy().view(STATS_DTYPE)


def verify_batch(ref: torch.Tensor, cands, atol: float, rtol: float,
                 stats_out: torch.Tensor | None = None) -> torch.Tensor:
    """rkv_verify_batch: K candidates against one reference, same dtype, no input tensor.
    Returns the device buffer of K rkv_stats (uint8, K*88 bytes)."""
    K = len(cands)
    _require_case(ref, cands, "verify_batch", stats_out)
    n = ref.numel()
    if stats_out is None:
        stats_out = torch.empty(K * STATS_BYTES, dtype=torch.uint8, device=ref.device)
    ptrs = (ctypes.c_void_p * K)(*[c.data_ptr() for c in cands])
    set_stream()
    _check(lib().rkv_verify_batch(ctypes.c_void_p(ref.data_ptr()), ptrs, K, n, _dtype_code(ref),
                                  float(atol), float(rtol), ctypes.c_void_p(stats_out.data_ptr())),
           "rkv_verify_batch")
    return stats_out


def verify_batch_static(ref: torch.Tensor, cands, atol: float, rtol: float,
                        stats_out: torch.Tensor, stream=None) -> torch.Tensor:
    """rkv_verify_batch_static: like ``verify_batch`` but nothing is allocated, here or in
    the library -- the scratch is a fixed 8 MiB array inside the library, so the caller must
    pass ``stats_out`` (K*88 bytes, uint8, on the device).  For callers that cannot allocate
    device memory when they verify (all memory already in their own pool, or no allocator
    calls allowed on this thread).  Calls share that array: do not overlap them on the GPU."""
    K = len(cands)
    _require_case(ref, cands, "verify_batch_static", stats_out)
    ptrs = (ctypes.c_void_p * K)(*[c.data_ptr() for c in cands])
    _check(lib().rkv_verify_batch_static(ctypes.c_void_p(ref.data_ptr()), ptrs, K, ref.numel(),
                                         _dtype_code(ref), float(atol), float(rtol),
                                         ctypes.c_void_p(stats_out.data_ptr()),
                                         ctypes.c_void_p(_stream_ptr(stream))),
           "rkv_verify_batch_static")
    return stats_out


@dataclass
class TensorDesc:
    """One tensor of a case, as torch tensors (or generator specs)."""
    n: int
    cands: list                       # K device tensors
    atol: float
    rtol: float
    ref: torch.Tensor | None = None   # None -> regenerated from ref_gen
    input: torch.Tensor | None = None
    ref_gen: tuple | None = None      # (seed, stream_id, dist)
    input_gen: tuple | None = None
    ref_dtype: int | None = None      # for a generated reference; default fp32
    _keep: list = field(default_factory=list, repr=False)

    def to_c(self, where: str = "cuda") -> TensorDescC:
        """The C descriptor; `where` is the device type every tensor must live on ("cuda" for
        the device forms, "cpu" for the host-buffer form)."""
        d = TensorDescC()
        d.n = int(self.n)
        K = len(self.cands)
        if K < 1:
            raise ValueError("TensorDesc: no candidates")
        first = self.cands[0]
        _require(first, "TensorDesc: candidate 0", device=torch.device(where), numel=d.n)
        for k, c in enumerate(self.cands):
            _require(c, f"TensorDesc: candidate {k}", device=first.device, dtype=first.dtype, numel=d.n)
        if self.ref is not None:
            _require(self.ref, "TensorDesc: ref", device=first.device, numel=d.n)
        elif self.ref_gen is None:
            raise ValueError("TensorDesc: neither ref nor ref_gen given")
        if self.input is not None:     # a copy is a bit copy: the input has the candidates' dtype
            _require(self.input, "TensorDesc: input", device=first.device, dtype=first.dtype, numel=d.n)
        ptrs = (ctypes.c_void_p * K)(*[c.data_ptr() for c in self.cands])
        self._keep.append(ptrs)
        d.cands = ctypes.cast(ptrs, ctypes.POINTER(ctypes.c_void_p))
        d.cand_dtype = _dtype_code(self.cands[0])
        if self.ref is not None:
            d.ref = self.ref.data_ptr()
            d.ref_src = SRC_POINTER
            d.ref_dtype = _dtype_code(self.ref)
        else:
            seed, stream_id, dist = self.ref_gen
            d.ref_gen = GenSpec(int(seed), int(stream_id), int(dist), 0)
            d.ref_src = SRC_GENERATED
            d.ref_dtype = F32 if self.ref_dtype is None else int(self.ref_dtype)
        if self.input is not None:
            d.input = self.input.data_ptr()
            d.input_src = SRC_POINTER
        elif self.input_gen is not None:
            seed, stream_id, dist = self.input_gen
            d.input_gen = GenSpec(int(seed), int(stream_id), int(dist), 0)
            d.input_src = SRC_GENERATED
        else:
            d.input_src = SRC_NONE
        d.atol = float(self.atol)
        d.rtol = float(self.rtol)
        return d


def _desc_array(tensors) -> ctypes.Array:
    arr = (TensorDescC * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = t.to_c()
    return arr


def workspace_bytes(tensors, K: int) -> int:
    arr = _desc_array(tensors)
    return int(lib().rkv_workspace_bytes(arr, len(tensors), int(K)))


def verify_multi(tensors, K: int, workspace: torch.Tensor | None = None,
                 stats_out: torch.Tensor | None = None, joint_pass: torch.Tensor | None = None,
                 stream=None, descs=None):
    """rkv_verify_multi.  Returns (stats [K*T*88 bytes uint8], joint_pass [K] int32, workspace).

    ``descs`` may carry a prebuilt ctypes descriptor array (from ``prepare``) so
    that a timed loop does no Python marshalling.
    """
    T = len(tensors)
    arr = _desc_array(tensors) if descs is None else descs
    dev = tensors[0].cands[0].device
    if workspace is None:
        need = int(lib().rkv_workspace_bytes(arr, T, int(K)))
        if need == 0:
            raise RkvError(ERR_INVALID_ARG, "rkv_workspace_bytes")
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    else:
        _require(workspace, "verify_multi: workspace", device=dev, dtype=torch.uint8)
    if stats_out is None:
        stats_out = torch.empty(K * T * STATS_BYTES, dtype=torch.uint8, device=dev)
    else:
        _require(stats_out, "verify_multi: stats_out", device=dev, dtype=torch.uint8,
                 min_bytes=K * T * STATS_BYTES)
    if joint_pass is None:
        joint_pass = torch.empty(K, dtype=torch.int32, device=dev)
    else:
        _require(joint_pass, "verify_multi: joint_pass", device=dev, dtype=torch.int32, numel=K)
    for t in tensors:
        if len(t.cands) != K:
            raise ValueError(f"verify_multi: a tensor has {len(t.cands)} candidates, K = {K}")
    _check(lib().rkv_verify_multi(arr, T, int(K), ctypes.c_void_p(stats_out.data_ptr()),
                                  ctypes.c_void_p(joint_pass.data_ptr()),
                                  ctypes.c_void_p(workspace.data_ptr()), workspace.numel(),
                                  ctypes.c_void_p(_stream_ptr(stream))), "rkv_verify_multi")
    return stats_out, joint_pass, workspace


def prepare_sweep(cases):
    """Marshal the cases of a sweep once: `cases` is a list of lists of TensorDesc (one inner
    list per test case).  Returns an opaque object to pass as ``descs=`` to verify_sweep."""
    keep = []
    arr = (CaseDescC * len(cases))()
    for i, tensors in enumerate(cases):
        ta = _desc_array(tensors)
        keep.append(ta)
        arr[i].tensors = ctypes.cast(ta, ctypes.POINTER(TensorDescC))
        arr[i].T = len(tensors)
    return (arr, keep)


def verify_sweep(cases, K: int, workspace: torch.Tensor | None = None, stats_out: torch.Tensor | None = None,
                 case_pass: torch.Tensor | None = None, all_pass: torch.Tensor | None = None, stream=None,
                 descs=None):
    """rkv_verify_sweep: C test cases (lists of TensorDesc), the same K candidates in each, one
    launch.  Returns (stats, case_pass [C, K] int32, all_pass [K] int32, workspace); the stats of
    case c start at K * (tensors of the cases before it) * 88 bytes, entry [k * T_c + t] inside."""
    C = len(cases)
    arr, keep = prepare_sweep(cases) if descs is None else descs
    dev = cases[0][0].cands[0].device
    n_t = sum(len(c) for c in cases)
    for c in cases:
        for t in c:
            if len(t.cands) != K:
                raise ValueError(f"verify_sweep: a tensor has {len(t.cands)} candidates, K = {K}")
    if workspace is None:
        need = int(lib().rkv_sweep_workspace_bytes(arr, C, int(K)))
        if need == 0:
            raise RkvError(ERR_INVALID_ARG, "rkv_sweep_workspace_bytes")
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    else:
        _require(workspace, "verify_sweep: workspace", device=dev, dtype=torch.uint8)
    if stats_out is None:
        stats_out = torch.empty(K * n_t * STATS_BYTES, dtype=torch.uint8, device=dev)
    else:
        _require(stats_out, "verify_sweep: stats_out", device=dev, dtype=torch.uint8, min_bytes=K * n_t * STATS_BYTES)
    if case_pass is None:
        case_pass = torch.empty((C, K), dtype=torch.int32, device=dev)
    else:
        _require(case_pass, "verify_sweep: case_pass", device=dev, dtype=torch.int32, numel=C * K)
    if all_pass is None:
        all_pass = torch.empty(K, dtype=torch.int32, device=dev)
    else:
        _require(all_pass, "verify_sweep: all_pass", device=dev, dtype=torch.int32, numel=K)
    _check(lib().rkv_verify_sweep(arr, C, int(K), ctypes.c_void_p(stats_out.data_ptr()),
                                  ctypes.c_void_p(case_pass.data_ptr()), ctypes.c_void_p(all_pass.data_ptr()),
                                  ctypes.c_void_p(workspace.data_ptr()), workspace.numel(),
                                  ctypes.c_void_p(_stream_ptr(stream))), "rkv_verify_sweep")
    return stats_out, case_pass, all_pass, workspace


def debug_fault_drill(issue: int, wait_cycles: int) -> None:
    """Test hook (not in rkv.h): the next verification call withholds block 0's issue-th bulk
    copy and lets every bounded wait give up after wait_cycles clock cycles."""
    _check(lib().rkv_debug_fault_drill(int(issue), int(wait_cycles)), "rkv_debug_fault_drill")


def debug_bounds_build() -> bool:
    return bool(lib().rkv_debug_bounds_build())


def prepare(tensors):
    """Marshal the descriptors once; pass the result as ``descs=`` to verify_multi."""
    return _desc_array(tensors)


def device_status(workspace: torch.Tensor, stream=None) -> int:
    return int(lib().rkv_device_status(ctypes.c_void_p(workspace.data_ptr()),
                                       ctypes.c_void_p(_stream_ptr(stream))))


def verify_batch_host(ref: torch.Tensor, cands, atol: float, rtol: float) -> np.ndarray:
    """rkv_verify_batch_host: HOST tensors in, structured numpy stats out (synchronous)."""
    K = len(cands)
    _require_case(ref, cands, "verify_batch_host", device_type="cpu")
    n = ref.numel()
    out = np.zeros(K, dtype=STATS_DTYPE)
    ptrs = (ctypes.c_void_p * K)(*[c.data_ptr() for c in cands])
    set_stream()
    _check(lib().rkv_verify_batch_host(ctypes.c_void_p(ref.data_ptr()), ptrs, K, n,
                                       _dtype_code(ref), float(atol), float(rtol),
                                       out.ctypes.data_as(ctypes.c_void_p)),
           "rkv_verify_batch_host")
    return out


def verify_multi_host(tensors, K: int) -> tuple:
    """rkv_verify_multi_host: TensorDescs over HOST tensors in, (structured numpy stats of
    shape [K, T], joint_pass [K] uint32) out.  Synchronous."""
    T = len(tensors)
    arr = (TensorDescC * T)()
    for i, t in enumerate(tensors):
        if len(t.cands) != K:
            raise ValueError(f"verify_multi_host: a tensor has {len(t.cands)} candidates, K = {K}")
        arr[i] = t.to_c(where="cpu")
    out = np.zeros((K, T), dtype=STATS_DTYPE)
    joint = np.zeros(K, dtype=np.uint32)
    set_stream()
    _check(lib().rkv_verify_multi_host(arr, T, int(K), out.ctypes.data_as(ctypes.c_void_p),
                                       joint.ctypes.data_as(ctypes.c_void_p)), "rkv_verify_multi_host")
    return out, joint


def release_cached() -> None:
    lib().rkv_release_cached()


def screen_workspace_bytes() -> int:
    return int(lib().rkv_screen_workspace_bytes())


def screen_outputs(outs, range_lim: float = 0.01, std_lim: float = 0.01, spread_lim: float = 0.01,
                   stats_out: torch.Tensor | None = None, workspace: torch.Tensor | None = None,
                   stream=None) -> tuple:
    """rkv_screen_outputs: the task-soundness screens over the reference outputs of S seeds
    (2-D tensors of one shape and dtype on the device).  Returns (stats, workspace): the
    device buffer holding one rkv_screen_stats (uint8, 64 bytes) and the workspace used."""
    S = len(outs)
    rows, cols = outs[0].shape
    for o in outs:
        if tuple(o.shape) != (rows, cols) or o.dtype != outs[0].dtype or not o.is_contiguous():
            raise ValueError("outputs must be contiguous and agree in shape and dtype")
    dev = outs[0].device
    if stats_out is None:
        stats_out = torch.empty(SCREEN_BYTES, dtype=torch.uint8, device=dev)
    if workspace is None:
        workspace = torch.empty(screen_workspace_bytes(), dtype=torch.uint8, device=dev)
    ptrs = (ctypes.c_void_p * S)(*[o.data_ptr() for o in outs])
    _check(lib().rkv_screen_outputs(ptrs, S, int(rows), int(cols), _dtype_code(outs[0]), float(range_lim),
                                    float(std_lim), float(spread_lim), ctypes.c_void_p(stats_out.data_ptr()),
                                    ctypes.c_void_p(workspace.data_ptr()), workspace.numel(),
                                    ctypes.c_void_p(_stream_ptr(stream))), "rkv_screen_outputs")
    return stats_out, workspace


def screen_to_numpy(stats: torch.Tensor) -> np.ndarray:
    return stats.detach().cpu().numpy().view(SCREEN_DTYPE)


class CrossTable:
    """The checked pointer table of one rkv_cross_seed call (see prepare_cross)."""

    def __init__(self, ptrs, K, S, n, code, device, keep):
        self.ptrs, self.K, self.S, self.n, self.code, self.device, self.keep = ptrs, K, S, n, code, device, keep


def prepare_cross(outs) -> CrossTable:
    """Check outs[k][s] (candidate k's output for input seed s: device tensors of one size and
    dtype) once and marshal their addresses, for callers that repeat a call on the same tensors."""
    K, S = len(outs), len(outs[0])
    first = outs[0][0]
    _require(first, "cross_seed: outs[0][0]", device=torch.device("cuda"))
    code = _dtype_code(first)
    for k, row in enumerate(outs):
        if len(row) != S:
            raise ValueError("cross_seed: every candidate needs the same number of seeds")
        for s, t in enumerate(row):
            _require(t, f"cross_seed: outs[{k}][{s}]", device=first.device, dtype=first.dtype, numel=first.numel())
    ptrs = (ctypes.c_void_p * (K * S))(*[t.data_ptr() for row in outs for t in row])
    return CrossTable(ptrs, K, S, first.numel(), code, first.device, [list(row) for row in outs])


def cross_seed(outs, atol: float, rtol: float, spread_lim: float = 0.01, stats_out: torch.Tensor | None = None,
               workspace: torch.Tensor | None = None, stream=None, table: CrossTable | None = None) -> tuple:
    """rkv_cross_seed: outs[k][s] is candidate k's output for input seed s (device tensors of one
    size and dtype); with ``table`` (from prepare_cross on the same tensors) the checks and the
    marshalling are not repeated.  Returns (stats [K * 32 bytes, uint8], workspace)."""
    tb = table if table is not None else prepare_cross(outs)
    K, S, dev = tb.K, tb.S, tb.device
    if workspace is None:
        workspace = torch.empty(max(256, int(lib().rkv_cross_workspace_bytes(K, S))), dtype=torch.uint8, device=dev)
    if stats_out is None:
        stats_out = torch.empty(K * CROSS_BYTES, dtype=torch.uint8, device=dev)
    else:
        _require(stats_out, "cross_seed: stats_out", device=dev, dtype=torch.uint8, min_bytes=K * CROSS_BYTES)
    _check(lib().rkv_cross_seed(tb.ptrs, K, S, tb.n, tb.code, float(atol), float(rtol), float(spread_lim),
                                ctypes.c_void_p(stats_out.data_ptr()), ctypes.c_void_p(workspace.data_ptr()),
                                workspace.numel(), ctypes.c_void_p(_stream_ptr(stream))), "rkv_cross_seed")
    return stats_out, workspace


def cross_to_numpy(stats: torch.Tensor) -> np.ndarray:
    return stats.detach().cpu().numpy().view(CROSS_DTYPE)


def copy_of_inputs(inputs, cands, mask_out: torch.Tensor | None = None, workspace: torch.Tensor | None = None,
                   stream=None) -> tuple:
    """rkv_copy_of_inputs: bit m of mask[k] is set iff candidate k is a bit copy of inputs[m].
    Returns (mask [K] int32 on the device, workspace)."""
    K, M = len(cands), len(inputs)
    first = cands[0]
    _require(first, "copy_of_inputs: candidate 0", device=torch.device("cuda"))
    code = _dtype_code(first)
    for i, t in enumerate(list(inputs) + list(cands)):
        _require(t, f"copy_of_inputs: tensor {i}", device=first.device, dtype=first.dtype, numel=first.numel())
    dev = first.device
    if workspace is None:
        workspace = torch.empty(max(256, int(lib().rkv_copy_workspace_bytes(K, M))), dtype=torch.uint8, device=dev)
    if mask_out is None:
        mask_out = torch.empty(K, dtype=torch.int32, device=dev)
    else:
        _require(mask_out, "copy_of_inputs: mask_out", device=dev, dtype=torch.int32, numel=K)
    ip = (ctypes.c_void_p * M)(*[t.data_ptr() for t in inputs])
    cp = (ctypes.c_void_p * K)(*[t.data_ptr() for t in cands])
    _check(lib().rkv_copy_of_inputs(ip, M, cp, K, first.numel(), code, ctypes.c_void_p(mask_out.data_ptr()),
                                    ctypes.c_void_p(workspace.data_ptr()), workspace.numel(),
                                    ctypes.c_void_p(_stream_ptr(stream))), "rkv_copy_of_inputs")
    return mask_out, workspace
