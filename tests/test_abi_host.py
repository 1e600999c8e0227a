"""CPU-only checks of the C ABI: the library loads, exports every declared
symbol, validates arguments before touching CUDA, and plans slabs sensibly.
No kernel is launched here."""
import ctypes
import math
import os
import re

import pytest
import torch

from paper_2509_14279_b200 import binding as rkv
from paper_2509_14279_b200 import build as rkv_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HAS_GPU = torch.cuda.is_available()


@pytest.fixture(scope="module", autouse=True)
def built():
    rkv_build.build()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "rkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rkv_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert {"rkv_gen_inputs", "rkv_verify_batch", "rkv_verify_multi", "rkv_workspace_bytes",
            "rkv_gen_inputs_ex", "rkv_verify_batch_host", "rkv_plan_items"} <= set(names)
    L = ctypes.CDLL(rkv.LIB_PATH)
    for name in names:
        assert hasattr(L, name), name


def test_version_and_status_strings():
    assert rkv.version() >= 100
    seen = set()
    for code in range(0, -8, -1):
        s = rkv.status_string(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 8
    assert rkv.status_string(-99) == "unknown status"


def test_stats_struct_is_88_bytes():
    text = open(os.path.join(ROOT, "include", "rkv.h")).read()
    assert "88 bytes" in text
    assert rkv.STATS_BYTES == 88
    assert ctypes.sizeof(rkv.TensorDescC) == 8 * 4 + 24 * 2 + 4 * 4 + 8


@pytest.mark.parametrize("K", [1, 2, 8, 63, 64, 65, 128, 256, 1000])
@pytest.mark.parametrize("n", [1, 127, 3584, 3585, 4096, 262144, 1200000, 4000000, 1 << 24, (1 << 25) + 3, (1 << 30) + 17])
@pytest.mark.parametrize("dtype", [rkv.F32, rkv.BF16, rkv.F16])
def test_item_plan_properties(n, K, dtype):
    sms = 148
    grid = 2 * sms
    tile, n_tiles, warm, parts_warm, parts_main, tail, parts_tail = rkv.plan_items(n, K, sms, dtype)
    assert tile == (3584 if dtype == rkv.F32 else 7168)
    assert (n_tiles - 1) * tile < n <= n_tiles * tile
    assert 1 <= warm <= n_tiles
    assert 1 <= parts_warm <= K and -(-K // parts_warm) <= 64
    if warm < grid:
        # few tiles: the candidates are split so that every block gets an item, if K allows
        assert warm * parts_warm >= min(grid, warm * K)
    if n_tiles <= grid:
        assert warm == n_tiles           # everything fits the first wave of blocks: nobody to warm up for
    else:
        # the square root of the tile count, at most 18
        assert warm == min(18, math.isqrt(n_tiles))
    if warm < n_tiles:
        # a short warm-up group, then the fewest parts of at most 64 (more while the tiles are fewer
        # than the blocks)
        assert warm * warm <= n_tiles
        main = n_tiles - warm - tail
        assert parts_main == max(-(-K // 64), min(K, -(-grid // main) if main < grid else 1))
        # a long tensor ends with half a tile per block in parts a quarter that size
        if n_tiles - warm >= 4 * grid:
            assert tail == grid // 2 and parts_tail == min(K, 4 * parts_main)
            assert -(-K // parts_tail) <= 16
        else:
            assert tail == 0 and parts_tail == 0
        assert warm + tail < n_tiles
    else:
        assert parts_main == 0 and tail == 0 and parts_tail == 0


def test_item_plan_rejects_bad_arguments():
    for args in [(0, 4, 148), (1000, 0, 148), (1000, 4, 0)]:
        with pytest.raises(rkv.RkvError) as e:
            rkv.plan_items(*args)
        assert e.value.status == rkv.ERR_INVALID_ARG
    with pytest.raises(rkv.RkvError) as e:
        rkv.plan_items(1 << 40, 4, 148)
    assert e.value.status == rkv.ERR_UNSUPPORTED


def _desc(n=1024, ref=0x1000, cand=0x2000, K=1, atol=1e-5, rtol=1e-5, cand_dtype=0, ref_dtype=0,
          ref_src=1, input_src=0, inp=0, ref_dist=0):
    d = rkv.TensorDescC()
    d.n = n
    d.ref = ref
    d.input = inp
    ptrs = (ctypes.c_void_p * K)(*[cand + 0x100000 * k for k in range(K)])
    d.cands = ctypes.cast(ptrs, ctypes.POINTER(ctypes.c_void_p))
    d.cand_dtype, d.ref_dtype, d.ref_src, d.input_src = cand_dtype, ref_dtype, ref_src, input_src
    d.ref_gen = rkv.GenSpec(0, 0, ref_dist, 0)
    d.atol, d.rtol = atol, rtol
    return d, ptrs


def _call_multi(d, K=1, stats=0x3000, ws=0x4000, ws_bytes=1 << 30):
    arr = (rkv.TensorDescC * 1)(d)
    return rkv.lib().rkv_verify_multi(arr, 1, K, ctypes.c_void_p(stats), None, ctypes.c_void_p(ws),
                                      ws_bytes, None)


def test_verify_multi_validates_before_any_cuda_call():
    bad = [
        (dict(n=0), rkv.ERR_INVALID_ARG),
        (dict(n=1 << 40), rkv.ERR_UNSUPPORTED),
        (dict(ref=0), rkv.ERR_INVALID_ARG),
        (dict(ref=0x1004), rkv.ERR_ALIGNMENT),
        (dict(cand=0x2008), rkv.ERR_ALIGNMENT),
        (dict(cand=0), rkv.ERR_INVALID_ARG),
        (dict(atol=float("nan")), rkv.ERR_INVALID_ARG),
        (dict(rtol=float("inf")), rkv.ERR_INVALID_ARG),
        (dict(atol=-1e-5), rkv.ERR_INVALID_ARG),
        (dict(cand_dtype=3), rkv.ERR_INVALID_ARG),
        (dict(ref_src=2, ref_dtype=2), rkv.ERR_UNSUPPORTED),      # no fp16 rounding in the generator
        (dict(ref_dtype=-1), rkv.ERR_INVALID_ARG),
        (dict(ref_src=0), rkv.ERR_INVALID_ARG),
        (dict(ref_src=2, ref_dist=9), rkv.ERR_INVALID_ARG),
        (dict(input_src=1, inp=0), rkv.ERR_INVALID_ARG),
        (dict(input_src=1, inp=0x5002), rkv.ERR_ALIGNMENT),
        (dict(input_src=3), rkv.ERR_INVALID_ARG),
    ]
    for kw, want in bad:
        d, keep = _desc(**kw)
        assert _call_multi(d) == want, kw
    d, keep = _desc()
    assert _call_multi(d, K=0) == rkv.ERR_INVALID_ARG
    assert _call_multi(d, stats=0) == rkv.ERR_INVALID_ARG
    assert _call_multi(d, ws=0) == rkv.ERR_WORKSPACE
    assert _call_multi(d, ws=0x4010) == rkv.ERR_ALIGNMENT
    arr = (rkv.TensorDescC * 1)(d)
    assert rkv.lib().rkv_verify_multi(arr, 65, 1, ctypes.c_void_p(0x3000), None,
                                      ctypes.c_void_p(0x4000), 1 << 30, None) == rkv.ERR_UNSUPPORTED
    assert rkv.lib().rkv_verify_multi(None, 1, 1, ctypes.c_void_p(0x3000), None,
                                      ctypes.c_void_p(0x4000), 1 << 30, None) == rkv.ERR_INVALID_ARG


def test_sweep_validates_before_any_cuda_call():
    L = rkv.lib()
    d, keep = _desc()
    arr = (rkv.TensorDescC * 1)(d)

    def call(cases, C, K=1, stats=0x3000, ws=0x4000, ws_bytes=1 << 30):
        return L.rkv_verify_sweep(cases, C, K, ctypes.c_void_p(stats), None, None, ctypes.c_void_p(ws), ws_bytes, None)

    one = (rkv.CaseDescC * 1)()
    one[0].tensors = ctypes.cast(arr, ctypes.POINTER(rkv.TensorDescC))
    one[0].T = 1
    assert call(None, 1) == rkv.ERR_INVALID_ARG
    assert call(one, 0) == rkv.ERR_INVALID_ARG
    assert call(one, 1, K=0) == rkv.ERR_INVALID_ARG
    assert call(one, 1, stats=0) == rkv.ERR_INVALID_ARG
    assert call(one, 1, ws=0) == rkv.ERR_WORKSPACE
    assert call(one, 1, ws=0x4010) == rkv.ERR_ALIGNMENT
    one[0].T = 0
    assert call(one, 1) == rkv.ERR_INVALID_ARG
    one[0].T = 65
    assert call(one, 1) == rkv.ERR_UNSUPPORTED
    one[0].T = 1
    many = (rkv.CaseDescC * 4097)()
    for i in range(4097):
        many[i].tensors = ctypes.cast(arr, ctypes.POINTER(rkv.TensorDescC))
        many[i].T = 1
    assert call(many, 4097) == rkv.ERR_UNSUPPORTED                 # more than 4096 tensors over all cases
    bad, keep2 = _desc(ref=0x1004)
    arr2 = (rkv.TensorDescC * 1)(bad)
    one[0].tensors = ctypes.cast(arr2, ctypes.POINTER(rkv.TensorDescC))
    assert call(one, 1) == rkv.ERR_ALIGNMENT
    assert L.rkv_sweep_workspace_bytes(None, 1, 1) == 0


def test_gen_and_batch_validate_before_any_cuda_call():
    L = rkv.lib()
    assert L.rkv_gen_inputs_ex(0, 0, 0, 16, 0, 0, None, None) == rkv.ERR_INVALID_ARG
    assert L.rkv_gen_inputs_ex(0, 0, 5, 16, 0, 0, ctypes.c_void_p(0x1000), None) == rkv.ERR_INVALID_ARG
    assert L.rkv_gen_inputs_ex(0, 0, 0, 0, 0, 0, ctypes.c_void_p(0x1000), None) == rkv.ERR_INVALID_ARG
    assert L.rkv_gen_inputs_ex(0, 0, 0, 16, 3, 0, ctypes.c_void_p(0x1000), None) == rkv.ERR_INVALID_ARG
    assert L.rkv_gen_inputs_ex(0, 0, 0, 16, 0, 3, ctypes.c_void_p(0x1000), None) == rkv.ERR_INVALID_ARG
    assert L.rkv_gen_inputs_ex(0, 0, 0, 16, 0, 0, ctypes.c_void_p(0x1008), None) == rkv.ERR_ALIGNMENT
    shape = (ctypes.c_int64 * 2)(4, 0)
    assert L.rkv_gen_inputs(0, 0, shape, 2, 0, ctypes.c_void_p(0x1000)) == rkv.ERR_INVALID_ARG
    assert L.rkv_gen_inputs(0, 0, None, 2, 0, ctypes.c_void_p(0x1000)) == rkv.ERR_INVALID_ARG
    ptrs = (ctypes.c_void_p * 2)(0x2000, 0x3000)
    assert L.rkv_verify_batch(None, ptrs, 2, 16, 0, 1e-5, 1e-5, ctypes.c_void_p(0x9000)) == rkv.ERR_INVALID_ARG
    assert L.rkv_verify_batch(ctypes.c_void_p(0x1000), ptrs, 2, 16, 0, 1e-5, 1e-5, None) == rkv.ERR_INVALID_ARG
    assert L.rkv_verify_batch(ctypes.c_void_p(0x1000), ptrs, 0, 16, 0, 1e-5, 1e-5,
                              ctypes.c_void_p(0x9000)) == rkv.ERR_INVALID_ARG
    assert L.rkv_verify_batch_host(None, ptrs, 2, 16, 0, 1e-5, 1e-5, ctypes.c_void_p(0x9000)) == rkv.ERR_INVALID_ARG
    assert L.rkv_device_status(None, None) == rkv.ERR_INVALID_ARG


@pytest.mark.skipif(HAS_GPU, reason="only meaningful without a device")
def test_no_device_is_an_error_not_a_fallback():
    d, keep = _desc()
    assert _call_multi(d) == rkv.ERR_CUDA
    assert rkv.lib().rkv_gen_inputs_ex(0, 0, 0, 16, 0, 0, ctypes.c_void_p(0x1000), None) == rkv.ERR_CUDA
    arr = (rkv.TensorDescC * 1)(d)
    assert rkv.lib().rkv_workspace_bytes(arr, 1, 1) == 0


def test_population_plans_are_seeded_and_cover_the_kinds():
    from paper_2509_14279_b200 import population as pop
    a = pop.plan_mixed(64, 1 << 20, seed=1, fault_rate=0.4)
    b = pop.plan_mixed(64, 1 << 20, seed=1, fault_rate=0.4)
    assert a == b and a != pop.plan_mixed(64, 1 << 20, seed=2, fault_rate=0.4)
    kinds = {c.kind for c in a}
    assert pop.NOISE in kinds and len(kinds & set(pop.FAULT_KINDS)) >= 3
    c3 = pop.plan_mixed(64, 1 << 20, seed=2, fault_rate=0.01, bf16=True)
    assert any(c.kind in pop.FAULT_KINDS for c in c3)              # at least one fault is forced
    m = pop.plan_multi(128, (1 << 20, 4096, 4096), seed=3, fault_rate=0.1)
    assert len(m) == 128 and all(len(r) == 3 for r in m)
    assert all(sum(c.kind in pop.FAULT_KINDS for c in r) <= 1 for r in m)


def test_screen_outputs_validates_before_any_cuda_call():
    L = rkv.lib()
    assert rkv.SCREEN_BYTES == 64
    text = open(os.path.join(ROOT, "include", "rkv.h")).read()
    assert "rkv_screen_stats;               /* 64 bytes */" in text

    def call(ptr_values=(0x1000, 0x2000), S=None, rows=8, cols=8, dtype=0, lims=(0.01, 0.01, 0.01),
             stats=0x9000, ws=0x4000, ws_bytes=1 << 30):
        ptrs = (ctypes.c_void_p * max(1, len(ptr_values)))(*ptr_values)
        return L.rkv_screen_outputs(ptrs, len(ptr_values) if S is None else S, rows, cols, dtype, lims[0],
                                    lims[1], lims[2], ctypes.c_void_p(stats), ctypes.c_void_p(ws), ws_bytes, None)

    assert call(S=0) == rkv.ERR_INVALID_ARG
    assert call(rows=0) == rkv.ERR_INVALID_ARG
    assert call(cols=0) == rkv.ERR_INVALID_ARG
    assert call(dtype=2) == rkv.ERR_INVALID_ARG
    assert call(stats=0) == rkv.ERR_INVALID_ARG
    assert call(ptr_values=(0x1000, 0)) == rkv.ERR_INVALID_ARG
    assert call(ptr_values=(0x1000, 0x2004)) == rkv.ERR_ALIGNMENT
    assert call(ptr_values=tuple(0x1000 * (i + 1) for i in range(17))) == rkv.ERR_UNSUPPORTED
    assert call(rows=1 << 20, cols=1 << 20) == rkv.ERR_UNSUPPORTED
    assert call(lims=(-0.01, 0.01, 0.01)) == rkv.ERR_INVALID_ARG
    assert call(lims=(0.01, float("nan"), 0.01)) == rkv.ERR_INVALID_ARG
    assert call(lims=(0.01, 0.01, -1.0)) == rkv.ERR_INVALID_ARG
    assert call(ws=0) == rkv.ERR_WORKSPACE
    assert call(ws=0x4008) == rkv.ERR_ALIGNMENT
    assert L.rkv_screen_outputs(None, 2, 8, 8, 0, 0.01, 0.01, 0.01, ctypes.c_void_p(0x9000),
                                ctypes.c_void_p(0x4000), 1 << 30, None) == rkv.ERR_INVALID_ARG


def test_binding_refuses_mismatched_tensors_before_the_c_call():
    """A candidate of the wrong size, dtype or device, a strided view or too small a result
    buffer must raise on the host: the C ABI sees pointers only and would read past the end."""
    ref = torch.zeros(1024)
    good = torch.zeros(1024)
    with pytest.raises(ValueError, match="candidate 1.*1000 elements"):
        rkv._require_case(ref, [good, torch.zeros(1000)], "t", device_type="cpu")
    with pytest.raises(TypeError, match="candidate 0.*dtype"):
        rkv._require_case(ref, [good.to(torch.bfloat16)], "t", device_type="cpu")
    with pytest.raises(ValueError, match="not contiguous"):
        rkv._require_case(ref, [torch.zeros(2048)[::2]], "t", device_type="cpu")
    with pytest.raises(TypeError, match="float32, bfloat16 or float16"):
        rkv._require_case(ref.double(), [good.double()], "t", device_type="cpu")
    with pytest.raises(ValueError, match="no candidates"):
        rkv._require_case(ref, [], "t", device_type="cpu")
    with pytest.raises(ValueError, match="stats_out.*needs at least"):
        rkv._require_case(ref, [good, good], "t", stats_out=torch.zeros(100, dtype=torch.uint8), device_type="cpu")
    rkv._require_case(ref, [good, good], "t", stats_out=torch.zeros(176, dtype=torch.uint8), device_type="cpu")
    # the device forms refuse host tensors, the host form refuses nothing it should take
    with pytest.raises(ValueError, match="expected a cuda tensor"):
        rkv.verify_batch(ref, [good], 1e-5, 1e-5)
    with pytest.raises(ValueError, match="expected a cuda tensor"):
        rkv.verify_batch_static(ref, [good], 1e-5, 1e-5, torch.zeros(88, dtype=torch.uint8))
    with pytest.raises(ValueError, match="expected cuda"):
        rkv.TensorDesc(n=1024, cands=[good], atol=1e-5, rtol=1e-5, ref=ref).to_c()
    with pytest.raises(TypeError):
        rkv._require(3.0, "x")
    # the pointer table of the cross-seed check is refused the same way, before anything is marshalled
    with pytest.raises(ValueError, match="on cpu, expected cuda"):
        rkv.prepare_cross([[good, good]])
    with pytest.raises(ValueError, match="on cpu, expected cuda"):
        rkv.cross_seed([[good, good]], 1e-5, 1e-5)


def test_cross_checks_validate_before_any_cuda_call():
    L = rkv.lib()
    assert rkv.CROSS_BYTES == 32
    vp = ctypes.c_void_p

    def cross(ptrs=(0x1000, 0x2000), K=1, S=2, n=64, dtype=0, atol=1e-5, rtol=1e-5, lim=0.01, stats=0x9000,
              ws=0x4000, ws_bytes=1 << 30):
        arr = (vp * max(1, len(ptrs)))(*ptrs)
        return L.rkv_cross_seed(arr, K, S, n, dtype, atol, rtol, lim, vp(stats), vp(ws), ws_bytes, None)

    assert cross(K=0) == rkv.ERR_INVALID_ARG
    assert cross(S=0) == rkv.ERR_INVALID_ARG
    assert cross(n=0) == rkv.ERR_INVALID_ARG
    assert cross(dtype=3) == rkv.ERR_INVALID_ARG
    assert cross(atol=-1.0) == rkv.ERR_INVALID_ARG
    assert cross(rtol=float("nan")) == rkv.ERR_INVALID_ARG
    assert cross(lim=-0.5) == rkv.ERR_INVALID_ARG
    assert cross(stats=0) == rkv.ERR_INVALID_ARG
    assert cross(S=17) == rkv.ERR_UNSUPPORTED
    assert cross(K=4097) == rkv.ERR_UNSUPPORTED
    assert cross(n=1 << 40) == rkv.ERR_UNSUPPORTED
    assert cross(ptrs=(0x1000, 0)) == rkv.ERR_INVALID_ARG
    assert cross(ptrs=(0x1000, 0x2004)) == rkv.ERR_ALIGNMENT
    assert cross(ws=0) == rkv.ERR_WORKSPACE
    assert L.rkv_cross_seed(None, 1, 2, 64, 0, 1e-5, 1e-5, 0.01, vp(0x9000), vp(0x4000), 1 << 30, None) == rkv.ERR_INVALID_ARG

    def copy(inputs=(0x1000,), cands=(0x2000,), n=64, dtype=0, mask=0x9000, ws=0x4000, ws_bytes=1 << 30, M=None, K=None):
        ia = (vp * max(1, len(inputs)))(*inputs)
        ca = (vp * max(1, len(cands)))(*cands)
        return L.rkv_copy_of_inputs(ia, len(inputs) if M is None else M, ca, len(cands) if K is None else K, n, dtype,
                                    vp(mask), vp(ws), ws_bytes, None)

    assert copy(M=0) == rkv.ERR_INVALID_ARG
    assert copy(K=0) == rkv.ERR_INVALID_ARG
    assert copy(n=0) == rkv.ERR_INVALID_ARG
    assert copy(dtype=7) == rkv.ERR_INVALID_ARG
    assert copy(mask=0) == rkv.ERR_INVALID_ARG
    assert copy(inputs=(0x1000,) * 9) == rkv.ERR_UNSUPPORTED
    assert copy(inputs=(0,)) == rkv.ERR_INVALID_ARG
    assert copy(cands=(0x2008,)) == rkv.ERR_ALIGNMENT
    assert copy(ws=0) == rkv.ERR_WORKSPACE
    assert copy(ws_bytes=8) == rkv.ERR_WORKSPACE
    assert L.rkv_copy_workspace_bytes(0, 1) == 0 and L.rkv_copy_workspace_bytes(4, 2) >= 4 * 4 + 6 * 8
    assert L.rkv_cross_workspace_bytes(1, 17) == 0
