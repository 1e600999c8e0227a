"""GPU parity: rkv_gen_inputs / rkv_gen_inputs_ex against the oracle, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_14279_b200 import binding as rkv
from paper_2509_14279_b200 import population as pop

pytestmark = pytest.mark.gpu

SIZES = [1, 2, 3, 4, 5, 7, 8, 9, 31, 32, 33, 255, 256, 257, 1023, 1025, 4095, 4096, 4097, 100003]


def bits(t: torch.Tensor) -> np.ndarray:
    a = pop.bits_numpy(t)
    return a.view(np.uint32) if a.dtype == np.float32 else a


@pytest.mark.parametrize("dist", oracle.DISTS)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_gen_matches_oracle_small_and_ragged(dist, dtype):
    td = torch.float32 if dtype == "f32" else torch.bfloat16
    od = oracle.F32 if dtype == "f32" else oracle.BF16
    for n in SIZES:
        for seed, stream in [(0, 0), (0xFEDCBA9876543210, (7 << 32) | 5)]:
            g = rkv.gen_inputs_ex(seed, stream, dist, n, dtype=td)
            want = oracle.gen(seed, stream, dist, n, dtype=od)
            want = want.view(np.uint32) if od == oracle.F32 else want
            assert np.array_equal(bits(g), want), (dist, dtype, n, seed)


@pytest.mark.parametrize("dist", oracle.DISTS)
def test_gen_matches_oracle_large(dist):
    n = (1 << 22) + 12
    g = rkv.gen_inputs_ex(5, 0, dist, n)
    want = oracle.gen(5, 0, dist, n)
    assert np.array_equal(bits(g), want.view(np.uint32))
    g16 = rkv.gen_inputs_ex(5, 0, dist, n, dtype=torch.bfloat16)
    assert np.array_equal(bits(g16), oracle.gen(5, 0, dist, n, dtype=oracle.BF16))


def test_gen_window_and_block_index_beyond_32_bits():
    for first in (4, 4096, (1 << 34) - 8, (1 << 36) + 4):
        for dist in (oracle.NORMAL, oracle.SPARSE90, oracle.STUDENT_T2):
            g = rkv.gen_inputs_ex(9, 2, dist, 1000, first_elem=first)
            want = oracle.gen(9, 2, dist, 1000, first_elem=first)
            assert np.array_equal(bits(g), want.view(np.uint32))


def test_gen_inputs_shape_form_is_stream_zero():
    g = rkv.gen_inputs(0, rkv.DIST_NORMAL, (256, 1024))
    assert g.shape == (256, 1024)
    want = oracle.gen(0, 0, oracle.NORMAL, 256 * 1024)
    assert np.array_equal(bits(g), want.view(np.uint32))


def test_gen_rejects_bad_arguments():
    out = torch.empty(64, device="cuda")
    with pytest.raises(rkv.RkvError) as e:
        rkv.gen_inputs_ex(0, 0, 7, 64, out=out)
    assert e.value.status == rkv.ERR_INVALID_ARG
    with pytest.raises(rkv.RkvError) as e:
        rkv.gen_inputs_ex(0, 0, 0, 64, first_elem=2, out=out)
    assert e.value.status == rkv.ERR_INVALID_ARG
    with pytest.raises(rkv.RkvError) as e:
        rkv.gen_inputs_ex(0, 0, 0, 32, out=out[1:33])
    assert e.value.status == rkv.ERR_ALIGNMENT
