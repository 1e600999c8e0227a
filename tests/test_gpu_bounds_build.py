"""The small-case suite under the range-checked build of the library.

`python -m paper_2509_14279_b200.build --debug-bounds` compiles the same sources with
RKV_DEBUG_BOUNDS: the verification kernel then checks every index into global memory and
into its shared-memory tables before using it, records the first violation in the
workspace header and skips the access (status RKV_ERR_BOUNDS; nothing traps or asserts).
This stands in for a memory checker: sizes around every tile and vector boundary, candidate
counts around the part limits, all storage types, stored and regenerated references.  The
run happens in a child process because a process loads one build of the library.
"""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
import numpy as np, torch
sys.path.insert(0, %(root)r); sys.path.insert(0, %(tests)r)
import oracle
from paper_2509_14279_b200 import binding as rkv
from paper_2509_14279_b200 import population as pop
from rkv_testlib import assert_stats_equal, build_case_cpu, mixed_plan, oracle_gen_tensor
assert rkv.debug_bounds_build(), "not the range-checked build"
TD = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}
checked = 0
for n in (1, 2, 3, 4, 5, 31, 32, 33, 3583, 3584, 3585, 4095, 4096, 4097, 7167, 7168, 7169, 3584 * 300 + 1):
    for K in (1, 2, 7, 8, 9, 65):
        if n > 10000 and K not in (2, 65):
            continue
        for cdt, rdt in (("f32", "f32"), ("bf16", "f32"), ("f16", "f16")):
            ref = oracle_gen_tensor(n + K, 0, oracle.NORMAL, n, "f32").to(TD[rdt])
            inp = oracle_gen_tensor(n + K, 2, oracle.NORMAL, n, "f32").to(TD[cdt])
            cands = build_case_cpu(mixed_plan(K, n, seed=n + K, bf16=cdt != "f32"), ref, inp, cdt)
            tol = (1e-5, 1e-5) if cdt == "f32" else (1e-2, 1.6e-2)
            d = rkv.TensorDesc(n=n, cands=[c.cuda() for c in cands], atol=tol[0], rtol=tol[1], ref=ref.cuda(),
                               input=inp.cuda())
            stats, joint, ws = rkv.verify_multi([d], K)
            st = rkv.device_status(ws)
            assert st == rkv.OK, (n, K, cdt, st, ws[:64].cpu().numpy().view(np.uint32)[8:14])
            got = rkv.stats_to_numpy(stats)
            for k in range(K):
                w = oracle.verify(pop.bits_numpy(ref), pop.bits_numpy(cands[k]), tol[0], tol[1], input=pop.bits_numpy(inp))
                assert_stats_equal(got[k], w, f"n={n} K={K} {cdt}/{rdt} k={k}")
            checked += 1
            if cdt != "f16":      # the same case with reference and input regenerated
                d2 = rkv.TensorDesc(n=n, cands=d.cands, atol=tol[0], rtol=tol[1], ref_gen=(n + K, 0, rkv.DIST_NORMAL),
                                    input_gen=(n + K, 2, rkv.DIST_NORMAL), ref_dtype=rkv.F32)
                s2, _, ws2 = rkv.verify_multi([d2], K)
                assert rkv.device_status(ws2) == rkv.OK
                assert rkv.stats_to_numpy(s2).tobytes() == got.tobytes(), (n, K, cdt)
print("bounds build ok:", checked, "cases")
"""


def test_small_cases_pass_every_range_check():
    from paper_2509_14279_b200 import build as rkv_build
    lib = rkv_build.build(debug_bounds=True)
    env = dict(os.environ, RKV_LIB=lib)
    code = CHILD % {"root": ROOT, "tests": os.path.join(ROOT, "tests")}
    r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "bounds build ok" in r.stdout
