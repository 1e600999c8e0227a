"""The N > 1 path on CPU: two gloo ranks shard the candidates of one case, each
verifies its shard (the oracle stands in for the GPU library here), and the
gathered verdicts and the max-over-ranks time equal the single-process result."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2509_14279_b200 import population as pop
from paper_2509_14279_b200 import shard


def test_k_range_is_a_balanced_partition():
    for K in (0, 1, 7, 8, 64, 129):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                seen.extend(shard.k_range(K, world, r))
            assert seen == list(range(K))
            sizes = [len(shard.k_range(K, world, r)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard.k_range(4, 2, 2)


def _case(K, n, seed):
    ref = oracle.gen(seed, 0, oracle.NORMAL, n)
    inp = oracle.gen(seed, 2, oracle.NORMAL, n)
    plan = pop.plan_mixed(K, n, seed, 0.4)
    cands = [pop.materialize(c, torch.from_numpy(ref), torch.from_numpy(inp)).numpy() for c in plan]
    return ref, inp, cands


def _worker(rank, world, port, K, n, seed, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ref, inp, cands = _case(K, n, seed)             # same seeded case on every rank
        mine = shard.k_range(K, world, rank)
        local = [int(oracle.verify(ref, cands[k], 1e-5, 1e-5, input=inp)["verdict"] == 0) for k in mine]
        everyone = shard.gather_joint_pass(local, K)
        slowest = shard.max_over_ranks(10.0 + rank)      # pretend rank r took 10 + r ms
        total = shard.sum_over_ranks(float(len(mine)))
        np.save(os.path.join(out_dir, f"rank{rank}.npy"),
                np.array(everyone + [int(slowest), int(total)], dtype=np.int64))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("K", [7, 8])
def test_two_ranks_shard_the_candidates_and_agree(tmp_path, K):
    n, seed, world = 5000, 4, 2
    mp.spawn(_worker, args=(world, _free_port(), K, n, seed, str(tmp_path)), nprocs=world, join=True)
    ref, inp, cands = _case(K, n, seed)
    want = [int(oracle.verify(ref, c, 1e-5, 1e-5, input=inp)["verdict"] == 0) for c in cands]
    assert 0 < sum(want) < K
    for r in range(world):
        got = np.load(os.path.join(str(tmp_path), f"rank{r}.npy")).tolist()
        assert got[:K] == want
        assert got[K] == 10 + world - 1          # the slowest rank's time
        assert got[K + 1] == K                   # every candidate verified exactly once


def test_bench_starts_its_own_ranks_when_no_launcher_did(tmp_path):
    """`bench.py --gpus 2` with WORLD_SIZE unset re-executes itself under torch.distributed.run with two
    ranks on 127.0.0.1.  The reference arm runs on CPU: rank 0 prints the one JSON line with n_gpus = 2,
    rank 1 exits 0 without work."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "1", "--workload", "c1"], env=env, capture_output=True, text=True,
                       timeout=600, cwd=str(tmp_path))
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["n_gpus"] == 2 and out["value"] > 0
