#!/usr/bin/env python
"""Benchmark of the verification hot path.

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--workload c2]

One step = one pass of the whole path over one batch of synthetic input: for
each value distribution of the workload, regenerate the reference and the input
tensor with the Philox generator (rkv_gen_inputs) and verify all K candidates
against them in one fused launch (rkv_verify_multi, followed by its finalize
kernel).  The metric is verified GB/s: candidate + reference bytes checked per
second, whole job.  Candidates are built once, untimed, and stay resident in
HBM; every launch streams several GB, far more than the 126 MB L2.

With --gpus N > 1 (launched under torch.distributed.run) every rank runs the
same workload on its own GPU with its own seeded candidates (candidates are
independent units: no data-path collective); the time is the max over ranks.

--impl reference times the CPU oracle on the host cores instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "verified_GBps"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", default="c2", choices=["c1", "c2", "c3", "c4", "c5", "s1"],
                    help="c1..c5: the verification workloads (c2 is the benchmark); s1: the task-soundness "
                         "screens over 8 outputs of 4096 x 4096 fp32 (its own metric, not the benchmark)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--max-dists", type=int, default=0, help="use only the first D distributions")
    ap.add_argument("--cands", type=int, default=0,
                    help="override K (a smaller case for profiler captures; not a bench value)")
    return ap.parse_args()


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def kernel_source_hash() -> str:
    h = hashlib.sha256()
    for f in ("rkv_verify.cu", "rkv_philox.cuh", "rkv_internal.h"):
        with open(os.path.join(ROOT, "paper_2509_14279_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def recorded_traffic(workload: str, algo_bytes: float):
    """DRAM bytes per launch of the dominant kernel, from the committed ncu summary
    (``profiles/verify_kernel_<workload>.md`` holds the measured DRAM bytes per
    algorithmic byte of a smaller capture of the same kernel; traffic grows in proportion
    to the bytes streamed).  None if there is no summary or the kernel changed since."""
    p = os.path.join(ROOT, "profiles", f"verify_kernel_{workload}.md")
    try:
        rec = {}
        with open(p) as fh:
            for line in fh:
                if line.startswith("- ") and ":" in line:
                    k, v = line[2:].split(":", 1)
                    rec[k.strip()] = v.strip().strip("`")
        if rec.get("kernel_source_hash") != kernel_source_hash():
            return None
        return float(rec["dram_bytes_per_algorithmic_byte"]) * algo_bytes
    except Exception:
        return None


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples during the timed region."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-i", str(self.index), "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------
# workload construction (device side, untimed)
# ----------------------------------------------------------------------------

def build_workload(name: str, rank: int, max_dists: int = 0, cands_override: int = 0):
    """Returns a list of cases; each case = dict(dist, gens, descs, K, bytes, ...)."""
    import torch

    from paper_2509_14279_b200 import binding as rkv
    from paper_2509_14279_b200 import population as pop

    W = pop.WORKLOADS[name]
    if cands_override:
        import dataclasses
        W = dataclasses.replace(W, K=cands_override)
    dists = W.dists[:max_dists] if max_dists else W.dists
    cases = []
    seed0 = W.seeds[0] + 1000 * rank
    for dist_name in dists:
        dist = pop.DIST_IDS[dist_name]
        descs, gens, algo_bytes, launches = [], [], 0, 0
        for t, n in enumerate(W.numels):
            cdt = W.cand_dtype
            if cdt == "mixed":
                cdt = "f32" if t == 0 else "bf16"
            tdt = torch.float32 if cdt == "f32" else torch.bfloat16
            csz = 4 if cdt == "f32" else 2
            ref_stream = 0 if W.fused else (t << 32)
            inp_stream = 2 if W.fused else (t << 32) | 2
            ref = rkv.gen_inputs_ex(seed0, ref_stream, dist, n)
            inp = rkv.gen_inputs_ex(seed0, inp_stream, dist, n, dtype=tdt)
            if len(W.numels) > 1 and not W.fused:
                plans = pop.plan_multi(W.K, W.numels, seed0 + dist, W.fault_rate)
                plan = [plans[k][t] for k in range(W.K)]
            elif name == "c1":
                plan = pop.plan_c1(n, seed0)
            else:
                plan = pop.plan_mixed(W.K, n, seed0 + dist + 17 * t, W.fault_rate, bf16=(cdt == "bf16"))
            cands = [pop.materialize(c, ref, inp, cdt) for c in plan]
            atol, rtol = W.tols[t] if len(W.tols) > 1 else W.tols[0]
            if W.fused:
                descs.append(rkv.TensorDesc(n=n, cands=cands, atol=atol, rtol=rtol,
                                            ref_gen=(seed0, ref_stream, dist),
                                            input_gen=(seed0, inp_stream, dist)))
                algo_bytes += W.K * n * csz
                del ref, inp
            else:
                descs.append(rkv.TensorDesc(n=n, cands=cands, atol=atol, rtol=rtol, ref=ref, input=inp))
                gens.append((seed0, ref_stream, dist, n, ref))
                gens.append((seed0, inp_stream, dist, n, inp))
                algo_bytes += W.K * n * csz + n * 4
                launches += 2
            del cands
        variants = {(d.cands[0].dtype, None if d.ref is None else d.ref.dtype) for d in descs}
        launches += len(variants) + 1      # one verify kernel per storage variant + finalize
        cases.append({"dist": dist_name, "descs": descs, "gens": gens, "K": W.K, "plan_last": plan,
                      "algo_bytes": algo_bytes, "launches": launches})
    torch.cuda.synchronize()
    return W, cases


def run_native(args):
    import torch
    import torch.distributed as dist

    from paper_2509_14279_b200 import binding as rkv

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    rkv.lib()                                     # fail loudly if the CUDA library is missing

    W, cases = build_workload(args.workload, rank, args.max_dists, args.cands)
    # marshal once; allocate workspace and outputs once
    for c in cases:
        c["arr"] = rkv.prepare(c["descs"])
        c["stats"], c["joint"], c["ws"] = rkv.verify_multi(c["descs"], c["K"], descs=c["arr"])
    torch.cuda.synchronize()

    def one_step(events=None):
        for c in cases:
            for (seed, stream_id, d, n, out) in c["gens"]:
                rkv.gen_inputs_ex(seed, stream_id, d, n, out=out)
            if events is not None:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
            rkv.verify_multi(c["descs"], c["K"], workspace=c["ws"], stats_out=c["stats"],
                             joint_pass=c["joint"], descs=c["arr"])
            if events is not None:
                e1.record()
                events.append((e0, e1, c["algo_bytes"]))

    def barrier():
        if world > 1:
            dist.barrier()

    for _ in range(max(args.warmup, 3)):
        one_step()
    torch.cuda.synchronize()
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.15)
    torch.cuda.synchronize()
    barrier()
    events = []
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(args.steps):
        one_step(events)
    t1.record()
    torch.cuda.synchronize()
    barrier()
    elapsed_ms = t0.elapsed_time(t1)
    clocks = sampler.stop() if rank == 0 else None
    from paper_2509_14279_b200 import shard
    elapsed_ms = shard.max_over_ranks(elapsed_ms, device="cuda")

    step_bytes = sum(c["algo_bytes"] for c in cases)
    value = world * step_bytes * args.steps / (elapsed_ms * 1e-3) / 1e9

    # roofline of the dominant kernel: verify launches timed one by one inside the timed region
    durs = [e0.elapsed_time(e1) * 1e-3 for (e0, e1, _) in events]
    launch_bytes = statistics.mean(b for (_, _, b) in events)
    achieved = launch_bytes / statistics.mean(durs) / 1e9
    peak, peak_kind = measured_peak()
    roofline = {"bound": "hbm", "kernel": "verify_kernel", "achieved": round(achieved, 1),
                "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                "frac": round(achieved / peak, 4),
                "frac_of_nominal_8TBps": round(achieved / NOMINAL_HBM_GBS, 4),
                "algorithmic_bytes_per_launch": launch_bytes,
                "avg_launch_ms": round(statistics.mean(durs) * 1e3, 4),
                "note": "events bracket rkv_verify_multi: table upload + workspace clear + verify_kernel "
                        "(one per storage variant) + finalize_kernel",
                "traffic": recorded_traffic(args.workload, launch_bytes)}

    # verdict sanity on the last case: every planted fault that fails at any scale must fail
    from paper_2509_14279_b200 import population as pop
    last = cases[-1]
    jp = last["joint"].cpu().tolist()
    bad = [k for k, c in enumerate(last["plan_last"]) if c.kind in pop.SCALE_FREE_FAULT_KINDS and jp[k] == 1]
    verdict_check = "ok" if not bad and rkv.device_status(last["ws"]) == 0 else f"FAULTS PASSED: {bad}"

    out = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": round(elapsed_ms / args.steps, 4),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": f"{W.name}: K={W.K} candidates, shapes {list(W.shapes)}, "
                               f"cand {W.cand_dtype}, {len(cases)} distributions per step"
                               f"{', fused regeneration' if W.fused else ''}",
                   "distributions": [c["dist"] for c in cases],
                   "bytes_per_step": step_bytes, "l2": "inputs larger than L2 (each launch streams > 4 GB)",
                   "parallelism": f"replicas x{world}" if world > 1 else "single gpu"},
        "gpu_launches": sum(c["launches"] for c in cases) * args.steps,
        "roofline": roofline, "clocks": clocks, "verdict_check": verdict_check,
    }
    if rank == 0:
        if not args.no_e2e:
            out["e2e"] = run_e2e(args, W, cases[0], world)
        if not args.no_cpu_baseline and world == 1:
            out["cpu_baseline"] = cpu_baseline_sample(W)
        print(json.dumps(out), flush=True)
    elif not args.no_e2e:
        run_e2e(args, W, cases[0], world)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_e2e(args, W, case, world):
    """Same metric through rkv_verify_batch_host: pinned HOST buffers in, HOST
    results out, copies inside the timed region.  One distribution per step."""
    import torch
    import torch.distributed as dist

    from paper_2509_14279_b200 import binding as rkv

    d = case["descs"][0]
    if d.ref is None:
        ref_dev = rkv.gen_inputs_ex(d.ref_gen[0], d.ref_gen[1], d.ref_gen[2], d.n)
    else:
        ref_dev = d.ref
    cand_dt = d.cands[0].dtype
    ref_h = ref_dev.reshape(-1).to(cand_dt).cpu().pin_memory()
    cands_h = [c.cpu().pin_memory() for c in d.cands]
    esz = cands_h[0].element_size()
    h2d = (len(cands_h) + 1) * d.n * esz
    d2h = len(cands_h) * rkv.STATS_BYTES
    steps = max(2, min(args.steps, 5))
    for _ in range(2):
        rkv.verify_batch_host(ref_h, cands_h, d.atol, d.rtol)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(steps):
        rkv.verify_batch_host(ref_h, cands_h, d.atol, d.rtol)
    torch.cuda.synchronize()
    el = time.perf_counter() - t0
    from paper_2509_14279_b200 import shard
    el = shard.max_over_ranks(el, device="cuda")
    return {"value": round(world * h2d * steps / el / 1e9, 2), "unit": UNIT,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": steps,
            "sample": f"one distribution ({case['dist']}) per step, pinned host buffers, "
                      "through rkv_verify_batch_host"}


# ----------------------------------------------------------------------------
# CPU oracle timing (reported baseline / reference arm)
# ----------------------------------------------------------------------------

def _oracle_sample_step(W, dist_id, n_s, k_s, threads, seed):
    """One bounded sample: generate reference + input (n_s elements) and verify
    k_s candidates with the oracle.  Returns (seconds, bytes verified)."""
    from concurrent.futures import ThreadPoolExecutor

    import numpy as np
    import torch

    import oracle
    from paper_2509_14279_b200 import population as pop

    bf16 = W.cand_dtype == "bf16"
    t0 = time.perf_counter()
    ref = oracle.gen(seed, 0, dist_id, n_s)
    inp = oracle.gen(seed, 2, dist_id, n_s, dtype=oracle.BF16 if bf16 else oracle.F32)
    t_gen = time.perf_counter() - t0
    plan = pop.plan_mixed(k_s, n_s, seed, W.fault_rate, bf16=bf16)
    tr, ti = torch.from_numpy(ref), pop.from_bits(inp)
    cands = [pop.bits_numpy(pop.materialize(c, tr, ti, "bf16" if bf16 else "f32")) for c in plan]
    atol, rtol = W.tols[0]
    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(lambda c: oracle.verify(ref, c, atol, rtol, input=inp), cands))
    t_ver = time.perf_counter() - t0
    nbytes = k_s * n_s * (2 if bf16 else 4) + n_s * 4
    return t_gen + t_ver, nbytes


def cpu_baseline_sample(W, budget_s: float = 12.0):
    """The oracle on the host cores, on a bounded sample of the workload: the first
    distribution, a 4 Mi-element slice of the tensor, 16 candidates, repeated until
    about `budget_s` seconds of oracle time have been spent."""
    import oracle
    from paper_2509_14279_b200 import population as pop

    oracle.lib()
    cores = os.cpu_count() or 1
    threads = min(cores, 16)
    n_s = min(W.numels[0], 1 << 22)
    k_s = 16
    secs, nbytes, reps = 0.0, 0, 0
    while secs < budget_s and reps < 200:
        s, b = _oracle_sample_step(W, pop.DIST_IDS[W.dists[0]], n_s, k_s, threads, W.seeds[0] + reps)
        secs += s
        nbytes += b
        reps += 1
    return {"value": round(nbytes / secs / 1e9, 4), "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{W.dists[0]}: {reps} x (generate reference+input of {n_s} elements on 1 thread, "
                      f"verify {k_s} candidates of {n_s} elements on {threads} threads); {secs:.1f} s of oracle time",
            "host_cores_available": cores}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank != 0:
        return
    import oracle
    from paper_2509_14279_b200 import population as pop

    oracle.lib()
    W = pop.WORKLOADS[args.workload]
    cores = os.cpu_count() or 1
    threads = min(cores, 16)
    n_s = min(W.numels[0], 1 << 20)
    k_s = 8
    dists = [pop.DIST_IDS[d] for d in W.dists]
    for i in range(max(args.warmup, 1)):
        _oracle_sample_step(W, dists[i % len(dists)], n_s, k_s, threads, W.seeds[0])
    total_s, total_b = 0.0, 0
    for i in range(args.steps):
        s, b = _oracle_sample_step(W, dists[i % len(dists)], n_s, k_s, threads, W.seeds[0] + i)
        total_s += s
        total_b += b
    value = total_b / total_s / 1e9
    sample = (f"per step: one distribution (rotating), generate reference+input of {n_s} elements and "
              f"verify {k_s} candidates, {threads} threads")
    out = {
        "impl": "reference", "metric": METRIC, "value": round(value, 4), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 1), "ms_per_step": round(total_s / args.steps * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": f"{W.name}: K={W.K} candidates, shapes {list(W.shapes)}, cand {W.cand_dtype} "
                               "(CPU oracle on a bounded sample per step)"},
        "cpu_baseline": {"value": round(value, 4), "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": round(value, 4), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


def run_screen(args):
    """Workload s1: rkv_screen_outputs over the reference outputs of 8 seeds, 4096 x 4096 fp32
    each (512 MiB streamed per call, > L2).  One step = one call (screen_kernel + merge)."""
    import torch

    from paper_2509_14279_b200 import binding as rkv

    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    rkv.lib()
    S, rows, cols = 8, 4096, 4096
    outs = [rkv.gen_inputs_ex(21, s, rkv.DIST_NORMAL, rows * cols).reshape(rows, cols) for s in range(S)]
    stats, ws = rkv.screen_outputs(outs)
    for _ in range(max(args.warmup, 3)):
        rkv.screen_outputs(outs, stats_out=stats, workspace=ws)
    torch.cuda.synchronize()
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    time.sleep(0.15)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(args.steps):
        rkv.screen_outputs(outs, stats_out=stats, workspace=ws)
    t1.record()
    torch.cuda.synchronize()
    ms = t0.elapsed_time(t1) / args.steps
    clocks = sampler.stop()
    nbytes = S * rows * cols * 4
    achieved = nbytes / (ms * 1e-3) / 1e9
    peak, peak_kind = measured_peak()
    got = rkv.screen_to_numpy(stats)[0]
    out = {
        "metric": "screened_GBps", "value": round(achieved, 2), "unit": "GB/s", "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": round(ms, 4), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"s1: task-soundness screens, S={S} outputs of {rows}x{cols} fp32 (normal)",
                   "bytes_per_step": nbytes, "l2": "inputs larger than L2 (512 MiB per call)",
                   "parallelism": "single gpu"},
        "gpu_launches": 2 * args.steps,
        "roofline": {"bound": "hbm", "kernel": "screen_kernel", "achieved": round(achieved, 1), "peak": peak,
                     "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": round(achieved / peak, 4),
                     "algorithmic_bytes_per_launch": nbytes, "avg_launch_ms": round(ms, 4),
                     "note": "events bracket the calls: screen_kernel + screen_finalize_kernel", "traffic": None},
        "clocks": clocks,
        "result_check": "ok" if int(got["flags"]) == 0 and int(got["n_values"]) == S * rows * cols else "UNEXPECTED",
    }
    if not args.no_cpu_baseline:
        import numpy as np

        import oracle
        sub = [o[:512].contiguous().cpu().numpy() for o in outs]
        t = time.perf_counter()
        oracle.screen(sub)
        el = time.perf_counter() - t
        out["cpu_baseline"] = {"value": round(S * 512 * cols * 4 / el / 1e9, 4), "unit": "GB/s", "cores": 1,
                               "kind": "oracle", "sample": f"the first 512 rows of the {S} outputs, {el:.2f} s"}
    print(json.dumps(out), flush=True)


def main():
    args = parse_args()
    if args.workload == "s1":
        if args.impl == "reference" or int(os.environ.get("WORLD_SIZE", "1")) > 1:
            print(json.dumps({"impl": args.impl, "unavailable": "workload s1 runs on one GPU, native arm only"}))
            return
        run_screen(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_native(args)


if __name__ == "__main__":
    main()
