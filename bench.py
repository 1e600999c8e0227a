#!/usr/bin/env python
"""Benchmark of the verification hot path.

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--workload c5]

One step = one pass of the whole path over one batch of synthetic input.  The default
workload is c5, the large sweep: for each of the five value distributions, 128 fp32 and
128 bf16 candidate tensors of 2^24 elements are verified in one fused call
(rkv_verify_multi) against a reference -- and an input tensor for the copy flag -- that
the kernel regenerates from the Philox stream instead of reading (fused generate +
verify).  The four seeds 10..13 are spread over the distributions; when memory allows,
two such sets are resident and the steps alternate between them, so that every
distribution meets two seeds and every step all four.  Workloads that read their
reference from memory (c1..c4) regenerate it with rkv_gen_inputs_ex inside the step.

The metric is verified GB/s: candidate (+ reference, when it is read) bytes checked per
second, whole job.  Candidates are built once, untimed, and stay resident in HBM; every
launch streams several GB, far more than the 126 MB L2.

The same line carries, per workload c1..c4, the timing of the verify call alone
(`per_workload`), the generator's own throughput (`generator`), the end-to-end number
through the host-buffer entry point (`e2e`) and the CPU oracle timed on the host cores
(`cpu_baseline`).

With --gpus N > 1 every rank runs the same workload on its own GPU with its own seeded
candidates (candidates are independent units: no data-path collective); the time is the
max over ranks.  Started without a launcher (WORLD_SIZE unset) the script starts the N
ranks itself under torch.distributed.run.

--impl reference times the CPU oracle on the host cores instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import socket
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
DTYPE_NOTE = {"f32": "f32", "bf16": "f32 arithmetic on bf16 candidates (upcast exactly)",
              "mixed": "f32 arithmetic on f32 and bf16 candidates (bf16 upcast exactly)"}


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", default="c5", choices=["c1", "c2", "c3", "c4", "c5", "s1", "x1", "w1"],
                    help="c1..c5: the verification workloads (c5, the large sweep, is the benchmark); "
                         "s1: task-soundness screens; x1: cross-seed variation check; w1: config sweep of 256 small "
                         "cases (each its own metric, not the benchmark)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-workload", action="store_true")
    ap.add_argument("--no-generator", action="store_true")
    ap.add_argument("--sets", type=int, default=0,
                    help="resident candidate sets of c5 the steps alternate between (0: two if memory allows)")
    ap.add_argument("--max-dists", type=int, default=0, help="use only the first D distributions")
    ap.add_argument("--cands", type=int, default=0,
                    help="override K (a smaller case for profiler captures; not a bench value)")
    return ap.parse_args(argv)


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


def generator_inst_per_elem():
    """Lane-instructions per generated element and distribution, from the committed ncu count
    (``profiles/gen_kernel_f32.md``); None once the generator's sources changed since."""
    try:
        h = hashlib.sha256()
        for f in ("rkv_gen.cu", "rkv_philox.cuh"):
            with open(os.path.join(ROOT, "paper_2509_14279_b200", "csrc", f), "rb") as fh:
                h.update(fh.read())
        rec, inst = {}, {}
        with open(os.path.join(ROOT, "profiles", "gen_kernel_f32.md")) as fh:
            for line in fh:
                if line.startswith("- lane_inst_per_elem "):
                    k, v = line[len("- lane_inst_per_elem "):].split(":", 1)
                    inst[k.strip()] = float(v)
                elif line.startswith("- kernel_source_hash:"):
                    rec["hash"] = line.split(":", 1)[1].strip().strip("`")
        return inst if rec.get("hash") == h.hexdigest()[:16] else None
    except Exception:
        return None


def sm_max_mhz(index: int) -> float:
    """clocks.max.sm of the device (read only), 1965 MHz if nvidia-smi does not answer."""
    try:
        r = subprocess.run(["nvidia-smi", "--query-gpu=clocks.max.sm", "--format=csv,noheader,nounits", "-i", str(index)],
                           capture_output=True, text=True, timeout=20)
        return float(r.stdout.strip().splitlines()[0])
    except Exception:
        return 1965.0


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
                    rec.setdefault(k.strip(), v.strip().strip("`"))
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
# multi-GPU launch
# ----------------------------------------------------------------------------

def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def relaunch_if_needed(args) -> None:
    """`bench.py --gpus N` started without a launcher starts its N ranks itself: one
    process per GPU under torch.distributed.run, rendezvous on 127.0.0.1."""
    if args.gpus <= 1 or "WORLD_SIZE" in os.environ:
        return
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()),
           os.path.abspath(__file__), *sys.argv[1:]]
    sys.stdout.flush()
    os.execv(sys.executable, cmd)


# ----------------------------------------------------------------------------
# workload construction (device side, untimed)
# ----------------------------------------------------------------------------

def build_case(W, dist_name: str, seed: int, rank: int = 0):
    """One verification case of workload W: the candidates of every tensor for one value
    distribution and one seed, resident on the device.  Returns a dict with the
    descriptors, the generator launches a step repeats (`gens`), the candidate plans per
    tensor (`plans[t][k]`) and the algorithmic bytes of one verify call."""
    import torch

    from paper_2509_14279_b200 import binding as rkv
    from paper_2509_14279_b200 import population as pop

    dist = pop.DIST_IDS[dist_name]
    seed0 = seed + 1000 * rank
    descs, gens, plans, algo_bytes, launches = [], [], [], 0, 0
    multi = pop.plan_multi(W.K, W.numels, seed0 + dist, W.fault_rate) \
        if (len(W.numels) > 1 and not W.fused) else None
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
        if multi is not None:
            plan = [multi[k][t] for k in range(W.K)]
        elif W.name == "c1":
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
        plans.append(plan)
        del cands
    launches += 2                              # verify_kernel (one launch for all tensors) + finalize_case_kernel
    if W.fused and any(n >= 2048 * (3584 if (W.cand_dtype == "f32" or (W.cand_dtype == "mixed" and t == 0)) else 7168)
                       for t, n in enumerate(W.numels)):
        launches += 1                          # copy_check_kernel: regenerated input, a tensor with a warm-up group
    return {"dist": dist_name, "seed": seed, "descs": descs, "gens": gens, "K": W.K, "plans": plans,
            "plan_last": plans[-1], "algo_bytes": algo_bytes, "launches": launches}


def case_list(W, n_sets: int = 1, max_dists: int = 0):
    """(distribution, seed) pairs of a workload, one list per resident set.  The seeds of
    the workload are spread over its distributions; set j shifts the assignment by 2j."""
    dists = W.dists[:max_dists] if max_dists else W.dists
    S = len(W.seeds)
    return [[(d, W.seeds[(i + 2 * j) % S]) for i, d in enumerate(dists)] for j in range(n_sets)]


def build_workload(name: str, rank: int, max_dists: int = 0, cands_override: int = 0, n_sets: int = 1):
    """Returns (W, sets): sets[j] is the list of resident cases a step of set j verifies."""
    import dataclasses

    import torch

    from paper_2509_14279_b200 import population as pop

    W = pop.WORKLOADS[name]
    if cands_override:
        W = dataclasses.replace(W, K=cands_override)
    sets = [[build_case(W, d, s, rank) for (d, s) in pairs] for pairs in case_list(W, n_sets, max_dists)]
    torch.cuda.synchronize()
    return W, sets


def prepare_case(c):
    """Marshal once; allocate workspace and outputs once (one untimed call)."""
    from paper_2509_14279_b200 import binding as rkv
    c["arr"] = rkv.prepare(c["descs"])
    c["stats"], c["joint"], c["ws"] = rkv.verify_multi(c["descs"], c["K"], descs=c["arr"])


def step_case(c, events=None):
    """The part of a step that belongs to one case: regenerate what is read from memory,
    then verify every candidate in one call."""
    import torch

    from paper_2509_14279_b200 import binding as rkv
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


def verdict_check(c) -> str:
    """Every planted fault that fails at any scale must fail; the device status must be clean."""
    from paper_2509_14279_b200 import binding as rkv
    from paper_2509_14279_b200 import population as pop
    jp = c["joint"].cpu().tolist()
    bad = []
    for plan in c["plans"]:
        bad += [k for k, cand in enumerate(plan) if cand.kind in pop.SCALE_FREE_FAULT_KINDS and jp[k] == 1]
    if rkv.device_status(c["ws"]) != 0:
        return "DEVICE STATUS NOT OK"
    return "ok" if not bad else f"FAULTS PASSED: {sorted(set(bad))}"


def roofline_of(durs_s, launch_bytes, workload, note):
    peak, peak_kind = measured_peak()
    mean = statistics.mean(durs_s)
    achieved = launch_bytes / mean / 1e9
    return {"bound": "hbm", "kernel": "verify_kernel", "achieved": round(achieved, 1),
            "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
            "frac": round(achieved / peak, 4),
            "frac_of_nominal_8TBps": round(achieved / NOMINAL_HBM_GBS, 4),
            "algorithmic_bytes_per_launch": launch_bytes,
            "avg_launch_ms": round(mean * 1e3, 4),
            "median_launch_ms": round(statistics.median(durs_s) * 1e3, 4),
            "best_launch_ms": round(min(durs_s) * 1e3, 4),
            "launches_timed": len(durs_s),
            "note": note,
            "traffic": recorded_traffic(workload, launch_bytes)}


def time_workload_alone(name: str, rank: int, launches: int = 20):
    """c1..c4 beside the headline: every distribution of the workload is built, its verify
    call timed `launches` times with CUDA events (3 warm-up calls), and freed again before
    the next one is built, so that at most one case (<= 18 GB) is resident."""
    import torch

    from paper_2509_14279_b200 import population as pop

    W = pop.WORKLOADS[name]
    durs, nbytes, checks = [], [], []
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if name == "c1" else None
    for (d, s) in case_list(W)[0]:
        c = build_case(W, d, s, rank)
        prepare_case(c)
        for _ in range(3):
            step_case(c)
        ev = []
        for _ in range(launches):
            if flush is not None:
                flush.zero_()                     # a 9 MB case would otherwise sit in L2
            step_case(c, ev)
        torch.cuda.synchronize()
        durs += [e0.elapsed_time(e1) * 1e-3 for (e0, e1, _) in ev]
        nbytes.append(c["algo_bytes"])
        checks.append(verdict_check(c))
        del c, ev
        torch.cuda.empty_cache()
    r = roofline_of(durs, statistics.mean(nbytes), name,
                    "events bracket rkv_verify_multi: table upload + workspace clear + verify_kernel (+ copy_check_kernel with a regenerated input) + finalize_case_kernel")
    return {"workload": f"{W.name}: K={W.K}, shapes {list(W.shapes)}, cand {W.cand_dtype}, "
                        f"{len(W.dists)} distributions",
            "ms_per_call": r["avg_launch_ms"], "median_ms": r["median_launch_ms"], "best_ms": r["best_launch_ms"],
            "launches_timed": r["launches_timed"], "GBps": r["achieved"], "frac": r["frac"],
            "frac_of_nominal_8TBps": r["frac_of_nominal_8TBps"], "bytes_per_call": r["algorithmic_bytes_per_launch"],
            "traffic": r["traffic"], "l2": "flushed between calls" if flush is not None else "inputs larger than L2",
            "verdict_check": "ok" if all(x == "ok" for x in checks) else str(checks)}


def time_generator(with_oracle: bool):
    """rkv_gen_inputs on 2^24 fp32 elements per distribution: elements/s, bytes written per
    second against the copy peak (the kernel is ALU-bound, not write-bound); beside it the
    oracle's generator on one thread and on all host cores."""
    import torch

    from paper_2509_14279_b200 import binding as rkv
    from paper_2509_14279_b200 import population as pop

    n = 1 << 24
    peak, peak_kind = measured_peak()
    inst = generator_inst_per_elem()
    props = torch.cuda.get_device_properties(0)
    # one warp instruction per scheduler and clock: SMs x 4 schedulers x 32 lanes x the SM clock
    alu_peak = props.multi_processor_count * 4 * 32 * sm_max_mhz(0) * 1e6
    out = torch.empty(n, dtype=torch.float32, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    res = {}
    for name, d in pop.DIST_IDS.items():
        for _ in range(3):
            rkv.gen_inputs_ex(7, 0, d, n, out=out)
        ev = []
        for _ in range(20):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            rkv.gen_inputs_ex(7, 0, d, n, out=out)
            e1.record()
            ev.append((e0, e1))
        torch.cuda.synchronize()
        durs = [a.elapsed_time(b) * 1e-3 for a, b in ev]
        mean = statistics.mean(durs)
        res[name] = {"gpu_elems_per_s": round(n / mean, 1), "us_per_launch": round(mean * 1e6, 2),
                     "best_us": round(min(durs) * 1e6, 2), "written_GBps": round(n * 4 / mean / 1e9, 1),
                     "frac": round(n * 4 / mean / 1e9 / peak, 4)}
        if inst and name in inst:
            res[name]["lane_inst_per_elem"] = inst[name]
            res[name]["alu_frac"] = round(n / mean * inst[name] / alu_peak, 4)
    out_d = {"kernel": "gen_kernel", "bound": "alu", "elements": n, "dtype": "f32", "peak": peak,
             "peak_kind": f"of {peak_kind}", "alu_peak_lane_inst_per_s": alu_peak, "per_distribution": res,
             "note": "frac = bytes written / event time / copy peak; the kernel is bound by its arithmetic "
                     "(Philox rounds, polynomial log/sincos, IEEE divide and square root), not by the stores; "
                     "alu_frac = elements/s x lane-instructions per element (ncu count, profiles/gen_kernel_f32.md) "
                     "/ (SMs x 4 schedulers x 32 lanes x max SM clock)"}
    if with_oracle:
        import oracle
        n_o = 1 << 21
        cores = os.cpu_count() or 1
        for name, d in pop.DIST_IDS.items():
            t = time.perf_counter()
            oracle.gen(7, 0, d, n_o)
            t1 = time.perf_counter() - t
            t = time.perf_counter()
            _oracle_gen_parallel(7, 0, d, n_o * min(cores, 16), oracle.F32, min(cores, 16))
            ta = time.perf_counter() - t
            res[name]["oracle_elems_per_s_1_thread"] = round(n_o / t1, 1)
            res[name]["oracle_elems_per_s_all_cores"] = round(n_o * min(cores, 16) / ta, 1)
        out_d["oracle_threads"] = min(cores, 16)
    return out_d


def run_native(args):
    import torch
    import torch.distributed as dist

    from paper_2509_14279_b200 import binding as rkv
    from paper_2509_14279_b200 import shard

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    rkv.lib()                                     # fail loudly if the CUDA library is missing

    def barrier():
        if world > 1:
            dist.barrier()

    # the other workloads first, one case resident at a time
    per_workload = []
    if rank == 0 and world == 1 and not args.no_per_workload and not args.cands and not args.max_dists:
        for name in ("c1", "c2", "c3", "c4", "c5"):
            if name != args.workload:
                per_workload.append(time_workload_alone(name, rank))
    generator = None
    if rank == 0 and world == 1 and not args.no_generator and not args.cands:
        generator = time_generator(with_oracle=not args.no_cpu_baseline)
    torch.cuda.empty_cache()

    from paper_2509_14279_b200 import population as pop
    W0 = pop.WORKLOADS[args.workload]
    n_sets = args.sets
    if n_sets == 0:
        case_bytes = sum(W0.K * n * (2 if (W0.cand_dtype == "bf16" or (W0.cand_dtype == "mixed" and t == 1)) else 4)
                         for t, n in enumerate(W0.numels)) * len(W0.dists)
        free, _ = torch.cuda.mem_get_info()
        n_sets = 2 if (len(W0.seeds) > 1 and 2 * case_bytes + (24 << 30) < free) else 1
    W, sets = build_workload(args.workload, rank, args.max_dists, args.cands, n_sets)
    for cases in sets:
        for c in cases:
            prepare_case(c)
    torch.cuda.synchronize()

    def one_step(i, events=None):
        for c in sets[i % len(sets)]:
            step_case(c, events)

    warmup = max(args.warmup, 3)
    for i in range(warmup):
        one_step(i)
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
    for i in range(args.steps):
        one_step(warmup + i, events)
    t1.record()
    torch.cuda.synchronize()
    barrier()
    elapsed_ms = t0.elapsed_time(t1)
    clocks = sampler.stop() if rank == 0 else None
    elapsed_ms = shard.max_over_ranks(elapsed_ms, device="cuda")

    total_bytes = sum(b for (_, _, b) in events)
    step_bytes = total_bytes / args.steps
    value = world * total_bytes / (elapsed_ms * 1e-3) / 1e9

    # roofline of the dominant kernel: verify calls timed one by one inside the timed region
    durs = [e0.elapsed_time(e1) * 1e-3 for (e0, e1, _) in events]
    launch_bytes = statistics.mean(b for (_, _, b) in events)
    roofline = roofline_of(durs, launch_bytes, args.workload,
                           "events bracket rkv_verify_multi: table upload + workspace clear + verify_kernel "
                           "(one launch over every tensor and storage type) + copy_check_kernel (regenerated input) + finalize_case_kernel")

    checks = [verdict_check(c) for cases in sets for c in cases]
    pairs = [[f"{c['dist']}/seed {c['seed']}" for c in cases] for cases in sets]
    out = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": round(elapsed_ms / args.steps, 4),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": DTYPE_NOTE[W.cand_dtype], "data": "synthetic",
        "config": {"workload": f"{W.name}: K={W.K} candidates per tensor, shapes {list(W.shapes)}, "
                               f"cand {W.cand_dtype}, {len(sets[0])} distributions per step"
                               f"{', fused regeneration of reference and input' if W.fused else ''}",
                   "distribution_seed_pairs_per_set": pairs,
                   "sets": f"{len(sets)} resident set(s); step i runs set i mod {len(sets)}",
                   "bytes_per_step": step_bytes,
                   "bytes_counted": "candidate bytes only (reference and input are regenerated, not read)"
                                    if W.fused else "candidate + reference bytes",
                   "l2": "inputs larger than L2 (each call streams > 4 GB)",
                   "parallelism": f"replicas x{world}" if world > 1 else "single gpu"},
        "gpu_launches": sum(c["launches"] for i in range(args.steps) for c in sets[(warmup + i) % len(sets)]),
        "roofline": roofline, "clocks": clocks,
        "verdict_check": "ok" if all(x == "ok" for x in checks) else str(checks),
    }
    if per_workload:
        out["per_workload"] = per_workload
    if generator:
        out["generator"] = generator
    if rank == 0:
        if not args.no_e2e:
            out["e2e"] = run_e2e(args, W, sets[0][0], world)
        if not args.no_cpu_baseline and world == 1:
            out["cpu_baseline"] = cpu_baseline_sample(W)
        print(json.dumps(out), flush=True)
    elif not args.no_e2e:
        run_e2e(args, W, sets[0][0], world)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_e2e(args, W, case, world):
    """Same metric through rkv_verify_multi_host: pinned HOST buffers in, HOST results out,
    every copy inside the timed region.  One distribution per step."""
    import torch
    import torch.distributed as dist

    from paper_2509_14279_b200 import binding as rkv
    from paper_2509_14279_b200 import shard

    host_descs, h2d = [], 0
    for d in case["descs"]:
        cands_h = [c.cpu().pin_memory() for c in d.cands]
        ref_h = None if d.ref is None else d.ref.reshape(-1).cpu().pin_memory()
        inp_h = None if d.input is None else d.input.reshape(-1).cpu().pin_memory()
        host_descs.append(rkv.TensorDesc(n=d.n, cands=cands_h, atol=d.atol, rtol=d.rtol, ref=ref_h, input=inp_h,
                                         ref_gen=d.ref_gen, input_gen=d.input_gen, ref_dtype=d.ref_dtype))
        h2d += sum(c.numel() * c.element_size() for c in cands_h)
        h2d += 0 if ref_h is None else ref_h.numel() * ref_h.element_size()
        h2d += 0 if inp_h is None else inp_h.numel() * inp_h.element_size()
    K, T = case["K"], len(host_descs)
    d2h = K * T * rkv.STATS_BYTES + K * 4
    steps = max(2, min(args.steps, 4))
    for _ in range(2):
        got, joint = rkv.verify_multi_host(host_descs, K)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(steps):
        got, joint = rkv.verify_multi_host(host_descs, K)
    torch.cuda.synchronize()
    el = time.perf_counter() - t0
    el = shard.max_over_ranks(el, device="cuda")
    same = bool((joint == case["joint"].cpu().numpy()).all())
    return {"value": round(world * h2d * steps / el / 1e9, 2), "unit": UNIT,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": steps,
            "verdicts_match_device_run": same,
            "sample": f"one distribution ({case['dist']}, seed {case['seed']}) per step, every tensor and "
                      "candidate of it, pinned host buffers, through rkv_verify_multi_host"}


# ----------------------------------------------------------------------------
# CPU oracle timing (reported baseline / reference arm)
# ----------------------------------------------------------------------------

def _oracle_gen_parallel(seed, stream_id, dist_id, n, dtype, threads):
    """The oracle's generator over `threads` chunks (it is a pure function of the index)."""
    from concurrent.futures import ThreadPoolExecutor

    import numpy as np

    import oracle
    chunk = (-(-n // threads) + 3) // 4 * 4
    spans = [(s, min(chunk, n - s)) for s in range(0, n, chunk)]
    with ThreadPoolExecutor(max_workers=threads) as ex:
        parts = list(ex.map(lambda sp: oracle.gen(seed, stream_id, dist_id, sp[1], dtype=dtype, first_elem=sp[0]),
                            spans))
    return np.concatenate(parts)


def _oracle_sample(W, dist_id, n_s, k_s, threads, seed):
    """One bounded sample of workload W on the oracle: generate the reference and the input
    tensors of n_s elements, then verify k_s candidates per tensor.  Returns
    (seconds generating, seconds verifying, bytes verified)."""
    from concurrent.futures import ThreadPoolExecutor

    import torch

    import oracle
    from paper_2509_14279_b200 import population as pop

    t_gen, t_ver, nbytes = 0.0, 0.0, 0
    kinds = ["f32", "bf16"] if W.cand_dtype == "mixed" else [W.cand_dtype]
    for t, cdt in enumerate(kinds):
        bf16 = cdt == "bf16"
        t0 = time.perf_counter()
        ref = _oracle_gen_parallel(seed, 0, dist_id, n_s, oracle.F32, threads)
        inp = _oracle_gen_parallel(seed, 2, dist_id, n_s, oracle.BF16 if bf16 else oracle.F32, threads)
        t_gen += time.perf_counter() - t0
        plan = pop.plan_mixed(k_s, n_s, seed + t, W.fault_rate, bf16=bf16)
        tr, ti = torch.from_numpy(ref), pop.from_bits(inp)
        cands = [pop.bits_numpy(pop.materialize(c, tr, ti, cdt)) for c in plan]
        atol, rtol = W.tols[t] if len(W.tols) > 1 else W.tols[0]
        t0 = time.perf_counter()
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(lambda c: oracle.verify(ref, c, atol, rtol, input=inp), cands))
        t_ver += time.perf_counter() - t0
        nbytes += k_s * n_s * (2 if bf16 else 4) + (0 if W.fused else n_s * 4)
    return t_gen, t_ver, nbytes


def cpu_baseline_sample(W, budget_s: float = 8.0):
    """The oracle as it stands on the host cores, on a bounded sample of the workload: the
    first distribution, a 4 Mi-element slice of each tensor, 16 candidates per tensor;
    first on one thread, then on all cores (at most 16 threads), each until about
    `budget_s` seconds of oracle time have been spent."""
    import platform

    import oracle
    from paper_2509_14279_b200 import population as pop

    oracle.lib()
    cores = os.cpu_count() or 1
    threads = min(cores, 16)
    n_s = min(W.numels[0], 1 << 22)
    k_s = 16
    model = platform.processor() or ""
    try:
        with open("/proc/cpuinfo") as fh:
            for line in fh:
                if line.startswith("model name"):
                    model = line.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    res = {}
    for label, th in (("one_thread", 1), ("all_cores", threads)):
        g = v = 0.0
        b = reps = 0
        while g + v < budget_s and reps < 200:
            tg, tv, nb = _oracle_sample(W, pop.DIST_IDS[W.dists[0]], n_s, k_s, th, W.seeds[0] + reps)
            g, v, b, reps = g + tg, v + tv, b + nb, reps + 1
        res[label] = {"threads": th, "GBps": round(b / (g + v) / 1e9, 4), "verify_only_GBps": round(b / v / 1e9, 4),
                      "seconds": round(g + v, 2), "reps": reps}
    return {"value": res["all_cores"]["GBps"], "unit": UNIT, "cores": threads, "kind": "oracle",
            "one_thread": res["one_thread"], "all_cores": res["all_cores"],
            "cpu_model": model, "host_cores_available": cores,
            "sample": f"{W.dists[0]}: per repetition, generate reference+input of {n_s} elements and verify "
                      f"{k_s} candidates of {n_s} elements per tensor ({'f32 and bf16' if W.cand_dtype == 'mixed' else W.cand_dtype}); "
                      f"GBps counts the same bytes as the GPU metric over generation + verification time"}


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
        _oracle_sample(W, dists[i % len(dists)], n_s, k_s, threads, W.seeds[0])
    total_s, total_b = 0.0, 0
    for i in range(args.steps):
        tg, tv, b = _oracle_sample(W, dists[i % len(dists)], n_s, k_s, threads, W.seeds[i % len(W.seeds)])
        total_s += tg + tv
        total_b += b
    value = total_b / total_s / 1e9
    sample = (f"per step: one distribution (rotating) and one seed (rotating), generate reference+input of {n_s} "
              f"elements and verify {k_s} candidates per tensor, {threads} threads")
    out = {
        "impl": "reference", "metric": METRIC, "value": round(value, 4), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 1), "ms_per_step": round(total_s / args.steps * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": DTYPE_NOTE[W.cand_dtype],
        "data": "synthetic",
        "config": {"workload": f"{W.name}: K={W.K} candidates per tensor, shapes {list(W.shapes)}, cand {W.cand_dtype} "
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
    relaunch_if_needed(args)
    if args.workload in ("s1", "x1", "w1"):
        if args.impl == "reference" or int(os.environ.get("WORLD_SIZE", "1")) > 1:
            if int(os.environ.get("RANK", "0")) == 0:
                print(json.dumps({"impl": args.impl,
                                  "unavailable": f"workload {args.workload} runs on one GPU, native arm only"}))
            return
        if args.workload == "s1":
            run_screen(args)
        else:
            import bench_extra
            (bench_extra.run_cross if args.workload == "x1" else bench_extra.run_sweep)(args, measured_peak, ClockSampler)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_native(args)


if __name__ == "__main__":
    main()
