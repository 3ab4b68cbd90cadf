#!/usr/bin/env python
"""Benchmark of the Draco encode -> corrupt -> locate -> decode path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One step = one pass of the whole path over one batch of synthetic gradients resident in HBM:
encode all n workers' vectors, apply the adversaries, locate them, decode the sum.  The default
workload is the ResNet-152-sized cyclic-code configuration (n = 45, s = 5, d = 60.2 M).  With
N > 1 (torchrun, one rank per GPU) every rank holds its own d-slice of that size (weak scaling);
the only exchange is one all-reduce of the n complex projections inside the locator.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample.
Besides the contract keys the line carries `stages` (per-stage CUDA-event times), `clocks` (nvidia-smi
sampled every 20 ms during the timed steps) and `graph_replay` (the same step captured once into a CUDA
graph and replayed: what the launch overhead costs on small workloads).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import draco_inputs as di  # noqa: E402

METRIC = "coded_gradient_throughput"
UNIT = "GB/s"

WORKLOADS = {
    # name: (code, n, s, d, gradient std, adversary models, params)
    "cyc_n45_s5_d60.2M": ("cyc", 45, 5, 60_200_000, 1.0, ["revgrad"], [100.0]),
    "rep_n45_s3_d11.7M": ("rep", 45, 3, 11_700_000, 0.1, ["revgrad", "const"], [100.0, 1e4]),
    "cycp_n45_s5_d60.2M": ("cycp", 45, 5, 60_200_000, 1.0, ["revgrad"], [100.0]),   # packed transport: 30.1 M complex entries
    "cyc_n15_s2_d1M": ("cyc", 15, 2, 1_000_000, 1.0, ["gauss"], [1e3]),
    "rep_n15_s2_d100k": ("rep", 15, 2, 100_000, 1.0, ["revgrad"], [100.0]),
}
DEFAULT_WORKLOAD = "cyc_n45_s5_d60.2M"
MODEL_ID = {"revgrad": di.ADV_REVGRAD, "const": di.ADV_CONST, "gauss": di.ADV_GAUSS}
SEED = 0xD2AC0


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "MEASURED_PEAKS.json hbm_gbs (of measured)"
    except Exception:
        return 6650.0, "fallback 6.65 TB/s (of fallback)"


def adversaries(workload, rank=0):
    code, n, s, d, std, models, params = WORKLOADS[workload]
    adv = di.choose_adversaries(SEED + 1 + 1000 * 0, n, s)          # same nodes on every rank
    model = [MODEL_ID[models[k % len(models)]] for k in range(s)]
    param = [params[k % len(params)] for k in range(s)]
    return adv, model, param


def algorithmic_bytes(code, n, s, d, n_adv):
    """Bytes each stage must move (per step, one GPU)."""
    if code == "cycp":
        h = (d + 1) // 2
        return {"encode": 4 * n * d + 8 * n * h, "locate": 8 * n * h + 4 * h, "decode": 8 * (n - n_adv) * h + 4 * d,
                "corrupt": 2 * 8 * n_adv * h, "coded": 8 * n * h}
    if code == "cyc":
        return {"encode": 4 * n * d + 8 * n * d, "locate": 8 * n * d + 4 * d, "decode": 8 * (n - n_adv) * d + 4 * d,
                "corrupt": 2 * 8 * n_adv * d, "coded": 8 * n * d}
    return {"encode": 4 * n * d + 4 * n * d, "locate": 0, "decode": 4 * n * d + 4 * d, "corrupt": 2 * 4 * n_adv * d,
            "coded": 4 * n * d}


# --------------------------------------------------------------------------- CPU oracle arm
def oracle_step(workload, d_sample, seed):
    """The oracle, as it stands, on the first d_sample coordinates of the workload."""
    from oracle import draco_oracle as orc
    code, n, s, d, std, models, params = WORKLOADS[workload]
    adv, model, param = adversaries(workload)
    G = di.gradient_rows(seed, n, d, 0.0, std, i0=0, i1=d_sample)
    f = di.projection_vector(seed + 3, d, i0=0, i1=d_sample)
    t0 = time.perf_counter()
    if code == "cycp":         # the sample's own two halves are packed together
        R = orc.cyc_encode_packed(G, n, s)
        di.apply_adversaries(R, adv, model, param, seed=seed + 2)
        out = orc.cyc_locate(R, f[: R.shape[1]], n, s)
        orc.cyc_decode_packed(R, n, s, out["flags"], d_sample)
        ok = sorted(np.flatnonzero(out["flags"])) == adv.tolist()
    elif code == "cyc":
        R = orc.cyc_encode(G, n, s)
        di.apply_adversaries(R, adv, model, param, seed=seed + 2)
        out = orc.cyc_decode_full(R, f, n, s)
        ok = sorted(np.flatnonzero(out["flags"])) == adv.tolist()
    else:
        R = orc.rep_encode(G, n, s)
        di.apply_adversaries(R, adv, model, param, seed=seed + 2)
        out = orc.rep_decode(R, n, s)
        ok = sorted(np.flatnonzero(out["flags"])) == adv.tolist()
    dt = time.perf_counter() - t0
    return dt, ok


def oracle_threads():
    """Threads the oracle's numerical libraries (numpy's BLAS) may use right now."""
    try:
        from threadpoolctl import threadpool_info
        infos = threadpool_info()
        return max([i.get("num_threads", 1) for i in infos] + [1])
    except Exception:
        return 1


def cpu_baseline(workload, target_seconds=8.0):
    """The oracle as it stands on a bounded sample of the workload, once with every host core its libraries take
    and once limited to one thread (the two figures the measurement plan names), core count stated."""
    code, n, s, d, std, models, params = WORKLOADS[workload]
    probe = min(d, 200_000)
    oracle_step(workload, probe, SEED)                                   # builds and caches the code tables
    dt, _ = oracle_step(workload, probe, SEED)
    d_sample = int(min(d, max(probe, probe * target_seconds / max(dt, 1e-3))))
    dt_all, ok = oracle_step(workload, d_sample, SEED)
    cores = oracle_threads()
    dt_one = None
    try:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=1):
            dt_one, ok1 = oracle_step(workload, d_sample, SEED)
        ok = ok and ok1
    except Exception:
        pass
    per = 8 if code == "cyc" else 4                      # coded bytes per gradient coordinate (packed: 8 per 2)
    out = {"value": per * n * d_sample / dt_all / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
           "host_cores": os.cpu_count(),
           "sample": f"first {d_sample} of {d} coordinates, all {n} workers, one pass in {dt_all:.2f} s with {cores} threads"
                     + (f" and {dt_one:.2f} s with 1 thread" if dt_one else "")
                     + f" (numpy fp64/complex128; flags correct: {ok})"}
    if dt_one:
        out["value_1_thread"] = per * n * d_sample / dt_one / 1e9
    return out


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    workload = args.workload
    code, n, s, d, std, models, params = WORKLOADS[workload]
    probe = min(d, 50_000)
    oracle_step(workload, probe, SEED)                                   # builds and caches the code tables
    dt, _ = oracle_step(workload, probe, SEED)
    budget = 150.0 / max(1, args.steps + args.warmup)                  # seconds per step
    d_sample = int(min(d, max(10_000, probe * min(budget, 3.0) / max(dt, 1e-3))))
    for _ in range(args.warmup):
        oracle_step(workload, d_sample, SEED)
    times = []
    for _ in range(args.steps):
        dt, ok = oracle_step(workload, d_sample, SEED)
        times.append(dt)
    per = 8 if code == "cyc" else 4
    mean = sum(times) / len(times)
    value = per * n * d_sample / mean / 1e9
    sample = f"first {d_sample} of {d} coordinates per step, all {n} workers (numpy fp64/complex128 oracle)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": mean * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload, "code": code, "n": n, "s": s, "d": d, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# --------------------------------------------------------------------------- GPU arm
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.path = tempfile.mktemp(prefix="draco_clocks_", suffix=".csv")
        self.proc = None
        try:
            self.fh = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"], stdout=self.fh,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_min_mhz": None, "sm_max_mhz": None, "power_w_max": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.fh.close()
        sm, mx, pw, reasons = [], [], [], set()
        try:
            for ln in open(self.path):
                p = [x.strip() for x in ln.split(",")]
                if len(p) < 9:
                    continue
                try:
                    sm.append(float(p[1]))
                    mx.append(float(p[2]))
                except ValueError:
                    continue
                try:
                    pw.append(float(p[3]))
                except ValueError:
                    pass
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_min_mhz=min(sm), sm_max_mhz=max(mx), samples=len(sm))
        if pw:
            out["power_w_max"] = max(pw)
        out["reasons"] = sorted(reasons)
        return out


def stage_launches(code, n, n_adv):
    """Kernels launched per step: encode 1; corrupt 1 (all adversaries in one launch); cyclic locate = projection
    (two launches over half the rows each when n > 64) + reduction of the block partials fused with the solve;
    decode = decode vector + recovery (repetition: vote + finish, no separate locate)."""
    cyc = code in ("cyc", "cycp")
    return {"encode": 1, "corrupt": 1 if n_adv else 0, "locate": ((2 if n > 64 else 1) + LOCATE_TAIL_LAUNCHES) if cyc else 0,
            "decode": 2}


LOCATE_TAIL_LAUNCHES = 2     # cyc_reduce_partials_kernel, cyc_solve_kernel


def measure_workload(args, workload, world, rank, with_graph, with_e2e):
    """Times `args.steps` steps of one workload on this rank's GPU (inputs resident in HBM) and, optionally, the
    CUDA-graph replay and the host-buffer pipeline.  Returns the pieces of the JSON line."""
    import torch
    import torch.distributed as dist

    import paper_1803_09877_b200 as dr
    from paper_1803_09877_b200.sharding import locate_sharded, merge_flags

    code, n, s, d, std, models, params = WORKLOADS[workload]
    cyc = code in ("cyc", "cycp")
    packed = code == "cycp"
    vlen = (d + 1) // 2 if packed else d                 # entries per worker vector
    adv, model, param = adversaries(workload)
    plan = dr.Plan(n, s, d, dr.CYC_PACKED if packed else dr.CYC if cyc else dr.REP)
    stream = torch.cuda.current_stream()
    steps, warmup = args.steps, max(args.warmup, 3)

    # inputs resident in HBM; rank r holds coordinates [r d, (r+1) d) of a d * world vector
    G = torch.empty((n, d), dtype=torch.float32, device="cuda")
    dr.generate(G, n, d, mean=0.0, std=std, seed=SEED + 17 * rank)
    f = None
    if cyc:
        f = torch.empty(vlen, dtype=torch.float32, device="cuda")
        dr.generate(f, 1, vlen, mean=1.0, std=1.0, seed=SEED + 3 + 17 * rank)
    Z = torch.empty((n, (2 if cyc else 1) * vlen), dtype=torch.float32, device="cuda")
    u = torch.empty(d, dtype=torch.float32, device="cuda")
    flags = torch.empty(n, dtype=torch.uint8, device="cuda")
    e = torch.empty(3 * n, dtype=torch.float64, device="cuda")        # projection record: n (re, im) pairs + n squared norms

    names = ["encode", "corrupt", "locate", "decode"]

    def step(ev=None):
        def mark(i):
            if ev is not None:
                ev[i].record(stream)
        mark(0)
        plan.encode(G, Z)
        mark(1)
        plan.corrupt(Z, adv, model, param, seed=SEED + 2)
        mark(2)
        if cyc:
            if world > 1:      # d-sharded: local projection, all-reduce of the 3 n doubles, local solve
                locate_sharded(plan, Z, f, flags, e)
            else:
                plan.locate(Z, f, flags)
            mark(3)
            plan.decode(Z, flags, u)
        else:
            mark(3)
            plan.locate_decode(Z, None, flags, u)
            if world > 1:      # a node is flagged if any shard saw it disagree
                merge_flags(flags)
        mark(4)

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warmup):
        step()
    sync_all()
    got = sorted(np.flatnonzero(flags.cpu().numpy()).tolist())
    if got != adv.tolist():
        raise SystemExit(f"{workload}: flags {got} differ from the planted adversaries {adv.tolist()}")

    events = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(steps)]
    sampler = ClockSampler(torch.cuda.current_device()) if rank == 0 else None
    time.sleep(0.3)
    sync_all()
    t_start = torch.cuda.Event(enable_timing=True)
    t_stop = torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for k in range(steps):
        step(events[k])
    t_stop.record(stream)
    sync_all()
    clocks = sampler.stop() if sampler else None
    total_ms = t_start.elapsed_time(t_stop)
    if world > 1:
        t = torch.tensor([total_ms], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    ms_per_step = total_ms / steps
    per_step = {nm: [events[k][i].elapsed_time(events[k][i + 1]) for k in range(steps)] for i, nm in enumerate(names)}
    stage_ms = {nm: statistics.mean(v) for nm, v in per_step.items()}
    stage_min = {nm: min(v) for nm, v in per_step.items()}
    stage_med = {nm: statistics.median(v) for nm, v in per_step.items()}

    ab = algorithmic_bytes(code, n, s, d, len(adv))
    value = ab["coded"] * world / (ms_per_step * 1e-3) / 1e9
    peak, peak_src = measured_peak_gbs()
    if cyc:
        dom, dom_kernel = "encode", f"cyc_encode_stream_kernel<S={s}, packed={str(packed).lower()}>"
    else:
        dom, dom_kernel = "decode", "rep_vote_kernel"
    achieved = ab[dom] / (stage_ms[dom] * 1e-3) / 1e9
    # DRAM bytes per gradient coordinate of the dominant kernel, from the ncu captures summarised under profiles/
    # (dram__bytes_read.sum + dram__bytes_write.sum at d = 4 M / 8 M; every byte is touched once, so traffic scales with d).
    # Valid for n = 45 with the configured s only; null for any other shape, and null for a kernel that has changed
    # since its counters were taken.
    traffic_per_coord = DOMINANT_TRAFFIC_PER_COORD.get((code, n, s))
    traffic = traffic_per_coord * d if traffic_per_coord else None
    stages = {}
    for nm in names:
        if stage_ms[nm] > 0 and ab.get(nm, 0) > 0:
            g = ab[nm] / (stage_ms[nm] * 1e-3) / 1e9
            stages[nm] = {"ms": round(stage_ms[nm], 4), "ms_median": round(stage_med[nm], 4), "ms_min": round(stage_min[nm], 4),
                          "algorithmic_GB": round(ab[nm] / 1e9, 4), "GB/s": round(g, 1), "frac_of_peak": round(g / peak, 4),
                          "frac_of_nominal_8TBps": round(g / 8000.0, 4)}
        else:
            stages[nm] = {"ms": round(stage_ms[nm], 4)}
    launches = sum(stage_launches(code, n, len(adv)).values()) * steps
    roofline = {"bound": "hbm", "kernel": dom_kernel, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": traffic, "peak_source": peak_src,
                "nominal_peak": 8000.0, "frac_of_nominal": achieved / 8000.0,
                "algorithmic_bytes_per_launch": ab[dom], "avg_launch_ms": stage_ms[dom]}
    config = {"workload": workload, "code": code, "n": n, "s": s, "d_per_gpu": d, "adversaries": len(adv),
              "adversary_models": models, "l2": "inputs larger than L2 (no flush needed)"
              if ab["coded"] > 4e8 else "working set near L2 size: not an HBM number",
              "value_is": "bytes of coded gradients (n d complex64 / fp32) per step / step time"}

    # the same step captured once into a CUDA graph and replayed (one GPU only: the sharded step has a collective)
    graph_replay = None
    if with_graph and world == 1:
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        cg = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(cg, stream=side):
                step()
        stream.wait_stream(side)
        for _ in range(3):
            cg.replay()
        sync_all()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(stream)
        for _ in range(steps):
            cg.replay()
        g1.record(stream)
        sync_all()
        got = sorted(np.flatnonzero(flags.cpu().numpy()).tolist())
        if got != adv.tolist():
            raise SystemExit(f"graph replay: flags {got} differ from the planted adversaries {adv.tolist()}")
        gms = g0.elapsed_time(g1) / steps
        graph_replay = {"ms_per_step": gms, "value": ab["coded"] / (gms * 1e-3) / 1e9, "unit": UNIT,
                        "stream_launch_ms_per_step": ms_per_step}
        del cg

    # end to end through the host-buffer entry point (rank-local; H2D of G and f, D2H of u and flags)
    e2e = None
    if with_e2e:
        del events
        Gh = torch.empty((n, d), dtype=torch.float32, pin_memory=True)
        Gh.copy_(G)
        fh = torch.empty(vlen, dtype=torch.float32, pin_memory=True)
        if cyc:
            fh.copy_(f)
        uh = torch.empty(d, dtype=torch.float32, pin_memory=True)
        flh = torch.empty(n, dtype=torch.uint8, pin_memory=True)
        torch.cuda.synchronize()
        reps = max(2, min(steps, 5))
        plan.pipeline_host(Gh, fh if cyc else None, adv, model, param, SEED + 2, Z, uh, flh)   # warm-up, allocs
        sync_all()
        t0 = time.perf_counter()
        for _ in range(reps):
            plan.pipeline_host(Gh, fh if cyc else None, adv, model, param, SEED + 2, Z, uh, flh)
        sync_all()
        dt = (time.perf_counter() - t0) / reps
        if world > 1:
            t = torch.tensor([dt], dtype=torch.float64, device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            dt = float(t.item())
        if sorted(np.flatnonzero(flh.numpy()).tolist()) != adv.tolist():
            raise SystemExit("host pipeline: flags differ from the planted adversaries")
        e2e = {"value": ab["coded"] * world / dt / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": 4 * n * d + (4 * vlen if cyc else 0), "d2h_bytes_per_step": 4 * d + n,
               "ms_per_step": dt * 1e3, "steps": reps}
        del Gh, fh, uh, flh
    out = {"value": value, "ms_per_step": ms_per_step, "config": config, "roofline": roofline, "stages": stages,
           "clocks": clocks, "e2e": e2e, "graph_replay": graph_replay, "gpu_launches": launches,
           "dtype": "f32 (complex64 vectors; f64 centre taps, projection sums and recovery)" if cyc
           else "f32 (u32 bit patterns in the vote)"}
    plan.close()
    del G, Z, u, f, flags, e
    torch.cuda.empty_cache()
    return out


# ncu dram__bytes_read.sum + dram__bytes_write.sum per gradient coordinate of the dominant kernel (profiles/)
DOMINANT_TRAFFIC_PER_COORD = {("cyc", 45, 5): 525.1, ("cycp", 45, 5): 353.9, ("rep", 45, 3): 183.0}
SECONDARY_WORKLOADS = ["rep_n45_s3_d11.7M", "cycp_n45_s5_d60.2M"]


def launch_plan(args, argv):
    """How `bench.py --gpus N` starts its N ranks when it was not itself started by torchrun: the command and the
    extra environment of one torchrun process group on this node (rendezvous on 127.0.0.1)."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--standalone", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--local-addr", "127.0.0.1", os.path.abspath(__file__)] + [a for a in argv if a != "--dry-run"]
    env = {"MASTER_ADDR": "127.0.0.1", "OMP_NUM_THREADS": "1"}
    return cmd, env


def run_gpu(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    ranks = None
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        try:
            uuid = str(torch.cuda.get_device_properties(local).uuid)
        except Exception:                       # older runtimes have no uuid field: fall back to the device ordinal
            uuid = f"ordinal-{local}"
        mine = {"rank": rank, "device": local, "uuid": uuid}
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        ranks = gathered
        if len({g["uuid"] for g in gathered}) != world:
            raise SystemExit(f"ranks share a GPU: {gathered}")
    main = measure_workload(args, args.workload, world, rank, with_graph=not args.no_graph, with_e2e=not args.no_e2e)
    secondary = None
    if world == 1 and not args.no_secondary and args.workload == DEFAULT_WORKLOAD:
        secondary = {}
        for wl in SECONDARY_WORKLOADS:
            r = measure_workload(args, wl, world, rank, with_graph=False, with_e2e=False)
            secondary[wl] = {"value": r["value"], "unit": UNIT, "ms_per_step": r["ms_per_step"], "stages": r["stages"],
                             "roofline": r["roofline"], "gpu_launches": r["gpu_launches"], "clocks": r["clocks"],
                             "config": r["config"]}
    if rank == 0:
        cb = cpu_baseline(args.workload) if (world == 1 and not args.no_cpu_baseline) else None
        line = {"metric": METRIC, "value": main["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": main["ms_per_step"], "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": main["dtype"], "data": "synthetic",
                "config": main["config"], "roofline": main["roofline"], "stages": main["stages"], "clocks": main["clocks"],
                "e2e": main["e2e"], "graph_replay": main["graph_replay"], "gpu_launches": main["gpu_launches"],
                "cpu_baseline": cb, "secondary": secondary, "ranks": ranks}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()



# --------------------------------------------------------------------------- sweep over both codes
def run_sweep(args):
    """Both codes over n x s x d: per point the stage times, GB/s of coded gradients consumed / produced,
    achieved HBM GB/s against the roofline, and correctness for 0, s and more than s adversaries
    (the last must fail visibly).  One JSON line per point goes to --sweep-out; one summary line to stdout."""
    import torch

    import paper_1803_09877_b200 as dr

    torch.cuda.set_device(0)
    peak, peak_src = measured_peak_gbs()
    free_bytes = torch.cuda.mem_get_info()[0]
    ns = [int(x) for x in args.sweep_n.split(",")]
    ss = [int(x) for x in args.sweep_s.split(",")]
    ds = [int(float(x)) for x in args.sweep_d.split(",")]
    rng = np.random.default_rng(7)
    out_lines, skipped = [], []

    def timed(fn, reps=3):
        fn()
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
        for i in range(reps):
            ev[i].record()
            fn()
        ev[reps].record()
        torch.cuda.synchronize()
        return statistics.median(ev[i].elapsed_time(ev[i + 1]) for i in range(reps))

    for code in args.sweep_codes.split(","):
        cyc = code == "cyc"
        for n in ns:
            for s in ss:
                if 2 * s + 1 > n:
                    continue
                for d in ds:
                    need = 4 * n * d * (3 if cyc else 2) + 16 * d
                    if need > 0.92 * free_bytes:
                        skipped.append({"code": code, "n": n, "s": s, "d": d, "reason": f"needs {need / 1e9:.0f} GB"})
                        continue
                    seed = SEED + 100 * n + s
                    plan = dr.Plan(n, s, d, dr.CYC if cyc else dr.REP)
                    G = torch.empty((n, d), dtype=torch.float32, device="cuda")
                    dr.generate(G, n, d, seed=seed)
                    f = torch.empty(d, dtype=torch.float32, device="cuda")
                    dr.generate(f, 1, d, mean=1.0, std=1.0, seed=seed + 3)
                    Z = torch.empty((n, (2 if cyc else 1) * d), dtype=torch.float32, device="cuda")
                    u = torch.empty(d, dtype=torch.float32, device="cuda")
                    flags = torch.empty(n, dtype=torch.uint8, device="cuda")
                    idx = np.unique(rng.integers(0, d, 2000))
                    exact = di.gradient_rows(seed, n, d, idx=idx).astype(np.float64).sum(axis=0)
                    scale = max(float(np.abs(exact).max()), 1e-30)
                    groups = plan.groups() if not cyc else []
                    checks = {}
                    for label in ("0", "s", ">s"):
                        if label == "0":
                            adv, model, param = [], [], []
                        elif label == "s":
                            adv = di.choose_adversaries(seed + 1, n, s).tolist()
                            model, param = [di.ADV_REVGRAD] * s, [100.0] * s
                        elif cyc:
                            adv = di.choose_adversaries(seed + 2, n, s + 1).tolist()
                            model, param = [di.ADV_REVGRAD] * (s + 1), [100.0] * (s + 1)
                        else:                      # enough identical colluders to win group 0's vote
                            c = groups[0][1] // 2 + 1
                            adv, model, param = list(range(c)), [di.ADV_CONST] * c, [1e4] * c
                        plan.encode(G, Z)
                        if adv:
                            plan.corrupt(Z, adv, model, param, seed=seed + 4)
                        plan.locate_decode(Z, f if cyc else None, flags, u)
                        info = plan.info()
                        got = sorted(np.flatnonzero(flags.cpu().numpy()).tolist())
                        err = float(np.abs(u[idx].cpu().numpy().astype(np.float64) - exact).max() / scale)
                        checks[label] = {"planted": len(adv), "flags_match": got == sorted(adv), "err": err,
                                         "status": info["status"], "no_majority": info["no_majority"]}
                    adv = di.choose_adversaries(seed + 1, n, s).tolist()
                    reps = 20 if d >= 11_000_000 else 5
                    enc_ms = timed(lambda: plan.encode(G, Z), reps)
                    if adv:
                        plan.corrupt(Z, adv, [di.ADV_REVGRAD] * s, [100.0] * s, seed=seed + 4)
                    dec_ms = timed(lambda: plan.locate_decode(Z, f if cyc else None, flags, u), reps)
                    ab = algorithmic_bytes(code, n, s, d, len(adv))
                    enc_hbm = ab["encode"] / (enc_ms * 1e-3) / 1e9
                    dec_hbm = (ab["locate"] + ab["decode"]) / (dec_ms * 1e-3) / 1e9
                    tol = 1e-5 if not cyc else (1e-4 if n <= 15 else None)
                    ok_s = checks["s"]["flags_match"] and checks["0"]["flags_match"]
                    line = {"code": code, "n": n, "s": s, "d": d, "encode_ms": enc_ms, "decode_ms": dec_ms, "timed_reps": reps,
                            "coded_GBps_produced": ab["coded"] / (enc_ms * 1e-3) / 1e9,
                            "coded_GBps_consumed": ab["coded"] / (dec_ms * 1e-3) / 1e9,
                            "encode_hbm_GBps": enc_hbm, "encode_frac": enc_hbm / peak,
                            "decode_hbm_GBps": dec_hbm, "decode_frac": dec_hbm / peak,
                            "l2_note": "fits in L2: not an HBM number" if ab["coded"] < 2.5e8 else "",
                            "checks": checks, "flags_ok_upto_s": ok_s, "sum_tolerance": tol,
                            "sum_ok_upto_s": None if tol is None else (checks["0"]["err"] <= tol and checks["s"]["err"] <= tol),
                            # beyond s the decoder either reports a failed self-check (status != 0), or is visibly off
                            # (wrong flags, wrong sum), or - adversaries that do not collude - decodes all the same
                            "beyond_s_fails": (not checks[">s"]["flags_match"]) or checks[">s"]["err"] > 1e-3
                            or checks[">s"]["status"] != 0,
                            "beyond_s_silent_error": checks[">s"]["err"] > 1e-3 and checks[">s"]["status"] == 0
                            and (tol is not None)}
                    out_lines.append(line)
                    with open(args.sweep_out, "a") as fh:
                        fh.write(json.dumps(line) + "\n")
                    del G, Z, u, f, plan
                    torch.cuda.empty_cache()
    big = [x for x in out_lines if not x["l2_note"] and x["d"] >= 11_000_000]
    summary = {"mode": "sweep", "points": len(out_lines), "skipped": skipped, "peak_GBps": peak, "peak_source": peak_src,
               "flags_ok_upto_s": sum(bool(x["flags_ok_upto_s"]) for x in out_lines),
               "beyond_s_fails": sum(bool(x["beyond_s_fails"]) for x in out_lines),
               "beyond_s_silent_error": sum(bool(x.get("beyond_s_silent_error")) for x in out_lines),
               "min_decode_frac_large_d": min((x["decode_frac"] for x in big), default=None),
               "min_encode_frac_large_d": min((x["encode_frac"] for x in big), default=None), "out": args.sweep_out}
    print(json.dumps(summary))

def sweep_table(path: str) -> str:
    """Markdown table of a finished sweep (the JSON lines that --sweep wrote)."""
    rows = [json.loads(l) for l in open(path) if l.strip()]
    rows = [r for r in rows if "n" in r and "encode_ms" in r]
    def dfmt(d):
        return f"{d / 1e6:.1f} M"
    out = ["| code | n | s | d | encode ms | encode GB/s (frac) | locate+decode ms | decode GB/s (frac) | coded GB/s produced / consumed "
           "| err 0 adv | err s adv | flags ≤ s | > s fails |", "|---|---|---|---|---|---|---|---|---|---|---|---|---|"]
    for r in rows:
        c = r["checks"]
        out.append(f"| {r['code']} | {r['n']} | {r['s']} | {dfmt(r['d'])} | {r['encode_ms']:.3f} | {r['encode_hbm_GBps']:.0f} ({r['encode_frac']:.2f}) "
                   f"| {r['decode_ms']:.3f} | {r['decode_hbm_GBps']:.0f} ({r['decode_frac']:.2f}) "
                   f"| {r['coded_GBps_produced']:.0f} / {r['coded_GBps_consumed']:.0f} | {c['0']['err']:.1e} | {c['s']['err']:.1e} "
                   f"| {'yes' if r['flags_ok_upto_s'] else 'NO'} | {'yes' if r['beyond_s_fails'] else 'decoded'} |")
    return "\n".join(out) + "\n"



def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--d", type=int, default=None, help="override the workload's d (profiling on a small case)")
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay of the step")
    ap.add_argument("--sweep", action="store_true", help="both codes over n x s x d (one GPU); JSON lines to --sweep-out")
    ap.add_argument("--sweep-codes", default="rep,cyc")
    ap.add_argument("--sweep-n", default="15,45,105")
    ap.add_argument("--sweep-s", default="1,2,5,7")
    ap.add_argument("--sweep-d", default="1e6,11.7e6,60.2e6,138e6")
    ap.add_argument("--sweep-table", default=None, help="render the JSON lines of a finished sweep as a markdown table on stdout (no GPU)")
    ap.add_argument("--sweep-out", default=None, help="file the sweep appends its JSON lines to (default: a new temporary file)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true", help="skip the repetition-code and packed-transport workloads "
                    "that follow the default workload on one GPU")
    ap.add_argument("--dry-run", action="store_true", help="print how N ranks would be launched (JSON) and exit")
    args = ap.parse_args()
    if args.sweep_table:
        sys.stdout.write(sweep_table(args.sweep_table))
        return
    if args.d is not None:
        w = list(WORKLOADS[args.workload])
        w[3] = args.d
        args.workload = f"{args.workload}@d={args.d}"
        WORKLOADS[args.workload] = tuple(w)
    if (args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.sweep and args.impl == "ours") or args.dry_run:
        # started by hand as `python bench.py --gpus N`: become N ranks, one per GPU, under torchrun
        cmd, env = launch_plan(args, sys.argv[1:])
        if args.dry_run:
            single = [sys.executable, os.path.abspath(__file__)] + [a for a in sys.argv[1:] if a != "--dry-run"]
            print(json.dumps({"launch": cmd if (args.gpus > 1 and args.impl == "ours") else single,
                              "env": env if (args.gpus > 1 and args.impl == "ours") else {},
                              "ranks": args.gpus if args.impl == "ours" else 1}))
            return
        os.environ.update(env)
        os.execvp(cmd[0], cmd)
    if args.sweep:
        if args.sweep_out is None:
            fd, args.sweep_out = tempfile.mkstemp(prefix="draco_sweep_", suffix=".jsonl")
            os.close(fd)
        os.makedirs(os.path.dirname(os.path.abspath(args.sweep_out)), exist_ok=True)
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
