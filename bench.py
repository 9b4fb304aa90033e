#!/usr/bin/env python
"""Benchmark of the ConEF step on B200.

A "step" is one pass of the whole hot path over one batch of synthetic
gradients: decode -> p -> Q -> residual -> store through C -> sum of the
messages, for all N simulated workers and all tensors (every phase and every
reduce call of include/conef.h).  Default workload: the GPT-2-XL-shaped list
(1.56 G parameters, 8 workers resident in one GPU's HBM, rank-4 low-rank Q,
int4 blocks of 128 with fp16 scales).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line.  The headline is the --workload (default gpt2-xl); the other four
configurations (and the run-by-run variant of the count sketch) are timed after it and reported
under "configs".  With --gpus N > 1 (under torchrun) every rank runs an independent replica of
the workload (the path has no cross-GPU exchange in this arrangement); the value is the sum over
ranks divided by the slowest rank's time.  --sharded instead runs ONE worker per rank, N = world
size, with the small messages all-reduced over NCCL between the phases (Alg. 2 line 7).
--impl reference times the CPU oracle on a bounded sample.
"""
from __future__ import annotations

import argparse
import datetime
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2312_08538_b200 import multirank, workloads as wl  # noqa: E402

METRIC = "conef_step_params_per_sec"
UNIT = "elements/s"

# Algorithmic bytes per compressed element moved by each kernel of the step
# (what the method itself must read and write once: fp32 gradient + stored state).
def state_bytes_per_elem(c):
    if c["kind"] == "int8":
        return 1.0 + (4.0 if c.get("scale_dtype", "fp32") == "fp32" else 2.0) / c["block"]
    if c["kind"] == "int4":
        return 0.5 + (4.0 if c.get("scale_dtype", "fp32") == "fp32" else 2.0) / c["block"]
    if c["kind"] == "identity":
        return 4.0
    if c["kind"] == "stochquant":
        return (2.0 if c.get("levels", 16) > 127 else 1.0) + 4.0 / c["block"]
    return 4.0 * c["cs_rows"] / c["cs_col_div"]


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons.  It is started before the warm-up (the
    tool takes a moment to come up) and only the samples whose timestamp falls inside the timed
    region are kept."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.t0 = self.t1 = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def mark_begin(self):
        self.t0 = datetime.datetime.now()

    def mark_end(self):
        self.t1 = datetime.datetime.now()

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.1)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        inside, every = [], []
        mx, reasons = None, set()
        pad = datetime.timedelta(milliseconds=25)
        for r in self.rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 8:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f")
                clk = float(f[1])
                mx = float(f[2])
            except ValueError:
                continue
            every.append(clk)
            if self.t0 and self.t1 and self.t0 - pad <= ts <= self.t1 + pad:
                inside.append(clk)
                for n, v in zip(names, f[4:8]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
        use = sorted(inside if inside else every)
        return {"sm_mhz": use[len(use) // 2] if use else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(inside), "samples_total": len(every)}


def visible_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ----------------------------------------------------------------- CPU oracle sample

def oracle_sample_tensors(cfg, limit=4, budget=4.2e7):
    """A bounded sample of the workload for the CPU oracle: the first few
    compressed tensors (skipping embeddings) up to ~4e7 elements per worker."""
    picked, tot = [], 0
    for (r, c, k) in cfg["tensors"]:
        if not (k and c > 1) or r > 40000:
            continue
        if tot + r * c > budget and picked:
            break
        picked.append((r, c, k))
        tot += r * c
        if len(picked) >= limit:
            break
    return picked


def _oracle_run(cfg, tensors, steps, warmup):
    """Seconds per step of one oracle over `tensors` (all workers)."""
    from tests import parity_util as pu
    s = dict(cfg)
    s["tensors"] = list(tensors)
    q0 = wl.q_init(s, "cpu").numpy() if s["q"]["kind"] == "lowrank" else None
    o = pu.make_oracle(s, q_init=q0)
    grads = [wl.gradient(s, i, 0, "cpu").numpy() for i in range(s["n_workers"])]
    times = []
    for t in range(warmup + steps):
        t0 = time.perf_counter()
        res = o.step(t, grads)
        for which in ("values", "P", "Q", "dense1d"):
            o.reduced(res, which)
        if t >= warmup:
            times.append(time.perf_counter() - t0)
    return sum(times) / len(times)


def cpu_info():
    model = "unknown"
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                model = line.split(":", 1)[1].strip()
                break
    except OSError:
        pass
    from oracle import conef_oracle as orc
    try:
        cc = subprocess.run(["gcc", "--version"], capture_output=True, text=True).stdout.splitlines()[0]
    except Exception:
        cc = "gcc"
    return {"nproc": os.cpu_count(), "cpu_model": model, "compiler": cc, "flags": " ".join(orc.CFLAGS)}


def run_oracle_sample(cfg, steps, warmup, threads=1):
    """The oracle, as it stands, on a bounded sample.  threads = 1: one oracle over the sample's
    tensors.  threads > 1: the sample's tensors are dealt out to that many oracles that run side
    by side, one thread each (tensors are independent of one another; the C routines release the
    interpreter lock), and the rate is the whole sample over the wall time."""
    sample = oracle_sample_tensors(cfg, limit=max(4, threads))
    if threads > 1:
        while len(sample) < threads:       # as many tensors as threads, repeating the sample's shapes
            sample = sample + sample[:threads - len(sample)]
    elems = cfg["n_workers"] * sum(r * c for r, c, _ in sample)
    if threads <= 1:
        per_step = _oracle_run(cfg, sample, steps, warmup)
        used = 1
    else:
        from concurrent.futures import ThreadPoolExecutor
        parts = [sample[i::threads] for i in range(threads)]
        parts = [p for p in parts if p]
        used = len(parts)
        t0 = time.perf_counter()
        with ThreadPoolExecutor(max_workers=used) as ex:
            list(ex.map(lambda p: _oracle_run(cfg, p, steps, 0), parts))
        per_step = (time.perf_counter() - t0) / steps
    desc = f"{len(sample)} tensors {sample} x {cfg['n_workers']} workers = {elems} element-steps per step"
    return elems / per_step, per_step, desc, used


# ----------------------------------------------------------------- one workload on this rank's GPU

def config_of(name, cfg, N, comp, total):
    return {"workload": name, "n_workers": N, "tensors": len(cfg["tensors"]),
            "params": total, "compressed_params": comp, "q": cfg["q"]["kind"],
            "rank": cfg["q"].get("rank"), "c": cfg["c"]["kind"], "block": cfg["c"].get("block"),
            "scale_dtype": cfg["c"].get("scale_dtype"), "cs_chunk": cfg["c"].get("cs_chunk"), "lr": cfg["lr"],
            "unit_counted": "n_workers x compressed (2-D) parameters per step",
            "l2": "inputs larger than L2 (gradients of all workers are re-read from HBM each step)"
                  if N * total * 4 > 126e6 else "inputs smaller than L2: a buffer larger than L2 is written between steps"}


# DRAM bytes per element of the low-rank passes from their ncu captures (dram__bytes_read.sum +
# dram__bytes_write.sum over the elements of the captured launch; the two-block GPT-2-XL slice,
# rank 4, int4/128/fp16: profiles/k_rows_p1_gpt2-xl-slice.md, profiles/k_fast_pass_gpt2-xl-slice.md).
# Traffic grows in proportion to the elements, so the capture of the small case is scaled to
# the timed launch; null for configurations that were not captured.
# (pass 2 at full size: the capture's 4.655 less the extra partial rows of the slice's shorter tiles)
NCU_BYTES_PER_ELEM = {"pass1": 4.592, "pass2": 4.586, "pass3": 5.055}


def measure(name, args, dev, world, steps, warmup, want_e2e):
    """Times `steps` steps of workload `name` after `warmup`; returns the fields of a bench line."""
    from paper_2312_08538_b200 import binding as B
    import torch.distributed as dist
    cfg = wl.config(name)
    N = cfg["n_workers"]
    comp = wl.compressed_elems(cfg["tensors"])
    total = wl.total_elems(cfg["tensors"])
    lowrank = cfg["q"]["kind"] == "lowrank"
    q0 = wl.q_init(cfg, dev) if lowrank else None
    eng = B.ConEF(cfg["tensors"], N, cfg["q"], cfg["c"], cfg["lr"], q_init=q0, device=dev)
    if args.generic:
        eng.set_fast_path(False)
    grads = [wl.gradient(cfg, i, 0, dev) for i in range(N)]
    kinds = [B.MSG_P, B.MSG_Q] if lowrank else [B.MSG_VALUES]
    if eng.message_elems(B.MSG_DENSE1D) > 0:
        kinds.append(B.MSG_DENSE1D)
    outs = {k: torch.empty(eng.message_elems(k), dtype=torch.float32, device=dev) for k in kinds}
    stream = torch.cuda.current_stream()
    # small workloads fit L2: a buffer larger than L2 is rewritten between steps (outside the phases' events)
    flush = torch.empty(192 << 20, dtype=torch.uint8, device=dev) if N * total * 4 <= 126e6 else None

    fused = False
    if lowrank:
        eng.set_fused(args.fused, args.tile_periods, args.ctas_per_sm)
        fused = bool(eng.fused_info()["active"])
    if fused:
        phases = ["pass1", "gram_schmidt", "pass23", "reduce_q"]
    else:
        phases = ["pass1", "gram_schmidt", "pass2", "pass3", "reduce_q"] if lowrank else ["step", "reduce"]
    phase_ms = {p: 0.0 for p in phases}

    def one_step(t, marks=None):
        def mark():
            if marks is not None:
                e = torch.cuda.Event(enable_timing=True)
                e.record(stream)
                marks.append(e)
        if flush is not None:
            flush.fill_(t & 0xFF)
        mark()
        eng.step(t, grads, 0)
        mark()
        if lowrank:
            eng.reduce_messages(B.MSG_P, outs[B.MSG_P])
            mark()
            if fused:
                eng.step(t, grads, 1)
            else:
                eng.step(t, grads, 2)
                mark()
                eng.step(t, grads, 3)
            mark()
            eng.reduce_messages(B.MSG_Q, outs[B.MSG_Q])
        else:
            eng.reduce_messages(B.MSG_VALUES, outs[B.MSG_VALUES])
        if B.MSG_DENSE1D in outs:
            eng.reduce_messages(B.MSG_DENSE1D, outs[B.MSG_DENSE1D])
        mark()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(visible_gpu_index(dev.index or 0))
    sampler.start()
    t = 0
    for _ in range(warmup):
        one_step(t)
        t += 1
    barrier()
    launches0 = eng.launch_count()
    all_marks = []
    barrier()
    sampler.mark_begin()
    for _ in range(steps):
        marks = []
        one_step(t, marks)
        all_marks.append(marks)
        t += 1
    barrier()
    sampler.mark_end()
    clocks = sampler.stop()
    launches = eng.launch_count() - launches0
    # a step is timed from its first event to its last (the L2 flush of a small workload sits before the first)
    total_ms = sum(m[0].elapsed_time(m[-1]) for m in all_marks)
    for marks in all_marks:
        for p, (a, b) in zip(phases, zip(marks[:-1], marks[1:])):
            phase_ms[p] += a.elapsed_time(b)
    for p in phase_ms:
        phase_ms[p] /= steps
    status = eng.last_status()
    value, ms_per_step = multirank.throughput(total_ms / steps, N * comp, dev)

    # ---- roofline of the dominant kernel, timed live by the events above.  Algorithmic bytes per
    # compressed element: what the method itself must read and write once per kernel (fp32
    # gradient + stored state in; state out where the kernel stores).  "planned" is their sum
    # over the step's kernels (p is recomputed in every low-rank pass instead of being kept);
    # "floor" is every array touched once in the whole step.
    sb = state_bytes_per_elem(cfg["c"])
    peak, peak_kind = measured_peak()
    if lowrank:
        alg = {"pass1": 4.0 + sb, "pass23": 4.0 + 2 * sb} if fused else \
              {"pass1": 4.0 + sb, "pass2": 4.0 + sb, "pass3": 4.0 + 2 * sb}
        dom = max(alg, key=lambda k: phase_ms[k])
    else:
        alg = {"step": 4.0 + 2 * sb}
        dom = "step"
    planned = (3 * (4.0 + sb) + sb) if lowrank else (4.0 + 2 * sb)
    floor = 4.0 + 2 * sb
    units = N * comp
    achieved = alg[dom] * units / (phase_ms[dom] * 1e-3) / 1e9
    step_alg_gbs = planned * units / (ms_per_step * 1e-3) / 1e9
    floor_gbs = floor * units / (ms_per_step * 1e-3) / 1e9
    captured = lowrank and cfg["c"]["kind"] == "int4" and cfg["q"].get("rank") == 4 and not args.generic
    traffic = NCU_BYTES_PER_ELEM[dom] * units if captured and dom in NCU_BYTES_PER_ELEM else None
    per_kernel = {k: {"ms": phase_ms[k], "algorithmic_bytes_per_elem": alg[k],
                      "achieved_gbs": alg[k] * units / (phase_ms[k] * 1e-3) / 1e9,
                      "frac": alg[k] * units / (phase_ms[k] * 1e-3) / 1e9 / peak} for k in alg}
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": traffic,
                "algorithmic_bytes_per_launch": alg[dom] * units,
                "phase_ms": phase_ms, "per_kernel": per_kernel,
                "planned_bytes_per_elem": planned, "floor_bytes_per_elem": floor,
                "step_algorithmic_gbs": step_alg_gbs, "step_frac_of_peak": step_alg_gbs / peak,
                "step_frac_of_peak_is": "planned bytes (every kernel's own reads and writes) / step time / peak",
                "floor_gbs": floor_gbs, "floor_frac": floor_gbs / peak,
                "floor_frac_is": "floor bytes (every array touched once per step) / step time / peak"}

    # ---- end to end: the same step with the gradients coming from pinned host memory
    e2e = None
    if want_e2e:
        per_worker = grads[0].numel()
        host = torch.empty(per_worker, dtype=torch.float32, pin_memory=True)
        host.copy_(grads[0])
        res_host = {k: torch.empty(v.numel(), dtype=torch.float32, pin_memory=True) for k, v in outs.items()}
        h2d = per_worker * 4 * N
        d2h = sum(v.numel() * 4 for v in outs.values())

        def e2e_step(tt):
            for i in range(N):
                grads[i].copy_(host, non_blocking=True)   # one pinned staging buffer serves the N workers
            one_step(tt)
            for k in outs:
                res_host[k].copy_(outs[k], non_blocking=True)

        e2e_steps = max(1, min(steps, 3))
        e2e_step(t)
        t += 1
        barrier()
        a = torch.cuda.Event(enable_timing=True)
        bb = torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(e2e_steps):
            e2e_step(t)
            t += 1
        bb.record(stream)
        barrier()
        e2e_value, e2e_ms = multirank.throughput(a.elapsed_time(bb) / e2e_steps, N * comp, dev)
        e2e = {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "steps": e2e_steps, "ms_per_step": e2e_ms,
               "note": "every worker's gradient is copied from ONE pinned host buffer (worker 0's values): "
                       "the bytes moved and the work are those of N distinct gradients, the values are not"}
    return {"value": value, "ms_per_step": ms_per_step, "config": config_of(name, cfg, N, comp, total),
            "roofline": roofline, "e2e": e2e, "gpu_launches": launches, "clocks": clocks, "device_status": status,
            "state_bytes_per_worker": eng.state_bytes_per_worker(), "dense_error_bytes_per_worker": comp * 4,
            "fused_passes_2_3": fused}


def measure_sharded(name, args, dev, world, steps, warmup):
    """One worker per rank: N = world size, the messages all-reduced across ranks (NCCL) between the
    phases.  Returns the fields of a bench line."""
    from paper_2312_08538_b200 import binding as B
    import torch.distributed as dist
    cfg = wl.config(name)
    rank = dist.get_rank() if world > 1 else 0
    comp = wl.compressed_elems(cfg["tensors"])
    total = wl.total_elems(cfg["tensors"])
    lowrank = cfg["q"]["kind"] == "lowrank"
    q0 = wl.q_init(cfg, dev) if lowrank else None
    eng = B.ConEF(cfg["tensors"], 1, cfg["q"], cfg["c"], cfg["lr"], q_init=q0, device=dev)
    sh = multirank.ShardedConEF(eng, lowrank, world_size=world,
                                all_reduce=None if world > 1 else (lambda t_: None))
    grad = wl.gradient(cfg, rank, 0, dev)
    ms = multirank.timed_steps(lambda t_: sh.step(t_, grad), steps, warmup, multirank.CudaClock(dev),
                               barrier=(dist.barrier if world > 1 else None))
    value, ms_per_step = multirank.throughput(ms, comp, dev)
    c = config_of(name, cfg, world, comp, total)
    c["arrangement"] = "one worker per rank, messages all-reduced across ranks"
    return {"value": value, "ms_per_step": ms_per_step, "config": c, "device_status": eng.last_status(),
            "gpu_launches": eng.launch_count()}


# ----------------------------------------------------------------- main

OTHER_CONFIGS = ["tiny", "resnet50", "gpt2-small", "transformer-big", "transformer-big-chunksketch"]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="gpt2-xl")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="time the headline workload only")
    ap.add_argument("--sharded", action="store_true", help="one worker per rank, messages all-reduced across ranks")
    ap.add_argument("--generic", action="store_true", help="generic kernels only")
    ap.add_argument("--fused", action="store_true", help="low-rank passes 2 and 3 in the persistent task-list kernel")
    ap.add_argument("--tile-periods", type=int, default=0, help="tile length of the fused low-rank kernel (0: default)")
    ap.add_argument("--ctas-per-sm", type=int, default=0, help="resident CTAs per SM of the fused low-rank kernel (0: default)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    cfg = wl.config(args.workload)

    if args.impl == "reference":
        if rank != 0:
            return
        N = cfg["n_workers"]
        steps = max(1, min(args.steps, 3))
        v, per_step, sample, used = run_oracle_sample(cfg, steps, min(args.warmup, 1))
        config = config_of(args.workload, cfg, N, wl.compressed_elems(cfg["tensors"]), wl.total_elems(cfg["tensors"]))
        info = cpu_info()
        line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
                "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": per_step * 1e3,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
                "data": "synthetic", "config": config,
                "cpu_baseline": dict({"value": v, "unit": UNIT, "cores": used, "kind": "oracle", "sample": sample}, **info),
                "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    if args.sharded:
        m = measure_sharded(args.workload, args, dev, world, args.steps, args.warmup)
        if rank == 0:
            line = {"metric": METRIC, "value": m["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
                    "warmup": args.warmup, "ms_per_step": m["ms_per_step"], "higher_is_better": True,
                    "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                    "config": m["config"], "gpu_launches": m["gpu_launches"], "device_status": m["device_status"]}
            print(json.dumps(line))
        if world > 1:
            dist.destroy_process_group()
        return

    head = measure(args.workload, args, dev, world, args.steps, args.warmup, not args.no_e2e)
    torch.cuda.empty_cache()

    # ---- the other configurations, each timed the same way (they take well under a second each)
    configs = {}
    if world == 1 and not args.no_configs:
        for name in OTHER_CONFIGS:
            if name == args.workload:
                continue
            m = measure(name, args, dev, world, max(args.steps, 5), max(args.warmup, 3), False)
            torch.cuda.empty_cache()
            r = m["roofline"]
            configs[name] = {"ms_per_step": m["ms_per_step"], "value": m["value"], "unit": UNIT,
                             "n_workers": m["config"]["n_workers"], "compressed_params": m["config"]["compressed_params"],
                             "q": m["config"]["q"], "c": m["config"]["c"], "cs_chunk": m["config"]["cs_chunk"],
                             "l2": m["config"]["l2"],
                             "roofline": {"kernel": r["kernel"], "frac": r["frac"], "achieved": r["achieved"],
                                          "step_frac_of_peak": r["step_frac_of_peak"], "floor_frac": r["floor_frac"],
                                          "phase_ms": r["phase_ms"]},
                             "gpu_launches": m["gpu_launches"], "device_status": m["device_status"], "clocks": m["clocks"]}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        # the oracle as it stands: one thread, then one oracle per host core side by side
        v1, s1, sample1, _ = run_oracle_sample(cfg, 1, 0, threads=1)
        ncpu = os.cpu_count() or 1
        va, sa, samplea, used = run_oracle_sample(cfg, 1, 0, threads=ncpu) if ncpu > 1 else (v1, s1, sample1, 1)
        cpu = dict({"value": va, "unit": UNIT, "cores": used, "kind": "oracle", "sample": samplea, "seconds": sa,
                    "single_thread": {"value": v1, "cores": 1, "sample": sample1, "seconds": s1}}, **cpu_info())

    if rank == 0:
        line = {"metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": head["config"], "roofline": head["roofline"], "cpu_baseline": cpu, "e2e": head["e2e"],
                "gpu_launches": head["gpu_launches"], "clocks": head["clocks"], "device_status": head["device_status"],
                "state_bytes_per_worker": head["state_bytes_per_worker"],
                "dense_error_bytes_per_worker": head["dense_error_bytes_per_worker"],
                "fused_passes_2_3": head["fused_passes_2_3"], "configs": configs}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
