#!/usr/bin/env python
"""Benchmark of the ConEF step on B200.

A "step" is one pass of the whole hot path over one batch of synthetic
gradients: decode -> p -> Q -> residual -> store through C -> sum of the
messages, for all N simulated workers and all tensors (every phase and every
reduce call of include/conef.h).  Default workload: the GPT-2-XL-shaped list
(1.56 G parameters, 8 workers resident in one GPU's HBM, rank-4 low-rank Q,
int4 blocks of 128 with fp16 scales).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line.  With --gpus N > 1 (under torchrun) every rank runs an
independent replica of the workload (the path has no cross-GPU exchange in
this build); the value is the sum over ranks divided by the slowest rank's
time.  --impl reference times the CPU oracle on a bounded sample.
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

def oracle_sample_cfg(cfg):
    """A bounded sample of the workload for the CPU oracle: the first few
    compressed tensors (skipping embeddings) up to ~4e7 elements per worker."""
    picked, tot = [], 0
    for (r, c, k) in cfg["tensors"]:
        if not (k and c > 1) or r > 40000:
            continue
        if tot + r * c > 4.2e7 and picked:
            break
        picked.append((r, c, k))
        tot += r * c
        if len(picked) >= 4:
            break
    s = dict(cfg)
    s["tensors"] = picked
    return s


def run_oracle_sample(cfg, steps, warmup):
    from tests import parity_util as pu
    s = oracle_sample_cfg(cfg)
    q0 = wl.q_init(s, "cpu").numpy() if s["q"]["kind"] == "lowrank" else None
    o = pu.make_oracle(s, q_init=q0)
    grads = [wl.gradient(s, i, 0, "cpu").numpy() for i in range(s["n_workers"])]
    elems = s["n_workers"] * wl.compressed_elems(s["tensors"])
    times = []
    for t in range(warmup + steps):
        t0 = time.perf_counter()
        res = o.step(t, grads)
        for which in ("values", "P", "Q", "dense1d"):
            o.reduced(res, which)
        dt = time.perf_counter() - t0
        if t >= warmup:
            times.append(dt)
    per_step = sum(times) / len(times)
    sample = f"{len(s['tensors'])} tensors {s['tensors']} x {s['n_workers']} workers = {elems} element-steps per step"
    return elems / per_step, per_step, sample


# ----------------------------------------------------------------- main

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="gpt2-xl")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
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
    N = cfg["n_workers"]
    comp = wl.compressed_elems(cfg["tensors"])
    total = wl.total_elems(cfg["tensors"])
    config = {"workload": args.workload, "n_workers": N, "tensors": len(cfg["tensors"]),
              "params": total, "compressed_params": comp, "q": cfg["q"]["kind"],
              "rank": cfg["q"].get("rank"), "c": cfg["c"]["kind"], "block": cfg["c"].get("block"),
              "scale_dtype": cfg["c"].get("scale_dtype"), "cs_chunk": cfg["c"].get("cs_chunk"), "lr": cfg["lr"],
              "unit_counted": "n_workers x compressed (2-D) parameters per step",
              "l2": "inputs larger than L2 (gradients of all workers are re-read from HBM each step)"}

    if args.impl == "reference":
        if rank != 0:
            return
        steps = max(1, min(args.steps, 3))
        v, per_step, sample = run_oracle_sample(cfg, steps, min(args.warmup, 1))
        line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
                "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": per_step * 1e3,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
                "data": "synthetic", "config": config,
                "cpu_baseline": {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
                "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return

    from paper_2312_08538_b200 import binding as B

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

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

    sampler = ClockSampler(visible_gpu_index(local_rank))
    sampler.start()
    t = 0
    for _ in range(args.warmup):
        one_step(t)
        t += 1
    barrier()
    launches0 = eng.launch_count()
    all_marks = []
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.mark_begin()
    e0.record(stream)
    for _ in range(args.steps):
        marks = []
        one_step(t, marks)
        all_marks.append(marks)
        t += 1
    e1.record(stream)
    barrier()
    sampler.mark_end()
    clocks = sampler.stop()
    total_ms = e0.elapsed_time(e1)
    launches = eng.launch_count() - launches0
    for marks in all_marks:
        for p, (a, b) in zip(phases, zip(marks[:-1], marks[1:])):
            phase_ms[p] += a.elapsed_time(b)
    for p in phase_ms:
        phase_ms[p] /= args.steps
    status = eng.last_status()

    value, ms_per_step = multirank.throughput(total_ms / args.steps, N * comp, dev)

    # ---- roofline of the dominant kernel, timed live by the events above
    sb = state_bytes_per_elem(cfg["c"])
    peak, peak_kind = measured_peak()
    if lowrank:
        alg = {"pass1": 4.0 + sb, "pass23": 4.0 + 2 * sb} if fused else {"pass1": 4.0 + sb, "pass2": 4.0 + sb, "pass3": 4.0 + 2 * sb}
        dom = max(alg, key=lambda k: phase_ms[k])
        bytes_per_launch = alg[dom] * N * comp
        dur = phase_ms[dom]
    else:
        dom = "step"
        bytes_per_launch = (4.0 + 2 * sb) * N * comp
        dur = phase_ms["step"]
    achieved = bytes_per_launch / (dur * 1e-3) / 1e9
    step_alg_gbs = (sum(alg.values()) if lowrank else (4.0 + 2 * sb)) * N * comp / (ms_per_step * 1e-3) / 1e9
    # DRAM bytes per element of the dominant kernel from its ncu capture (dram__bytes_read.sum +
    # dram__bytes_write.sum over the elements of the captured launch; the capture of the two-block
    # GPT-2-XL slice, rank 4, int4/128/fp16, summarised under profiles/).  Traffic grows in proportion to the elements, so the capture of the
    # small case is scaled to this launch; null for configurations that were not captured.
    NCU_BYTES_PER_ELEM = {"pass1": 4.578, "pass2": 4.580, "pass3": 5.054}
    captured = lowrank and cfg["c"]["kind"] == "int4" and cfg["q"].get("rank") == 4 and not args.generic
    traffic = NCU_BYTES_PER_ELEM[dom] * N * comp if captured and dom in NCU_BYTES_PER_ELEM else None
    per_kernel = {}
    if lowrank:
        for k in alg:
            a_k = alg[k] * N * comp / (phase_ms[k] * 1e-3) / 1e9
            per_kernel[k] = {"ms": phase_ms[k], "algorithmic_bytes_per_elem": alg[k], "achieved_gbs": a_k,
                             "frac": a_k / peak}
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": traffic,
                "algorithmic_bytes_per_launch": bytes_per_launch,
                "phase_ms": phase_ms, "per_kernel": per_kernel, "step_algorithmic_gbs": step_alg_gbs,
                "step_frac_of_peak": step_alg_gbs / peak}

    if cfg["c"]["kind"] == "countsketch" and cfg["c"].get("cs_chunk", 0) and not lowrank and not args.generic:
        # The run-by-run count sketch is bound by instruction issue (five 64-bit hashes per element),
        # not by HBM: report warp instructions per second against the issue peak of the part,
        # 148 SMs x 4 schedulers x 1 instruction per clock at the 1965 MHz maximum SM clock.  The
        # instruction count per 32 elements is the ncu figure of the captured launch (profiles/).
        CSK_INST_PER_32 = 350.0
        issue_peak = 148 * 4 * 1.965      # G warp instructions / s
        inst = CSK_INST_PER_32 * N * comp / 32.0
        a_i = inst / (phase_ms["step"] * 1e-3) / 1e9
        roofline.update({"bound": "alu", "kernel": "k_sketch_chunk", "achieved": a_i, "peak": issue_peak,
                         "unit": "Gwarp-inst/s", "frac": a_i / issue_peak,
                         "peak_kind": "derived: 148 SMs x 4 schedulers x 1.965 GHz",
                         "traffic": 8.09 * N * comp, "hbm_algorithmic_gbs": achieved, "hbm_frac": achieved / peak})

    # ---- end to end: the same step with the gradients coming from pinned host memory
    e2e = None
    if not args.no_e2e:
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

        e2e_steps = max(1, min(args.steps, 3))
        e2e_step(t); t += 1
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
        e2e = {"value": e2e_value, "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
               "ms_per_step": e2e_ms}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, per_step, sample = run_oracle_sample(cfg, 1, 0)
        cpu = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
               "seconds": per_step}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": config, "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e,
                "gpu_launches": launches, "clocks": clocks, "device_status": status,
                "state_bytes_per_worker": eng.state_bytes_per_worker(),
                "dense_error_bytes_per_worker": comp * 4}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
