#!/usr/bin/env python
"""Benchmark of the verify step: verified positions per second.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl reference]

A step is one whole verify step (massv_verify_attn + massv_accept +
massv_kv_commit) on one batch of the synthetic workload.  The default workload
is the Qwen2.5-VL-7B-shaped batch-1 greedy step.  One JSON line is printed by
rank 0.  With N > 1 every rank runs an independent replica of the workload on
its own GPU (the path has no cross-GPU exchange), so scaling is weak.

`--impl reference` times the CPU oracle instead (it is the only reference
implementation there is): same workload, metric and unit, on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "verified positions/sec per verify step"
UNIT = "positions/s"
DEFAULT_WORKLOAD = "qwen7b_b1_t0"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
L2_FLUSH_BYTES = 512 << 20
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, from the ncu
# capture summarised under profiles/ (per workload; None where no capture of the current kernel exists)
NCU_TRAFFIC_BYTES = {"qwen7b_b1_t0": 1.090398e9 + 3.058e6}   # mean of three launches


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Polls nvidia-smi for SM clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id):
        self.gpu_id, self.proc, self.path = gpu_id, None, f"/tmp/massv_clocks_{os.getpid()}.csv"

    def start(self):
        try:
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu_id), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=self.out, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.out.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 7:
                    continue
                try:
                    sm.append(float(parts[0])); mx.append(float(parts[1]))
                except ValueError:
                    continue
                for n, v in zip(names, parts[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
        try:
            os.remove(self.path)
        except OSError:
            pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def time_oracle(cfg, w_cpu, max_seconds=30.0, max_reps=3):
    """Time the CPU oracle, as it stands, on whole verify steps of the workload."""
    import oracle
    times = []
    t_total = time.perf_counter()
    for _ in range(max_reps):
        t0 = time.perf_counter()
        oracle.verify_step(w_cpu, cfg.temperature)
        times.append(time.perf_counter() - t0)
        if time.perf_counter() - t_total > max_seconds:
            break
    t = min(times)
    return cfg.m / t, t, len(times), oracle.num_threads()


def bounded_cpu_workload(cfg, w):
    """Host copy of the workload, cut down to a few sequences when a whole batch
    would take the oracle more than a few tens of seconds."""
    import torch
    macs = float(cfg.m) * cfg.vocab * cfg.hidden
    keep = cfg.batch
    if macs > 2.0e10:
        keep = max(1, int(cfg.batch * 2.0e10 / macs))
    from dataclasses import replace
    sub_cfg = replace(cfg, batch=keep)
    sub = {}
    for k, v in w.items():
        if k in ("k_pages", "v_pages", "lm_head"):
            sub[k] = v.cpu()
        else:
            sub[k] = v[:keep].contiguous().cpu()
    return sub_cfg, sub, keep


def run_reference(args):
    """The reference arm: the CPU oracle on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import torch
    import oracle
    from workloads import generate, get_config
    oracle.build()
    cfg = get_config(args.config)
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    w = generate(cfg, device=dev)
    sub_cfg, w_cpu, keep = bounded_cpu_workload(cfg, w)
    del w
    for _ in range(min(args.warmup, 1)):
        oracle.verify_step(w_cpu, sub_cfg.temperature)
    steps = max(1, min(args.steps, 3))
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.verify_step(w_cpu, sub_cfg.temperature)
    dt = (time.perf_counter() - t0) / steps
    value = sub_cfg.m / dt
    sample = f"{keep} of {cfg.batch} sequences of {cfg.name}, whole verify step, {steps} timed passes"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": min(args.warmup, 1), "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "batch": cfg.batch, "gamma": cfg.gamma, "temperature": cfg.temperature},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", default=DEFAULT_WORKLOAD)
    ap.add_argument("--impl", default="massv", choices=["massv", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--attn-kernel", type=int, default=0, choices=[0, 1, 2],
                    help="attention split kernel: 0 = chosen by shape, 1 = warp-level MMA, 2 = tcgen05")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path (use --impl reference for the oracle)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    import __graft_entry__ as entry
    if rank == 0:
        entry.build()
    if world > 1:
        dist.barrier()
    import paper_2505_10526_b200 as mv
    from workloads import generate, get_config, kv_bytes
    from paper_2505_10526_b200.step import STEP_INPUTS as STEP_KEYS

    cfg = get_config(args.config)
    w = generate(cfg, device=dev)
    step = mv.VerifyStep.for_workload(cfg, w, attn_kernel=args.attn_kernel)
    seq0 = w["seq_lens"].clone()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def one_step(ev=None, split=False):
        """One verify step.  Events bracket the step; every tenth step (split=True) two more
        events separate the three calls and the library records four more around its two dominant
        kernels (the LM-head GEMM and the attention split kernel), which gives the breakdown and
        the kernels' own durations but also keeps kernels from overlapping with their neighbours."""
        if ev:
            ev[0].record(stream)
        if split:
            mv.massv_set_timing_events(lm_head=(ev[4], ev[5]), attn=(ev[6], ev[7]))
        step.attn(w)
        if split:
            ev[1].record(stream)
        step.accept(w)
        if split:
            ev[2].record(stream)
            mv.massv_set_timing_events(None, None)
        step.commit(w["seq_lens"])
        if ev:
            ev[3].record(stream)

    def between_steps():
        w["seq_lens"].copy_(seq0)          # undo the commit so every step does identical work
        flush.fill_(1)                     # evict L2 (126 MB) between timed steps

    for _ in range(max(args.warmup, 3)):
        one_step()
        between_steps()
    torch.cuda.synchronize()
    assert int(step.dev_status.item()) == 0, "device-side error during warm-up"

    K = args.steps
    SPLIT_EVERY = 10
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(8 if i % SPLIT_EVERY == 0 else 4)] for i in range(K)]
    for evs in events:          # torch creates CUDA events lazily: the library needs the handles of its four
        for e in evs[4:]:
            e.record(stream)
    uuid = None
    try:
        uuid = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        pass
    sampler = ClockSampler(uuid if uuid else local_rank)
    launches0 = mv.massv_launch_count()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    wall0 = time.perf_counter()
    for i in range(K):
        one_step(events[i], split=(i % SPLIT_EVERY == 0))
        between_steps()
    torch.cuda.synchronize()
    wall = time.perf_counter() - wall0
    clocks = sampler.stop()
    if world > 1:
        dist.barrier()
    launches = mv.massv_launch_count() - launches0
    split_ev = [e for i, e in enumerate(events) if i % SPLIT_EVERY == 0]
    t_attn = sum(e[0].elapsed_time(e[1]) for e in split_ev) / len(split_ev)
    t_accept = sum(e[1].elapsed_time(e[2]) for e in split_ev) / len(split_ev)
    t_commit = sum(e[2].elapsed_time(e[3]) for e in split_ev) / len(split_ev)
    t_lm_kernel = sum(e[4].elapsed_time(e[5]) for e in split_ev) / len(split_ev)        # LM-head kernel alone
    t_attn_kernel = sum(e[6].elapsed_time(e[7]) for e in split_ev) / len(split_ev)      # attention split kernel alone
    t_step = sum(e[0].elapsed_time(e[3]) for e in events) / K        # ms on the device, per step
    from paper_2505_10526_b200.replicas import aggregate_throughput
    ms_per_step, value = aggregate_throughput(cfg.m, t_step, dev)
    assert int(step.dev_status.item()) == 0, "device-side error during the timed region"

    # ---- end to end: per-step inputs start in pinned host memory, results end there
    host_inputs = step.host_inputs_like({k: w[k].cpu() for k in STEP_KEYS if k in w and (cfg.temperature > 0 or k not in
                                         ("draft_probs", "u_accept", "u_sample"))})      # views of one pinned buffer
    resident = {k: w[k] for k in ("k_pages", "v_pages", "page_table", "seq_lens", "lm_head")}
    for _ in range(3):
        step.run_host(host_inputs, resident, commit=True)
        between_steps()
    torch.cuda.synchronize()
    Ke = max(10, min(K, 200))
    e2e_t = 0.0
    for _ in range(Ke):
        t0 = time.perf_counter()
        step.run_host(host_inputs, resident, commit=True)
        e2e_t += time.perf_counter() - t0
        between_steps()
        torch.cuda.synchronize()
    e2e_ms_per_step, e2e_value = aggregate_throughput(cfg.m, e2e_t / Ke * 1e3, dev)
    h2d, d2h = step.host_bytes_per_step(host_inputs)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks, peak_src = load_peaks()
    lm_bytes = cfg.vocab * cfg.hidden * 2 + cfg.m * cfg.hidden * 2
    lm_flops = 2.0 * cfg.m * cfg.vocab * cfg.hidden
    attn_bytes = kv_bytes(cfg, seq0.tolist())
    ridge = peaks["bf16_tflops"] * 1e12 / (peaks["hbm_gbs"] * 1e9)
    # the dominant kernel, timed alone by events the library records around it (massv_set_timing_events)
    if cfg.m > ridge:   # the LM-head contraction is bound by the tensor pipe
        roofline = {"kernel": "lm_head_umma_kernel", "bound": "tensor",
                    "achieved": lm_flops / (t_lm_kernel * 1e-3) / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"}
    else:
        roofline = {"kernel": "lm_head_umma_kernel", "bound": "hbm",
                    "achieved": lm_bytes / (t_lm_kernel * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    roofline["frac"] = roofline["achieved"] / roofline["peak"]
    roofline["peak_source"] = f"of {peak_src}"
    roofline["traffic"] = NCU_TRAFFIC_BYTES.get(cfg.name)
    roofline["algorithmic"] = lm_bytes if roofline["bound"] == "hbm" else lm_flops
    roofline["ms_per_launch"] = t_lm_kernel
    roofline["frac_of_whole_accept_call"] = roofline["algorithmic"] / (t_accept * 1e-3) / (1e12 if roofline["bound"] == "tensor" else 1e9) / roofline["peak"]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "batch": cfg.batch, "gamma": cfg.gamma, "temperature": cfg.temperature,
                   "n_q_heads": cfg.n_q_heads, "n_kv_heads": cfg.n_kv_heads, "head_dim": cfg.head_dim,
                   "hidden": cfg.hidden, "vocab": cfg.vocab, "mean_context": float(seq0.float().mean()),
                   "attn_kernel": {0: "by shape", 1: "warp_mma", 2: "tcgen05"}[args.attn_kernel],
                   "l2": f"flushed between timed steps by a {L2_FLUSH_BYTES >> 20} MiB write; LM-head weights alone exceed L2",
                   "parallelism": f"replicas x{world}"},
        "breakdown_ms": {"verify_attn": t_attn, "accept": t_accept, "kv_commit": t_commit,
                         "lm_head_kernel": t_lm_kernel, "attn_split_kernel": t_attn_kernel,
                         "note": "from every 10th timed step, which carries the extra events"},
        "attn_hbm": {"achieved": attn_bytes / (t_attn * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": attn_bytes / (t_attn * 1e-3) / 1e9 / peaks["hbm_gbs"],
                     "frac_split_kernel_alone": attn_bytes / (t_attn_kernel * 1e-3) / 1e9 / peaks["hbm_gbs"]},
        "mean_accept_len": float(step.accept_len.float().mean()),
        "roofline": roofline, "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_ms_per_step,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": int(launches), "wall_s_timed_region": wall,
    }
    if not args.no_cpu_baseline and world == 1:
        sub_cfg, w_cpu, keep = bounded_cpu_workload(cfg, w)
        v, t, reps, cores = time_oracle(sub_cfg, w_cpu)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"{keep} of {cfg.batch} sequences of {cfg.name}, whole verify step, best of {reps} ({t:.2f} s)"}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
