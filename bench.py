#!/usr/bin/env python
"""Benchmark of the verify step: verified positions per second.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--no-sweep] [--impl reference]
    python bench.py --sharded-world W [--config NAME]      (kernel times of one vocabulary shard)

A step is one whole verify step (massv_verify_attn + massv_accept +
massv_kv_commit) on one batch of a synthetic workload.  The default workload is
the long-context Qwen2.5-VL-7B-shaped batch of 64 sequences at gamma = 5, T = 1
(the paper's inference settings); the JSON line rank 0 prints also carries a
`sweep` with one entry per other workload of the table (batch 1, batch 16, the
Gemma3-12B shape, the other long-context points), each with its breakdown and a
roofline block per dominant kernel.  With N > 1 every rank runs an independent
replica of the workload on its own GPU (the path has no cross-GPU exchange), so
scaling is weak.

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
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "verified positions/sec per verify step"
UNIT = "positions/s"
DEFAULT_WORKLOAD = "qwen7b_long_g5_t1"
SWEEP = ["qwen7b_b1_t0", "qwen7b_b16_t1", "gemma12b_b32_t1", "qwen7b_long_g3_t0", "qwen7b_long_g3_t1",
         "qwen7b_long_g5_t0", "qwen7b_long_g7_t0", "qwen7b_long_g7_t1"]
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}
L2_FLUSH_BYTES = 512 << 20
MIN_SPLIT_STEPS = 5

# DRAM traffic of one launch of a kernel over its algorithmic bytes (dram__bytes_read.sum +
# dram__bytes_write.sum of an ncu capture, summarised under profiles/), keyed by (kernel, shape
# family).  Captures of the long-context attention kernel are taken at batch 16 (a few GB on the
# device) and scaled by the K/V bytes of the launch: the kernel streams every K/V byte once, so its
# traffic grows in proportion.  None: no capture of the kernel as it stands.
NCU_TRAFFIC_RATIO = {
    ("attn", "qwen"): (693.56 + 5.1) / 691.5,  # profiles/attn_umma_kernel_qwen7b_long_b16.md (batch 16, scaled by K/V bytes)
    ("attn", "gemma"): 1.384 / 1.34,          # profiles/attn_split_kernel_gemma12b_b32_t1.md (read 1.378 GB + 6.2 MB written)
    ("lm_head", "qwen"): 1.0934 / 1.0900,     # profiles/lm_head_umma_kernel_qwen7b_b1_t0.md (the weight-bound launches, M <= 256)
    ("lm_head", "gemma"): (2.04619 + 0.14287) / 2.01474,   # profiles/lm_head_umma_kernel_gemma12b_b32_t1.md (weights once + the fp32 logits that left L2)
    ("residual", "qwen"): (74.30 + 1.35) / 77.86,   # profiles/residual_sample_kernel_qwen7b_lmhead_g5_t1.md
    ("residual", "gemma"): (62.99 + 0.08) / 67.11,    # profiles/lm_head_umma_kernel_gemma12b_b32_t1.md (second table)
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU from a background thread (NVML, a few
    milliseconds apart; `nvidia-smi -lms` when NVML cannot be loaded).  `mark()` brackets the timed
    region, so that the summary can tell the samples taken inside it from the rest."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index, uuid=None, period_s=0.004):
        self.index, self.uuid, self.period = index, uuid, period_s
        self.samples, self.marks = [], []
        self._stop = threading.Event()
        self._thread = self._proc = None
        self.source = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nvml = pynvml
            self._h = (pynvml.nvmlDeviceGetHandleByUUID(self.uuid.encode() if hasattr(self.uuid, "encode") else self.uuid)
                       if self.uuid else pynvml.nvmlDeviceGetHandleByIndex(self.index))
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
            self.source = "nvml"
            self._thread = threading.Thread(target=self._poll_nvml, daemon=True)
            self._thread.start()
            return
        except Exception:
            self._nvml = None
        try:
            self._path = f"/tmp/massv_clocks_{os.getpid()}.csv"
            self._out = open(self._path, "w")
            fields = ("timestamp,clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
                      "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
                      "clocks_event_reasons.sw_power_cap")
            self._proc = subprocess.Popen(["nvidia-smi", "-i", str(self.uuid or self.index), f"--query-gpu={fields}",
                                           "--format=csv,noheader,nounits", "-lms", "20"],
                                          stdout=self._out, stderr=subprocess.DEVNULL)
            self._t_start = time.time()
            self.source = "nvidia-smi"
        except OSError:
            self._proc = None

    def _poll_nvml(self):
        n = self._nvml
        get_reasons = getattr(n, "nvmlDeviceGetCurrentClocksEventReasons", None) or n.nvmlDeviceGetCurrentClocksThrottleReasons
        while not self._stop.is_set():
            try:
                mhz = float(n.nvmlDeviceGetClockInfo(self._h, n.NVML_CLOCK_SM))
                bits = int(get_reasons(self._h))
                self.samples.append((time.perf_counter(), mhz, bits))
            except Exception:
                pass
            self._stop.wait(self.period)

    def mark(self):
        self.marks.append(time.perf_counter() if self.source != "nvidia-smi" else time.time())

    def stop(self):
        if self.source == "nvml":
            self._stop.set()
            self._thread.join(timeout=2)
            rows = self.samples
            sm_max = self.sm_max
        elif self.source == "nvidia-smi" and self._proc is not None:
            self._proc.terminate()
            try:
                self._proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self._proc.kill()
            self._out.close()
            rows, sm_max = [], None
            import datetime
            with open(self._path) as f:
                for line in f:
                    parts = [p.strip() for p in line.split(",")]
                    if len(parts) < 7:
                        continue
                    try:
                        t = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                        mhz, sm_max = float(parts[1]), float(parts[2])
                    except ValueError:
                        continue
                    bits = 0
                    for bit, v in zip((0x8, 0x40, 0x20, 0x4), parts[3:7]):
                        if v.lower().startswith("active"):
                            bits |= bit
                    rows.append((t, mhz, bits))
            try:
                os.remove(self._path)
            except OSError:
                pass
        else:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["no clock source available"]}
        inside = rows
        if len(self.marks) >= 2:
            inside = [r for r in rows if self.marks[0] <= r[0] <= self.marks[1]]
        window = "timed region"
        if len(inside) < 3:           # a region of a few milliseconds: fall back to every sample taken under load
            inside, window = rows, "warm-up + timed region + end-to-end runs"
        bits = 0
        for r in inside:
            bits |= r[2]
        return {"sm_mhz": statistics.median(r[1] for r in inside) if inside else None, "sm_max_mhz": sm_max,
                "samples": len(inside), "samples_all": len(rows), "window": window, "source": self.source,
                "reasons": sorted(name for bit, name in self.REASONS.items() if bits & bit)}


def config_block(cfg, mean_context, attn_kernel, world):
    """The `config` object of the JSON line; both arms print the same keys for the same workload."""
    return {"workload": cfg.name, "batch": cfg.batch, "gamma": cfg.gamma, "temperature": cfg.temperature,
            "n_q_heads": cfg.n_q_heads, "n_kv_heads": cfg.n_kv_heads, "head_dim": cfg.head_dim,
            "hidden": cfg.hidden, "vocab": cfg.vocab, "mean_context": float(mean_context),
            "attn_kernel": {0: "by shape", 1: "warp_mma", 2: "tcgen05"}[attn_kernel],
            "l2": f"flushed between timed steps by a {L2_FLUSH_BYTES >> 20} MiB write; K/V and LM-head weights exceed L2 anyway",
            "parallelism": f"replicas x{world}"}


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


def bounded_cpu_workload(cfg, w, budget_macs=2.0e10):
    """Host copy of the workload, cut down to its first few sequences when a whole batch would take
    the oracle more than a few tens of seconds (the LM head's multiply-adds set the cost)."""
    from dataclasses import replace
    macs = float(cfg.m) * cfg.vocab * cfg.hidden
    keep = cfg.batch
    if macs > budget_macs:
        keep = max(1, int(cfg.batch * budget_macs / macs))
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
    mean_ctx = float(w["seq_lens"].float().mean())
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
    sample = f"first {keep} of {cfg.batch} sequences of {cfg.name}, whole verify step, {steps} timed passes"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": min(args.warmup, 1), "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_block(cfg, mean_ctx, args.attn_kernel, args.gpus),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def _stats(xs):
    return {"mean": sum(xs) / len(xs), "median": statistics.median(xs), "best": min(xs)}


def roofline_block(kernel, bound, algorithmic, ms, peaks, peak_src, family):
    """achieved = algorithmic bytes (or flops) of one launch / its mean duration between the two events
    the library records around it; fractions of the measured peak, of the sustained tensor peak where
    that applies, and of the nominal figure."""
    if bound == "tensor":
        achieved, peak, unit = algorithmic / (ms["mean"] * 1e-3) / 1e12, peaks["bf16_tflops"], "TFLOP/s"
    else:
        achieved, peak, unit = algorithmic / (ms["mean"] * 1e-3) / 1e9, peaks["hbm_gbs"], "GB/s"
    r = {"kernel": kernel, "bound": bound, "achieved": achieved, "peak": peak, "unit": unit, "frac": achieved / peak,
         "peak_source": f"of {peak_src}" + (" (burst: the kernel is timed alone)" if bound == "tensor" else ""),
         "frac_of_nominal": achieved / (NOMINAL["bf16_tflops"] if bound == "tensor" else NOMINAL["hbm_gbs"]),
         "algorithmic": algorithmic, "ms_per_launch": ms["mean"], "ms_per_launch_median": ms["median"],
         "ms_per_launch_best": ms["best"]}
    if bound == "tensor" and peaks.get("bf16_tflops_sustained"):
        r["frac_of_sustained"] = achieved / peaks["bf16_tflops_sustained"]
    key = {"attn_umma_kernel": "attn", "attn_split_kernel": "attn", "lm_head_umma_kernel": "lm_head", "lm_head_duo_kernel": "lm_head",
           "residual_sample_kernel": "residual"}[kernel]
    ratio = NCU_TRAFFIC_RATIO.get((key, family))
    r["traffic"] = None if (ratio is None or bound == "tensor") else ratio * algorithmic
    return r


def measure(mv, cfg, dev, K, W, attn_kernel, peaks, peak_src, world, sampler=None, want_e2e=False, want_tvd=False):
    """Generate one workload and time it: K steps bracketed by events on the launching stream, the L2
    flushed between steps; at least MIN_SPLIT_STEPS of them also carry the events that separate the
    three calls, and as many others the events the library records around its dominant kernels (kept
    apart: an event between two kernels of a call keeps them from overlapping and costs a few us)."""
    import torch
    from workloads import generate, kv_bytes
    from paper_2505_10526_b200.binding import TIMED_ATTN, TIMED_LM_HEAD, TIMED_RESIDUAL
    from paper_2505_10526_b200.replicas import aggregate_throughput, barrier
    from paper_2505_10526_b200.step import STEP_INPUTS

    w = generate(cfg, device=dev)
    step = mv.VerifyStep.for_workload(cfg, w, attn_kernel=attn_kernel, want_logits=want_tvd and cfg.temperature > 0)
    seq0 = w["seq_lens"].clone()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    sampling = cfg.temperature > 0
    n_ev = 10 if sampling else 8

    PLAIN, CALLS, KERNELS = 0, 1, 2

    def one_step(ev=None, split=PLAIN):
        if ev:
            ev[0].record(stream)
        if split == KERNELS:
            mv.massv_set_kernel_timing(TIMED_LM_HEAD, (ev[4], ev[5]))
            mv.massv_set_kernel_timing(TIMED_ATTN, (ev[6], ev[7]))
            if sampling:
                mv.massv_set_kernel_timing(TIMED_RESIDUAL, (ev[8], ev[9]))
        step.attn(w)
        if split == CALLS:
            ev[1].record(stream)
        step.accept(w)
        if split == CALLS:
            ev[2].record(stream)
        if split == KERNELS:
            for k in (TIMED_LM_HEAD, TIMED_ATTN, TIMED_RESIDUAL):
                mv.massv_set_kernel_timing(k, None)
        step.commit(w["seq_lens"])
        if ev:
            ev[3].record(stream)

    def between_steps():
        w["seq_lens"].copy_(seq0)          # undo the commit so every step does identical work
        flush.fill_(1)                     # evict L2 (126 MB) between timed steps

    def new_events(n):
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
        for e in evs[4:]:                  # torch creates CUDA events lazily: the library needs their handles
            e.record(stream)
        return evs

    warm_ev = {}
    for kind in (CALLS, KERNELS):                      # the first instrumented steps belong to the warm-up
        warm_ev[kind] = new_events(n_ev)
        one_step(warm_ev[kind], split=kind)
        between_steps()
    for _ in range(max(W, 3)):
        one_step()
        between_steps()
    torch.cuda.synchronize()
    assert int(step.dev_status.item()) == 0, "device-side error during warm-up"

    # every `period`-th step separates the calls, the step after it times the kernels, the rest are plain
    period = max(2, K // MIN_SPLIT_STEPS)
    is_split = [CALLS if i % period == 0 else KERNELS if i % period == 1 else PLAIN for i in range(K)]
    events = [new_events(n_ev if is_split[i] == KERNELS else 4) for i in range(K)]
    launches0 = mv.massv_launch_count()
    barrier()
    torch.cuda.synchronize()
    if sampler:
        sampler.mark()
    wall0 = time.perf_counter()
    for i in range(K):
        one_step(events[i], split=is_split[i])
        between_steps()
    torch.cuda.synchronize()
    wall = time.perf_counter() - wall0
    if sampler:
        sampler.mark()
    barrier()
    launches = mv.massv_launch_count() - launches0
    assert int(step.dev_status.item()) == 0, "device-side error during the timed region"

    per_step = [e[0].elapsed_time(e[3]) for e in events]
    # (a run of a single step has no step of the other kind: the warm-up's stands in)
    sp = [e for e, s in zip(events, is_split) if s == CALLS] or [warm_ev[CALLS]]
    spk = [e for e, s in zip(events, is_split) if s == KERNELS] or [warm_ev[KERNELS]]
    t_attn = _stats([e[0].elapsed_time(e[1]) for e in sp])
    t_accept = _stats([e[1].elapsed_time(e[2]) for e in sp])
    t_commit = _stats([e[2].elapsed_time(e[3]) for e in sp])
    t_lm = _stats([e[4].elapsed_time(e[5]) for e in spk])
    t_attn_k = _stats([e[6].elapsed_time(e[7]) for e in spk])
    t_res = _stats([e[8].elapsed_time(e[9]) for e in spk]) if sampling else None
    st = _stats(per_step)
    ms_per_step, value = aggregate_throughput(cfg.m, st["mean"], dev)

    family = "gemma" if cfg.head_dim == 256 else "qwen"
    lm_bytes = cfg.vocab * cfg.hidden * 2 + cfg.m * cfg.hidden * 2
    lm_flops = 2.0 * cfg.m * cfg.vocab * cfg.hidden
    attn_bytes = kv_bytes(cfg, seq0.tolist())
    ridge = peaks["bf16_tflops"] * 1e12 / (peaks["hbm_gbs"] * 1e9)
    attn_name = "attn_umma_kernel" if (attn_kernel == 2 or (attn_kernel == 0 and cfg.head_dim <= 128)) else "attn_split_kernel"
    rl = {"attn": roofline_block(attn_name, "hbm", attn_bytes, t_attn_k, peaks, peak_src, family),
          # 257 .. 384 token rows take the one-pass kernel (two sub-tiles of the rows in tensor memory at once)
          "lm_head": roofline_block("lm_head_duo_kernel" if 256 < cfg.m <= 384 else "lm_head_umma_kernel", "tensor" if cfg.m > ridge else "hbm",
                                    lm_flops if cfg.m > ridge else lm_bytes, t_lm, peaks, peak_src, family)}
    rl["attn"]["frac_whole_call"] = attn_bytes / (t_attn["mean"] * 1e-3) / 1e9 / peaks["hbm_gbs"]
    rl["lm_head"]["frac_whole_accept_call"] = rl["lm_head"]["algorithmic"] / (t_accept["mean"] * 1e-3) / \
        (1e12 if cfg.m > ridge else 1e9) / rl["lm_head"]["peak"]
    if sampling:
        rl["residual"] = roofline_block("residual_sample_kernel", "hbm", cfg.batch * cfg.vocab * 8, t_res, peaks, peak_src, family)
    shares = {"attn": t_attn_k["mean"], "lm_head": t_lm["mean"]}
    if sampling:
        shares["residual"] = t_res["mean"]
    dominant = max(shares, key=shares.get)

    entry = {
        "workload": cfg.name, "value": value, "unit": UNIT, "ms_per_step": ms_per_step,
        "ms_per_step_median": st["median"], "ms_per_step_best": st["best"], "steps": K,
        "breakdown_ms": {"verify_attn": t_attn["mean"], "accept": t_accept["mean"], "kv_commit": t_commit["mean"],
                         "lm_head_kernel": t_lm["mean"], "attn_kernel": t_attn_k["mean"],
                         "residual_kernel": t_res["mean"] if sampling else None,
                         "split_steps": len(sp), "kernel_steps": len(spk),
                         "note": "calls: means over the timed steps with an event between the calls; kernels: means over other "
                                 "steps, in which the library records events around the kernel (no overlap with its neighbours)"},
        "rooflines": rl, "dominant": dominant, "share_of_step": {k: v / st["mean"] for k, v in shares.items()},
        "mean_accept_len": float(step.accept_len.float().mean()), "gpu_launches": int(launches),
        "wall_s_timed_region": wall, "mean_context": float(seq0.float().mean()),
    }

    if want_tvd and sampling and cfg.gamma >= 1:
        # the paper's distribution-alignment diagnostic (Eq. 6) on the logits the step just wrote, with the row
        # statistics the acceptance call left in its workspace (one read of the logits)
        ws = mv.alloc_workspace(mv.massv_tvd_workspace_size(step.cdesc), dev)
        tvd = torch.empty((cfg.batch, cfg.gamma), dtype=torch.float32, device=dev)
        acc = torch.empty_like(tvd)
        times = []
        for i in range(3 + 10):
            flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            mv.massv_tvd_after_accept(step.cdesc, step.logits, w["draft_probs"], step.accept_ws, tvd, acc, ws, step.dev_status)
            b.record(stream)
            torch.cuda.synchronize()
            if i >= 3:
                times.append(a.elapsed_time(b))
        ts = _stats(times)
        alg = cfg.batch * cfg.gamma * cfg.vocab * 8
        entry["tvd"] = {"ms_per_call": ts["mean"], "ms_per_call_median": ts["median"], "ms_per_call_best": ts["best"],
                        "algorithmic": alg, "achieved": alg / (ts["mean"] * 1e-3) / 1e9, "unit": "GB/s",
                        "frac": alg / (ts["mean"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
                        "mean_tvd": float(tvd.mean()), "mean_accept_prob": float(acc.mean())}

    if want_e2e:
        # ---- end to end: per-step inputs start in pinned host memory, results end there
        def e2e_run(keys):
            host = step.host_inputs_like({k: w[k].cpu() for k in keys})
            resident = {k: v for k, v in w.items() if k not in keys}
            for _ in range(3):
                step.run_host(host, resident, commit=True)
                between_steps()
            torch.cuda.synchronize()
            Ke = max(10, min(K, 50))
            ts = []
            for _ in range(Ke):
                t0 = time.perf_counter()
                step.run_host(host, resident, commit=True)
                ts.append((time.perf_counter() - t0) * 1e3)
                between_steps()
                torch.cuda.synchronize()
            s = _stats(ts)
            ms, val = aggregate_throughput(cfg.m, s["mean"], dev)
            h2d, d2h = step.host_bytes_per_step(host)
            del host
            return {"value": val, "unit": UNIT, "ms_per_step": ms, "ms_per_step_median": s["median"],
                    "ms_per_step_best": s["best"], "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": Ke}
        all_keys = [k for k in STEP_INPUTS if k in w and (sampling or k not in ("draft_probs", "u_accept", "u_sample"))]
        entry["e2e"] = e2e_run(all_keys)
        entry["e2e"]["inputs_from_host"] = all_keys
        # a drafter on the same GPU leaves its tokens, distributions and the uniforms on the device:
        # only the target's own per-step tensors come from the host
        own = ["q", "k_new", "v_new", "hidden"]
        entry["e2e_q_resident"] = e2e_run(own)
        entry["e2e_q_resident"]["inputs_from_host"] = own
    entry["_handles"] = (w, step)       # the caller may still want the workload (CPU baseline)
    return entry


def run_sharded(args):
    """Kernel times of one rank of the vocabulary-sharded acceptance: all ranks of a world on ONE GPU in
    lockstep (no kernel waits on another rank's), rank 0's calls bracketed by events, L2 flushed.  The
    exchanges between the phases are not in these figures."""
    import torch
    import __graft_entry__ as entry
    entry.build()
    from paper_2505_10526_b200.sharded import ShardedAccept, run_lockstep
    from workloads import generate, get_config
    world = args.sharded_world
    cfg = get_config(args.config if args.config != DEFAULT_WORKLOAD else "qwen7b_b16_t1")
    if cfg.vocab % world:
        raise SystemExit("the vocabulary must divide evenly among the ranks")
    w = generate(cfg, device="cuda", with_attention=False)
    Vs = cfg.vocab // world
    ranks = [ShardedAccept(cfg.batch, cfg.gamma, cfg.hidden, Vs, cfg.temperature, world, r) for r in range(world)]
    inputs = []
    for r in range(world):
        kw = dict(hidden=w["hidden"], lm_head_shard=w["lm_head"][r * Vs:(r + 1) * Vs].contiguous(),
                  draft_tokens=w["draft_tokens"])
        if cfg.temperature > 0:
            kw.update(draft_probs_shard=w["draft_probs"][:, :, r * Vs:(r + 1) * Vs].contiguous(),
                      u_accept=w["u_accept"], u_sample=w["u_sample"])
        inputs.append(kw)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    spans = {}
    W, K = max(args.warmup, 3), min(args.steps, 50)
    for it in range(W + K):
        flush.zero_()
        ranks[0].marks = [] if it >= W else None
        res = run_lockstep(ranks, inputs, transport="publish")
        torch.cuda.synchronize()
        for t, l in res[1:]:
            assert torch.equal(t, res[0][0]) and torch.equal(l, res[0][1]), "ranks disagree"
        if ranks[0].marks:
            ev = dict(ranks[0].marks)
            for name in ("lm_head", "scan", "pick", "set_token"):
                if name + ":start" in ev:
                    spans.setdefault(name, []).append(ev[name + ":start"].elapsed_time(ev[name + ":stop"]))
    assert all(int(r.dev_status.item()) == 0 for r in ranks)
    med = {k: round(statistics.median(v), 4) for k, v in spans.items()}
    r0 = ranks[0]
    print(json.dumps({"metric": "kernel time of one vocabulary shard's acceptance calls", "unit": "ms", "n_gpus": 1,
                      "steps": K, "warmup": W, "data": "synthetic", "dtype": "bf16",
                      "config": {"workload": cfg.name, "world": world, "shard_vocab": Vs, "transport": "publish",
                                 "l2": "flushed between steps"},
                      "rank0_kernel_ms": med, "rank0_kernel_ms_total": round(sum(med.values()), 4),
                      "exchange_bytes_per_rank": {"stats": r0.stats.numel() * 4, "masses": r0.masses.numel() * 8,
                                                  "token": r0.token.numel() * 4},
                      "mean_accept_len": float(res[0][1].float().mean())}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", default=DEFAULT_WORKLOAD)
    ap.add_argument("--impl", default="massv", choices=["massv", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="time the --config workload only")
    ap.add_argument("--sweep-steps", type=int, default=0, help="timed steps per sweep entry (default: min(steps, 30))")
    ap.add_argument("--attn-kernel", type=int, default=0, choices=[0, 1, 2],
                    help="attention split kernel: 0 = chosen by shape, 1 = warp-level MMA, 2 = tcgen05")
    ap.add_argument("--sharded-world", type=int, default=0,
                    help="instead of the verify step, time one rank's calls of the vocabulary-sharded acceptance")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.sharded_world:
        run_sharded(args)
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
    from workloads import get_config

    peaks, peak_src = load_peaks()
    uuid = None
    try:
        uuid = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        pass
    sampler = ClockSampler(local_rank, uuid)
    sampler.start()                        # before the warm-up, so that a timed region of milliseconds still gets samples

    cfg = get_config(args.config)
    K, W = args.steps, max(args.warmup, 3)
    main_e = measure(mv, cfg, dev, K, W, args.attn_kernel, peaks, peak_src, world, sampler=sampler, want_e2e=True,
                     want_tvd=True)
    clocks = sampler.stop()
    w, step = main_e.pop("_handles")

    sweep = []
    if not args.no_sweep and world == 1 and args.config == DEFAULT_WORKLOAD:
        cpu_w = None
        if not args.no_cpu_baseline:
            cpu_w = bounded_cpu_workload(cfg, w)       # host copy before the device memory is handed back
        del w, step
        torch.cuda.empty_cache()
        Ks = args.sweep_steps or min(K, 30)
        for name in SWEEP:
            e = measure(mv, get_config(name), dev, Ks, W, args.attn_kernel, peaks, peak_src, world,
                        want_tvd=(name == "qwen7b_long_g7_t1"))
            e.pop("_handles")
            torch.cuda.empty_cache()
            sweep.append(e)
    else:
        cpu_w = None if (args.no_cpu_baseline or world > 1) else bounded_cpu_workload(cfg, w)
        del w, step

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    dom = main_e["dominant"]
    roofline = dict(main_e["rooflines"][dom])
    roofline["share_of_step"] = main_e["share_of_step"][dom]
    line = {
        "metric": METRIC, "value": main_e["value"], "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": main_e["ms_per_step"], "ms_per_step_median": main_e["ms_per_step_median"],
        "ms_per_step_best": main_e["ms_per_step_best"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": config_block(cfg, main_e["mean_context"], args.attn_kernel, world),
        "breakdown_ms": main_e["breakdown_ms"], "mean_accept_len": main_e["mean_accept_len"],
        "roofline": roofline, "rooflines": main_e["rooflines"], "clocks": clocks,
        "e2e": main_e["e2e"], "e2e_q_resident": main_e["e2e_q_resident"],
        "gpu_launches": main_e["gpu_launches"], "wall_s_timed_region": main_e["wall_s_timed_region"],
    }
    if "tvd" in main_e:
        line["tvd"] = main_e["tvd"]
    if cpu_w is not None:
        sub_cfg, w_cpu, keep = cpu_w
        v, t, reps, cores = time_oracle(sub_cfg, w_cpu)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"first {keep} of {cfg.batch} sequences of {cfg.name}, whole verify step, best of {reps} ({t:.2f} s)"}
    if sweep:
        line["sweep"] = sweep
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
