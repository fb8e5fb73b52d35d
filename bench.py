#!/usr/bin/env python
"""Benchmark of the BAOC hot path on B200.

One "step" is one pass of the whole per-step path over one batch of synthetic
gradients: the statistics pass (streaming kernel + combine) followed by the
fused mixed-configuration optimizer step under an assignment that the library
itself produced (short sampling window -> finalize -> risk -> budgeted
allocation).  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama_1b] [--impl ours|reference]

``--impl reference`` times the CPU oracle (a deliberately plain double-precision
program) on a bounded sample of the same workload, on the host cores.
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

CONFIG_NAMES = ["adamw32", "adamw8", "rms", "factored", "sgdm"]
EXTENDED_NAMES = CONFIG_NAMES + ["sgd", "adamw16", "rms16", "sgdm16", "rms8", "sgdm8", "factored16", "factored8",
                                 "adamw8_dynamic", "adafactor"]
METRIC = "hot-path throughput: statistics pass + mixed-config optimizer step"
UNIT = "params/s"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


def _ncu_traffic(kernel, algorithmic_bytes):
    """DRAM bytes per launch of `kernel`, scaled from the recorded ncu capture of a smaller case by the algorithmic
    bytes of this launch (traffic is proportional to the parameters processed).  None when there is no record or
    the kernel sources have changed since the counters were taken."""
    import hashlib
    pkg = os.path.join(ROOT, "paper_2605_04711_b200")
    try:
        rec = json.load(open(os.path.join(pkg, "ncu_traffic.json")))
        h = hashlib.sha256()
        for name in rec["kernel_sources"]:               # the files that define the two kernels and what they include
            h.update(name.encode())
            h.update(open(os.path.join(pkg, "csrc", name), "rb").read())
        if h.hexdigest() != rec["kernel_sources_sha256"] or kernel not in rec:
            return None
        k = rec[kernel]
        return float(k["dram_bytes"]) / float(k["algorithmic_bytes"]) * float(algorithmic_bytes)
    except Exception:
        return None


class ClockSampler(threading.Thread):
    """Samples SM clocks and clock-event (throttle) reasons while the timed region runs: NVML in-process every
    10 ms where the module loads, else the nvidia-smi query every 200 ms.  Read-only."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    REASON_BITS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20),
                   ("sw_power_cap", 0x4))

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index = index
        self.sm, self.reasons, self.sm_max, self.power = [], set(), None, []
        self._halt = threading.Event()
        self._nvml = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._dev = pynvml.nvmlDeviceGetHandleByIndex(self._physical_index(index))
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(self._dev, pynvml.NVML_CLOCK_SM))
            self._nvml = pynvml
        except Exception:
            self._nvml = None

    @staticmethod
    def _physical_index(local: int) -> int:
        vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
        ids = [x for x in vis.split(",") if x.strip() != ""]
        if local < len(ids) and ids[local].strip().isdigit():
            return int(ids[local])
        return local

    def _sample_nvml(self):
        n = self._nvml
        self.sm.append(float(n.nvmlDeviceGetClockInfo(self._dev, n.NVML_CLOCK_SM)))
        try:
            bits = int(n.nvmlDeviceGetCurrentClocksEventReasons(self._dev))
        except Exception:
            bits = int(n.nvmlDeviceGetCurrentClocksThrottleReasons(self._dev))
        for name, bit in self.REASON_BITS:
            if bits & bit:
                self.reasons.add(name)
        try:
            self.power.append(n.nvmlDeviceGetPowerUsage(self._dev) / 1000.0)
        except Exception:
            pass

    def _sample_smi(self):
        out = subprocess.run(["nvidia-smi", f"--id={self._physical_index(self.index)}", f"--query-gpu={self.FIELDS}",
                              "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=5).stdout
        parts = [x.strip() for x in out.strip().split(",")]
        if len(parts) >= 7:
            self.sm.append(float(parts[0]))
            self.sm_max = float(parts[1])
            self.power.append(float(parts[2]))
            for k, (name, _) in enumerate(self.REASON_BITS):
                if parts[3 + k].lower().startswith("active"):
                    self.reasons.add(name)

    def run(self):
        while not self._halt.is_set():
            try:
                if self._nvml is not None:
                    self._sample_nvml()
                else:
                    self._sample_smi()
            except Exception:
                pass
            self._halt.wait(0.01 if self._nvml is not None else 0.2)

    def stop(self):
        self._halt.set()
        self.join(timeout=6)

    def summary(self):
        if not self.sm:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": ["no samples"], "samples": 0}
        return {"sm_mhz": statistics.median(self.sm), "sm_min_mhz": min(self.sm), "sm_max_mhz": self.sm_max,
                "reasons": sorted(self.reasons), "samples": len(self.sm),
                "power_w_max": max(self.power) if self.power else None,
                "source": "nvml" if self._nvml is not None else "nvidia-smi"}


# ----------------------------------------------------------------------------
# CPU oracle timing (the reference arm and the cpu_baseline leg)
# ----------------------------------------------------------------------------

def _sample_blocks(wl, target_params, slice_rows=False):
    """A bounded sample of the workload: blocks in order until the target is met.  Without slicing, blocks larger than
    the target are skipped; with slicing, a matrix larger than a quarter of the target is cut to its first rows (whole
    rows, so it stays a matrix and every path, the factored one included, can run on it).  Returns
    ([(block index, rows, cols)], parameters)."""
    picked, total = [], 0
    cap = max(1, target_params // 4)
    for i, b in enumerate(wl.blocks):
        rows, cols = b.rows, b.cols
        if slice_rows and b.numel > cap:
            rows = max(1, cap // cols) if cols > 1 else cap
        elif b.numel > target_params:
            continue
        picked.append((i, rows, cols))
        total += rows * cols
        if total >= target_params:
            break
    return picked, total


def time_oracle(wl, assign, steps, warmup, target_params, configs=None, slice_rows=False):
    """Time the oracle's statistics step + optimizer step on a sample of blocks.  Returns (params/s, info).
    configs: the candidate tuples ``assign`` indexes (the binding's structs); default: the oracle's five.
    assign None: the sampled blocks take the candidates in turn (vectors skip the factored one)."""
    import numpy as np
    from threadpoolctl import threadpool_limits
    from oracle import baoc_oracle as O
    from paper_2605_04711_b200 import workloads as W

    if configs is None:
        cfgs = O.default_configs()
        # same hyper-parameter values as the library's fp32 fields
        for c in cfgs:
            for k in ("lr", "beta1", "beta2", "eps", "weight_decay"):
                setattr(c, k, float(np.float32(getattr(c, k))))
    else:
        cfgs = [O.Config(c.adaptive, c.momentum, c.decoupled_wd, c.factored, c.bits, lr=float(c.lr), beta1=float(c.beta1),
                         beta2=float(c.beta2), eps=float(c.eps), weight_decay=float(c.weight_decay),
                         quantizer="dynamic" if c.quantizer else "linear", af_beta2_schedule=bool(c.af_flags & 1),
                         af_clip=1.0 if c.af_flags & 2 else 0.0, af_relative_step=bool(c.af_flags & 4),
                         af_eps1=1e-30 if c.af_flags & 8 else 0.0) for c in configs]
    picked, total = _sample_blocks(wl, target_params, slice_rows)
    opts = O.Opts()
    kinds = []
    with threadpool_limits(limits=1):
        grads = [[W.block_grad(wl, i, t).double().numpy()[:r * c] for i, r, c in picked] for t in (1, 2)]
        theta = [W.block_param(wl, i).double().numpy()[:r * c] for i, r, c in picked]
        sstates = [O.stats_init(r * c) for _, r, c in picked]
        ostates = []
        for j, (i, r, c_) in enumerate(picked):
            c = int(assign[i]) if assign is not None else (j % len(cfgs))
            if cfgs[c].factored and c_ <= 1:
                c = 2
            ostates.append((c, O.step_init(cfgs[c], r * c_, r, c_)))
            kinds.append(O.config_kind(cfgs[c]))
        times = []
        for s in range(warmup + steps):
            t0 = time.perf_counter()
            for j, (i, r, c_) in enumerate(picked):
                g = grads[s % 2][j]
                O.stats_step(sstates[j], g, opts)
                c, st = ostates[j]
                theta[j] = O.step(theta[j], g, st, cfgs[c], r, c_)
            dt = time.perf_counter() - t0
            if s >= warmup:
                times.append(dt)
    sec = sum(times) / len(times)
    sliced = sum(1 for i, r, c in picked if r * c < wl.blocks[i].numel)
    info = {"kind": "oracle", "cores": 1, "unit": UNIT, "value": total / sec,
            "sample": f"{len(picked)} blocks / {total} params of {wl.name} (blocks in order up to {target_params} params"
                      + (f", {sliced} matrices cut to their first rows" if slice_rows else ", larger blocks skipped")
                      + f"; update paths {'/'.join(sorted(set(kinds)))}), one statistics step + one optimizer step per timed step, "
                      f"{len(times)} timed steps, numpy float64, 1 thread",
            "ms_per_step": sec * 1e3}
    return total / sec, info


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2605_04711_b200 import workloads as W
    wl = W.make_workload(args.workload, seed=0)
    # size the sample so that warmup + steps stay within a few minutes on one core (the oracle does about 3e7 parameters
    # per second); large matrices are cut to their first rows so that the sample holds matrices and every update path
    target = max(1 << 20, int(6.0e8 / max(args.steps + args.warmup, 1)))
    value, info = time_oracle(wl, None, args.steps, args.warmup, target, slice_rows=True)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": info["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "sample": info["sample"]},
            "cpu_baseline": {k: info[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------
# The CUDA arm
# ----------------------------------------------------------------------------

def run_ours(args):
    import numpy as np
    import torch

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    from paper_2605_04711_b200 import build
    build.build()
    from paper_2605_04711_b200 import harness, workloads as W

    sharded = bool(args.shard_blocks and world > 1)
    cap = 0
    if sharded:
        # strong scaling: whole blocks are dealt to the ranks (balanced by fp32-Adam step bytes).  The statistics and
        # the update need no collective; replicas hold full weights, so every step ends with an all-gather of the
        # updated parameters (each rank's flat buffer, allocated at the longest shard's length)
        wl = W.make_workload(args.workload, seed=0)
        part = harness.partition_blocks([26.0 * b.numel for b in wl.blocks], world)[rank]
        wl.blocks = [wl.blocks[i] for i in part]
        cap = int(harness.max_over_ranks(W.flat_layout(wl, 128)[1], dist, f"cuda:{local}"))
    else:
        wl = W.make_workload(args.workload, seed=rank)       # replicas: every rank streams its own copy of the workload
    from paper_2605_04711_b200 import binding
    extended = args.candidates == "extended" or args.assign in EXTENDED_NAMES[5:]
    names = EXTENDED_NAMES if extended else CONFIG_NAMES
    # optional: the statistics see a seeded sub-grid of every block (the paper's sparse coordinate sampling)
    samples = W.sample_subgrids(wl, args.sample_frac) if args.sample_frac < 1.0 else None
    sess = harness.Session(wl, configs=binding.extended_configs() if extended else None, n_grad_sets=2,
                           device=f"cuda:{local}", pinned_host_grads=True, samples=samples, param_capacity=cap,
                           factored_group_bytes=int(args.factored_group_mb * 2 ** 20))
    gathered = torch.empty(world * cap, dtype=torch.float32, device=f"cuda:{local}") if sharded else None
    # after a sharded step: all ranks receive all updated parameters
    exchange = (lambda: harness.all_gather_params(sess.params, gathered, dist)) if sharded else (lambda: None)
    sess.init_params()
    for t in (1, 2):
        k = sess.fill_grads(t)
        sess.host_copy_of_grads(k)
    sess._fixed_cache.clear()
    torch.cuda.synchronize()

    # short sampling window -> risk -> allocation -> configure (set-up, timed separately)
    ev = lambda: torch.cuda.Event(enable_timing=True)
    for t in range(1, args.window + 1):
        sess.sample_stats(t % 2)
    sess.h.risk(sess.param_table, as_dicts=False)                    # untimed: the first call also loads the finalize kernels
    e0, e1 = ev(), ev()
    e0.record()
    risk, stats = sess.h.risk(sess.param_table, as_dicts=False)      # the C call alone: it returns after its own copy back
    e1.record()
    torch.cuda.synchronize()
    finalize_ms = e0.elapsed_time(e1)
    stats = [s.as_dict() for s in stats]
    t0 = time.perf_counter()
    assign, objective, rc = sess.allocate(risk)
    alloc_ms = (time.perf_counter() - t0) * 1e3
    if args.assign != "auto":
        # one configuration for every block (vectors cannot be factored: they take the momentum-free one of the same width)
        c = names.index(args.assign)
        vec = {"factored": "rms", "factored16": "rms16", "factored8": "rms8", "adafactor": "rms"}
        assign = np.asarray([names.index(vec[args.assign]) if (args.assign in vec and b.cols <= 1) else c for b in wl.blocks],
                            np.int32)
    sess.configure(assign)
    info = sess.h.query()
    stats_bytes, step_bytes = info.stats_bytes_per_call, info.step_bytes_per_call
    counts = np.bincount(assign, minlength=len(sess.configs)).tolist()
    params_by_cfg = [int(sum(b.numel for b, a in zip(wl.blocks, assign) if a == c)) for c in range(len(sess.configs))]

    def one_step(s, t):
        sess.sample_stats(s % 2)
        sess.step(s % 2, t)
        exchange()

    step_t = 0
    for s in range(args.warmup):
        step_t += 1
        one_step(s, step_t)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
        torch.cuda.synchronize()

    # L2: a step of the large workloads streams many times the 126 MB of L2; a workload whose step moves less than
    # 1 GB gets L2 flushed (a 256 MB buffer overwritten) before every timed step, outside the timed intervals
    flush_l2 = (stats_bytes + step_bytes) < (1 << 30)
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=f"cuda:{local}") if flush_l2 else None
    launches0 = sess.h.query().kernel_launches
    sampler = ClockSampler(local)
    sampler.start()
    marks = [(ev(), ev(), ev()) for _ in range(args.steps)]
    for s in range(args.steps):
        step_t += 1
        if flush_l2:
            flush_buf.fill_(s & 0xff)
        a, b, c = marks[s]
        a.record()
        sess.sample_stats(s % 2)
        b.record()
        sess.step(s % 2, step_t)
        exchange()
        c.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
        torch.cuda.synchronize()
    sampler.stop()
    launches = sess.h.query().kernel_launches - launches0

    # the K steps run back to back on one stream; with the L2 flush in between only the steps themselves are counted
    total_ms = (sum(a.elapsed_time(c) for a, b, c in marks) if flush_l2 else marks[0][0].elapsed_time(marks[-1][2]))
    stats_ms = sum(a.elapsed_time(b) for a, b, c in marks) / args.steps
    step_ms = sum(b.elapsed_time(c) for a, b, c in marks) / args.steps
    dev = f"cuda:{local}"
    total_ms_max = harness.max_over_ranks(total_ms, dist, dev)
    ms_per_step = total_ms_max / args.steps
    all_params = harness.sum_over_ranks(wl.numel, dist, dev)      # parameters all ranks processed per step
    value = all_params / (ms_per_step * 1e-3)
    cnt, _ = sess.h.nonfinite()

    # per-kernel split of the step (events inside the library around the row/column kernels and the fused kernel), on a
    # few more steps; the same loop also brackets the whole baoc_step call, so parts and whole come from one loop.  The
    # loop reads its events back after every step (a host synchronisation), which the main timed loop does not have.
    sess.h.profile(True)
    red_ms, fused_ms, whole_ms = [], [], []
    for s in range(min(args.steps, 20)):
        step_t += 1
        sess.sample_stats(s % 2)
        w0, w1 = ev(), ev()
        w0.record()
        sess.step(s % 2, step_t)
        w1.record()
        a, b = sess.h.profile_last()
        torch.cuda.synchronize()
        red_ms.append(a)
        fused_ms.append(b)
        whole_ms.append(w0.elapsed_time(w1))
    sess.h.profile(False)
    red_ms, fused_ms = sum(red_ms) / len(red_ms), sum(fused_ms) / len(fused_ms)
    parts_whole_ms = sum(whole_ms) / len(whole_ms)

    # end to end: gradients start in pinned host memory, the per-block running statistics come back
    e2e_steps = max(1, min(args.e2e_steps, args.steps))
    d2h = 0
    torch.cuda.synchronize()
    ea, eb = ev(), ev()
    ea.record()
    for s in range(e2e_steps):
        step_t += 1
        sess.step_from_host(s % 2, True, step_t)
        exchange()
        running = sess.h.read_stats()
    eb.record()
    torch.cuda.synchronize()
    e2e_ms = ea.elapsed_time(eb) / e2e_steps
    e2e_ms = harness.max_over_ranks(e2e_ms, dist, dev)
    d2h = 8 * 8 * len(wl.blocks)
    h2d = 2 * wl.numel

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_kind = _peaks()
    stats_gbs = stats_bytes / (stats_ms * 1e-3) / 1e9
    step_gbs = step_bytes / (step_ms * 1e-3) / 1e9
    # the dominant kernel of the step gets the `roofline` object, the other one `roofline_other`
    n_factored = sum(n for n, c in zip(params_by_cfg, sess.configs) if c.factored)   # at any precision of their statistics
    # the library counts what it moves: 12 B per factored parameter (the gradient is read by the row/column reduction and
    # again by the update); the method itself needs 10 B (one read), which is also what the fused kernel alone moves
    algo_step_bytes = step_bytes - 2 * n_factored
    fused_bytes = algo_step_bytes
    fused_gbs = fused_bytes / (fused_ms * 1e-3) / 1e9
    algo_step_gbs = algo_step_bytes / (step_ms * 1e-3) / 1e9
    peak_note = peak_kind + " (burst copy, read + write; a read-dominated kernel can exceed it: the nominal 8 TB/s is the ceiling)"
    r_stats = {"kernel": "stats_step_kernel", "bound": "hbm", "achieved": stats_gbs, "peak": peak, "unit": "GB/s",
               "frac": stats_gbs / peak, "peak_kind": peak_note, "frac_of_8TBs": stats_gbs / 8000.0,
               "bytes_per_launch": int(stats_bytes), "ms": stats_ms,
               "bytes_per_param": 22 if samples is None else "26 per sampled coordinate",
               "timed": "events around baoc_sample_stats (includes its ~25 us combine kernel)",
               "traffic": args.traffic_stats if args.traffic_stats is not None else (_ncu_traffic("stats_step_kernel", stats_bytes) if samples is None else None)}
    r_fused = {"kernel": "fused_step_kernel", "bound": "hbm", "achieved": fused_gbs, "peak": peak, "unit": "GB/s",
               "frac": fused_gbs / peak, "peak_kind": peak_note, "frac_of_8TBs": fused_gbs / 8000.0,
               "bytes_per_launch": int(fused_bytes), "ms": fused_ms,
               "timed": "events inside baoc_step around the fused kernel alone, in the parts loop (see parts_loop)",
               "parts_loop": {"steps": len(whole_ms), "whole_step_ms": parts_whole_ms, "row_col_kernels_ms": red_ms,
                              "fused_kernel_ms": fused_ms,
                              "note": "one loop with a host synchronisation after every step; the main timed loop has none"},
               "whole_step": {"ms": step_ms, "timed": "events around baoc_step in the main timed loop",
                              "bytes_moved": int(step_bytes), "GBps_moved": step_gbs, "frac_moved": step_gbs / peak,
                              "bytes_algorithmic": int(algo_step_bytes), "GBps_algorithmic": algo_step_gbs,
                              "frac_algorithmic": algo_step_gbs / peak, "frac_algorithmic_of_8TBs": algo_step_gbs / 8000.0,
                              "note": "moved counts the factored blocks' gradient twice (12 B/param: row/column reduction, then "
                                      "update); algorithmic counts it once (10 B/param)"},
               "traffic": args.traffic_step if args.traffic_step is not None else _ncu_traffic("fused_step_kernel", fused_bytes)}
    roofline, other = (r_fused, r_stats) if fused_ms >= stats_ms else (r_stats, r_fused)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong" if sharded else "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.workload, "params": wl.numel, "blocks": len(wl.blocks), "grad_dtype": "bf16",
                   "param_dtype": "f32", "candidate_configs": names, "assignment": args.assign,
                   "assignment_blocks_per_config": counts, "assignment_params_per_config": params_by_cfg,
                   "mem_budget_frac_of_fp32_adam": wl.mem_budget_frac, "state_bytes": int(info.state_bytes),
                   "window_steps_before_timing": args.window, "stats_sample_frac": args.sample_frac, "factored_group_mb": args.factored_group_mb, "l2": ("flushed before every timed step (a 256 MB buffer overwritten, outside the timed intervals)" if flush_l2 else
                          f"inputs ({(stats_bytes + step_bytes) / 1e9:.1f} GB per step) far exceed the 126 MB L2"),
                   "parallelism": (f"whole blocks sharded over {world} GPUs; no collective in the statistics pass or the update; "
                                   f"NCCL all-gather of the updated parameters ({4 * cap} bytes per rank) inside the timed region"
                                   if sharded else f"replicas x{world}, no collective") if world > 1 else "single GPU",
                   "allocator_status": int(rc), "nonfinite_blocks": int(cnt)},
        "clocks": sampler.summary(),
        "gpu_launches": int(launches),
        "e2e": {"value": all_params / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                "d2h_bytes_per_step": int(d2h), "ms_per_step": e2e_ms, "steps": e2e_steps},
        "roofline": roofline,
        "roofline_other": other,
        "stats_pass": {"ms": stats_ms, "GBps": stats_gbs, "params_per_s": wl.numel / (stats_ms * 1e-3)},
        "mixed_step": {"ms": step_ms, "GBps": step_gbs, "GBps_algorithmic": algo_step_gbs, "params_per_s": wl.numel / (step_ms * 1e-3),
                       "includes_param_all_gather": sharded},
        "once_per_window": {"finalize_and_risk_ms": finalize_ms, "allocate_ms": alloc_ms, "objective": objective},
    }
    if world == 1 and not args.no_cpu_baseline:
        _, cb = time_oracle(wl, assign, 3, 1, args.cpu_sample_params, sess.configs)   # about 15 s of CPU work
        line["cpu_baseline"] = {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama_1b")
    ap.add_argument("--candidates", default="default", choices=["default", "extended"],
                    help="default: the five tuples of the headline path; extended: plus sgd and the bf16-state variants")
    ap.add_argument("--assign", default="auto", choices=["auto"] + EXTENDED_NAMES,
                    help="auto: the library's own budgeted allocation; else every block under that one configuration")
    ap.add_argument("--shard-blocks", action="store_true",
                    help="N > 1: deal whole blocks of ONE workload to the ranks (strong scaling) instead of one replica per rank")
    ap.add_argument("--sample-frac", type=float, default=1.0,
                    help="fraction of every block's coordinates the statistics see (1 = dense, the default; the paper's own "
                         "default is 0.001)")
    ap.add_argument("--factored-group-mb", type=float, default=0.0,
                    help="0: one row/column reduction and one update launch for all factored blocks; > 0: factored blocks in groups "
                         "of at most this many MiB of gradient, each reduced and updated back to back (second read from L2)")
    ap.add_argument("--window", type=int, default=4, help="statistics steps before the finalize that feeds the allocation")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-sample-params", type=int, default=100_000_000)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--traffic-stats", type=float, default=None, help="ncu DRAM bytes per launch of the statistics kernel, if known")
    ap.add_argument("--traffic-step", type=float, default=None)
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
