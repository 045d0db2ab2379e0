#!/usr/bin/env python
"""Benchmark of one decode step of parallel-sample shared-prefix attention on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg2] [--impl psa|reference]

A step = prefix + suffix + merge stages over one batch of seeded synthetic inputs (the shapes of
the paper's parallel-sampling set-up; nothing is read from disk).  Rank r works on its own
prompts (seed r): the path shards over independent prompts with no collective ("weak" scaling).
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import psa_workloads as wl  # noqa: E402

METRIC = "sample-tokens/sec per decode step"
UNIT = "sample-tokens/s"
L2_BYTES = 126e6
# DRAM bytes (read + write) per launch of the dominant kernel, from an ncu launch list of this very command
# (dram__bytes_read.sum + dram__bytes_write.sum).  Only valid for the kernel source it was taken with.
NCU_TRAFFIC = {"cfg2": {"kernel": "suffix_kernel", "bytes_per_launch": 68271539 + 18168,
                        "source": "paper_2502_02534_b200/csrc/suffix_sm100.cu", "sha256_16": "498b791d8050fd97"}}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def ncu_traffic(config_name):
    import hashlib
    t = NCU_TRAFFIC.get(config_name)
    if not t:
        return None
    try:
        with open(os.path.join(ROOT, t["source"]), "rb") as f:
            if hashlib.sha256(f.read()).hexdigest()[:16] != t["sha256_16"]:
                return None          # the kernel changed since the counters were taken
    except OSError:
        return None
    return t["bytes_per_launch"]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while work runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int, period_s: float = 0.005):
        self.samples, self.reason_bits, self.max_mhz = [], 0, None
        self._stop = threading.Event()
        self._thread = None
        self.period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _run(self):
        while not self._stop.is_set():
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
                self.reason_bits |= int(self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join()
        reasons = [name for bit, name in self.REASONS.items() if self.reason_bits & bit]
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": reasons, "samples": len(self.samples)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ---------------------------------------------------------------------------------------------- reference arm
def run_reference(args, cfg):
    """The CPU fp64 oracle as it stands, timed on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    w = wl.make_workload(cfg)
    B, Hq = int(np.sum(w["n_samples"])), w["num_q_heads"]
    n_rows = B * Hq
    t0 = time.perf_counter()
    oracle.attend(w)
    t_full = time.perf_counter() - t0
    budget = 150.0 / max(1, args.steps + args.warmup)
    if t_full <= budget:
        rows, sample = None, f"every row of {cfg.name} ({n_rows} rows) per step"
        rows_per_step = n_rows
    else:
        rows_per_step = max(Hq, int(n_rows * budget / t_full) // Hq * Hq)
        sel = np.random.default_rng(0).choice(B, rows_per_step // Hq, replace=False)
        rows = (np.sort(sel)[:, None] * Hq + np.arange(Hq)[None, :]).ravel()
        sample = f"{rows_per_step // Hq} of {B} samples of {cfg.name} (all {Hq} heads) per step"
    cores = 0
    for _ in range(args.warmup):
        oracle.attend(w, rows=rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        _, _, cores = oracle.attend(w, rows=rows)
    dt = (time.perf_counter() - t0) / max(1, args.steps)
    value = (rows_per_step / Hq) / dt
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": {"workload": cfg.name, "note": "CPU fp64 oracle on host cores"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------- psa arm
def run_psa(args, cfg):
    import torch
    import torch.distributed as dist
    import paper_2502_02534_b200 as psa
    from paper_2502_02534_b200.binding import host_staging_bytes

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- inputs: rank r samples its own prompts (seed r); several copies so no step finds its inputs in L2
    import dataclasses
    cfg_r = dataclasses.replace(cfg, seed=cfg.seed + rank)
    w = wl.make_workload(cfg_r)
    B, Hq, D = int(np.sum(w["n_samples"])), w["num_q_heads"], w["head_dim"]
    abytes, aflops = wl.algorithmic_bytes(w), wl.algorithmic_flops(w)
    input_bytes = sum(int(w[k].nbytes) for k in ("q", "prefix_k", "prefix_v", "pool_k", "pool_v"))
    n_copies = max(2, int(np.ceil(4 * L2_BYTES / input_bytes))) if input_bytes < 4 * L2_BYTES else 1

    def upload():
        d = {k: torch.from_numpy(np.ascontiguousarray(w[k]).view(np.int16)).cuda().view(torch.bfloat16)
             for k in ("q", "prefix_k", "prefix_v", "pool_k", "pool_v")}
        for k in ("page_indptr", "page_indices", "suffix_lens"):
            d[k] = torch.from_numpy(np.ascontiguousarray(w[k], dtype=np.int32)).cuda()
        return d

    copies = [upload() for _ in range(n_copies)]
    out = torch.empty((B, Hq, D), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((B, Hq), dtype=torch.float32, device="cuda")
    plan = psa.Plan(w["prefix_lens"], w["n_samples"], w["suffix_lens"], num_q_heads=Hq, num_kv_heads=w["num_kv_heads"],
                    head_dim=D, page_size=w["page_size"], sm_scale=w["sm_scale"], out_dtype="bf16")
    plan.bind_workspace()
    info = plan.info

    def step(i, stage="all"):
        d = copies[i % n_copies]
        psa.decode(plan, d["q"], d["prefix_k"], d["prefix_v"], d["pool_k"], d["pool_v"], d["page_indptr"],
                   d["page_indices"], d["suffix_lens"], out, lse, stage=stage)

    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()
    for i in range(max(3, n_copies)):        # first launches set kernel attributes; keep them out of any capture
        step(i)
    torch.cuda.synchronize()

    # ---- a decode step is launch-bound on the host (three tiny kernels), so the timed loop replays CUDA
    # graphs of several captured steps, as a serving loop would
    def capture(fn, count):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(count):
                fn(i)
        return g

    # one graph holds `per_graph` consecutive steps (one per input copy); a second one holds the remainder,
    # so that exactly args.steps steps are timed
    per_graph = max(n_copies, 8) if args.steps >= 8 else 1
    g_full = capture(step, per_graph)
    per_graph_steps = per_graph
    n_full, n_rest = divmod(args.steps, per_graph)
    g_rest = capture(step, n_rest) if n_rest else None
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(run_one, steps, warmup):
        for i in range(warmup):
            run_one(i)
        barrier()
        ev0.record()
        for i in range(steps):
            run_one(i)
        ev1.record()
        barrier()
        return ev0.elapsed_time(ev1)

    for _ in range(-(-args.warmup // per_graph)):
        g_full.replay()
    barrier()
    ev0.record()
    for _ in range(n_full):
        g_full.replay()
    if g_rest is not None:
        g_rest.replay()
    ev1.record()
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    plan.check_status()
    eager_steps = min(args.steps, 500)
    ms_eager = timed(step, eager_steps, min(args.warmup, 10)) / eager_steps

    # ---- per-stage durations: each stage alone, launched back to back over the same rotating copies
    stage_avg = {}
    reps = max(1, min(args.steps, 400) // max(n_copies, 8))
    per_graph = max(n_copies, 8)
    for name in ("prefix", "suffix", "merge"):
        g = capture(lambda i, name=name: step(i, name), per_graph)
        stage_avg[name] = timed(lambda i: g.replay(), reps, 2) / (reps * per_graph)
    plan.check_status()

    # ---- end to end through the host-buffer entry point: pinned host inputs, H2D + step + D2H every step
    pin = {k: torch.from_numpy(np.ascontiguousarray(w[k]).view(np.int16)).pin_memory()
           for k in ("q", "prefix_k", "prefix_v", "pool_k", "pool_v")}
    for k in ("page_indptr", "page_indices", "suffix_lens"):
        pin[k] = torch.from_numpy(np.ascontiguousarray(w[k], dtype=np.int32)).pin_memory()
    out_h = torch.empty((B, Hq, D), dtype=torch.bfloat16).pin_memory()
    lse_h = torch.empty((B, Hq), dtype=torch.float32).pin_memory()
    n_tok, n_pages, n_idx = w["prefix_k"].shape[0], w["pool_k"].shape[0], len(w["page_indices"])
    staging = torch.empty(host_staging_bytes(plan, n_tok, n_pages, n_idx), dtype=torch.uint8, device="cuda")
    h2d = sum(int(pin[k].numel() * pin[k].element_size()) for k in pin)
    d2h = int(out_h.numel() * 2 + lse_h.numel() * 4)

    def e2e_step():
        psa.decode_host(plan, pin["q"], pin["prefix_k"], pin["prefix_v"], pin["pool_k"], pin["pool_v"], pin["page_indptr"],
                        pin["page_indices"], pin["suffix_lens"], out_h, lse_h, staging)

    e2e_steps = max(1, min(args.steps, int(20.0 / max(1e-4, h2d / 20e9))))   # keep this leg to ~20 s at worst
    for _ in range(min(3, args.warmup)):
        e2e_step()
    barrier()
    ev0.record()
    for _ in range(e2e_steps):
        e2e_step()
    ev1.record()
    barrier()
    e2e_ms = ev0.elapsed_time(ev1) / e2e_steps
    clocks = sampler.stop()

    # ---- max over ranks
    from paper_2502_02534_b200.sharding import max_over_ranks
    ms_total, e2e_ms, ms_eager = max_over_ranks([ms_total, e2e_ms, ms_eager])
    ms_step = ms_total / args.steps
    value = world * B / (ms_step * 1e-3)

    if rank == 0:
        peaks, peaks_kind = load_peaks()
        hbm = float(peaks["hbm_gbs"])
        tf = float(peaks.get("bf16_tflops_sustained", peaks.get("bf16_tflops", 1400.0)))
        suf_gbs = abytes["suffix"] / (stage_avg["suffix"] * 1e-3) / 1e9 if stage_avg["suffix"] else None
        kernels = {}
        for name in ("prefix", "suffix"):
            t_roof_ms = max(abytes[name] / (hbm * 1e9), aflops[name] / (tf * 1e12)) * 1e3
            kernels[name] = {"ms": stage_avg[name], "algorithmic_bytes": abytes[name], "flops": aflops[name],
                             "t_roof_ms": t_roof_ms, "frac_of_roofline": t_roof_ms / stage_avg[name] if stage_avg[name] else None}
        # The planner may run a tensor-bound prefix stage on part of the SMs on purpose (few long items, so that the
        # suffix stage streams beside it); the tensor fraction on the SMs the stage actually occupies says how well
        # each of them is used.
        n_sms = torch.cuda.get_device_properties(local_rank).multi_processor_count
        blocks = info.num_prefix_items
        if stage_avg["prefix"] and blocks:
            share = min(1.0, blocks / n_sms)
            kernels["prefix"].update({"blocks": blocks, "sms": n_sms,
                                      "tensor_frac_on_sms_used": aflops["prefix"] / (tf * 1e12 * share) / (stage_avg["prefix"] * 1e-3)})
        kernels["merge"] = {"ms": stage_avg["merge"]}
        t_roof_step = max((abytes["prefix"] + abytes["suffix"]) / (hbm * 1e9), (aflops["prefix"] + aflops["suffix"]) / (tf * 1e12)) * 1e3
        # CPU baseline: the oracle as it stands, on this machine's host cores, one full step of the same workload
        import oracle
        best, cores = None, 0
        for _ in range(3):
            t0 = time.perf_counter()
            _, _, cores = oracle.attend(w)
            dt = time.perf_counter() - t0
            best = dt if best is None else min(best, dt)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": cfg.name, "prompts": cfg.num_prefixes, "samples": B, "q_heads": Hq,
                       "kv_heads": w["num_kv_heads"], "head_dim": D, "prefix_len": list(cfg.prefix_len),
                       "suffix_len": list(cfg.suffix_len), "page_size": 16,
                       "cold_l2": f"steps rotate over {n_copies} input copies ({n_copies * input_bytes / 1e6:.0f} MB > L2 126 MB)",
                       "launch": f"CUDA graph replay, {per_graph_steps} captured psa_decode steps per graph",
                       "sharding": "independent prompts per rank, no collective"},
            "plan": {"prefix_items": info.num_prefix_items, "suffix_items": info.num_suffix_items,
                     "prefix_tiles_per_item": info.prefix_tiles_per_item, "suffix_chunk_tokens": info.suffix_chunk_tokens},
            "gpu_launches": info.kernel_launches * args.steps,
            "e2e": {"value": world * B / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": e2e_ms, "steps": e2e_steps, "entry_point": "psa_decode_host"},
            "roofline": {"kernel": "suffix_kernel", "bound": "hbm", "achieved": suf_gbs, "peak": hbm, "unit": "GB/s",
                         "frac": suf_gbs / hbm if suf_gbs else None, "traffic": ncu_traffic(cfg.name), "peak_kind": f"of {peaks_kind}",
                         "algorithmic_bytes_per_launch": abytes["suffix"]},
            "kernels": kernels,
            "eager_ms_per_step": ms_eager,
            "step_roofline": {"t_roof_ms": t_roof_step, "frac": t_roof_step / ms_step},
            "cpu_baseline": {"value": B / best, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"one full {cfg.name} step ({B * Hq} rows), best of 3"},
            "clocks": clocks,
            "input_checksum": wl.checksum(w),
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", default="cfg2", choices=sorted(wl.CONFIGS))
    ap.add_argument("--impl", default="psa", choices=["psa", "reference"])
    args = ap.parse_args()
    args.warmup = max(3, args.warmup) if args.impl == "psa" else args.warmup
    cfg = wl.CONFIGS[args.config]
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_psa(args, cfg)


if __name__ == "__main__":
    main()
