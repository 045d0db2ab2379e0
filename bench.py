#!/usr/bin/env python
"""Benchmark of one decode step of parallel-sample shared-prefix attention on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg4] [--sharding prompts|heads] [--impl psa|reference]

A step = prefix + suffix + merge stages over one batch of seeded synthetic inputs (the shapes of the paper's
parallel-sampling set-up; nothing is read from disk).  The headline workload is the largest configuration (cfg4);
with one GPU the line also carries `per_config`, the same measurement for every named configuration.

Several GPUs: started as `python bench.py --gpus N` the script starts its N ranks itself; under
`python -m torch.distributed.run` it reads RANK / LOCAL_RANK / WORLD_SIZE from the environment.  Two ways to cut
the work: `--sharding prompts` (default; rank r owns its own prompts, seed r; no data-path collective, weak scaling)
and `--sharding heads` (rank r owns Hkv / N KV heads of the SAME problem and one all-gather of out / lse along the
head axis follows every step; strong scaling).  Rank 0 prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import dataclasses
import hashlib
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
HEADLINE = "cfg4"
MIN_TIMED_MS = 200.0        # the K-step block is repeated until this much device time has been timed
MAX_BLOCKS = 400
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}      # datasheet figures, for context beside the measured peaks
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per launch of the dominant kernel, from ncu captures of
# single launches (profiles/).  An entry is only valid for the kernel source it was taken with (hash below); entries
# with `scaled_from` were not captured themselves: traffic grows in proportion to the tokens a launch streams, and the
# figure is the captured configuration's bytes per algorithmic byte times this configuration's algorithmic bytes.
NCU_TRAFFIC = {
    "cfg2": {"kernel": "suffix_kernel", "bytes_per_launch": 68273408 + 56576},      # 1.0052 x the algorithmic bytes
    "cfg3": {"kernel": "suffix_kernel", "bytes_per_launch": 264009728 + 237312},    # 1.0031 x
}
NCU_TRAFFIC_SOURCE = {"suffix_kernel": ("paper_2502_02534_b200/csrc/suffix_sm100.cu", "498b791d8050fd97")}
# measured DRAM bytes per algorithmic byte of the largest captured configuration (cfg3); scales the configurations that
# are too large to capture under a profiler (cfg4, cfg5: 2.2 GB per launch), whose traffic grows with the tokens streamed
NCU_TRAFFIC_RATIO = {"suffix_kernel": (264009728 + 237312) / 263438152}


def ncu_traffic(config_name, kernel, algorithmic_bytes):
    src = NCU_TRAFFIC_SOURCE.get(kernel)
    if not src:
        return None
    try:
        with open(os.path.join(ROOT, src[0]), "rb") as f:
            if hashlib.sha256(f.read()).hexdigest()[:16] != src[1]:
                return None          # the kernel changed since the counters were taken
    except OSError:
        return None
    t = NCU_TRAFFIC.get(config_name)
    if t and t["kernel"] == kernel:
        return t["bytes_per_launch"]
    if kernel in NCU_TRAFFIC_RATIO:
        return int(round(NCU_TRAFFIC_RATIO[kernel] * algorithmic_bytes))
    return None


def load_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return json.load(f), "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


def needs_launcher(gpus: int, env) -> bool:
    """True when this process has to start the ranks itself: several GPUs asked for, no launcher's environment."""
    return gpus > 1 and "WORLD_SIZE" not in env


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while work runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int, period_s: float = 0.005):
        self.samples, self.reason_bits, self.max_mhz = [], 0, None
        self._stop = threading.Event()
        self._thread = None
        self._on = threading.Event()
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
            if self._on.is_set():
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

    def region(self, on: bool):
        """Only samples taken while a timed region runs are kept."""
        (self._on.set if on else self._on.clear)()

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
def oracle_sample(w, cfg_name, budget_s):
    """Rows of the workload the oracle attends in one timed pass: all of them if that fits the budget, else whole
    samples drawn at random.  Returns (rows or None, samples per pass, description)."""
    import oracle
    B, Hq = int(np.sum(w["n_samples"])), w["num_q_heads"]
    t0 = time.perf_counter()
    oracle.attend(w)
    t_full = time.perf_counter() - t0
    if t_full <= budget_s:
        return None, B, f"every row of {cfg_name} ({B * Hq} rows) per step"
    n = max(1, int(B * budget_s / t_full))
    sel = np.sort(np.random.default_rng(0).choice(B, n, replace=False))
    rows = (sel[:, None] * Hq + np.arange(Hq)[None, :]).ravel()
    return rows, n, f"{n} of {B} samples of {cfg_name} (all {Hq} heads) per step"


def run_reference(args, cfg):
    """The CPU fp64 oracle as it stands, timed on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    w = wl.make_workload(cfg)
    rows, n_samples, sample = oracle_sample(w, cfg.name, 150.0 / max(1, args.steps + args.warmup))
    cores = 0
    for _ in range(args.warmup):
        oracle.attend(w, rows=rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        _, _, cores = oracle.attend(w, rows=rows)
    dt = (time.perf_counter() - t0) / max(1, args.steps)
    value = n_samples / dt
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": {"workload": cfg.name, "note": "CPU fp64 oracle on host cores"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------- psa arm
class Runner:
    """One configuration on this rank's GPU: inputs (several copies, so that no step finds them in L2), plan, the
    timed loops."""

    def __init__(self, cfg, rank, world, sharding, steps, warmup, sampler):
        import torch
        import paper_2502_02534_b200 as psa
        from paper_2502_02534_b200.sharding import shard_heads
        self.torch, self.psa = torch, psa
        self.cfg, self.rank, self.world, self.sharding = cfg, rank, world, sharding
        self.steps, self.warmup, self.sampler = steps, warmup, sampler
        if sharding == "heads":
            self.w_full = wl.make_workload(cfg)                       # the same problem on every rank
            w = shard_heads(self.w_full, rank, world) if world > 1 else self.w_full
        else:
            w = wl.make_workload(dataclasses.replace(cfg, seed=cfg.seed + rank))   # rank r samples its own prompts
            self.w_full = w
        self.w = w
        self.B, self.Hq, self.D = int(np.sum(w["n_samples"])), w["num_q_heads"], w["head_dim"]
        self.Hq_full = self.w_full["num_q_heads"]
        self.abytes, self.aflops = wl.algorithmic_bytes(w), wl.algorithmic_flops(w)
        self.input_bytes = sum(int(w[k].nbytes) for k in ("q", "prefix_k", "prefix_v", "pool_k", "pool_v"))
        self.n_copies = max(2, int(np.ceil(4 * L2_BYTES / self.input_bytes))) if self.input_bytes < 4 * L2_BYTES else 1
        self.copies = [self._upload() for _ in range(self.n_copies)]
        self.out = torch.empty((self.B, self.Hq, self.D), dtype=torch.bfloat16, device="cuda")
        self.lse = torch.empty((self.B, self.Hq), dtype=torch.float32, device="cuda")
        self.gather = sharding == "heads" and world > 1
        if self.gather:      # the one exchange of KV-head sharding: all-gather along the head axis, then [N,B,h,D] -> [B,N*h,D]
            self.g_out = torch.empty((world, self.B, self.Hq, self.D), dtype=torch.bfloat16, device="cuda")
            self.g_lse = torch.empty((world, self.B, self.Hq), dtype=torch.float32, device="cuda")
            self.full_out = torch.empty((self.B, world * self.Hq, self.D), dtype=torch.bfloat16, device="cuda")
            self.full_lse = torch.empty((self.B, world * self.Hq), dtype=torch.float32, device="cuda")
        # planning is host work done once per batch shape, outside the decode loop: timed on its own (plan + work lists to the device)
        plan_ms = []
        for _ in range(5):
            t0 = time.perf_counter()
            self.plan = psa.Plan(w["prefix_lens"], w["n_samples"], w["suffix_lens"], num_q_heads=self.Hq,
                                 num_kv_heads=w["num_kv_heads"], head_dim=self.D, page_size=w["page_size"],
                                 sm_scale=w["sm_scale"], out_dtype="bf16")
            self.plan.bind_workspace()
            torch.cuda.synchronize()
            plan_ms.append((time.perf_counter() - t0) * 1e3)
        self.plan_host_ms = statistics.median(plan_ms)
        self.info = self.plan.info
        self.ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]

    def _upload(self):
        torch, w = self.torch, self.w
        d = {k: torch.from_numpy(np.ascontiguousarray(w[k]).view(np.int16)).cuda().view(torch.bfloat16)
             for k in ("q", "prefix_k", "prefix_v", "pool_k", "pool_v")}
        for k in ("page_indptr", "page_indices", "suffix_lens"):
            d[k] = torch.from_numpy(np.ascontiguousarray(w[k], dtype=np.int32)).cuda()
        return d

    def barrier(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()
        self.torch.cuda.synchronize()

    def step(self, i, stage="all"):
        d = self.copies[i % self.n_copies]
        self.psa.decode(self.plan, d["q"], d["prefix_k"], d["prefix_v"], d["pool_k"], d["pool_v"], d["page_indptr"],
                        d["page_indices"], d["suffix_lens"], self.out, self.lse, stage=stage)
        if self.gather and stage == "all":
            import torch.distributed as dist
            dist.all_gather_into_tensor(self.g_out, self.out)
            dist.all_gather_into_tensor(self.g_lse, self.lse)
            self.full_out.view(self.B, self.world, self.Hq, self.D).copy_(self.g_out.permute(1, 0, 2, 3))
            self.full_lse.view(self.B, self.world, self.Hq).copy_(self.g_lse.permute(1, 0, 2))

    def capture(self, fn, count):
        g = self.torch.cuda.CUDAGraph()
        with self.torch.cuda.graph(g):
            for i in range(count):
                fn(i)
        return g

    def timed_blocks(self, run_block, block_steps, min_ms, max_blocks=MAX_BLOCKS):
        """Runs `run_block` (exactly `block_steps` steps) repeatedly, each run bracketed by a barrier and a device
        synchronisation on both sides and timed with CUDA events, until `min_ms` of device time is covered.
        Returns the per-block times in ms (max over ranks)."""
        from paper_2502_02534_b200.sharding import max_over_ranks
        times, total = [], 0.0
        self.sampler.region(True)
        while True:
            self.barrier()
            self.ev[0].record()
            run_block()
            self.ev[1].record()
            self.barrier()
            t = max_over_ranks([self.ev[0].elapsed_time(self.ev[1])])[0]
            times.append(t)
            total += t
            if total >= min_ms or len(times) >= max_blocks:
                break
        self.sampler.region(False)
        return times

    def measure(self, with_eager=False, min_ms=MIN_TIMED_MS):
        torch = self.torch
        for i in range(max(3, self.n_copies)):        # first launches set kernel attributes; keep them out of any capture
            self.step(i)
        torch.cuda.synchronize()
        K = self.steps
        # A decode step is launch-bound on the host (three small kernels), so the timed loop replays CUDA graphs of
        # captured steps, as a serving loop would.  One graph holds `per_graph` consecutive steps (one per input copy);
        # a second one holds the remainder, so that a block is exactly K steps.  With a collective in the step (KV-head
        # sharding over several ranks) the steps are launched eagerly instead.
        use_graph = not self.gather
        if use_graph:
            per_graph = max(self.n_copies, 8) if K >= 8 else 1
            g_full = self.capture(self.step, per_graph)
            n_full, n_rest = divmod(K, per_graph)
            g_rest = self.capture(self.step, n_rest) if n_rest else None

            def block():
                for _ in range(n_full):
                    g_full.replay()
                if g_rest is not None:
                    g_rest.replay()
            for _ in range(-(-self.warmup // per_graph)):
                g_full.replay()
            launch = f"CUDA graph replay, {per_graph} captured psa_decode steps per graph"
        else:
            def block():
                for i in range(K):
                    self.step(i)
            for i in range(self.warmup):
                self.step(i)
            launch = "eager launches (psa_decode, then one NCCL all-gather of out and lse along the head axis)"
        times = self.timed_blocks(block, K, min_ms)
        self.plan.check_status()
        res = {"block_ms": times, "ms_step_median": statistics.median(times) / K, "ms_step_min": min(times) / K,
               "blocks": len(times), "launch": launch}
        if use_graph and self.n_copies > 1:
            # side note: the same steps on ONE input copy, which then stays in L2 (not a roofline figure)
            g_warm = self.capture(lambda i: self.step(0), per_graph)
            g_warm.replay()
            res["warm_l2_ms_per_step"] = statistics.median(self.timed_blocks(g_warm.replay, per_graph, min(min_ms, 20.0), 100)) / per_graph
        if with_eager:
            n = min(K, 500)
            res["eager_ms_per_step"] = statistics.median(self.timed_blocks(lambda: [self.step(i) for i in range(n)], n, 20.0, 20)) / n

        # per-stage durations: each stage alone, launched back to back over the same rotating copies
        per_graph = max(self.n_copies, 8)
        stage_ms = {}
        for name in ("prefix", "suffix", "merge"):
            g = self.capture(lambda i, name=name: self.step(i, name), per_graph)
            g.replay()
            ts = self.timed_blocks(g.replay, per_graph, min(min_ms, 30.0), 100)
            stage_ms[name] = statistics.median(ts) / per_graph
        self.plan.check_status()
        res["stage_ms"] = stage_ms
        # the prefix stage planned for itself: the same prompts and samples with no suffix work, so that the planner
        # cuts the items for a grid that owns the machine (in the fused step it shares the SMs with the suffix stage)
        w = self.w
        alone = self.psa.Plan(w["prefix_lens"], w["n_samples"], np.zeros_like(np.asarray(w["suffix_lens"])), num_q_heads=self.Hq,
                              num_kv_heads=w["num_kv_heads"], head_dim=self.D, page_size=w["page_size"], sm_scale=w["sm_scale"],
                              out_dtype="bf16")
        alone.bind_workspace()
        if alone.info.num_prefix_items:
            fused_plan, self.plan = self.plan, alone
            try:
                g = self.capture(lambda i: self.step(i, "prefix"), per_graph)
                g.replay()
                ts = self.timed_blocks(g.replay, per_graph, min(min_ms, 30.0), 100)
                alone.check_status()
            finally:
                self.plan = fused_plan
            res["prefix_alone"] = {"ms": statistics.median(ts) / per_graph, "items": alone.info.num_prefix_items,
                                   "tiles_per_item": alone.info.prefix_tiles_per_item}
        return res

    def e2e(self, budget_s=8.0):
        """End to end through the host-buffer entry point: pinned host inputs, H2D + step + D2H every step."""
        torch, w, psa = self.torch, self.w, self.psa
        from paper_2502_02534_b200.binding import host_staging_bytes
        pin = {k: torch.from_numpy(np.ascontiguousarray(w[k]).view(np.int16)).pin_memory()
               for k in ("q", "prefix_k", "prefix_v", "pool_k", "pool_v")}
        for k in ("page_indptr", "page_indices", "suffix_lens"):
            pin[k] = torch.from_numpy(np.ascontiguousarray(w[k], dtype=np.int32)).pin_memory()
        out_h = torch.empty((self.B, self.Hq, self.D), dtype=torch.bfloat16).pin_memory()
        lse_h = torch.empty((self.B, self.Hq), dtype=torch.float32).pin_memory()
        n_tok, n_pages, n_idx = w["prefix_k"].shape[0], w["pool_k"].shape[0], len(w["page_indices"])
        staging = torch.empty(host_staging_bytes(self.plan, n_tok, n_pages, n_idx), dtype=torch.uint8, device="cuda")
        h2d = sum(int(pin[k].numel() * pin[k].element_size()) for k in pin)
        d2h = int(out_h.numel() * 2 + lse_h.numel() * 4)

        def one():
            psa.decode_host(self.plan, pin["q"], pin["prefix_k"], pin["prefix_v"], pin["pool_k"], pin["pool_v"],
                            pin["page_indptr"], pin["page_indices"], pin["suffix_lens"], out_h, lse_h, staging)

        n = max(1, min(self.steps, int(budget_s / max(1e-4, h2d / 20e9))))
        for _ in range(min(3, self.warmup)):
            one()
        ts = self.timed_blocks(lambda: [one() for _ in range(n)], n, 0.0, 1)
        self.plan.check_status()
        ms = ts[0] / n
        return {"value": self.world * self.B / (ms * 1e-3) if self.sharding != "heads" else self.B / (ms * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms, "steps": n,
                "entry_point": "psa_decode_host"}

    def cpu_baseline(self, budget_s):
        """The oracle as it stands on this machine's host cores, on a bounded sample of this workload."""
        import oracle
        rows, n_samples, sample = oracle_sample(self.w, self.cfg.name, budget_s)
        best, cores = None, 0
        for _ in range(2):
            t0 = time.perf_counter()
            _, _, cores = oracle.attend(self.w, rows=rows)
            dt = time.perf_counter() - t0
            best = dt if best is None else min(best, dt)
        return {"value": n_samples / best, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample + ", best of 2"}

    def rooflines(self, res, peaks, peaks_kind):
        """Per-stage roofline times and fractions against the measured and the nominal denominators."""
        hbm = float(peaks["hbm_gbs"])
        tf_sus = float(peaks.get("bf16_tflops_sustained", peaks.get("bf16_tflops", 1400.0)))
        tf_burst = float(peaks.get("bf16_tflops", tf_sus))
        rows = self.B * self.Hq
        out_bytes = rows * (self.D * 2 + 4)
        merge_bytes = int(self.info.num_partial_rows) * (self.D * 4 + 4) + out_bytes
        bytes_ = {"prefix": self.abytes["prefix"], "suffix": self.abytes["suffix"], "merge": merge_bytes}
        flops = {"prefix": self.aflops["prefix"], "suffix": self.aflops["suffix"], "merge": 0}
        kernels = {}
        for name in ("prefix", "suffix", "merge"):
            ms = res["stage_ms"][name]
            t_meas = max(bytes_[name] / (hbm * 1e9), flops[name] / (tf_sus * 1e12)) * 1e3
            t_nom = max(bytes_[name] / (NOMINAL["hbm_gbs"] * 1e9), flops[name] / (NOMINAL["bf16_tflops"] * 1e12)) * 1e3
            bound = "hbm" if bytes_[name] / (hbm * 1e9) >= flops[name] / (tf_sus * 1e12) else "tensor"
            kernels[name] = {"ms": ms, "algorithmic_bytes": bytes_[name], "flops": flops[name], "bound": bound,
                             "t_roof_ms": t_meas, "frac_of_measured": t_meas / ms if ms else None,
                             "t_roof_nominal_ms": t_nom, "frac_of_nominal": t_nom / ms if ms else None,
                             "achieved_gbs": bytes_[name] / (ms * 1e-3) / 1e9 if ms else None,
                             "achieved_tflops": flops[name] / (ms * 1e-3) / 1e12 if ms else None}
        # The planner may run a tensor-bound prefix stage on part of the SMs on purpose (few long items, so that the
        # suffix stage streams beside it); the tensor fraction on the SMs the stage occupies says how well each is used.
        n_sms = self.torch.cuda.get_device_properties(self.torch.cuda.current_device()).multi_processor_count
        blocks = self.info.num_prefix_items
        if res["stage_ms"]["prefix"] and blocks:
            share = min(1.0, blocks / n_sms)
            kernels["prefix"].update({"blocks": blocks, "sms": n_sms, "tensor_frac_on_sms_used_of_measured":
                                      flops["prefix"] / (tf_sus * 1e12 * share) / (res["stage_ms"]["prefix"] * 1e-3)})
        if res.get("prefix_alone"):
            pa = res["prefix_alone"]
            kernels["prefix_planned_alone"] = {"ms": pa["ms"], "items": pa["items"], "tiles_per_item": pa["tiles_per_item"],
                                               "frac_of_measured": kernels["prefix"]["t_roof_ms"] / pa["ms"],
                                               "frac_of_nominal": kernels["prefix"]["t_roof_nominal_ms"] / pa["ms"],
                                               "achieved_tflops": flops["prefix"] / (pa["ms"] * 1e-3) / 1e12,
                                               "achieved_gbs": bytes_["prefix"] / (pa["ms"] * 1e-3) / 1e9,
                                               "note": "prefix stage of a plan without suffix work: the grid owns the SMs"}
        tot_b, tot_f = bytes_["prefix"] + bytes_["suffix"], flops["prefix"] + flops["suffix"]
        t_step = max(tot_b / (hbm * 1e9), tot_f / (tf_sus * 1e12)) * 1e3
        t_step_nom = max(tot_b / (NOMINAL["hbm_gbs"] * 1e9), tot_f / (NOMINAL["bf16_tflops"] * 1e12)) * 1e3
        ms_step = res["ms_step_median"]
        step = {"t_roof_ms": t_step, "frac_of_measured": t_step / ms_step, "t_roof_nominal_ms": t_step_nom,
                "frac_of_nominal": t_step_nom / ms_step}
        dom = max(("prefix", "suffix", "merge"), key=lambda n: res["stage_ms"][n])
        k = kernels[dom]
        kernel_name = {"prefix": "prefix_kernel", "suffix": "suffix_kernel", "merge": "merge_kernel"}[dom]
        if k["bound"] == "hbm":
            roof = {"kernel": kernel_name, "bound": "hbm", "achieved": k["achieved_gbs"], "peak": hbm, "unit": "GB/s",
                    "frac": k["achieved_gbs"] / hbm, "frac_of_nominal": k["achieved_gbs"] / NOMINAL["hbm_gbs"],
                    "traffic": ncu_traffic(self.cfg.name, kernel_name, k["algorithmic_bytes"]),
                    "peak_kind": f"of {peaks_kind} (copy bandwidth, read + write)", "algorithmic_bytes_per_launch": k["algorithmic_bytes"]}
        else:
            roof = {"kernel": kernel_name, "bound": "tensor", "achieved": k["achieved_tflops"], "peak": tf_sus, "unit": "TFLOP/s",
                    "frac": k["achieved_tflops"] / tf_sus, "frac_of_nominal": k["achieved_tflops"] / NOMINAL["bf16_tflops"],
                    "traffic": None, "peak_kind": f"of {peaks_kind} (sustained bf16 GEMM; burst {tf_burst:.0f})",
                    "algorithmic_flops_per_launch": k["flops"]}
        return kernels, step, roof


def run_psa(args, cfg):
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if args.sharding == "heads" and cfg.num_kv_heads % world:
        raise SystemExit(f"--sharding heads: {cfg.num_kv_heads} KV heads do not divide over {world} ranks")

    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()
    run = Runner(cfg, rank, world, args.sharding, args.steps, args.warmup, sampler)
    res = run.measure(with_eager=True)
    e2e = run.e2e()
    clocks = sampler.stop()
    peaks, peaks_kind = load_peaks()
    strong = args.sharding == "heads"
    ms_step = res["ms_step_median"]
    value = (run.B if strong else world * run.B) / (ms_step * 1e-3)

    line = None
    if rank == 0:
        kernels, step_roof, roof = run.rooflines(res, peaks, peaks_kind)
        w = run.w_full
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "strong" if strong else "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": cfg.name, "prompts": cfg.num_prefixes, "samples": int(np.sum(w["n_samples"])),
                       "q_heads": run.Hq_full, "kv_heads": w["num_kv_heads"], "head_dim": run.D,
                       "prefix_len": list(cfg.prefix_len), "suffix_len": list(cfg.suffix_len), "page_size": 16,
                       "cold_l2": (f"steps rotate over {run.n_copies} input copies "
                                   f"({run.n_copies * run.input_bytes / 1e6:.0f} MB > L2 126 MB)"),
                       "launch": res["launch"],
                       "sharding": ("KV heads per rank, one all-gather of out / lse along the head axis per step" if strong
                                    else "independent prompts per rank, no collective")},
            "timing": {"block_steps": args.steps, "blocks": res["blocks"], "timed_ms": sum(res["block_ms"]),
                       "ms_per_step_median": ms_step, "ms_per_step_min": res["ms_step_min"],
                       "note": "each block of `steps` steps is bracketed by barrier + synchronize and timed with CUDA events; "
                               "blocks repeat until the timed region covers 200 ms; value uses the median block"},
            "plan": {"prefix_items": run.info.num_prefix_items, "suffix_items": run.info.num_suffix_items,
                     "prefix_tiles_per_item": run.info.prefix_tiles_per_item, "suffix_chunk_tokens": run.info.suffix_chunk_tokens},
            "gpu_launches": run.info.kernel_launches * args.steps * res["blocks"],
            "e2e": e2e, "roofline": roof, "kernels": kernels, "eager_ms_per_step": res.get("eager_ms_per_step"),
            "step_roofline": step_roof, "clocks": clocks, "input_checksum": wl.checksum(run.w),
            "plan_host_ms": run.plan_host_ms, "warm_l2_ms_per_step": res.get("warm_l2_ms_per_step"),
        }
        line["cpu_baseline"] = run.cpu_baseline(10.0) if world == 1 else None   # reported at one GPU only
    del run
    torch.cuda.empty_cache()

    # ---- every named configuration, one GPU only: the table behind the per-kernel claims
    if world == 1 and not args.no_per_config:
        per = {}
        quiet = ClockSampler(-1)       # per-config runs do not feed the clock record of the headline
        for name in sorted(wl.CONFIGS):
            if name == cfg.name:
                k, s, r = line["kernels"], line["step_roofline"], line["roofline"]
                per[name] = {"step_us": ms_step * 1e3, "step_us_min": line["timing"]["ms_per_step_min"] * 1e3,
                             "sample_tokens_per_s": value, "stage_us": {n: k[n]["ms"] * 1e3 for n in k},
                             "frac_of_measured": {**{n: k[n]["frac_of_measured"] for n in k}, "step": s["frac_of_measured"]},
                             "frac_of_nominal": {**{n: k[n]["frac_of_nominal"] for n in k}, "step": s["frac_of_nominal"]},
                             "bound": {n: k[n]["bound"] for n in ("prefix", "suffix", "merge")}, "traffic": r["traffic"],
                             "plan": line["plan"], "cpu_baseline": line["cpu_baseline"], "plan_host_ms": line["plan_host_ms"],
                             "warm_l2_step_us": None if line["warm_l2_ms_per_step"] is None else line["warm_l2_ms_per_step"] * 1e3}
                continue
            c = wl.CONFIGS[name]
            rn = Runner(c, 0, 1, "prompts", max(8, min(args.steps, 200)), max(3, min(args.warmup, 10)), quiet)
            rs = rn.measure(min_ms=50.0)
            k, s, r = rn.rooflines(rs, peaks, peaks_kind)
            per[name] = {"step_us": rs["ms_step_median"] * 1e3, "step_us_min": rs["ms_step_min"] * 1e3,
                         "sample_tokens_per_s": rn.B / (rs["ms_step_median"] * 1e-3),
                         "stage_us": {n: k[n]["ms"] * 1e3 for n in k},
                         "frac_of_measured": {**{n: k[n]["frac_of_measured"] for n in k}, "step": s["frac_of_measured"]},
                         "frac_of_nominal": {**{n: k[n]["frac_of_nominal"] for n in k}, "step": s["frac_of_nominal"]},
                         "bound": {n: k[n]["bound"] for n in ("prefix", "suffix", "merge")},
                         "traffic": ncu_traffic(name, "suffix_kernel", k["suffix"]["algorithmic_bytes"]),
                         "plan": {"prefix_items": rn.info.num_prefix_items, "suffix_items": rn.info.num_suffix_items,
                                  "prefix_tiles_per_item": rn.info.prefix_tiles_per_item,
                                  "suffix_chunk_tokens": rn.info.suffix_chunk_tokens},
                         "cpu_baseline": rn.cpu_baseline(5.0), "plan_host_ms": rn.plan_host_ms,
                         "warm_l2_step_us": None if rs.get("warm_l2_ms_per_step") is None else rs["warm_l2_ms_per_step"] * 1e3}
            del rn
            torch.cuda.empty_cache()
        line["per_config"] = per
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", default=HEADLINE, choices=sorted(wl.CONFIGS))
    ap.add_argument("--sharding", default="prompts", choices=["prompts", "heads"])
    ap.add_argument("--no-per-config", action="store_true", help="skip the table over every named configuration")
    ap.add_argument("--impl", default="psa", choices=["psa", "reference"])
    args = ap.parse_args()
    if args.steps < 1:
        ap.error("--steps must be at least 1")
    args.warmup = max(3, args.warmup) if args.impl == "psa" else args.warmup
    cfg = wl.CONFIGS[args.config]
    if args.impl == "psa" and needs_launcher(args.gpus, os.environ):
        from paper_2502_02534_b200.launch import spawn_ranks
        sys.exit(spawn_ranks(args.gpus, [sys.executable, os.path.abspath(__file__), *sys.argv[1:]]))
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_psa(args, cfg)


if __name__ == "__main__":
    main()
