"""Time one stage (or the whole step) of a named configuration with the planner's knobs forced by hand.

    python -m paper_2502_02534_b200.stage_timer --config cfg3 --stage prefix --prefix-only --prefix-kernel 3 --tiles 15

For tuning the planner's choices (block shape, key tiles per item, rows per item, suffix chunk) and as the small,
self-contained command profilers are pointed at: `--prefix-only` draws the configuration without suffix tokens, so
that only the prompt K/V (tens of MB) is held on the device and the prefix grid owns the SMs.  Inputs are the seeded
synthetic workloads of `psa_workloads`; launches are timed one by one with CUDA events (`--graph N`: N launches per
replayed CUDA graph instead).  Prints one line per repetition and the plan the library made.
"""
from __future__ import annotations

import argparse
import dataclasses
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def main(argv=None):
    import torch
    import psa_workloads as wl
    import paper_2502_02534_b200 as psa
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--config", default="cfg3", choices=sorted(wl.CONFIGS))
    ap.add_argument("--stage", default="all", choices=["all", "prefix", "suffix", "merge"])
    ap.add_argument("--prefix-only", action="store_true", help="no suffix tokens at all (small memory; prefix and merge stages only)")
    ap.add_argument("--prefix-kernel", type=int, default=0, help="PSA_PREFIX_KERNEL_*: 0 auto, 1 small, 2 long, 3 decoupled, 4 coupled")
    ap.add_argument("--tiles", type=int, default=0, help="128-key tiles per prefix item (0 = planner)")
    ap.add_argument("--rows", type=int, default=0, help="query rows per prefix item: 0 (planner), 128 or 256")
    ap.add_argument("--chunk", type=int, default=0, help="tokens per suffix item (0 = planner)")
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--graph", type=int, default=0, help="launches per CUDA graph replay (0 = eager launches)")
    args = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise RuntimeError("a CUDA device is needed: the library has no CPU path")

    cfg = wl.CONFIGS[args.config]
    if args.prefix_only:
        cfg = dataclasses.replace(cfg, suffix_len=(0, 0))
    w = wl.make_workload(cfg)
    B, Hq, D = int(np.sum(w["n_samples"])), w["num_q_heads"], w["head_dim"]
    bf = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda().view(torch.bfloat16)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()
    dev = {k: bf(w[k]) for k in ("q", "prefix_k", "prefix_v", "pool_k", "pool_v")}
    dev.update({k: i32(w[k]) for k in ("page_indptr", "page_indices", "suffix_lens")})
    plan = psa.Plan(w["prefix_lens"], w["n_samples"], w["suffix_lens"], num_q_heads=Hq, num_kv_heads=w["num_kv_heads"], head_dim=D,
                    sm_scale=w["sm_scale"], prefix_kernel=args.prefix_kernel, prefix_tiles_per_item=args.tiles,
                    prefix_rows_per_item=args.rows, suffix_chunk_tokens=args.chunk)
    plan.bind_workspace()
    out = torch.empty((B, Hq, D), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((B, Hq), dtype=torch.float32, device="cuda")

    def launch():
        psa.decode(plan, dev["q"], dev["prefix_k"], dev["prefix_v"], dev["pool_k"], dev["pool_v"], dev["page_indptr"],
                   dev["page_indices"], dev["suffix_lens"], out, lse, stage=args.stage)

    info = plan.info
    print(f"{args.config} stage={args.stage} prefix items {info.num_prefix_items} (<= {info.prefix_tiles_per_item} tiles of 128 keys), "
          f"suffix items {info.num_suffix_items} (chunks of {info.suffix_chunk_tokens} tokens)", flush=True)
    for _ in range(3):
        launch()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    per, run = 1, launch
    if args.graph > 0:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for _ in range(args.graph):
                launch()
        per, run = args.graph, g.replay
        run()
        torch.cuda.synchronize()
    for _ in range(args.reps):
        e0.record()
        run()
        e1.record()
        torch.cuda.synchronize()
        print(f"  {e0.elapsed_time(e1) * 1e3 / per:9.2f} us per launch", flush=True)
    plan.check_status()


if __name__ == "__main__":
    main()
