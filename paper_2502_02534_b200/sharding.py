"""Multi-GPU plumbing.  Nothing here computes attention.

Two ways to cut the path, both without any communication inside the attention itself:
  * by prompt (`partition_prompts`, `shard_workload`): each rank owns a contiguous range of prompts with all of their
    samples, plans and decodes it alone; no data-path collective at all, only timing crosses ranks.
  * by KV head (`shard_heads`, `gather_heads`): each rank holds the prefix K/V and the suffix pools of its KV heads
    and the matching query heads of every sample, runs the whole step on `[B, Hq / world, D]`, and ONE exchange
    follows: an all-gather of the outputs along the head axis (B * Hq * D elements in total).  This keeps the
    shared prefix shared on every rank; sharding by sample would replicate its read.
"""
from __future__ import annotations

import numpy as np


def partition_prompts(prefix_lens, n_samples, suffix_lens, world: int):
    """Split prompts 0..P-1 into `world` contiguous ranges of roughly equal KV traffic
    (prefix tokens + the prompt's suffix tokens).  Returns [(begin, end)] * world."""
    prefix_lens = np.asarray(prefix_lens, dtype=np.int64)
    n_samples = np.asarray(n_samples, dtype=np.int64)
    suffix_lens = np.asarray(suffix_lens, dtype=np.int64)
    first = np.concatenate([[0], np.cumsum(n_samples)])
    cost = np.array([prefix_lens[p] * (n_samples[p] > 0) + suffix_lens[first[p]:first[p + 1]].sum()
                     for p in range(len(prefix_lens))], dtype=np.float64)
    total = cost.sum()
    cum = np.concatenate([[0.0], np.cumsum(cost)])
    cuts = [0]
    for r in range(1, world):
        target = total * r / world
        cut = int(np.searchsorted(cum, target, side="left"))
        # nearest boundary to the target, never moving backwards
        if cut > 0 and abs(cum[cut - 1] - target) <= abs(cum[min(cut, len(cost))] - target):
            cut -= 1
        cuts.append(min(max(cut, cuts[-1]), len(cost)))
    cuts.append(len(cost))
    return [(cuts[r], cuts[r + 1]) for r in range(world)]


def shard_workload(w: dict, rank: int, world: int) -> dict:
    """The sub-problem of one rank: its prompts, their samples, their page lists.  The suffix
    pool is kept whole (page ids stay valid); everything else is sliced."""
    begin, end = partition_prompts(w["prefix_lens"], w["n_samples"], w["suffix_lens"], world)[rank]
    n_samples = np.asarray(w["n_samples"])
    prefix_lens = np.asarray(w["prefix_lens"])
    first = np.concatenate([[0], np.cumsum(n_samples)])
    tok = np.concatenate([[0], np.cumsum(prefix_lens)])
    s0, s1 = int(first[begin]), int(first[end])
    indptr = np.asarray(w["page_indptr"])
    sub = dict(w)
    sub.update(
        prefix_lens=prefix_lens[begin:end].copy(), n_samples=n_samples[begin:end].copy(),
        suffix_lens=np.asarray(w["suffix_lens"])[s0:s1].copy(),
        q=w["q"][s0:s1], prefix_k=w["prefix_k"][tok[begin]:tok[end]], prefix_v=w["prefix_v"][tok[begin]:tok[end]],
        page_indptr=(indptr[s0:s1 + 1] - indptr[s0]).astype(np.int32),
        page_indices=np.asarray(w["page_indices"])[indptr[s0]:indptr[s1]].copy(),
        sample_range=(s0, s1),
    )
    return sub


def shard_heads(w: dict, rank: int, world: int) -> dict:
    """The sub-problem of one rank under KV-head sharding: KV heads [rank * Hkv / world, (rank + 1) * Hkv / world) and
    their query heads, for every sample.  Lengths, page table and sample order are unchanged."""
    Hq, Hkv = int(w["num_q_heads"]), int(w["num_kv_heads"])
    if Hkv % world:
        raise ValueError(f"{Hkv} KV heads do not divide over {world} ranks")
    hk = Hkv // world
    G = Hq // Hkv
    k0, k1 = rank * hk, (rank + 1) * hk
    sub = dict(w)
    sub.update(
        num_q_heads=hk * G, num_kv_heads=hk,
        q=np.ascontiguousarray(np.asarray(w["q"])[:, k0 * G:k1 * G]),
        prefix_k=np.ascontiguousarray(np.asarray(w["prefix_k"])[:, k0:k1]),
        prefix_v=np.ascontiguousarray(np.asarray(w["prefix_v"])[:, k0:k1]),
        pool_k=np.ascontiguousarray(np.asarray(w["pool_k"])[:, k0:k1]),
        pool_v=np.ascontiguousarray(np.asarray(w["pool_v"])[:, k0:k1]),
        head_range=(k0 * G, k1 * G),
    )
    return sub


def gather_heads(out_local, lse_local):
    """The one exchange step of KV-head sharding: all-gather of every rank's `out [B, Hq / world, D]` and
    `lse [B, Hq / world]` (torch tensors, on the device of the process group's backend) along the head axis.
    Returns (out [B, Hq, D], lse [B, Hq]); without a process group the inputs come back unchanged."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return out_local, lse_local
    world = dist.get_world_size()
    outs = [torch.empty_like(out_local) for _ in range(world)]
    lses = [torch.empty_like(lse_local) for _ in range(world)]
    dist.all_gather(outs, out_local.contiguous())
    dist.all_gather(lses, lse_local.contiguous())
    return torch.cat(outs, dim=1), torch.cat(lses, dim=1)


def max_over_ranks(values):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]
