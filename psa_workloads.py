"""Seeded synthetic inputs for shared-prefix decode attention.

Shapes only: this module draws lengths, random bf16 tensors and page tables.  It holds
none of the attention arithmetic and is the one module both the CUDA tests and the CPU
oracle tests read their inputs from.

A workload is a plain dict of numpy arrays:

  prefix_lens [P] int32, n_samples [P] int32, suffix_lens [B] int32,
  q [B, Hq, D] uint16 (bf16 bits),
  prefix_k / prefix_v [sum L, Hkv, D] uint16 (prompts packed back to back),
  pool_k / pool_v [n_pool_pages, Hkv, page_size, D] uint16,
  page_indptr [B+1] int32, page_indices [n_pages] int32,
  num_q_heads, num_kv_heads, head_dim, page_size, sm_scale.

The five named configurations follow the parallel-sampling set-up the paper describes
(one prompt of selected demonstrations sampled many times, bounded output length):
they stand in for that hosted-API workload, which is not reproducible offline.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

BF16_NAN = np.uint16(0x7FC0)


@dataclass(frozen=True)
class PsaConfig:
    name: str
    num_prefixes: int
    samples_per_prefix: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    prefix_len: tuple          # (lo, hi): lo == hi fixed, else log-uniform integers, both ends inclusive
    suffix_len: tuple          # (lo, hi) uniform integers, both ends inclusive
    page_size: int = 16
    permute_pages: bool = False
    seed: int = 0


CONFIGS = {
    "cfg1": PsaConfig("cfg1", 1, 8, 8, 2, 64, (512, 512), (1, 128)),
    "cfg2": PsaConfig("cfg2", 1, 32, 32, 8, 128, (4096, 4096), (0, 1024)),
    "cfg3": PsaConfig("cfg3", 1, 64, 32, 8, 128, (16384, 16384), (0, 2048)),
    "cfg4": PsaConfig("cfg4", 1, 256, 64, 8, 128, (8192, 8192), (0, 4096), permute_pages=True),
    "cfg5": PsaConfig("cfg5", 16, 16, 32, 8, 128, (1024, 32768), (0, 4096)),
}


def _rng(seed: int, stream: int) -> np.random.Generator:
    # one master seed per configuration, one counter-based sub-stream per tensor
    return np.random.Generator(np.random.Philox(key=seed * 1000 + stream))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    u = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (u >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(shape, seed: int, stream: int, chunk: int = 1 << 24) -> np.ndarray:
    """N(0,1) samples rounded to bf16 bits, drawn in bounded chunks."""
    n = int(np.prod(shape, dtype=np.int64))
    out = np.empty(n, dtype=np.uint16)
    g = _rng(seed, stream)
    for a in range(0, n, chunk):
        b = min(n, a + chunk)
        out[a:b] = f32_to_bf16_bits(g.standard_normal(b - a, dtype=np.float32))
    return out.reshape(shape)


def draw_lengths(cfg: PsaConfig):
    g = _rng(cfg.seed, 0)
    lo, hi = cfg.prefix_len
    if lo == hi:
        prefix_lens = np.full(cfg.num_prefixes, lo, dtype=np.int32)
    else:
        u = g.uniform(math.log(lo), math.log(hi), size=cfg.num_prefixes)
        prefix_lens = np.clip(np.rint(np.exp(u)), lo, hi).astype(np.int32)
    n_samples = np.full(cfg.num_prefixes, cfg.samples_per_prefix, dtype=np.int32)
    B = int(n_samples.sum())
    slo, shi = cfg.suffix_len
    suffix_lens = g.integers(slo, shi + 1, size=B, dtype=np.int64).astype(np.int32)
    return prefix_lens, n_samples, suffix_lens


def build_page_table(suffix_lens, page_size, permute, seed, slack_fraction=0.125):
    """CSR page table: ceil(S/page) pages per sample, handed out in sample order, then
    (optionally) one random permutation of all physical page ids across the whole pool."""
    n_pages = (np.asarray(suffix_lens, dtype=np.int64) + page_size - 1) // page_size
    indptr = np.zeros(len(suffix_lens) + 1, dtype=np.int32)
    np.cumsum(n_pages, out=indptr[1:])
    used = int(indptr[-1])
    pool_pages = max(1, used + int(math.ceil(used * slack_fraction)))
    if permute:
        phys = _rng(seed, 6).permutation(pool_pages)[:used].astype(np.int32)
    else:
        phys = np.arange(used, dtype=np.int32)
    return indptr, phys, pool_pages


def poison_unused(w: dict) -> None:
    """Overwrite every pool slot no sample owns (page tails and slack pages) with bf16 NaN
    so that any read of it shows up in the result."""
    page = int(w["page_size"])
    pool_pages = w["pool_k"].shape[0]
    valid = np.zeros((pool_pages, page), dtype=bool)
    for s, S in enumerate(w["suffix_lens"]):
        pages = w["page_indices"][w["page_indptr"][s]: w["page_indptr"][s + 1]]
        for i, pg in enumerate(pages):
            valid[pg, : min(page, int(S) - i * page)] = True
    mask = ~valid
    for name in ("pool_k", "pool_v"):
        a = w[name]
        a.transpose(0, 2, 1, 3)[mask] = BF16_NAN


def make_workload(cfg: PsaConfig, poison: bool = False, lengths=None) -> dict:
    """Draw one workload.  ``lengths`` = (prefix_lens, n_samples, suffix_lens) overrides the
    configuration's length distributions (used by edge-case tests)."""
    if lengths is None:
        prefix_lens, n_samples, suffix_lens = draw_lengths(cfg)
    else:
        prefix_lens, n_samples, suffix_lens = (np.asarray(a, dtype=np.int32) for a in lengths)
    B = int(n_samples.sum())
    assert len(suffix_lens) == B
    Hq, Hkv, D, page = cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.page_size
    indptr, indices, pool_pages = build_page_table(suffix_lens, page, cfg.permute_pages, cfg.seed)
    total_prefix = int(prefix_lens.sum())
    w = dict(
        name=cfg.name,
        prefix_lens=prefix_lens, n_samples=n_samples, suffix_lens=suffix_lens,
        num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, page_size=page,
        sm_scale=1.0 / math.sqrt(D),
        q=normal_bf16((B, Hq, D), cfg.seed, 1),
        prefix_k=normal_bf16((total_prefix, Hkv, D), cfg.seed, 2),
        prefix_v=normal_bf16((total_prefix, Hkv, D), cfg.seed, 3),
        pool_k=normal_bf16((pool_pages, Hkv, page, D), cfg.seed, 4),
        pool_v=normal_bf16((pool_pages, Hkv, page, D), cfg.seed, 5),
        page_indptr=indptr, page_indices=indices,
    )
    if poison:
        poison_unused(w)
    return w


def make_cascade_workload(cfg: PsaConfig, shared_len: int, poison: bool = False, lengths=None) -> dict:
    """A two-level cascade: ``shared_len`` tokens attended by EVERY sample (the base prompt and demonstrations that
    all tasks share) followed by the configuration's per-prompt prefixes (the task text shared by a task's samples).
    Same dict as make_workload, with the prefix arrays holding group 0 (shared) then the per-prompt groups, and
      prefix_lens [P+1], n_samples [P+1], group_first_sample [P+1]
    describing the groups (group g: prefix_lens[g] tokens, samples first..first+n)."""
    w = make_workload(cfg, poison=poison, lengths=lengths)
    B = len(w["suffix_lens"])
    Hkv, D = cfg.num_kv_heads, cfg.head_dim
    first = np.concatenate([[0], np.cumsum(w["n_samples"])[:-1]]).astype(np.int32)
    w["prefix_k"] = np.concatenate([normal_bf16((shared_len, Hkv, D), cfg.seed, 7), w["prefix_k"]])
    w["prefix_v"] = np.concatenate([normal_bf16((shared_len, Hkv, D), cfg.seed, 8), w["prefix_v"]])
    w["prefix_lens"] = np.concatenate([[shared_len], w["prefix_lens"]]).astype(np.int32)
    w["n_samples"] = np.concatenate([[B], w["n_samples"]]).astype(np.int32)
    w["group_first_sample"] = np.concatenate([[0], first]).astype(np.int32)
    return w


def flatten_cascade(w: dict) -> dict:
    """The same problem without sharing: one prefix per SAMPLE that physically holds every token the sample's
    groups cover, in group order.  Used to check grouped results against ungrouped ones."""
    B = len(w["suffix_lens"])
    tok = np.concatenate([[0], np.cumsum(w["prefix_lens"])])
    ks, vs, lens = [], [], []
    for s in range(B):
        n = 0
        for g in range(len(w["prefix_lens"])):
            f = int(w["group_first_sample"][g])
            if f <= s < f + int(w["n_samples"][g]):
                ks.append(w["prefix_k"][tok[g]:tok[g + 1]]); vs.append(w["prefix_v"][tok[g]:tok[g + 1]])
                n += int(w["prefix_lens"][g])
        lens.append(n)
    flat = {k: v for k, v in w.items() if k != "group_first_sample"}
    Hkv, D = int(w["num_kv_heads"]), int(w["head_dim"])
    flat["prefix_k"] = np.concatenate(ks) if ks else np.zeros((0, Hkv, D), np.uint16)
    flat["prefix_v"] = np.concatenate(vs) if vs else np.zeros((0, Hkv, D), np.uint16)
    flat["prefix_lens"] = np.asarray(lens, dtype=np.int32)
    flat["n_samples"] = np.ones(B, dtype=np.int32)
    return flat


def checksum(w: dict) -> int:
    """Order-sensitive 64-bit checksum of the tensors, to tell runs apart in logs."""
    acc = 1469598103934665603
    for name in ("q", "prefix_k", "prefix_v", "pool_k", "pool_v", "page_indices", "suffix_lens"):
        a = np.ascontiguousarray(w[name]).view(np.uint8)
        pad = (-a.size) % 8
        if pad:
            a = np.concatenate([a.ravel(), np.zeros(pad, np.uint8)])
        acc = (acc * 1099511628211 + int(np.bitwise_xor.reduce(a.ravel().view(np.uint64)))) & 0xFFFFFFFFFFFFFFFF
    return acc


def algorithmic_bytes(w: dict) -> dict:
    """KV bytes each part of the step must read once (bf16 K and V), plus page-table entries."""
    Hkv, D = int(w["num_kv_heads"]), int(w["head_dim"])
    prefix = 4 * int(np.sum(w["prefix_lens"], dtype=np.int64)) * Hkv * D
    suffix = 4 * int(np.sum(w["suffix_lens"], dtype=np.int64)) * Hkv * D + 4 * int(w["page_indptr"][-1])
    return {"prefix": prefix, "suffix": suffix}


def algorithmic_flops(w: dict) -> dict:
    """QK^T and PV multiply-adds (2 flops each) per part of the step."""
    Hq, D = int(w["num_q_heads"]), int(w["head_dim"])
    first = np.concatenate([[0], np.cumsum(w["n_samples"])])
    pre = sum(4 * int(n) * Hq * int(L) * D for n, L in zip(w["n_samples"], w["prefix_lens"]))
    suf = 4 * Hq * D * int(np.sum(w["suffix_lens"], dtype=np.int64))
    del first
    return {"prefix": pre, "suffix": suf}
