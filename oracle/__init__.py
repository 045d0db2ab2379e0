"""TEST INFRASTRUCTURE ONLY: the CPU fp64 oracle for shared-prefix decode attention.

``attend`` is a ctypes front for ``psa_oracle.c`` (the plain softmax(QK^T)V
definition of the paper's "attn" benchmark group, two passes, fp64).
``recurrences`` holds the paper's streaming forms of the same operator, used to
pin the definition.  Nothing in the product imports this package; only the
tests, the smoke check and the CPU-baseline leg of the benchmark do.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "psa_oracle.c"
_LIB = _HERE / "libpsa_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the C oracle with gcc (OpenMP threads). Returns the library path."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", str(tmp), str(_SRC), "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


class _Problem(ctypes.Structure):
    _fields_ = [
        ("num_prefixes", ctypes.c_int),
        ("prefix_lens", ctypes.c_void_p),
        ("n_samples", ctypes.c_void_p),
        ("first_sample", ctypes.c_void_p),
        ("num_samples", ctypes.c_int32),
        ("num_q_heads", ctypes.c_int),
        ("num_kv_heads", ctypes.c_int),
        ("head_dim", ctypes.c_int),
        ("page_size", ctypes.c_int),
        ("sm_scale", ctypes.c_double),
        ("q", ctypes.c_void_p),
        ("prefix_k", ctypes.c_void_p),
        ("prefix_v", ctypes.c_void_p),
        ("prefix_stride_tok", ctypes.c_int64),
        ("prefix_stride_head", ctypes.c_int64),
        ("pool_k", ctypes.c_void_p),
        ("pool_v", ctypes.c_void_p),
        ("pool_stride_page", ctypes.c_int64),
        ("pool_stride_head", ctypes.c_int64),
        ("pool_stride_tok", ctypes.c_int64),
        ("page_indptr", ctypes.c_void_p),
        ("page_indices", ctypes.c_void_p),
        ("suffix_lens", ctypes.c_void_p),
    ]


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(str(build()))
        _lib.psa_oracle_attend.restype = ctypes.c_int
        _lib.psa_oracle_attend.argtypes = [
            ctypes.POINTER(_Problem), ctypes.c_void_p, ctypes.c_int64,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_int),
        ]
        _lib.psa_oracle_weights.restype = ctypes.c_int64
        _lib.psa_oracle_weights.argtypes = [
            ctypes.POINTER(_Problem), ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_int64,
        ]
    return _lib


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _problem(w: dict):
    """Marshal a workload dict (see the input generators) into the C struct.

    Returned list keeps the numpy arrays alive for the duration of the call.
    """
    keep = {}
    for name, dt in (("prefix_lens", np.int32), ("n_samples", np.int32), ("suffix_lens", np.int32),
                     ("page_indptr", np.int32), ("page_indices", np.int32)):
        keep[name] = _c(w[name], dt)
    for name in ("q", "prefix_k", "prefix_v", "pool_k", "pool_v"):
        a = w[name]
        assert a.dtype == np.uint16, f"{name} must hold bf16 bit patterns (uint16)"
        keep[name] = np.ascontiguousarray(a)
    # prefix groups: explicit (cascade: first_sample given) or one group per prompt, samples in order
    if "group_first_sample" in w:
        keep["first_sample"] = _c(w["group_first_sample"], np.int32)
    else:
        keep["first_sample"] = np.concatenate([[0], np.cumsum(keep["n_samples"])[:-1]]).astype(np.int32) if len(keep["n_samples"]) else np.zeros(0, np.int32)
    n_total_samples = len(keep["suffix_lens"])
    Hq, Hkv, D = int(w["num_q_heads"]), int(w["num_kv_heads"]), int(w["head_dim"])
    page = int(w["page_size"])
    # default layouts: prefix [sum L, Hkv, D]; pool [pages, Hkv, page, D]
    pst = w.get("prefix_strides", (Hkv * D, D))
    qst = w.get("pool_strides", (Hkv * page * D, page * D, D))
    pb = _Problem(
        len(keep["prefix_lens"]), keep["prefix_lens"].ctypes.data, keep["n_samples"].ctypes.data,
        keep["first_sample"].ctypes.data, n_total_samples,
        Hq, Hkv, D, page, float(w["sm_scale"]),
        keep["q"].ctypes.data, keep["prefix_k"].ctypes.data, keep["prefix_v"].ctypes.data,
        int(pst[0]), int(pst[1]),
        keep["pool_k"].ctypes.data, keep["pool_v"].ctypes.data, int(qst[0]), int(qst[1]), int(qst[2]),
        keep["page_indptr"].ctypes.data, keep["page_indices"].ctypes.data, keep["suffix_lens"].ctypes.data,
    )
    return pb, keep


def attend(w: dict, rows=None, n_threads: int = 0):
    """fp64 attention of every (sample, query head) row, or of ``rows`` (flat s*Hq+h).

    Returns (out [n_rows, D] float64, lse [n_rows] float64, threads_used).
    """
    lib = _load()
    pb, keep = _problem(w)
    B = len(keep["suffix_lens"])
    if rows is None:
        n_rows, rows_ptr = B * pb.num_q_heads, None
    else:
        rows = _c(rows, np.int64)
        n_rows, rows_ptr = len(rows), rows.ctypes.data
    out = np.zeros((n_rows, pb.head_dim), dtype=np.float64)
    lse = np.zeros((n_rows,), dtype=np.float64)
    used = ctypes.c_int(0)
    rc = lib.psa_oracle_attend(ctypes.byref(pb), rows_ptr, n_rows, out.ctypes.data, lse.ctypes.data,
                               int(n_threads), ctypes.byref(used))
    if rc != 0:
        raise RuntimeError("psa_oracle_attend failed (bad row index or out of memory)")
    return out, lse, used.value


def weights(w: dict, s: int, h: int):
    """Softmax weights of row (s, h) over its prefix-then-suffix context, fp64."""
    lib = _load()
    pb, keep = _problem(w)
    cap = int(np.sum(keep["prefix_lens"])) + int(np.max(keep["suffix_lens"], initial=0)) + 1
    buf = np.zeros((cap,), dtype=np.float64)
    n = lib.psa_oracle_weights(ctypes.byref(pb), int(s), int(h), buf.ctypes.data, cap)
    if n < 0:
        raise RuntimeError("psa_oracle_weights failed")
    return buf[:n].copy()


def append_kv(w: dict, new_k: np.ndarray, new_v: np.ndarray) -> dict:
    """The step after the path, as plainly as possible: sample s's new K/V rows ([B, Hkv, D] bf16 bits) go to
    position S_s of its page list (page S_s // page_size, slot S_s % page_size) and S_s grows by one.
    Returns a new workload dict with copied pools and lengths; the input is left alone."""
    page = int(w["page_size"])
    out = dict(w)
    out["pool_k"] = np.array(w["pool_k"], copy=True)
    out["pool_v"] = np.array(w["pool_v"], copy=True)
    lens = np.array(w["suffix_lens"], dtype=np.int32, copy=True)
    for s in range(len(lens)):
        S = int(lens[s])
        pages = w["page_indices"][int(w["page_indptr"][s]): int(w["page_indptr"][s + 1])]
        if S // page >= len(pages):
            raise IndexError(f"sample {s} has no page for position {S}")
        pg = int(pages[S // page])
        out["pool_k"][pg, :, S % page, :] = new_k[s]
        out["pool_v"][pg, :, S % page, :] = new_v[s]
        lens[s] = S + 1
    out["suffix_lens"] = lens
    return out


def append_kv_alloc(w: dict, new_k: np.ndarray, new_v: np.ndarray, free_pages, free_count: int):
    """append_kv with pages taken from a stack, sample by sample in order.  `page_indptr` gives every sample its SLOTS
    (capacity); a slot without a page holds a negative id; `free_pages[:free_count]` are ids nobody owns, the top of the
    stack at the end.  A sample whose length is a multiple of the page size pops one id for its next slot; a sample that
    cannot be served -- stack empty, no slot left, or already at `suffix_bounds[s]` when the workload carries bounds -- is
    skipped.  Returns (new workload, new free_count, list of skipped samples); the input is left alone."""
    page = int(w["page_size"])
    out = dict(w)
    out["pool_k"] = np.array(w["pool_k"], copy=True)
    out["pool_v"] = np.array(w["pool_v"], copy=True)
    out["page_indices"] = np.array(w["page_indices"], dtype=np.int32, copy=True)
    lens = np.array(w["suffix_lens"], dtype=np.int32, copy=True)
    bounds = w.get("suffix_bounds")
    free = [int(x) for x in np.asarray(free_pages)[:free_count]]
    skipped = []
    for s in range(len(lens)):
        S = int(lens[s])
        first, cap = int(w["page_indptr"][s]), int(w["page_indptr"][s + 1]) - int(w["page_indptr"][s])
        slot = S // page
        if (bounds is not None and S >= int(bounds[s])) or slot >= cap:
            skipped.append(s)
            continue
        if S % page == 0:                      # the token opens a new page
            if not free:
                skipped.append(s)
                continue
            out["page_indices"][first + slot] = free.pop()
        pg = int(out["page_indices"][first + slot])
        if pg < 0:
            skipped.append(s)
            continue
        out["pool_k"][pg, :, S % page, :] = new_k[s]
        out["pool_v"][pg, :, S % page, :] = new_v[s]
        lens[s] = S + 1
    out["suffix_lens"] = lens
    return out, len(free), skipped


def causal_attend(q, k, v, prompt_lens, sm_scale, rows=None, n_threads: int = 0):
    """Prefill: causal self-attention of packed prompts.  q [T, Hq, D], k / v [T, Hkv, D] as bf16 bits (uint16).
    Returns (out [n_rows, D], lse [n_rows]) in float64; rows = token * Hq + head."""
    lib = _load()
    lib.psa_oracle_causal.restype = ctypes.c_int
    lib.psa_oracle_causal.argtypes = [ctypes.c_int, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_double,
                                      ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
                                      ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int]
    q, k, v = (np.ascontiguousarray(a) for a in (q, k, v))
    assert q.dtype == np.uint16 and k.dtype == np.uint16 and v.dtype == np.uint16
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    lens = _c(prompt_lens, np.int32)
    assert int(lens.sum()) == T == k.shape[0] == v.shape[0]
    if rows is None:
        n_rows, rows_ptr = T * Hq, None
    else:
        rows = _c(rows, np.int64)
        n_rows, rows_ptr = len(rows), rows.ctypes.data
    out = np.zeros((n_rows, D), dtype=np.float64)
    lse = np.zeros((n_rows,), dtype=np.float64)
    rc = lib.psa_oracle_causal(len(lens), lens.ctypes.data, Hq, Hkv, D, float(sm_scale), q.ctypes.data, k.ctypes.data,
                               v.ctypes.data, rows_ptr, n_rows, out.ctypes.data, lse.ctypes.data, int(n_threads))
    if rc != 0:
        raise RuntimeError("psa_oracle_causal failed")
    return out, lse
