"""TEST INFRASTRUCTURE ONLY: the paper's streaming forms of softmax(S).V, in fp64.

The paper prints three algebraically equal ways to fold a stream of
(logit, value) pairs into the attention output (figure "attn tasks": Task 0
normalises at every step, Task 1 splits the running maximum from the running
sum, Task 2 defers the division to the end).  They are restated here from the
mathematics, one scalar step at a time, so the tests can tie the two-pass
definition in ``psa_oracle.c`` to the paper's own operator.  ``merge_partials``
is the identity that the deferred-division form implies for contexts processed
in pieces.  Pure Python loops: small inputs only.
"""
from __future__ import annotations

import math

import numpy as np


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) exactly: bf16 is the top half of an fp32."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def gather_context(w: dict, s: int, h: int):
    """Dense fp64 copies of one row's query, keys and values (prefix first, then the
    sample's own paged tokens), found by walking the page table here in Python."""
    Hq, Hkv, D, page = (int(w[k]) for k in ("num_q_heads", "num_kv_heads", "head_dim", "page_size"))
    G = Hq // Hkv
    kv = h // G
    n_samples = np.asarray(w["n_samples"])
    prefix_lens = np.asarray(w["prefix_lens"])
    # prefix groups: explicit first samples (cascade) or consecutive prompts
    first = np.asarray(w["group_first_sample"]) if "group_first_sample" in w else np.concatenate([[0], np.cumsum(n_samples)[:-1]])
    tok = np.concatenate([[0], np.cumsum(prefix_lens)])
    S = int(w["suffix_lens"][s])
    q = bf16_bits_to_f64(np.asarray(w["q"]).reshape(-1, Hq, D)[s, h])
    pk = np.asarray(w["prefix_k"]).reshape(-1, Hkv, D)
    pv = np.asarray(w["prefix_v"]).reshape(-1, Hkv, D)
    K, V = [], []
    for g in range(len(prefix_lens)):
        if int(first[g]) <= s < int(first[g]) + int(n_samples[g]):
            K += [pk[t, kv] for t in range(int(tok[g]), int(tok[g + 1]))]
            V += [pv[t, kv] for t in range(int(tok[g]), int(tok[g + 1]))]
    L = len(K)
    poolk = np.asarray(w["pool_k"]).reshape(-1, Hkv, page, D)
    poolv = np.asarray(w["pool_v"]).reshape(-1, Hkv, page, D)
    for t in range(S):
        pg = int(w["page_indices"][int(w["page_indptr"][s]) + t // page])
        K.append(poolk[pg, kv, t % page])
        V.append(poolv[pg, kv, t % page])
    if L + S == 0:
        return q, np.zeros((0, D)), np.zeros((0, D))
    return q, bf16_bits_to_f64(np.stack(K)), bf16_bits_to_f64(np.stack(V))


def logits(w: dict, s: int, h: int):
    """(x [n], V [n, D]) with x_j = sm_scale * q.k_j, fp64."""
    q, K, V = gather_context(w, s, h)
    return float(w["sm_scale"]) * (K @ q), V


def _running_maximum(x):
    """M_t = max(x_0 .. x_t) and the factor exp(M_{t-1} - M_t) by which everything accumulated before step t shrinks
    when the maximum moves (0 at t = 0: the state starts at m = -inf, l = 0, o = 0)."""
    x = np.asarray(x, dtype=np.float64)
    M = np.maximum.accumulate(x) if len(x) else x
    before = np.concatenate([[-math.inf], M[:-1]]) if len(x) else x
    with np.errstate(invalid="ignore"):
        keep = np.where(before == -math.inf, 0.0, np.exp(before - M))
    return M, keep


def task0_maxsum(x, V):
    """Task 0 ("MaxSum"): one operator carries (m, l, o) with o normalised after EVERY key.  In closed form the state
    after t keys is m_t = max_j x_j, l_t = sum_j exp(x_j - m_t), o_t = sum_j exp(x_j - m_t) v_j / l_t (j <= t); stepping
    from t - 1 to t, l_t = l_{t-1} exp(m_{t-1} - m_t) + exp(x_t - m_t) and the normalised o moves toward v_t by the new
    key's share of the sum, o_t = o_{t-1} + (exp(x_t - m_t) / l_t) (v_t - o_{t-1})."""
    V = np.asarray(V, dtype=np.float64)
    M, keep = _running_maximum(x)
    weight = np.exp(np.asarray(x, dtype=np.float64) - M) if len(M) else M
    l, o = 0.0, np.zeros(V.shape[1])
    for t in range(len(M)):
        l = l * keep[t] + weight[t]
        o = o + (weight[t] / l) * (V[t] - o)
    return o, (float(M[-1]) if len(M) else -math.inf), l


def _exp_max_diff(x):
    """Stage one of Tasks 1 and 2 ("ExpMaxDiff") as a stream: for every key its weight e_t = exp(x_t - m_t) at the new
    running maximum, the factor d_t = exp(m_{t-1} - m_t) for what came before, and m_t."""
    M, keep = _running_maximum(x)
    e = np.exp(np.asarray(x, dtype=np.float64) - M) if len(M) else M
    return list(zip(e, keep, M))


def task1_divsum(x, V):
    """Task 1: "ExpMaxDiff" feeds "DivSum", which sees only (e_t, d_t, v_t): it keeps the sum l and the NORMALISED output,
    l_t = d_t l_{t-1} + e_t,  o_t = (d_t l_{t-1} o_{t-1} + e_t v_t) / l_t  (the two-operand weighted mean of the old
    output and the new value)."""
    V = np.asarray(V, dtype=np.float64)
    l, o, m = 0.0, np.zeros(V.shape[1]), -math.inf
    for (e, d, m), v_t in zip(_exp_max_diff(x), V):
        carried = d * l
        l = carried + e
        o = (carried * o + e * v_t) / l
    return o, float(m), l


def task2_deferred(x, V):
    """Task 2: "ExpMaxDiff" feeds two plain weighted sums, r_t = d_t r_{t-1} + e_t and acc_t = d_t acc_{t-1} + e_t v_t,
    divided ONCE at the end: the form every fast kernel of the library uses."""
    V = np.asarray(V, dtype=np.float64)
    r, acc, m = 0.0, np.zeros(V.shape[1]), -math.inf
    for (e, d, m), v_t in zip(_exp_max_diff(x), V):
        r = d * r + e
        acc = d * acc + e * v_t
    return acc / r, float(m), r


def merge_partials(outs, lses):
    """Combine normalised partial results of disjoint key sets.

    Partial i carries out_i = sum_j w_j v_j / Z_i and lse_i = ln sum_j exp(x_j).  Since
    the un-normalised accumulators of Task 2 simply add once brought to a common maximum,
    lse = ln sum_i exp(lse_i) and out = sum_i exp(lse_i - lse) out_i.  Pieces with
    lse_i = -inf are empty and contribute nothing; all empty gives (0, -inf)."""
    lses = [float(v) for v in lses]
    top = max(lses, default=-math.inf)
    D = len(outs[0]) if outs else 0
    if top == -math.inf:
        return np.zeros(D), -math.inf
    z = sum(math.exp(v - top) for v in lses)
    lse = top + math.log(z)
    out = np.zeros(D)
    for o, v in zip(outs, lses):
        if v != -math.inf:
            out += math.exp(v - lse) * np.asarray(o, dtype=np.float64)
    return out, lse
