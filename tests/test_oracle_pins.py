"""Pins for the CPU oracle: closed forms, brute force, a library softmax, invariants and
the paper's streaming recurrences.  Each test is chosen so that one plausible mistake in
``oracle/psa_oracle.c`` (dropped scale, wrong sign, wrong head mapping, wrong page slot,
transposed operand, missing normalisation) makes it fail."""
import math

import numpy as np
import pytest

import oracle
import psa_workloads as wl
from oracle import recurrences as rec

TOL = 1e-12


def bits(x):
    return wl.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def tiny_cfg(**kw):
    base = dict(name="tiny", num_prefixes=1, samples_per_prefix=3, num_q_heads=4, num_kv_heads=2,
                head_dim=8, prefix_len=(5, 5), suffix_len=(0, 9), page_size=4, seed=7)
    base.update(kw)
    return wl.PsaConfig(**base)


def dense_problem(q, K, V, sm_scale, page_size=4, as_suffix=0):
    """One sample, one head: the last ``as_suffix`` keys live in pages, the rest in the prefix."""
    n, D = K.shape
    L = n - as_suffix
    n_pages = (as_suffix + page_size - 1) // page_size
    pool_k = np.full((max(1, n_pages), 1, page_size, D), wl.BF16_NAN, np.uint16)
    pool_v = pool_k.copy()
    for t in range(as_suffix):
        pool_k[t // page_size, 0, t % page_size] = bits(K[L + t])
        pool_v[t // page_size, 0, t % page_size] = bits(V[L + t])
    return dict(prefix_lens=[L], n_samples=[1], suffix_lens=[as_suffix], num_q_heads=1, num_kv_heads=1,
                head_dim=D, page_size=page_size, sm_scale=sm_scale,
                q=bits(q).reshape(1, 1, D),
                prefix_k=bits(K[:L]).reshape(L, 1, D), prefix_v=bits(V[:L]).reshape(L, 1, D),
                pool_k=pool_k, pool_v=pool_v,
                page_indptr=np.array([0, n_pages], np.int32), page_indices=np.arange(n_pages, dtype=np.int32))


# ---------------------------------------------------------------- exact inputs
def test_bf16_widening_is_exact():
    # 0x3FC0 = 1.5, 0xC020 = -2.5, 0x3E80 = 0.25: one key, V carries the values through
    K = np.array([[1.0, 0.0]]); V = np.array([[1.5, -2.5]]); q = np.array([0.25, 0.0])
    w = dense_problem(q, K, V, 1.0)
    assert list(w["prefix_v"].ravel()) == [0x3FC0, 0xC020] and w["q"].ravel()[0] == 0x3E80
    out, lse, _ = oracle.attend(w)
    assert out[0, 0] == 1.5 and out[0, 1] == -2.5
    assert lse[0] == 0.25          # one key: lse = its logit = sm_scale * q.k


# ---------------------------------------------------------------- brute force, 1-3 keys
def test_one_key_gives_its_value_and_logit():
    q = np.array([0.5, -1.0, 2.0, 0.25]); k = np.array([[1.0, 2.0, -0.5, 4.0]]); v = np.array([[3.0, -1.0, 0.5, 8.0]])
    for scale in (1.0, 0.5, 0.125):
        out, lse, _ = oracle.attend(dense_problem(q, k, v, scale))
        assert np.array_equal(out[0], v[0])
        assert abs(lse[0] - scale * float(q @ k[0])) < TOL     # catches a dropped or squared scale


def test_two_and_three_keys_hand_expanded():
    q = np.array([1.0, -0.5]); K = np.array([[0.5, 1.0], [2.0, -1.0], [-1.0, 0.25]])
    V = np.array([[1.0, 10.0], [-2.0, 20.0], [4.0, -30.0]]); scale = 0.5
    x = [scale * (q[0] * K[j, 0] + q[1] * K[j, 1]) for j in range(3)]
    for n in (2, 3):
        e = [math.exp(x[j]) for j in range(n)]
        z = sum(e)
        want = [sum(e[j] * V[j, d] for j in range(n)) / z for d in range(2)]
        for suf in range(n + 1):                      # every prefix/suffix cut of the same keys
            out, lse, _ = oracle.attend(dense_problem(q, K[:n], V[:n], scale, as_suffix=suf))
            assert np.allclose(out[0], want, rtol=0, atol=TOL)
            assert abs(lse[0] - math.log(z)) < TOL


# ---------------------------------------------------------------- closed forms
def test_all_keys_equal_gives_mean_and_log_n():
    n, D = 13, 8
    q = np.arange(D) * 0.25 - 1.0
    K = np.tile(np.linspace(-1, 1, D), (n, 1))
    V = np.arange(n * D, dtype=np.float64).reshape(n, D) * 0.5
    scale = 0.5
    out, lse, _ = oracle.attend(dense_problem(q, K, V, scale, as_suffix=6))
    x = scale * float(bits_f64(q) @ bits_f64(K[0]))
    assert np.allclose(out[0], V.mean(axis=0), rtol=0, atol=1e-11)
    assert abs(lse[0] - (x + math.log(n))) < TOL


def bits_f64(x):
    return wl.bf16_bits_to_f32(bits(x)).astype(np.float64)


@pytest.mark.parametrize("a", [0.0, 1.0, 3.0, 50.0, 800.0])
def test_one_hot_key_closed_form(a):
    # key j* has logit a, every other key logit 0
    n, D, jstar = 9, 4, 5
    q = np.array([1.0, 0, 0, 0]); K = np.zeros((n, D)); K[jstar, 0] = a
    V = np.arange(n * D, dtype=np.float64).reshape(n, D) - 7.0
    out, lse, _ = oracle.attend(dense_problem(q, K, V, 1.0, as_suffix=3))
    if a < 700:
        ea = math.exp(a)
        want = (ea * V[jstar] + (V.sum(axis=0) - V[jstar])) / (ea + n - 1)
        assert np.allclose(out[0], want, rtol=0, atol=1e-11)
        assert abs(lse[0] - math.log(ea + n - 1)) < 1e-11
    else:   # exp(a) overflows fp64: only a max-subtracted softmax survives, and returns v_j* exactly
        assert np.array_equal(out[0], V[jstar]) and lse[0] == a


def test_weights_sum_to_one_and_match_library_softmax():
    from scipy.special import softmax as sp_softmax
    w = wl.make_workload(tiny_cfg(), poison=True)
    for s in range(3):
        for h in range(4):
            wt = oracle.weights(w, s, h)
            assert abs(wt.sum() - 1.0) < TOL and (wt >= 0).all()
            x, _ = rec.logits(w, s, h)
            assert np.allclose(wt, sp_softmax(x), rtol=0, atol=TOL)


def test_values_of_ones_and_convex_hull():
    w = wl.make_workload(tiny_cfg(), poison=True)
    out, _, _ = oracle.attend(w)
    for s in range(3):
        for h in range(4):
            _, V = rec.logits(w, s, h)
            o = out[s * 4 + h]
            assert (o <= V.max(axis=0) + TOL).all() and (o >= V.min(axis=0) - TOL).all()
    w["prefix_v"][:] = bits(1.0); w["pool_v"][:] = bits(1.0)
    out, _, _ = oracle.attend(w)
    assert np.allclose(out, 1.0, rtol=0, atol=TOL)      # sum_j w_j / Z = 1


# ---------------------------------------------------------------- library special case
def test_prefix_only_matches_torch_softmax_bmm_on_odd_shapes():
    torch = pytest.importorskip("torch")
    # the odd sizes of the paper's functional verifier: M=5, N=7, K=9, D=11
    n_keys, n_samples, D = 5, 7, 11
    cfg = tiny_cfg(samples_per_prefix=n_samples, num_q_heads=1, num_kv_heads=1, head_dim=D,
                   prefix_len=(n_keys, n_keys), suffix_len=(0, 0))
    w = wl.make_workload(cfg)
    out, lse, _ = oracle.attend(w)
    q = torch.from_numpy(rec.bf16_bits_to_f64(w["q"]))[:, 0]                 # [N, D]
    K = torch.from_numpy(rec.bf16_bits_to_f64(w["prefix_k"]))[:, 0]          # [M, D]
    V = torch.from_numpy(rec.bf16_bits_to_f64(w["prefix_v"]))[:, 0]
    S = (q @ K.T) * w["sm_scale"]                                            # [N, M]
    E1 = V.unsqueeze(0).expand(n_samples, n_keys, D)
    ref = torch.bmm(torch.softmax(S, 1).unsqueeze(1), E1).squeeze(1)
    assert np.allclose(out, ref.numpy(), rtol=0, atol=TOL)
    assert np.allclose(lse, torch.logsumexp(S, 1).numpy(), rtol=0, atol=TOL)


# ---------------------------------------------------------------- the paper's recurrences
@pytest.mark.parametrize("form", [rec.task0_maxsum, rec.task1_divsum, rec.task2_deferred])
def test_streaming_forms_equal_two_pass_definition(form):
    w = wl.make_workload(tiny_cfg(prefix_len=(11, 11), suffix_len=(1, 9)), poison=True)
    out, lse, _ = oracle.attend(w)
    for s in range(3):
        for h in range(4):
            x, V = rec.logits(w, s, h)
            o, m, l = form(x, V)
            assert np.allclose(o, out[s * 4 + h], rtol=0, atol=TOL)
            assert abs(m + math.log(l) - lse[s * 4 + h]) < TOL


def test_split_and_merge_equals_concatenation_exhaustively():
    w = wl.make_workload(tiny_cfg(samples_per_prefix=1, prefix_len=(4, 4), suffix_len=(3, 3)), poison=True)
    out, lse, _ = oracle.attend(w)
    x, V = rec.logits(w, 0, 1)
    n = len(x)
    assert n == 7

    def piece(a, b):
        if a == b:
            return np.zeros(V.shape[1]), -math.inf
        o, m, l = rec.task2_deferred(x[a:b], V[a:b])
        return o, m + math.log(l)

    for c1 in range(n + 1):                 # all 2-way and 3-way cuts, empty pieces included
        for c2 in range(c1, n + 1):
            parts = [piece(0, c1), piece(c1, c2), piece(c2, n)]
            o, l = rec.merge_partials([p[0] for p in parts], [p[1] for p in parts])
            assert np.allclose(o, out[1], rtol=0, atol=TOL) and abs(l - lse[1]) < TOL


def test_prefix_only_plus_suffix_only_merge_equals_full():
    w = wl.make_workload(tiny_cfg(), poison=True)
    full_o, full_l, _ = oracle.attend(w)
    wp = dict(w); wp["suffix_lens"] = np.zeros_like(w["suffix_lens"])
    ws = dict(w); ws["prefix_lens"] = np.zeros_like(w["prefix_lens"])
    ws["prefix_k"] = w["prefix_k"][:0]; ws["prefix_v"] = w["prefix_v"][:0]
    po, pl, _ = oracle.attend(wp)
    so, sl, _ = oracle.attend(ws)
    for r in range(len(full_l)):
        o, l = rec.merge_partials([po[r], so[r]], [pl[r], sl[r]])
        assert np.allclose(o, full_o[r], rtol=0, atol=TOL) and abs(l - full_l[r]) < TOL
    empty = np.flatnonzero(w["suffix_lens"] == 0)
    for s in empty:                          # an empty piece is (0, -inf) and is harmless
        assert (sl[s * 4:(s + 1) * 4] == -math.inf).all() and (so[s * 4:(s + 1) * 4] == 0).all()


def test_empty_context_gives_zero_and_minus_inf():
    cfg = tiny_cfg(samples_per_prefix=2, prefix_len=(0, 0), suffix_len=(0, 0))
    w = wl.make_workload(cfg)
    out, lse, _ = oracle.attend(w)
    assert (out == 0).all() and (lse == -math.inf).all()


# ---------------------------------------------------------------- indexing pins
def test_gqa_head_mapping_is_contiguous_groups():
    # V of KV head kv is the constant kv+1 everywhere: out of query head h must be h // G + 1
    cfg = tiny_cfg(num_q_heads=6, num_kv_heads=3)
    w = wl.make_workload(cfg, poison=True)
    for kv in range(3):
        w["prefix_v"][:, kv, :] = bits(kv + 1.0)
        pv = w["pool_v"][:, kv]
        pv[pv != wl.BF16_NAN] = bits(kv + 1.0)
    out, _, _ = oracle.attend(w)
    out = out.reshape(3, 6, -1)
    for h in range(6):
        assert np.allclose(out[:, h], h // 2 + 1.0, rtol=0, atol=TOL)


def test_page_table_walk_finds_every_token_once():
    # equal keys => uniform weights; V[...,0] = global token id => out[0] = mean id of the context
    cfg = tiny_cfg(num_prefixes=2, samples_per_prefix=2, prefix_len=(3, 9), suffix_len=(0, 11),
                   permute_pages=True, seed=3)
    w = wl.make_workload(cfg, poison=True)
    Hkv, page = 2, 4
    w["prefix_k"][:] = bits(0.5)
    pk = w["pool_k"]; pk[pk != wl.BF16_NAN] = bits(0.5)
    first = np.concatenate([[0], np.cumsum(w["n_samples"])]); offs = np.concatenate([[0], np.cumsum(w["prefix_lens"])])
    next_id = 0.0
    prefix_ids = []
    for p in range(2):
        ids = []
        for t in range(int(w["prefix_lens"][p])):
            w["prefix_v"][offs[p] + t, :, 0] = bits(next_id); ids.append(next_id); next_id += 1
        prefix_ids.append(ids)
    want = []
    for s in range(4):
        p = int(np.searchsorted(first, s, side="right") - 1)
        ids = list(prefix_ids[p])
        for t in range(int(w["suffix_lens"][s])):
            pg = w["page_indices"][w["page_indptr"][s] + t // page]
            w["pool_v"][pg, :, t % page, 0] = bits(next_id); ids.append(next_id); next_id += 1
        want.append(np.mean(ids) if ids else 0.0)
    assert next_id < 256            # every id is an exact bf16 integer
    out, lse, _ = oracle.attend(w)
    out = out.reshape(4, 4, -1)
    for s in range(4):
        assert np.allclose(out[s, :, 0], want[s], rtol=0, atol=1e-11)
    assert np.isfinite(out).all()   # NaN-poisoned tails and slack pages were never read


def test_sample_key_and_page_permutations():
    cfg = tiny_cfg(samples_per_prefix=4, suffix_len=(1, 9))
    w = wl.make_workload(cfg, poison=True)
    out, lse, _ = oracle.attend(w)
    B, Hq, D = 4, 4, 8
    # samples: permute rows of q, lengths and page lists
    perm = np.array([2, 0, 3, 1])
    w2 = dict(w)
    w2["q"] = w["q"][perm]; w2["suffix_lens"] = w["suffix_lens"][perm]
    lists = [w["page_indices"][w["page_indptr"][s]: w["page_indptr"][s + 1]] for s in range(B)]
    w2["page_indices"] = np.concatenate([lists[s] for s in perm]).astype(np.int32)
    w2["page_indptr"] = np.concatenate([[0], np.cumsum([len(lists[s]) for s in perm])]).astype(np.int32)
    o2, l2, _ = oracle.attend(w2)
    assert np.allclose(o2.reshape(B, Hq, D), out.reshape(B, Hq, D)[perm], rtol=0, atol=TOL)
    assert np.allclose(l2.reshape(B, Hq), lse.reshape(B, Hq)[perm], rtol=0, atol=TOL)
    # prefix keys: reorder tokens (K and V together)
    kp = np.random.default_rng(0).permutation(w["prefix_k"].shape[0])
    w3 = dict(w); w3["prefix_k"] = w["prefix_k"][kp]; w3["prefix_v"] = w["prefix_v"][kp]
    o3, l3, _ = oracle.attend(w3)
    assert np.allclose(o3, out, rtol=0, atol=TOL) and np.allclose(l3, lse, rtol=0, atol=TOL)
    # physical pages: relabel pages, move their contents, update the table
    n_pool = w["pool_k"].shape[0]
    pp = np.random.default_rng(1).permutation(n_pool)           # old id -> new id
    w4 = dict(w)
    w4["pool_k"] = np.empty_like(w["pool_k"]); w4["pool_v"] = np.empty_like(w["pool_v"])
    w4["pool_k"][pp] = w["pool_k"]; w4["pool_v"][pp] = w["pool_v"]
    w4["page_indices"] = pp[w["page_indices"]].astype(np.int32)
    o4, l4, _ = oracle.attend(w4)
    assert np.array_equal(o4, out) and np.array_equal(l4, lse)


def test_strided_layouts_give_the_same_result():
    cfg = tiny_cfg()
    w = wl.make_workload(cfg, poison=True)
    out, lse, _ = oracle.attend(w)
    Hkv, D, page = 2, 8, 4
    w2 = dict(w)        # head-major prefix [Hkv, L, D] and token-major pool [pages, page, Hkv, D]
    L = w["prefix_k"].shape[0]
    w2["prefix_k"] = np.ascontiguousarray(w["prefix_k"].transpose(1, 0, 2))
    w2["prefix_v"] = np.ascontiguousarray(w["prefix_v"].transpose(1, 0, 2))
    w2["prefix_strides"] = (D, L * D)
    w2["pool_k"] = np.ascontiguousarray(w["pool_k"].transpose(0, 2, 1, 3))
    w2["pool_v"] = np.ascontiguousarray(w["pool_v"].transpose(0, 2, 1, 3))
    w2["pool_strides"] = (page * Hkv * D, D, Hkv * D)
    o2, l2, _ = oracle.attend(w2)
    assert np.array_equal(o2, out) and np.array_equal(l2, lse)


def test_row_subset_equals_full_run_and_threads_do_not_matter():
    w = wl.make_workload(tiny_cfg(samples_per_prefix=5), poison=True)
    out, lse, _ = oracle.attend(w, n_threads=1)
    rows = np.array([17, 0, 9, 19, 3])
    o, l, used = oracle.attend(w, rows=rows, n_threads=3)
    assert np.array_equal(o, out[rows]) and np.array_equal(l, lse[rows])
    with pytest.raises(RuntimeError):
        oracle.attend(w, rows=np.array([20]))


def test_definition_matches_numpy_restatement_on_config1():
    w = wl.make_workload(wl.CONFIGS["cfg1"], poison=True)
    out, lse, _ = oracle.attend(w)
    assert np.isfinite(out).all() and np.isfinite(lse).all()
    rng = np.random.default_rng(5)
    for r in rng.choice(out.shape[0], 6, replace=False):
        s, h = divmod(int(r), 8)
        x, V = rec.logits(w, s, h)
        o, m, l = rec.task2_deferred(x, V)
        assert np.allclose(o, out[r], rtol=0, atol=TOL) and abs(m + math.log(l) - lse[r]) < TOL


# ---------------------------------------------------------------- cascades of shared prefixes
def test_cascade_equals_the_same_keys_without_sharing():
    """Grouped (cascade) contexts against the flat path pinned above: every sample's keys copied out physically."""
    cfg = tiny_cfg(num_prefixes=3, samples_per_prefix=2, prefix_len=(2, 9), suffix_len=(0, 7), seed=13)
    w = wl.make_cascade_workload(cfg, shared_len=6, poison=True)
    assert list(w["n_samples"]) == [6, 2, 2, 2] and list(w["group_first_sample"]) == [0, 0, 2, 4]
    out, lse, _ = oracle.attend(w)
    flat = wl.flatten_cascade(w)
    assert list(flat["prefix_lens"]) == [6 + int(w["prefix_lens"][1 + s // 2]) for s in range(6)]
    fo, fl, _ = oracle.attend(flat)
    assert np.allclose(out, fo, rtol=0, atol=TOL) and np.allclose(lse, fl, rtol=0, atol=TOL)
    for s in range(6):                       # and against the Python streaming form on the grouped layout
        x, V = rec.logits(w, s, 3)
        o, m, l = rec.task2_deferred(x, V)
        assert np.allclose(o, out[s * 4 + 3], rtol=0, atol=TOL) and abs(m + math.log(l) - lse[s * 4 + 3]) < TOL
        assert len(x) == 6 + int(w["prefix_lens"][1 + s // 2]) + int(w["suffix_lens"][s])


def test_cascade_counts_every_token_of_every_level_once():
    # equal keys => uniform weights; V[..., 0] = token id => out[0] = mean id over the sample's groups and suffix
    cfg = tiny_cfg(num_prefixes=2, samples_per_prefix=2, prefix_len=(3, 5), suffix_len=(0, 0), seed=2)
    w = wl.make_cascade_workload(cfg, shared_len=4)
    w["prefix_k"][:] = bits(0.25)
    n_tok = w["prefix_k"].shape[0]
    for t in range(n_tok):
        w["prefix_v"][t, :, 0] = bits(float(t))
    out, lse, _ = oracle.attend(w)
    tok = np.concatenate([[0], np.cumsum(w["prefix_lens"])])
    for s in range(4):
        ids = list(range(0, 4)) + list(range(int(tok[1 + s // 2]), int(tok[2 + s // 2])))
        assert np.allclose(out.reshape(4, 4, -1)[s, :, 0], np.mean(ids), rtol=0, atol=1e-11)
    # overlapping groups that are not nested also work: samples 1..2 get an extra group
    w2 = dict(w)
    lens = np.array(list(w["prefix_lens"]), np.int32)
    w2["prefix_lens"] = lens; w2["n_samples"] = np.array([4, 2, 2], np.int32); w2["group_first_sample"] = np.array([0, 1, 2], np.int32)
    out2, _, _ = oracle.attend(w2)
    want = {0: [0, 1, 2, 3], 1: list(range(0, 4 + int(lens[1]))), 2: list(range(0, int(tok[3]))), 3: [0, 1, 2, 3] + list(range(int(tok[2]), int(tok[3])))}
    for s in range(4):
        assert np.allclose(out2.reshape(4, 4, -1)[s, :, 0], np.mean(want[s]), rtol=0, atol=1e-11)


def test_append_puts_the_new_token_last_in_every_context():
    cfg = tiny_cfg(samples_per_prefix=4, suffix_len=(1, 9))
    w = wl.make_workload(cfg)                       # pages exist for lengths up to the drawn ones
    full = np.array(w["suffix_lens"]).copy()
    w["suffix_lens"] = np.maximum(full - 1, 0).astype(np.int32)   # one slot short of what the pages hold
    grow = full > 0
    new_k = wl.normal_bf16((4, 2, 8), 99, 1); new_v = wl.normal_bf16((4, 2, 8), 99, 2)
    w2 = oracle.append_kv(w, new_k, new_v) if grow.all() else None
    if w2 is None:
        pytest.skip("a sample drew length 0")
    assert list(w2["suffix_lens"]) == list(w["suffix_lens"] + 1) and w["pool_k"] is not w2["pool_k"]
    for s in range(4):
        for h in range(4):
            q, K, V = rec.gather_context(w2, s, h)
            q0, K0, V0 = rec.gather_context(w, s, h)
            assert np.array_equal(K[:-1], K0) and np.array_equal(V[:-1], V0)
            assert np.array_equal(K[-1], rec.bf16_bits_to_f64(new_k[s, h // 2])) and np.array_equal(V[-1], rec.bf16_bits_to_f64(new_v[s, h // 2]))
    with pytest.raises(IndexError):
        w3 = dict(w); w3["suffix_lens"] = (np.array(w["page_indptr"][1:]) - np.array(w["page_indptr"][:-1])) * 4
        oracle.append_kv(w3, new_k, new_v)


# ---------------------------------------------------------------- prefill (causal) oracle
def _prefill_inputs(lens, Hq=4, Hkv=2, D=8, seed=31):
    T = int(np.sum(lens))
    return (wl.normal_bf16((T, Hq, D), seed, 1), wl.normal_bf16((T, Hkv, D), seed, 2), wl.normal_bf16((T, Hkv, D), seed, 3))


def test_causal_oracle_equals_the_pinned_operator_on_growing_prefixes():
    """Token i of a prompt = one sample whose whole context is the prompt's first i+1 tokens, copied out."""
    lens = [5, 1, 7]
    q, k, v = _prefill_inputs(lens)
    out, lse = oracle.causal_attend(q, k, v, lens, 0.35)
    offs = np.concatenate([[0], np.cumsum(lens)])
    ks, vs, plens = [], [], []
    for p, L in enumerate(lens):
        for i in range(L):
            ks.append(k[offs[p]: offs[p] + i + 1]); vs.append(v[offs[p]: offs[p] + i + 1]); plens.append(i + 1)
    T = sum(lens)
    flat = dict(prefix_lens=np.array(plens, np.int32), n_samples=np.ones(T, np.int32), suffix_lens=np.zeros(T, np.int32),
                num_q_heads=4, num_kv_heads=2, head_dim=8, page_size=4, sm_scale=0.35, q=q,
                prefix_k=np.concatenate(ks), prefix_v=np.concatenate(vs),
                pool_k=np.zeros((1, 2, 4, 8), np.uint16), pool_v=np.zeros((1, 2, 4, 8), np.uint16),
                page_indptr=np.zeros(T + 1, np.int32), page_indices=np.zeros(0, np.int32))
    fo, fl, _ = oracle.attend(flat)
    assert np.allclose(out, fo, rtol=0, atol=TOL) and np.allclose(lse, fl, rtol=0, atol=TOL)
    # the first token of every prompt sees only itself
    for p in range(3):
        for h in range(4):
            r = offs[p] * 4 + h
            assert np.array_equal(out[r], rec.bf16_bits_to_f64(v[offs[p], h // 2]))


def test_causal_oracle_matches_torch_masked_softmax():
    torch = pytest.importorskip("torch")
    lens = [9]
    q, k, v = _prefill_inputs(lens, Hq=2, Hkv=1, D=11, seed=5)
    out, lse = oracle.causal_attend(q, k, v, lens, 0.3)
    Q = torch.from_numpy(rec.bf16_bits_to_f64(q)); K = torch.from_numpy(rec.bf16_bits_to_f64(k))[:, 0]; V = torch.from_numpy(rec.bf16_bits_to_f64(v))[:, 0]
    for h in range(2):
        S = (Q[:, h] @ K.T) * 0.3
        S = S.masked_fill(torch.triu(torch.ones(9, 9, dtype=torch.bool), diagonal=1), float("-inf"))
        ref = torch.softmax(S, 1) @ V
        assert np.allclose(out.reshape(9, 2, 11)[:, h], ref.numpy(), rtol=0, atol=TOL)
        assert np.allclose(lse.reshape(9, 2)[:, h], torch.logsumexp(S, 1).numpy(), rtol=0, atol=TOL)
    rows = np.array([3, 17, 0])
    o2, l2 = oracle.causal_attend(q, k, v, lens, 0.3, rows=rows)
    assert np.array_equal(o2, out[rows]) and np.array_equal(l2, lse[rows])
