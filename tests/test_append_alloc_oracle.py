"""Pins of the oracle for the append with page allocation (oracle.append_kv_alloc): a hand-written case with every
array spelled out, agreement with the plain append when every page is already assigned, and a brute-force read-back
of every sample's context through the page table."""
import numpy as np

import oracle
import psa_workloads as wl


def tiny():
    # 4 samples, page size 16, one KV head, D = 16; slots (capacity): 2, 1, 2, 1; lengths 16, 3, 0, 16
    Hkv, D, page = 1, 16, 16
    pool = np.zeros((8, Hkv, page, D), np.uint16)
    w = dict(page_size=page, num_kv_heads=Hkv, head_dim=D, pool_k=pool.copy(), pool_v=pool.copy(),
             page_indptr=np.array([0, 2, 3, 5, 6], np.int32), page_indices=np.array([4, -1, 2, -1, -1, 6], np.int32),
             suffix_lens=np.array([16, 3, 0, 16], np.int32))
    new_k = (np.arange(4 * Hkv * D, dtype=np.uint16) + 100).reshape(4, Hkv, D)
    new_v = (np.arange(4 * Hkv * D, dtype=np.uint16) + 900).reshape(4, Hkv, D)
    return w, new_k, new_v


def test_hand_written_case():
    w, new_k, new_v = tiny()
    out, count, skipped = oracle.append_kv_alloc(w, new_k, new_v, np.array([7, 0, 5, 1], np.int32), 3)   # stack: 7 0 5 | top = 5
    # sample 0 (S = 16) opens slot 1 with page 5; sample 1 (S = 3) writes into its page 2; sample 2 (S = 0) opens slot 0
    # with page 0; sample 3 (S = 16) has no slot left (capacity 1): skipped, and keeps the stack untouched
    assert out["page_indices"].tolist() == [4, 5, 2, 0, -1, 6]
    assert out["suffix_lens"].tolist() == [17, 4, 1, 16] and count == 1 and skipped == [3]
    assert np.array_equal(out["pool_k"][5, 0, 0], new_k[0, 0]) and np.array_equal(out["pool_v"][5, 0, 0], new_v[0, 0])
    assert np.array_equal(out["pool_k"][2, 0, 3], new_k[1, 0]) and np.array_equal(out["pool_k"][0, 0, 0], new_k[2, 0])
    touched = np.zeros(out["pool_k"].shape[:3], bool).transpose(0, 2, 1)
    touched[5, 0] = touched[2, 3] = touched[0, 0] = True
    assert (out["pool_k"].transpose(0, 2, 1, 3)[~touched] == 0).all()            # nothing else moved
    assert w["page_indices"].tolist() == [4, -1, 2, -1, -1, 6] and w["suffix_lens"].tolist() == [16, 3, 0, 16]   # input left alone
    # an empty stack: the two samples that need a page are skipped, the one that does not is served
    out, count, skipped = oracle.append_kv_alloc(w, new_k, new_v, np.zeros(0, np.int32), 0)
    assert skipped == [0, 2, 3] and count == 0 and out["suffix_lens"].tolist() == [16, 4, 0, 16]
    # planned bounds: a sample at its bound is skipped even though it has room
    w2 = dict(w, suffix_bounds=np.array([40, 3, 40, 40], np.int32))
    out, count, skipped = oracle.append_kv_alloc(w2, new_k, new_v, np.array([7, 0, 5, 1], np.int32), 4)
    assert skipped == [1, 3] and out["suffix_lens"].tolist() == [17, 3, 1, 16] and count == 2
    assert out["page_indices"].tolist() == [4, 1, 2, 5, -1, 6]


def test_equals_the_plain_append_when_every_page_is_assigned_and_contexts_read_back():
    cfg = wl.PsaConfig("a", 2, 4, 4, 2, 32, (5, 9), (0, 70), permute_pages=True, seed=3)
    w = wl.make_workload(cfg)
    B, Hkv, D, page = 8, 2, 32, 16
    # give every sample two more slots than it uses (20 steps open at most two pages), unassigned; free pages = the pool's slack
    lens = np.asarray(w["suffix_lens"])
    used = (lens + page - 1) // page
    cap = used + 2
    indptr = np.concatenate([[0], np.cumsum(cap)]).astype(np.int32)
    indices = np.full(int(indptr[-1]), -1, np.int32)
    for s in range(B):
        indices[indptr[s]:indptr[s] + used[s]] = w["page_indices"][w["page_indptr"][s]:w["page_indptr"][s + 1]]
    owned = set(int(x) for x in w["page_indices"])
    n_pool = w["pool_k"].shape[0]
    extra = np.zeros((2 * B, Hkv, page, D), np.uint16)
    wa = dict(w, page_indptr=indptr, page_indices=indices, pool_k=np.concatenate([w["pool_k"], extra]), pool_v=np.concatenate([w["pool_v"], extra]))
    free = np.array([p for p in range(n_pool + 2 * B) if p not in owned], np.int32)
    for step in range(20):
        new_k = wl.normal_bf16((B, Hkv, D), 50 + step, 1); new_v = wl.normal_bf16((B, Hkv, D), 50 + step, 2)
        before = np.asarray(wa["suffix_lens"]).copy()
        need = int(np.sum(before % page == 0))
        count0 = len(free)
        # the plain append on a copy whose lists already hold the pages this step will pop (in sample order, from the top)
        pre = dict(wa, page_indices=wa["page_indices"].copy())
        top = count0
        for s in range(B):
            if before[s] % page == 0:
                top -= 1
                pre["page_indices"][indptr[s] + before[s] // page] = free[top]
        plain = oracle.append_kv(pre, new_k, new_v)
        wa, count, skipped = oracle.append_kv_alloc(wa, new_k, new_v, free, count0)
        free = free[:count]
        assert skipped == [] and count == count0 - need
        assert np.array_equal(wa["pool_k"], plain["pool_k"]) and np.array_equal(wa["pool_v"], plain["pool_v"])
        assert np.array_equal(wa["suffix_lens"], plain["suffix_lens"]) and np.array_equal(wa["page_indices"], pre["page_indices"])
        # brute-force read-back: the last key / value of every context is the appended token
        for s in range(B):
            t = int(wa["suffix_lens"][s]) - 1
            pg = int(wa["page_indices"][indptr[s] + t // page])
            assert np.array_equal(wa["pool_k"][pg, :, t % page], new_k[s]) and np.array_equal(wa["pool_v"][pg, :, t % page], new_v[s])
        pages = [int(x) for x in wa["page_indices"] if x >= 0]
        assert len(pages) == len(set(pages)) and not (set(pages) & set(int(x) for x in free))      # no page has two owners
    # the grown contexts attend like a workload whose page lists were complete from the start
    ref_o, ref_l, _ = oracle.attend(wa)
    assert np.isfinite(ref_o).all() and np.isfinite(ref_l).all()
