"""Host-side logic that needs no GPU: the C-ABI library loads and exports every symbol the header
declares, the planner's work lists cover every key / token exactly once, and misuse is reported
through status codes."""
import os
import re

import numpy as np
import pytest

import psa_workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def make_plan(prefix_lens, n_samples, suffix_lens, Hq=32, Hkv=8, D=128, sms=148, **kw):
    from paper_2502_02534_b200 import Plan
    return Plan(prefix_lens, n_samples, suffix_lens, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, num_sms=sms, **kw)


def test_library_exports_every_declared_symbol():
    import paper_2502_02534_b200 as psa
    header = open(os.path.join(ROOT, "include", "psa.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(psa_[a-z_0-9]+)\s*\(", header))
    assert declared == set(psa.EXPORTED_SYMBOLS)
    lib = psa.library()
    for name in declared:
        assert hasattr(lib, name), name
    assert lib.psa_version() >= 100
    assert psa.status_string(0) == "ok" and "workspace" in psa.status_string(3)


@pytest.mark.parametrize("name", list(wl.CONFIGS))
@pytest.mark.parametrize("sms", [1, 7, 148])
def test_work_lists_cover_everything_exactly_once(name, sms):
    cfg = wl.CONFIGS[name]
    L, N, S = wl.draw_lengths(cfg)
    plan = make_plan(L, N, S, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, sms)
    G = cfg.num_q_heads // cfg.num_kv_heads
    info = plan.info
    pre, suf = plan.prefix_items(), plan.suffix_items()
    assert len(pre) == info.num_prefix_items and len(suf) == info.num_suffix_items
    tok_off = np.concatenate([[0], np.cumsum(L)]); first = np.concatenate([[0], np.cumsum(N)])
    # prefix: every (prompt, kv head, row, key) exactly once
    rows_seen = set()
    for p in range(len(L)):
        cover = np.zeros((cfg.num_kv_heads, int(N[p]) * G, int(L[p])), dtype=np.int8) if L[p] * N[p] * G <= 4e6 else None
        for it in pre[pre[:, 6] == p]:
            t0, nk, kv, s0, nr, prow, _, split = (int(v) for v in it)
            assert 0 < nk <= info.prefix_tiles_per_item * 128 and 0 < nr <= 256
            assert tok_off[p] <= t0 and t0 + nk <= tok_off[p + 1]
            assert (t0 - tok_off[p]) % 128 == 0
            r0 = (s0 - first[p]) * G
            assert first[p] <= s0 and r0 + nr <= N[p] * G
            if cover is not None:
                cover[kv, r0:r0 + nr, t0 - tok_off[p]:t0 - tok_off[p] + nk] += 1
            for r in range(prow, prow + nr):
                assert r not in rows_seen
                rows_seen.add(r)
        if cover is not None:
            assert (cover == 1).all()
    # suffix: every (sample, kv head, token) exactly once, chunk-aligned
    C = info.suffix_chunk_tokens
    assert C % 16 == 0
    seen = {}
    for s, kv, t0, prow in suf:
        assert t0 % C == 0 and t0 < S[s]
        assert (s, kv, t0) not in seen
        seen[(int(s), int(kv), int(t0))] = prow
        for r in range(prow, prow + G):
            assert r not in rows_seen
            rows_seen.add(r)
    assert len(seen) == sum(cfg.num_kv_heads * -(-int(x) // C) for x in S)
    assert rows_seen == set(range(info.num_partial_rows))
    assert plan.workspace_bytes >= info.num_partial_rows * (cfg.head_dim + 1) * 4


def test_planner_fills_the_machine_on_the_named_configurations():
    for name, cfg in wl.CONFIGS.items():
        if name == "cfg1":
            continue
        L, N, S = wl.draw_lengths(cfg)
        info = make_plan(L, N, S, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim).info
        # the two stages run side by side: the prefix stage takes a good part of the SMs (fewer, longer items when it is
        # tensor-bound and the suffix stage can use the bandwidth meanwhile), the rest is left to the suffix stage
        assert info.num_prefix_items >= 0.4 * 148, name
        # the suffix stage is bound by HBM as a whole: at least one block per SM, and enough of them in flight
        assert info.num_suffix_items >= 1.5 * 148, name


def test_planner_weighs_the_two_stages_against_each_other():
    """A tensor-bound prefix stage (many rows per KV head) beside a large suffix stage is cut into few long items that
    leave SMs to the suffix stage; without a suffix stage the same prefix is spread over the whole machine.  Suffix items
    stay whole samples as long as the longest one is a small part of the stage."""
    L, N = [8192], [256]
    big = make_plan(L, N, [2048] * 256, Hq=64, Hkv=8).info
    none = make_plan(L, N, [0] * 256, Hq=64, Hkv=8).info
    assert big.num_prefix_items <= 74 < 148 * 0.8 <= none.num_prefix_items
    assert big.prefix_tiles_per_item > none.prefix_tiles_per_item
    assert big.suffix_chunk_tokens >= 2048 and big.num_suffix_items == 256 * 8
    # one very long sample among short ones is still split, so that it does not become the tail of the stage
    lens = [64] * 63 + [60000]
    skew = make_plan([128], [64], lens, Hq=32, Hkv=8).info
    assert skew.suffix_chunk_tokens < 60000 and skew.num_suffix_items > 64 * 8


def test_bad_arguments_give_status_codes():
    from paper_2502_02534_b200 import PsaError
    ok = dict(prefix_lens=[10], n_samples=[2], suffix_lens=[1, 2])
    cases = [
        (dict(ok, Hq=6, Hkv=4), 1), (dict(ok, D=96), 2), (dict(ok, Hq=48, Hkv=1), 2), (dict(ok, page_size=32), 2),
        (dict(ok, sm_scale=-1.0), 1), (dict(ok, prefix_lens=[-1]), 1), (dict(ok, suffix_lens=[1, -2]), 1),
        (dict(ok, n_samples=[-2]), 1),
    ]
    for kw, status in cases:
        with pytest.raises(PsaError) as e:
            make_plan(**kw)
        assert e.value.status == status, kw
    plan = make_plan(**ok)
    assert plan.info.num_samples == 2


def test_empty_problems_plan_cleanly():
    plan = make_plan([], [], [])
    assert plan.info.num_prefix_items == 0 and plan.info.num_suffix_items == 0 and plan.info.kernel_launches == 0
    plan = make_plan([0, 5], [3, 0], [0, 0, 0])
    assert plan.info.num_prefix_items == 0 and plan.info.num_suffix_items == 0 and plan.info.kernel_launches == 1


def test_cascade_plan_covers_every_group_key_once_and_limits_levels():
    from paper_2502_02534_b200 import Plan, PsaError
    first, n, lens = [0, 0, 4, 2], [8, 4, 4, 3], [1000, 130, 77, 300]       # nested and overlapping groups
    S = [5] * 8
    plan = Plan([], [], S, num_q_heads=8, num_kv_heads=2, head_dim=128, num_sms=148, groups=(first, n, lens))
    items = plan.prefix_items()
    tok = np.concatenate([[0], np.cumsum(lens)])
    G = 4
    for g in range(4):
        cover = np.zeros((2, n[g] * G, lens[g]), dtype=np.int8)
        for t0, nk, kv, s0, nr, prow, grp, split in items[items[:, 6] == g]:
            r0 = (s0 - first[g]) * G
            assert first[g] <= s0 and r0 + nr <= n[g] * G and tok[g] <= t0 and t0 + nk <= tok[g + 1]
            cover[kv, r0:r0 + nr, t0 - tok[g]:t0 - tok[g] + nk] += 1
        assert (cover == 1).all()
    rows = np.concatenate([np.arange(p, p + nr) for _, _, _, _, nr, p, _, _ in items])
    assert len(set(rows.tolist())) == len(rows)
    with pytest.raises(PsaError):
        Plan([], [], S, num_q_heads=8, num_kv_heads=2, head_dim=128, num_sms=148, groups=([0], [9], [10]))
