"""GPU parity: the CUDA library (through its C ABI) against the CPU fp64 oracle, element by element,
on the same seeded inputs.  Tolerances: max |err| <= 1e-2 on out, <= 1e-3 on lse (absolute)."""
import math

import numpy as np
import pytest

import oracle
import psa_workloads as wl
from psa_testlib import assert_close, make_plan, run_gpu, to_device

pytestmark = pytest.mark.gpu


def cfg(**kw):
    base = dict(name="t", num_prefixes=1, samples_per_prefix=4, num_q_heads=8, num_kv_heads=2, head_dim=128,
                prefix_len=(300, 300), suffix_len=(0, 200), page_size=16, seed=11)
    base.update(kw)
    return wl.PsaConfig(**base)


def check(w, out_dtype="bf16", rows=None, what="", **plan_kw):
    plan = make_plan(w, out_dtype, **plan_kw) if plan_kw else None
    out, lse, plan = run_gpu(w, out_dtype, plan=plan)
    if rows is None:
        ref_o, ref_l, _ = oracle.attend(w)
    else:
        ref_o, ref_l, _ = oracle.attend(w, rows=rows)
        out, lse = out[rows], lse[rows]
    return assert_close(out, lse, ref_o, ref_l, what)


# ------------------------------------------------------------------ the named configurations
@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3"])
@pytest.mark.parametrize("out_dtype", ["bf16", "f32"])
def test_named_config_every_element(name, out_dtype):
    w = wl.make_workload(wl.CONFIGS[name], poison=True)
    check(w, out_dtype, what=f"{name}/{out_dtype}")


@pytest.mark.parametrize("name", ["cfg4", "cfg5"])
def test_full_size_config_every_element(name):
    """Full size, the launch configuration the benchmark times (default plan, bf16 output), every element against
    the oracle (a few seconds of CPU time each)."""
    w = wl.make_workload(wl.CONFIGS[name], poison=True)
    out, lse, plan = run_gpu(w, "bf16")
    ref_o, ref_l, _ = oracle.attend(w)
    assert_close(out, lse, ref_o, ref_l, name)


# ------------------------------------------------------------------ shapes around every tile / page edge
@pytest.mark.parametrize("D,G", [(128, 4), (128, 8), (128, 1), (128, 2), (64, 4), (64, 8), (64, 1), (64, 2)])
def test_head_dim_and_group_sizes(D, G):
    w = wl.make_workload(cfg(head_dim=D, num_q_heads=2 * G, num_kv_heads=2, samples_per_prefix=5,
                             prefix_len=(333, 333), suffix_len=(0, 150)), poison=True)
    check(w, "f32", what=f"D{D} G{G}")


@pytest.mark.parametrize("L", [0, 1, 15, 127, 128, 129, 255, 256, 257, 1000])
def test_prefix_lengths_around_tile_edges(L):
    w = wl.make_workload(cfg(prefix_len=(L, L), suffix_len=(1, 40)), poison=True)
    check(w, "f32", what=f"L{L}")


def test_suffix_lengths_around_page_and_chunk_edges():
    lens = [0, 1, 15, 16, 17, 31, 32, 33, 63, 64, 65, 127, 128, 129, 255, 256, 257, 511, 513, 1023, 1025]
    c = cfg(samples_per_prefix=len(lens), prefix_len=(64, 64))
    w = wl.make_workload(c, poison=True, lengths=([64], [len(lens)], lens))
    check(w, "f32", what="suffix edges")
    check(w, "bf16", what="suffix edges bf16")


@pytest.mark.parametrize("n_samples", [1, 31, 32, 33, 63, 64, 65, 70])
def test_row_counts_around_row_tile_edges(n_samples):
    # G = 4: 32 samples fill one 128-row tile, 64 fill the 256 rows of one item
    w = wl.make_workload(cfg(samples_per_prefix=n_samples, num_q_heads=4, num_kv_heads=1,
                             prefix_len=(200, 200), suffix_len=(0, 20)), poison=True)
    check(w, "f32", what=f"N{n_samples}")


def test_many_prompts_ragged_everything():
    rng = np.random.default_rng(4)
    P = 7
    prefix_lens = [0, 1, 130, 777, 128, 2049, 300]
    n_samples = [3, 0, 40, 2, 70, 1, 5]
    B = sum(n_samples)
    suffix_lens = rng.integers(0, 300, size=B)
    suffix_lens[:3] = 0                      # prompt 0 has no prefix: those rows have an empty context
    w = wl.make_workload(cfg(num_prefixes=P, permute_pages=True), poison=True,
                         lengths=(prefix_lens, n_samples, suffix_lens))
    eo, el = check(w, "f32", what="ragged")
    out, lse, _ = run_gpu(w, "bf16")
    assert (lse[: 3 * 8] == -math.inf).all() and (out[: 3 * 8] == 0).all()


def test_all_contexts_empty():
    w = wl.make_workload(cfg(prefix_len=(0, 0), suffix_len=(0, 0)))
    out, lse, _ = run_gpu(w, "bf16")
    assert (out == 0).all() and (lse == -math.inf).all()


def test_multi_split_prefix_and_multi_chunk_suffix_small_sm_count():
    # planning for few SMs and for many SMs must give the same numbers
    w = wl.make_workload(cfg(prefix_len=(3000, 3000), suffix_len=(100, 900), samples_per_prefix=6), poison=True)
    for sms in (1, 4, 148, 1000):
        check(w, "f32", what=f"sms{sms}", num_sms=sms)


# ------------------------------------------------------------------ every prefix block shape
@pytest.mark.parametrize("kernel", [1, 2, 3, 4])          # small, long, decoupled, coupled (PSA_PREFIX_KERNEL_*)
def test_every_prefix_block_shape_against_the_oracle(kernel):
    """The planner picks a block shape by the items' rows and lengths; here each shape is forced in turn over row counts
    and prefix lengths around its tile edges (64- and 128-key tiles, one and two row tiles, one and several key ranges
    per prompt), every element against the oracle.  Items of more than 128 rows take a two-row-tile shape regardless."""
    shapes = [(128, 4, 5, 333), (128, 4, 32, 64), (128, 4, 32, 65), (128, 8, 16, 1000), (64, 4, 20, 700), (64, 8, 7, 129),
              (128, 1, 100, 4097), (128, 2, 64, 63), (128, 4, 70, 777), (128, 4, 64, 2000), (64, 2, 150, 500), (128, 4, 40, 1),
              (128, 4, 40, 127), (128, 4, 40, 128), (128, 4, 40, 192), (128, 4, 40, 193)]
    # the decoupled shape is what the planner takes in steps without suffix work: forced, it is tested there as well
    for suffix in ([(0, 60), (0, 0)] if kernel == 3 else [(0, 60)]):
        for D, G, N, L in shapes:
            w = wl.make_workload(cfg(head_dim=D, num_q_heads=2 * G, num_kv_heads=2, samples_per_prefix=N, prefix_len=(L, L),
                                     suffix_len=suffix), poison=True)
            for tiles in (0, 1, 3):
                check(w, "f32", what=f"kernel {kernel} D{D} G{G} N{N} L{L} S{suffix} tiles {tiles}", prefix_kernel=kernel,
                      prefix_tiles_per_item=tiles)


def test_prefix_only_plan_takes_the_decoupled_block_and_matches():
    """A step without any suffix work (every S_s = 0) lets the prefix grid own the SMs; the planner then picks the
    decoupled block on alternate key tiles for rows that fill most of a row tile."""
    c = cfg(samples_per_prefix=30, num_q_heads=8, num_kv_heads=2, prefix_len=(1500, 1500), suffix_len=(0, 0))
    w = wl.make_workload(c, poison=True)
    check(w, "f32", what="prefix only")
    check(w, "bf16", what="prefix only bf16")


# ------------------------------------------------------------------ layouts, plan reuse
def test_strided_layouts_head_major_prefix_and_token_major_pool():
    import torch
    from paper_2502_02534_b200 import decode
    w = wl.make_workload(cfg(), poison=True)
    ref_o, ref_l, _ = oracle.attend(w)
    dev = to_device(w)
    Hkv, D, page = w["num_kv_heads"], w["head_dim"], w["page_size"]
    L = w["prefix_k"].shape[0]
    pk = dev["prefix_k"].permute(1, 0, 2).contiguous()      # [Hkv, L, D]
    pv = dev["prefix_v"].permute(1, 0, 2).contiguous()
    sk = dev["pool_k"].permute(0, 2, 1, 3).contiguous()     # [pages, 16, Hkv, D]
    sv = dev["pool_v"].permute(0, 2, 1, 3).contiguous()
    plan = make_plan(w, "f32")
    B, Hq = int(np.sum(w["n_samples"])), w["num_q_heads"]
    out = torch.full((B, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device="cuda")
    decode(plan, dev["q"], pk, pv, sk, sv, dev["page_indptr"], dev["page_indices"], dev["suffix_lens"], out, lse,
           prefix_strides=(D, L * D), pool_strides=(page * Hkv * D, D, Hkv * D))
    torch.cuda.synchronize()
    plan.check_status()
    assert_close(out.double().cpu().numpy().reshape(B * Hq, D), lse.double().cpu().numpy().reshape(-1), ref_o, ref_l, "strided")


def test_plan_reuse_with_shorter_actual_suffixes_and_growth():
    """A plan made for upper bounds serves every step whose lengths stay below them."""
    c = cfg(samples_per_prefix=6, suffix_len=(50, 400))
    w = wl.make_workload(c, poison=False)
    bounds = np.asarray(w["suffix_lens"]).copy()
    plan = make_plan(w, "f32", suffix_bounds=bounds)
    dev = to_device(w)
    import torch
    for shrink in (0, 1, 17, 49):
        w2 = dict(w)
        w2["suffix_lens"] = np.maximum(bounds - shrink, 0).astype(np.int32)
        dev["suffix_lens"] = torch.from_numpy(w2["suffix_lens"]).cuda()
        out, lse, _ = run_gpu(w2, "f32", plan=plan, dev=dev)
        ref_o, ref_l, _ = oracle.attend(w2)
        assert_close(out, lse, ref_o, ref_l, f"shrink{shrink}")


# ------------------------------------------------------------------ adversarial values
def test_late_large_logit_forces_accumulator_rescale():
    """A key far into the context with a logit ~40 above everything before it: the running maximum
    must move and the accumulated output must be rescaled (prefix in TMEM, suffix in registers)."""
    c = cfg(samples_per_prefix=3, prefix_len=(700, 700), suffix_len=(90, 90), num_q_heads=4, num_kv_heads=1)
    w = wl.make_workload(c, poison=True)
    D = w["head_dim"]
    q0 = wl.bf16_bits_to_f32(w["q"][0, 0])
    big = wl.f32_to_bf16_bits(q0 * (40.0 / (w["sm_scale"] * float(q0 @ q0))))
    w["prefix_k"][650, 0] = big                # tile 5 of the prefix
    pg = w["page_indices"][w["page_indptr"][1] + 80 // 16]
    q1 = wl.bf16_bits_to_f32(w["q"][1, 1])
    w["pool_k"][pg, 0, 80 % 16] = wl.f32_to_bf16_bits(q1 * (60.0 / (w["sm_scale"] * float(q1 @ q1))))
    ref_o, ref_l, _ = oracle.attend(w)
    assert ref_l[0] > 35 and ref_l[1 * 4 + 1] > 55
    out, lse, _ = run_gpu(w, "f32")
    assert_close(out, lse, ref_o, ref_l, "rescale")


def test_all_keys_equal_closed_form():
    c = cfg(samples_per_prefix=2, prefix_len=(257, 257), suffix_len=(33, 33), num_q_heads=4, num_kv_heads=1)
    w = wl.make_workload(c, poison=True)
    k = w["prefix_k"][0, 0].copy()
    w["prefix_k"][:] = k
    pk = w["pool_k"]
    pk[pk != wl.BF16_NAN] = 0
    for pg in w["page_indices"]:
        n = w["pool_k"][pg, 0].shape[0]
        for t in range(n):
            if w["pool_k"][pg, 0, t, 0] != wl.BF16_NAN:
                w["pool_k"][pg, 0, t] = k
    out, lse, _ = run_gpu(w, "f32")
    q = wl.bf16_bits_to_f32(w["q"]).astype(np.float64).reshape(-1, 128)
    x = w["sm_scale"] * (q @ wl.bf16_bits_to_f32(k).astype(np.float64))
    assert np.max(np.abs(lse - (x + math.log(257 + 33)))) <= 1e-3
    ref_o, ref_l, _ = oracle.attend(w)
    assert_close(out, lse, ref_o, ref_l, "equal keys")


def test_permuting_samples_permutes_rows_only():
    c = cfg(samples_per_prefix=8, permute_pages=True)
    w = wl.make_workload(c, poison=True)
    out, lse, _ = run_gpu(w, "f32")
    perm = np.array([5, 2, 7, 0, 3, 6, 1, 4])
    B, Hq, D = 8, w["num_q_heads"], w["head_dim"]
    w2 = dict(w)
    w2["q"] = w["q"][perm]; w2["suffix_lens"] = w["suffix_lens"][perm]
    lists = [w["page_indices"][w["page_indptr"][s]: w["page_indptr"][s + 1]] for s in range(B)]
    w2["page_indices"] = np.concatenate([lists[s] for s in perm]).astype(np.int32)
    w2["page_indptr"] = np.concatenate([[0], np.cumsum([len(lists[s]) for s in perm])]).astype(np.int32)
    o2, l2, _ = run_gpu(w2, "f32")
    # the work lists differ (chunks are ordered by length), so equality is up to summation order
    assert np.max(np.abs(o2.reshape(B, Hq, D) - out.reshape(B, Hq, D)[perm])) <= 1e-5
    assert np.max(np.abs(l2.reshape(B, Hq) - lse.reshape(B, Hq)[perm])) <= 1e-5


# ------------------------------------------------------------------ stages and the host-buffer entry point
def test_stage_entry_points_compose_to_decode():
    import torch
    from paper_2502_02534_b200 import decode
    w = wl.make_workload(cfg(), poison=True)
    dev = to_device(w)
    plan = make_plan(w, "f32")
    B, Hq, D = int(np.sum(w["n_samples"])), w["num_q_heads"], w["head_dim"]
    out = torch.zeros((B, Hq, D), dtype=torch.float32, device="cuda"); lse = torch.zeros((B, Hq), dtype=torch.float32, device="cuda")
    args = (plan, dev["q"], dev["prefix_k"], dev["prefix_v"], dev["pool_k"], dev["pool_v"], dev["page_indptr"],
            dev["page_indices"], dev["suffix_lens"], out, lse)
    for stage in ("suffix", "prefix", "merge"):
        decode(*args, stage=stage)
    torch.cuda.synchronize()
    ref_o, ref_l, _ = oracle.attend(w)
    assert_close(out.double().cpu().numpy().reshape(B * Hq, D), lse.double().cpu().numpy().reshape(-1), ref_o, ref_l, "stages")


def test_many_fused_steps_on_one_workspace_and_counter_wrap_around():
    """The merge stage of a fused step learns that the prefix stage is complete from two counters in the workspace
    (prefix launches, prefix blocks done) that no kernel ever resets.  Many steps in a row, a stand-alone prefix stage
    in between (it must not count), a CUDA-graph replay, and counters preset just below 2^32 so that they wrap
    during the run: every step must give the oracle's result."""
    import torch
    from paper_2502_02534_b200 import decode
    w = wl.make_workload(cfg(prefix_len=(900, 900), suffix_len=(0, 300), samples_per_prefix=40), poison=True)
    ref_o, ref_l, _ = oracle.attend(w)
    dev = to_device(w)
    plan = make_plan(w, "f32", num_sms=16)      # few SMs in the plan: several prefix blocks per SM, several waves
    plan.bind_workspace()
    n_blocks = plan.info.num_prefix_items
    assert n_blocks > 1 and plan.info.num_suffix_items > 0
    B, Hq, D = int(np.sum(w["n_samples"])), w["num_q_heads"], w["head_dim"]
    out = torch.empty((B, Hq, D), dtype=torch.float32, device="cuda")
    lse = torch.empty((B, Hq), dtype=torch.float32, device="cuda")

    def step(stage="all"):
        decode(plan, dev["q"], dev["prefix_k"], dev["prefix_v"], dev["pool_k"], dev["pool_v"], dev["page_indptr"],
               dev["page_indices"], dev["suffix_lens"], out, lse, stage=stage)

    def check(what):
        torch.cuda.synchronize()
        plan.check_status()
        assert_close(out.double().cpu().numpy().reshape(B * Hq, D), lse.double().cpu().numpy().reshape(-1), ref_o, ref_l, what)

    for i in range(25):
        out.fill_(float("nan")); lse.fill_(float("nan"))
        step()
        if i % 6 == 0:
            check(f"step {i}")
        if i % 5 == 0:
            step("prefix")                      # a stand-alone stage leaves the counters alone
    check("after 25 steps")
    words = plan.workspace[:64 * 4].view(torch.int32)
    assert int(words[8]) == 25 and int(words[9]) == 25 * n_blocks

    # preset the counters a few launches below the wrap of the 32-bit product launches x blocks
    launches = (2 ** 32 - 3 * n_blocks) // n_blocks
    words[8] = int(np.array(launches, dtype=np.uint32).view(np.int32)) if launches >= 2 ** 31 else launches
    words[9] = int(np.array((launches * n_blocks) % 2 ** 32, dtype=np.uint32).view(np.int32))
    torch.cuda.synchronize()
    for i in range(8):
        out.fill_(float("nan")); lse.fill_(float("nan"))
        step()
        check(f"wrap step {i}")

    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for _ in range(2):
            step()
        side.synchronize()
        with torch.cuda.graph(g, stream=side):
            for _ in range(6):
                step()
    out.fill_(float("nan"))
    g.replay(); g.replay()
    check("graph replays")


def test_decode_from_host_buffers():
    import torch
    from paper_2502_02534_b200 import decode_host
    from paper_2502_02534_b200.binding import host_staging_bytes
    w = wl.make_workload(wl.CONFIGS["cfg1"], poison=True)
    plan = make_plan(w, "bf16")
    plan.bind_workspace()
    B, Hq, D = int(np.sum(w["n_samples"])), w["num_q_heads"], w["head_dim"]
    nbytes = host_staging_bytes(plan, w["prefix_k"].shape[0], w["pool_k"].shape[0], len(w["page_indices"]))
    staging = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    out = torch.empty((B, Hq, D), dtype=torch.bfloat16).pin_memory(); lse = torch.empty((B, Hq), dtype=torch.float32).pin_memory()
    i32 = lambda a: np.ascontiguousarray(a, dtype=np.int32)
    decode_host(plan, w["q"], w["prefix_k"], w["prefix_v"], w["pool_k"], w["pool_v"], i32(w["page_indptr"]),
                i32(w["page_indices"]), i32(w["suffix_lens"]), out, lse, staging)
    torch.cuda.synchronize()
    plan.check_status()
    ref_o, ref_l, _ = oracle.attend(w)
    assert_close(out.float().double().numpy().reshape(B * Hq, D), lse.double().numpy().reshape(-1), ref_o, ref_l, "host")


def test_misuse_returns_status_codes_not_faults():
    import torch
    from paper_2502_02534_b200 import PsaError, decode
    w = wl.make_workload(cfg())
    dev = to_device(w)
    plan = make_plan(w)
    plan.bind_workspace()
    B, Hq, D = int(np.sum(w["n_samples"])), w["num_q_heads"], w["head_dim"]
    out = torch.zeros((B, Hq, D), dtype=torch.bfloat16, device="cuda"); lse = torch.zeros((B, Hq), dtype=torch.float32, device="cuda")
    good = [plan, dev["q"], dev["prefix_k"], dev["prefix_v"], dev["pool_k"], dev["pool_v"], dev["page_indptr"],
            dev["page_indices"], dev["suffix_lens"], out, lse]
    for idx in (1, 2, 4, 6, 9, 10):                    # a null pointer in each position
        bad = list(good); bad[idx] = None
        with pytest.raises(PsaError) as e:
            decode(*bad)
        assert e.value.status == 1
    with pytest.raises(PsaError) as e:                 # misaligned q
        bad = list(good); bad[1] = dev["q"].view(-1)[1:]
        decode(*bad)
    assert e.value.status == 1
    with pytest.raises(PsaError) as e:                 # stride not a multiple of 8 elements
        decode(*good, prefix_strides=(Hq * D + 1, D))
    assert e.value.status == 1
    small = plan.workspace[: plan.workspace_bytes - 256]
    keep = plan.workspace
    plan.workspace = small
    with pytest.raises(PsaError) as e:
        decode(*good)
    assert e.value.status == 3
    plan.workspace = keep
    decode(*good)                                      # and the context is still healthy
    torch.cuda.synchronize()
    plan.check_status()


# ------------------------------------------------------------------ seeded random shapes
@pytest.mark.parametrize("seed", list(range(12)))
def test_random_shapes_against_oracle(seed):
    """Random prompts / samples / lengths / head geometry, every element against the oracle.  The shapes cover
    all three prefix block shapes (<= 64 rows with long items, <= 128 rows, > 128 rows) and ragged everything."""
    rng = np.random.default_rng(1000 + seed)
    D = int(rng.choice([64, 128]))
    G = int(rng.choice([1, 2, 4, 8]))
    Hkv = int(rng.choice([1, 2, 3]))
    P = int(rng.integers(1, 5))
    style = seed % 3
    if style == 0:      # few samples, long prompts
        n_samples = rng.integers(0, max(2, 64 // G), size=P); prefix_lens = rng.integers(0, 3000, size=P)
    elif style == 1:    # around one row tile
        n_samples = rng.integers(1, max(2, 160 // G), size=P); prefix_lens = rng.integers(0, 700, size=P)
    else:               # several row tiles (R >= 512 for some prompt)
        n_samples = rng.integers(1, 40, size=P); n_samples[0] = 520 // G + int(rng.integers(0, 9))
        prefix_lens = rng.integers(1, 500, size=P)
    B = int(n_samples.sum())
    suffix_lens = rng.integers(0, int(rng.choice([40, 300, 1100])), size=B)
    c = wl.PsaConfig("fuzz", P, 1, G * Hkv, Hkv, D, (1, 1), (0, 1), permute_pages=bool(seed % 2), seed=seed)
    w = wl.make_workload(c, poison=True, lengths=(prefix_lens, n_samples, suffix_lens))
    check(w, "f32" if seed % 2 else "bf16", what=f"fuzz{seed} D{D} G{G} Hkv{Hkv} N{list(n_samples)} L{list(prefix_lens)}")


# ------------------------------------------------------------------ cascades of shared prefixes
@pytest.mark.parametrize("shared_len,n_prompts,n_samples", [(700, 4, 8), (129, 3, 40), (2000, 16, 4), (64, 2, 150)])
def test_two_level_cascade_against_oracle(shared_len, n_prompts, n_samples):
    """Level 0 (demonstrations shared by every task's samples) batched over ALL samples, level 1 per prompt."""
    c = cfg(num_prefixes=n_prompts, samples_per_prefix=n_samples, prefix_len=(50, 400), suffix_len=(0, 120),
            num_q_heads=8, num_kv_heads=2, permute_pages=True, seed=21)
    w = wl.make_cascade_workload(c, shared_len=shared_len, poison=True)
    eo, el = check(w, "f32", what=f"cascade {shared_len}/{n_prompts}x{n_samples}")
    # the cascade must agree with the same keys planned without sharing (one prefix per sample)
    if n_prompts * n_samples <= 64:
        flat = wl.flatten_cascade(w)
        out_c, lse_c, _ = run_gpu(w, "f32")
        out_f, lse_f, _ = run_gpu(flat, "f32")
        assert np.max(np.abs(out_c - out_f)) <= 2e-3 and np.max(np.abs(lse_c - lse_f)) <= 1e-4


def test_cascade_with_overlapping_unnested_groups_and_five_levels_rejected():
    from paper_2502_02534_b200 import Plan, PsaError
    c = cfg(num_prefixes=1, samples_per_prefix=6, prefix_len=(10, 10), suffix_len=(0, 30), seed=4)
    w = wl.make_workload(c, poison=True)
    lens = np.array([100, 37, 260], np.int32)
    w["prefix_lens"] = lens; w["n_samples"] = np.array([6, 3, 4], np.int32); w["group_first_sample"] = np.array([0, 1, 2], np.int32)
    w["prefix_k"] = wl.normal_bf16((int(lens.sum()), 2, 128), 5, 2); w["prefix_v"] = wl.normal_bf16((int(lens.sum()), 2, 128), 5, 3)
    check(w, "f32", what="overlapping groups")
    with pytest.raises(PsaError) as e:
        Plan([], [], [0, 0], num_q_heads=8, num_kv_heads=2, head_dim=128, num_sms=148,
             groups=([0, 0, 0, 0, 0], [2, 2, 2, 2, 2], [5, 5, 5, 5, 5]))
    assert e.value.status == 2
    with pytest.raises(PsaError) as e:
        Plan([], [], [0, 0], num_q_heads=8, num_kv_heads=2, head_dim=128, num_sms=148, groups=([1], [2], [5]))
    assert e.value.status == 1


def test_bounded_wait_reports_timeout_and_context_survives():
    """A wait that nothing satisfies gives up after its limit, raises PSA_ERR_TIMEOUT through the status word,
    and the next decode on the same context and workspace is correct."""
    import time
    from paper_2502_02534_b200 import PsaError
    w = wl.make_workload(cfg(), poison=True)
    dev = to_device(w)
    plan = make_plan(w, "f32")
    out, lse, _ = run_gpu(w, "f32", plan=plan, dev=dev)
    t0 = time.perf_counter()
    plan.selftest_bounded_wait(limit_ns=2_000_000)           # 2 ms
    with pytest.raises(PsaError) as e:
        plan.check_status()
    assert e.value.status == 5 and time.perf_counter() - t0 < 1.0
    plan.check_status()                                      # cleared
    out2, lse2, _ = run_gpu(w, "f32", plan=plan, dev=dev)
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)


def test_decode_append_decode_loop_reuses_one_plan():
    """Three decode steps with a token appended to every sample in between, one plan made for the final lengths:
    pools and lengths bit-exact against the oracle's append, attention within tolerance at every step."""
    import torch
    from paper_2502_02534_b200 import PsaError, append_kv
    steps = 3
    c = cfg(samples_per_prefix=9, suffix_len=(3, 200), permute_pages=True)
    w = wl.make_workload(c, poison=False)                      # page lists sized for the bounds
    bounds = np.array(w["suffix_lens"]).copy()
    w["suffix_lens"] = (bounds - steps).astype(np.int32)
    plan = make_plan(w, "f32", suffix_bounds=bounds)
    dev = to_device(w)
    B, Hkv, D = 9, w["num_kv_heads"], w["head_dim"]
    for k in range(steps + 1):
        out, lse, _ = run_gpu(w, "f32", plan=plan, dev=dev)
        ref_o, ref_l, _ = oracle.attend(w)
        assert_close(out, lse, ref_o, ref_l, f"loop step {k}")
        if k == steps:
            break
        new_k = wl.normal_bf16((B, Hkv, D), 70 + k, 1); new_v = wl.normal_bf16((B, Hkv, D), 70 + k, 2)
        w = oracle.append_kv(w, new_k, new_v)
        nk = torch.from_numpy(new_k.view(np.int16)).cuda().view(torch.bfloat16)
        nv = torch.from_numpy(new_v.view(np.int16)).cuda().view(torch.bfloat16)
        append_kv(plan, nk, nv, dev["pool_k"], dev["pool_v"], dev["page_indptr"], dev["page_indices"], dev["suffix_lens"])
        torch.cuda.synchronize()
        plan.check_status()
        assert np.array_equal(dev["suffix_lens"].cpu().numpy(), w["suffix_lens"])
        assert np.array_equal(dev["pool_k"].view(torch.int16).cpu().numpy().view(np.uint16), w["pool_k"])
        assert np.array_equal(dev["pool_v"].view(torch.int16).cpu().numpy().view(np.uint16), w["pool_v"])
    # every sample is at its bound now: one more append must change nothing and report PSA_ERR_BOUNDS
    before = dev["pool_k"].clone()
    append_kv(plan, nk, nv, dev["pool_k"], dev["pool_v"], dev["page_indptr"], dev["page_indices"], dev["suffix_lens"])
    torch.cuda.synchronize()
    with pytest.raises(PsaError) as e:
        plan.check_status()
    assert e.value.status == 6
    assert torch.equal(before, dev["pool_k"]) and np.array_equal(dev["suffix_lens"].cpu().numpy(), bounds)


def test_page_table_validator_flags_bad_tables_only():
    import torch
    from paper_2502_02534_b200 import PsaError
    w = wl.make_workload(cfg(samples_per_prefix=6, suffix_len=(20, 90), permute_pages=True))
    dev = to_device(w)
    plan = make_plan(w)
    n_pool = w["pool_k"].shape[0]
    plan.validate_page_table(dev["page_indptr"], dev["page_indices"], dev["suffix_lens"], n_pool)
    plan.check_status()                                                  # a good table passes
    def expect_bad(indptr, indices, lens, pool=n_pool):
        plan.validate_page_table(indptr, indices, lens, pool)
        with pytest.raises(PsaError) as e:
            plan.check_status()
        assert e.value.status == 6
    bad = dev["page_indices"].clone(); bad[3] = n_pool                   # page id outside the pool
    expect_bad(dev["page_indptr"], bad, dev["suffix_lens"])
    bad = dev["page_indices"].clone(); bad[0] = -1
    expect_bad(dev["page_indptr"], bad, dev["suffix_lens"])
    lens = dev["suffix_lens"].clone(); lens[2] += 1                      # above the planned bound
    expect_bad(dev["page_indptr"], dev["page_indices"], lens)
    indptr = dev["page_indptr"].clone(); indptr[1:] -= 1                 # sample 0 one page short (its length needs them all)
    expect_bad(indptr, dev["page_indices"], dev["suffix_lens"])
    expect_bad(dev["page_indptr"], dev["page_indices"], dev["suffix_lens"], pool=1)
    plan.validate_page_table(dev["page_indptr"], dev["page_indices"], dev["suffix_lens"], n_pool)
    plan.check_status()


def test_long_prefix_beside_tiny_suffixes_merge_waits_for_the_prefix_stage():
    """The suffix stage is over long before the prefix stage here, so the merge grid really has to wait on the prefix
    block counter (and, planned lengths aside, some samples have no suffix token at all at run time)."""
    import torch
    from paper_2502_02534_b200 import decode
    w = wl.make_workload(cfg(prefix_len=(6000, 6000), suffix_len=(1, 3), samples_per_prefix=40, num_q_heads=16, num_kv_heads=2),
                         poison=True)
    plan = make_plan(w, "f32", prefix_tiles_per_item=47, suffix_bounds=np.asarray(w["suffix_lens"]) + 4)   # few long prefix items
    w["suffix_lens"] = np.asarray(w["suffix_lens"]).copy(); w["suffix_lens"][::3] = 0
    ref_o, ref_l, _ = oracle.attend(w)
    for _ in range(3):
        out, lse, _ = run_gpu(w, "f32", plan=plan)
        assert_close(out, lse, ref_o, ref_l, "long prefix, tiny suffixes")


def test_two_plans_on_two_streams_with_their_own_workspaces():
    """Concurrent steps are allowed on distinct workspaces: two different problems, each on its own stream, interleaved
    call by call, several rounds without a synchronisation in between."""
    import torch
    from paper_2502_02534_b200 import decode
    probs = []
    for seed, n, L in ((31, 24, 1800), (32, 40, 700)):
        w = wl.make_workload(cfg(prefix_len=(L, L), suffix_len=(0, 500), samples_per_prefix=n, seed=seed), poison=True)
        plan = make_plan(w, "f32"); plan.bind_workspace()
        dev = to_device(w)
        B, Hq, D = n, w["num_q_heads"], w["head_dim"]
        out = torch.full((B, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
        lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device="cuda")
        probs.append((w, plan, dev, out, lse, torch.cuda.Stream()))
    torch.cuda.synchronize()
    for _ in range(6):
        for w, plan, dev, out, lse, st in probs:
            decode(plan, dev["q"], dev["prefix_k"], dev["prefix_v"], dev["pool_k"], dev["pool_v"], dev["page_indptr"],
                   dev["page_indices"], dev["suffix_lens"], out, lse, stream=st)
    torch.cuda.synchronize()
    for w, plan, dev, out, lse, st in probs:
        plan.check_status()
        ref_o, ref_l, _ = oracle.attend(w)
        B, Hq, D = out.shape
        assert_close(out.double().cpu().numpy().reshape(B * Hq, D), lse.double().cpu().numpy().reshape(-1), ref_o, ref_l, "two streams")


# ------------------------------------------------------------------ seeded draws over shapes and planner knobs
@pytest.mark.parametrize("seed", range(24))
def test_drawn_shapes_and_planner_knobs_against_the_oracle(seed):
    """Shapes nobody picked by hand: prompts, samples, heads, lengths, paging and the planner's knobs (block shape, key tiles
    and rows per item, suffix chunk, SM count) drawn from a seeded generator, every element against the oracle."""
    rng = np.random.default_rng(1000 + seed)
    D = int(rng.choice([64, 128]))
    G = int(rng.choice([1, 2, 4, 8]))
    Hkv = int(rng.choice([1, 2, 3]))
    P = int(rng.choice([1, 1, 2, 5]))
    N = int(rng.choice([1, 3, 16, 33, 64 // G + 1, 256 // G]))
    hi = int(rng.choice([1, 70, 200, 700, 2100]))
    lo = hi if rng.random() < 0.5 else max(1, hi // 4)
    s_hi = int(rng.choice([0, 17, 100, 400]))
    c = cfg(num_prefixes=P, samples_per_prefix=N, num_q_heads=G * Hkv, num_kv_heads=Hkv, head_dim=D, prefix_len=(lo, hi),
            suffix_len=(0, s_hi), permute_pages=bool(rng.random() < 0.5), seed=500 + seed)
    w = wl.make_workload(c, poison=True)
    knobs = {}
    if rng.random() < 0.7: knobs["prefix_kernel"] = int(rng.integers(0, 5))
    if rng.random() < 0.6: knobs["prefix_tiles_per_item"] = int(rng.choice([1, 2, 3, 5]))
    if rng.random() < 0.4: knobs["prefix_rows_per_item"] = int(rng.choice([128, 256]))
    if rng.random() < 0.5: knobs["suffix_chunk_tokens"] = int(rng.choice([64, 128, 256]))
    if rng.random() < 0.3: knobs["num_sms"] = int(rng.choice([1, 7, 148]))
    check(w, str(rng.choice(["f32", "bf16"])), what=f"seed {seed}: {c} {knobs}", **knobs)
