"""The allocation-free entry point, psa_decode_static, against psa_decode and against the oracle.

Some embedders of the library may not allocate device memory around a decode step (their
process's memory pool owns the GPU, or an allocation would stall a latency-critical loop), so
psa_decode_static keeps the step's scratch memory in a fixed array inside the library.  This
file is collected last on purpose: a run that stops at the first failure has then already run
every other test.  It passes on its own in a fresh process as well as after the other tests.

The one property the entry point exists for is checked directly: free device memory and torch's
allocator counters do not move across a call (from the second call on; the first call on a device
is when the driver may materialise the array, see include/psa.h).
"""
import numpy as np
import pytest

import oracle
import psa_workloads as wl
from psa_testlib import LSE_TOL, OUT_TOL, assert_close, make_plan, to_device

pytestmark = pytest.mark.gpu

# cudaMalloc hands memory out in granules; a module load may round the array up to the next one
GRANULE_SLACK = 2 << 20


def _buffers(B, Hq, D):
    import torch
    out = torch.full((B, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device="cuda")
    return out, lse


def _call(fn, plan, dev, out, lse):
    fn(plan, dev["q"], dev["prefix_k"], dev["prefix_v"], dev["pool_k"], dev["pool_v"], dev["page_indptr"],
       dev["page_indices"], dev["suffix_lens"], out, lse)


def _memory_state():
    import torch
    torch.cuda.synchronize()
    free, _ = torch.cuda.mem_get_info()
    return free, torch.cuda.memory_allocated(), torch.cuda.memory_reserved()


def test_static_workspace_matches_decode_and_oracle_on_two_calls_in_a_row_and_allocates_nothing():
    import torch
    from paper_2502_02534_b200 import decode, decode_static, static_check_status
    from paper_2502_02534_b200.binding import STATIC_WORKSPACE_BYTES
    # two different problems back to back: the second call finds the first one's lists and
    # partial results in the shared array and must not be disturbed by them
    cfg_a = wl.CONFIGS["cfg1"]
    cfg_b = wl.PsaConfig("two_prompts", 2, 5, 8, 2, 128, (100, 700), (0, 300), permute_pages=True, seed=5)
    first_call = True
    for cfg in (cfg_a, cfg_b):
        w = wl.make_workload(cfg, poison=True)
        dev = to_device(w)
        B, Hq, D = int(np.sum(w["n_samples"])), w["num_q_heads"], w["head_dim"]
        plan = make_plan(w, "f32")
        ref_o, ref_l = _buffers(B, Hq, D)
        _call(decode, plan, dev, ref_o, ref_l)          # also loads the kernels' modules, so that they do not count below
        torch.cuda.synchronize()
        plan.check_status()
        got_o, got_l = _buffers(B, Hq, D)
        before = _memory_state()
        _call(decode_static, plan, dev, got_o, got_l)
        after = _memory_state()
        static_check_status()
        # torch's allocator saw nothing, and the device's free memory did not move -- except that the very first
        # call of the process on this device may be the one in which the driver creates the array
        assert after[1:] == before[1:]
        taken = before[0] - after[0]
        if first_call:
            assert 0 <= taken <= STATIC_WORKSPACE_BYTES + GRANULE_SLACK
        else:
            assert taken == 0
        first_call = False
        # once more on the same problem: still nothing, and the same numbers
        again_o, again_l = _buffers(B, Hq, D)
        before = _memory_state()
        _call(decode_static, plan, dev, again_o, again_l)
        after = _memory_state()
        assert after == before
        static_check_status()
        assert torch.equal(again_o, got_o) and torch.equal(again_l, got_l)

        # against psa_decode with a caller workspace ...
        r_o, r_l = ref_o.double().cpu().numpy(), ref_l.double().cpu().numpy()
        g_o, g_l = got_o.double().cpu().numpy(), got_l.double().cpu().numpy()
        assert np.isfinite(g_o).all()
        assert np.array_equal(np.isneginf(g_l), np.isneginf(r_l))
        fin = np.isfinite(r_l)
        assert np.max(np.abs(g_o - r_o)) <= OUT_TOL
        assert np.max(np.abs(g_l[fin] - r_l[fin]), initial=0.0) <= LSE_TOL
        # ... and against the CPU oracle, element by element
        o_o, o_l, _ = oracle.attend(w)
        assert_close(g_o.reshape(B * Hq, D), g_l.reshape(B * Hq), o_o, o_l, f"static {cfg.name}")


def test_static_status_word_is_readable_and_clears():
    """A device-side error of the static path reaches the host: the unsatisfiable wait of the self-test reports
    PSA_ERR_TIMEOUT into the library's array, psa_static_check_status returns and clears it, and the next step on
    that array is correct."""
    import torch
    from paper_2502_02534_b200 import PsaError, decode_static, static_check_status, static_selftest_bounded_wait
    w = wl.make_workload(wl.CONFIGS["cfg1"], poison=True)
    dev = to_device(w)
    B, Hq, D = int(np.sum(w["n_samples"])), w["num_q_heads"], w["head_dim"]
    plan = make_plan(w, "f32")
    out, lse = _buffers(B, Hq, D)
    _call(decode_static, plan, dev, out, lse)
    static_check_status()
    static_selftest_bounded_wait(limit_ns=2_000_000)
    with pytest.raises(PsaError) as e:
        static_check_status()
    assert e.value.status == 5
    static_check_status()                                 # cleared
    out2, lse2 = _buffers(B, Hq, D)
    _call(decode_static, plan, dev, out2, lse2)
    static_check_status()
    assert torch.equal(out, out2) and torch.equal(lse, lse2)


def test_static_workspace_rejects_plans_beyond_its_size():
    import torch
    from paper_2502_02534_b200 import Plan, PsaError, decode_static
    from paper_2502_02534_b200.binding import STATIC_WORKSPACE_BYTES
    cfg = wl.CONFIGS["cfg4"]                           # 256 samples x 64 heads: ~30 MB of partial results
    L, N, S = wl.draw_lengths(cfg)                     # lengths only: the size check comes before any memory access
    plan = Plan(L, N, S, num_q_heads=cfg.num_q_heads, num_kv_heads=cfg.num_kv_heads, head_dim=cfg.head_dim)
    assert plan.workspace_bytes > STATIC_WORKSPACE_BYTES
    dummy = torch.zeros(1024, dtype=torch.bfloat16, device="cuda")
    idx = torch.zeros(1024, dtype=torch.int32, device="cuda")
    lse = torch.zeros(1024, dtype=torch.float32, device="cuda")
    with pytest.raises(PsaError) as e:
        decode_static(plan, dummy, dummy, dummy, dummy, dummy, idx, idx, idx, dummy, lse)
    assert e.value.status == 3 and "PSA_STATIC_WORKSPACE_BYTES" in str(e.value)
