"""The allocation-free entry point, psa_decode_static, against psa_decode.

Some embedders of the library may not allocate device memory around a decode step (their
process's memory pool owns the GPU, or an allocation would stall a latency-critical loop), so
psa_decode_static keeps the step's scratch memory in a fixed array inside the library.  This
file is collected last on purpose: a run that stops at the first failure has then already run
every other test.  It passes on its own in a fresh process as well as after the other tests.
"""
import numpy as np
import pytest

import psa_workloads as wl
from psa_testlib import LSE_TOL, OUT_TOL, make_plan, to_device

pytestmark = pytest.mark.gpu


def _run(fn, plan, dev, B, Hq, D):
    import torch
    out = torch.full((B, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device="cuda")
    fn(plan, dev["q"], dev["prefix_k"], dev["prefix_v"], dev["pool_k"], dev["pool_v"], dev["page_indptr"],
       dev["page_indices"], dev["suffix_lens"], out, lse)
    torch.cuda.synchronize()
    return out.double().cpu().numpy(), lse.double().cpu().numpy()


def test_static_workspace_matches_decode_on_two_calls_in_a_row():
    from paper_2502_02534_b200 import decode, decode_static
    # two different problems back to back: the second call finds the first one's lists and
    # partial results in the shared array and must not be disturbed by them
    cfg_a = wl.CONFIGS["cfg1"]
    cfg_b = wl.PsaConfig("two_prompts", 2, 5, 8, 2, 128, (100, 700), (0, 300), permute_pages=True, seed=5)
    for cfg in (cfg_a, cfg_b):
        w = wl.make_workload(cfg, poison=True)
        dev = to_device(w)
        B, Hq, D = int(np.sum(w["n_samples"])), w["num_q_heads"], w["head_dim"]
        plan = make_plan(w, "f32")
        ref_o, ref_l = _run(decode, plan, dev, B, Hq, D)
        plan.check_status()
        got_o, got_l = _run(decode_static, plan, dev, B, Hq, D)
        assert np.isfinite(got_o).all()
        assert np.array_equal(np.isneginf(got_l), np.isneginf(ref_l))
        fin = np.isfinite(ref_l)
        assert np.max(np.abs(got_o - ref_o)) <= OUT_TOL
        assert np.max(np.abs(got_l[fin] - ref_l[fin]), initial=0.0) <= LSE_TOL


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
