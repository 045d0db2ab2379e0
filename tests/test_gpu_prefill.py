"""GPU parity of psa_prefill (causal attention of packed prompts over themselves) against the CPU oracle."""
import numpy as np
import pytest

import oracle
import psa_workloads as wl
from psa_testlib import LSE_TOL, OUT_TOL

pytestmark = pytest.mark.gpu


def run_prefill(lens, Hq, Hkv, D, out_dtype="f32", seed=3, **plan_kw):
    import torch
    from paper_2502_02534_b200 import Plan, prefill
    T = int(np.sum(lens))
    q = wl.normal_bf16((T, Hq, D), seed, 1); k = wl.normal_bf16((T, Hkv, D), seed, 2); v = wl.normal_bf16((T, Hkv, D), seed, 3)
    dev = [torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16) for a in (q, k, v)]
    plan = Plan([], [], [], num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, out_dtype=out_dtype, prefill_prompt_lens=lens, **plan_kw)
    tdt = torch.float32 if out_dtype == "f32" else torch.bfloat16
    out = torch.full((T, Hq, D), float("nan"), dtype=tdt, device="cuda")
    lse = torch.full((T, Hq), float("nan"), dtype=torch.float32, device="cuda")
    prefill(plan, dev[0], dev[1], dev[2], out, lse)
    torch.cuda.synchronize()
    plan.check_status()
    return (q, k, v), out.float().double().cpu().numpy().reshape(T * Hq, D), lse.double().cpu().numpy().reshape(-1), plan


def compare(inputs, lens, out, lse, rows=None, what=""):
    q, k, v = inputs
    D = q.shape[2]
    ref_o, ref_l = oracle.causal_attend(q, k, v, lens, D ** -0.5, rows=rows)
    if rows is not None:
        out, lse = out[rows], lse[rows]
    assert np.isfinite(out).all() and np.isfinite(lse).all(), what
    assert np.max(np.abs(out - ref_o)) <= OUT_TOL, (what, float(np.max(np.abs(out - ref_o))))
    assert np.max(np.abs(lse - ref_l)) <= LSE_TOL, (what, float(np.max(np.abs(lse - ref_l))))


@pytest.mark.parametrize("lens", [[1], [33], [64], [65], [127, 129], [300, 1, 257], [1000], [0, 5, 0]])
@pytest.mark.parametrize("G,D", [(4, 128), (1, 64), (8, 128), (2, 64)])
def test_prefill_small_prompts_every_element(lens, G, D):
    inputs, out, lse, _ = run_prefill(lens, 2 * G, 2, D)
    if sum(lens) == 0:
        return
    compare(inputs, lens, out, lse, what=f"lens{lens} G{G} D{D}")


def test_prefill_long_prompt_sampled_rows_and_bf16_output():
    lens = [3000, 1500]
    inputs, out, lse, plan = run_prefill(lens, 8, 2, 128, out_dtype="bf16")
    rng = np.random.default_rng(0)
    T = sum(lens)
    toks = np.concatenate([[0, 1, 255, 256, 257, 2999, 3000, 3001, T - 1], rng.choice(T, 60, replace=False)])
    rows = (toks[:, None] * 8 + np.arange(8)[None, :]).ravel()
    compare(inputs, lens, out, lse, rows=rows, what="long")
    assert np.isfinite(out).all() and np.isfinite(lse).all()


def test_prefill_planned_for_few_and_many_sms_and_one_row_tile_items():
    lens = [700, 90]
    for kw in (dict(num_sms=2), dict(num_sms=1000), dict(prefix_rows_per_item=128), dict(prefix_tiles_per_item=1)):
        inputs, out, lse, _ = run_prefill(lens, 4, 1, 128, **kw)
        compare(inputs, lens, out, lse, what=str(kw))
