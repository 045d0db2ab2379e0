"""Helpers shared by the GPU parity tests: upload a workload, run the library, compare with the oracle."""
import numpy as np

OUT_TOL = 1e-2   # max |out_gpu - out_oracle|, absolute
LSE_TOL = 1e-3   # max |lse_gpu - lse_oracle|, absolute


def to_device(w):
    import torch
    dev = {}
    for name in ("q", "prefix_k", "prefix_v", "pool_k", "pool_v"):
        a = np.ascontiguousarray(w[name])
        dev[name] = torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    for name in ("page_indptr", "page_indices", "suffix_lens"):
        dev[name] = torch.from_numpy(np.ascontiguousarray(w[name], dtype=np.int32)).cuda()
    return dev


def make_plan(w, out_dtype="bf16", suffix_bounds=None, **kw):
    from paper_2502_02534_b200 import Plan
    if "group_first_sample" in w:      # a cascade of shared prefixes
        kw = dict(kw, groups=(w["group_first_sample"], w["n_samples"], w["prefix_lens"]))
    return Plan(w["prefix_lens"], w["n_samples"], w["suffix_lens"] if suffix_bounds is None else suffix_bounds,
                num_q_heads=w["num_q_heads"], num_kv_heads=w["num_kv_heads"], head_dim=w["head_dim"],
                page_size=w["page_size"], sm_scale=w["sm_scale"], out_dtype=out_dtype, **kw)


def run_gpu(w, out_dtype="bf16", plan=None, dev=None):
    """Returns (out [B*Hq, D] float64, lse [B*Hq] float64, plan)."""
    import torch
    from paper_2502_02534_b200 import decode
    dev = dev or to_device(w)
    plan = plan or make_plan(w, out_dtype)
    B, Hq, D = len(w["suffix_lens"]), w["num_q_heads"], w["head_dim"]
    tdt = torch.bfloat16 if out_dtype == "bf16" else torch.float32
    out = torch.full((B, Hq, D), float("nan"), dtype=tdt, device="cuda")
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device="cuda")
    if plan.workspace is None:
        plan.bind_workspace()
    decode(plan, dev["q"], dev["prefix_k"], dev["prefix_v"], dev["pool_k"], dev["pool_v"], dev["page_indptr"],
           dev["page_indices"], dev["suffix_lens"], out, lse)
    torch.cuda.synchronize()
    plan.check_status()
    return (out.float().double().cpu().numpy().reshape(B * Hq, D), lse.double().cpu().numpy().reshape(B * Hq), plan)


def assert_close(out, lse, ref_out, ref_lse, what=""):
    assert out.shape == ref_out.shape and lse.shape == ref_lse.shape
    assert np.isfinite(out).all(), f"{what}: non-finite values in out"
    neg_inf = np.isneginf(ref_lse)
    assert np.array_equal(np.isneginf(lse), neg_inf), f"{what}: -inf pattern of lse differs"
    assert np.isfinite(lse[~neg_inf]).all(), f"{what}: NaN/inf in lse"
    err_o = float(np.max(np.abs(out - ref_out))) if out.size else 0.0
    err_l = float(np.max(np.abs(lse[~neg_inf] - ref_lse[~neg_inf]))) if (~neg_inf).any() else 0.0
    assert err_o <= OUT_TOL, f"{what}: max |out err| {err_o:.3e} > {OUT_TOL}"
    assert err_l <= LSE_TOL, f"{what}: max |lse err| {err_l:.3e} > {LSE_TOL}"
    return err_o, err_l
