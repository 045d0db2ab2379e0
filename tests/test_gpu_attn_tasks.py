"""GPU parity of psa_attn_task (the paper's three attn task forms) against the fp64 recurrences of oracle/recurrences.py,
each form against ITS oracle form, and all three against one another."""
import math

import numpy as np
import pytest

import psa_workloads as wl
from oracle import recurrences

pytestmark = pytest.mark.gpu

ORACLE = {0: recurrences.task0_maxsum, 1: recurrences.task1_divsum, 2: recurrences.task2_deferred}


def run(task, R, M, D, seed, scale=None):
    import torch
    from paper_2502_02534_b200 import attn_task
    q = wl.normal_bf16((R, D), seed, 1); k = wl.normal_bf16((M, D), seed, 2); v = wl.normal_bf16((M, D), seed, 3)
    dev = [torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16) for a in (q, k, v)]
    scale = D ** -0.5 if scale is None else scale
    out, m, l = attn_task(task, dev[0], dev[1], dev[2], scale)
    torch.cuda.synchronize()
    f = recurrences.bf16_bits_to_f64
    return (f(q), f(k), f(v), scale), out.double().cpu().numpy(), m.double().cpu().numpy(), l.double().cpu().numpy()


@pytest.mark.parametrize("task", [0, 1, 2])
@pytest.mark.parametrize("R,M,D", [(5, 7, 64), (9, 11, 128), (3, 300, 32), (2, 1, 256), (6, 129, 96)])
def test_each_form_matches_its_oracle_form(task, R, M, D):
    (q, k, v, scale), out, m, l = run(task, R, M, D, seed=100 + task)
    for r in range(R):
        x = scale * (k @ q[r])
        o_ref, m_ref, l_ref = ORACLE[task](x, v)
        assert abs(m[r] - m_ref) <= 1e-5 * max(1.0, abs(m_ref))
        assert abs(l[r] - l_ref) <= 2e-4 * l_ref
        assert np.max(np.abs(out[r] - o_ref)) <= 2e-4


def test_the_three_forms_agree_and_match_the_definition_with_large_logits():
    """Scores of +-30 make a form that forgets a rescaling overflow or lose the early keys."""
    R, M, D = 4, 200, 64
    res = [run(t, R, M, D, seed=7, scale=4.0) for t in (0, 1, 2)]
    (q, k, v, scale) = res[0][0]
    for r in range(R):
        x = scale * (k @ q[r])
        w = np.exp(x - x.max()); ref = (w[:, None] * v).sum(0) / w.sum()
        lse = x.max() + math.log(w.sum())
        for _, out, m, l in res:
            assert np.max(np.abs(out[r] - ref)) <= 2e-4
            assert abs(m[r] + math.log(l[r]) - lse) <= 1e-4 * max(1.0, abs(lse))
    assert np.max(np.abs(res[0][1] - res[2][1])) <= 2e-4 and np.max(np.abs(res[1][1] - res[2][1])) <= 2e-4


def test_no_keys_returns_the_initial_state_and_misuse_a_status():
    import torch
    from paper_2502_02534_b200 import PsaError, attn_task
    q = torch.zeros((3, 64), dtype=torch.bfloat16, device="cuda"); kv = torch.zeros((0, 64), dtype=torch.bfloat16, device="cuda")
    for task in (0, 1, 2):
        out, m, l = attn_task(task, q, kv, kv, 1.0)
        assert (out == 0).all() and (m == -math.inf).all() and (l == 0).all()
    with pytest.raises(PsaError) as e:
        attn_task(3, q, kv, kv, 1.0)
    assert e.value.status == 1
    with pytest.raises(PsaError) as e:
        attn_task(0, q[:, :48].contiguous(), kv, kv, 1.0)
    assert e.value.status == 2
