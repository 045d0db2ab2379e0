"""KV-head sharding on ONE GPU: every rank's share of the problem goes through the CUDA kernels one after another,
the pieces are joined along the head axis the way the all-gather would, and the result is the unsharded oracle's.
(The exchange itself is covered on CPU by the gloo tests; here the point is that a head shard is a problem the
kernels solve correctly -- fewer KV heads, strided slices of nothing: every shard is a dense copy.)"""
import numpy as np
import pytest

import oracle
import psa_workloads as wl
from paper_2502_02534_b200.sharding import shard_heads, shard_workload
from psa_testlib import assert_close, run_gpu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("world", [2, 4, 8])
def test_head_shards_through_the_kernels_join_to_the_unsharded_oracle(world):
    cfg = wl.PsaConfig("hs", 2, 9, 32, 8, 128, (200, 900), (0, 260), permute_pages=True, seed=17)
    w = wl.make_workload(cfg, poison=True)
    B, Hq, D = int(np.sum(w["n_samples"])), w["num_q_heads"], w["head_dim"]
    ref_o, ref_l, _ = oracle.attend(w)
    outs, lses = [], []
    for rank in range(world):
        sub = shard_heads(w, rank, world)
        out, lse, _ = run_gpu(sub, "f32")
        hq = sub["num_q_heads"]
        assert sub["head_range"] == (rank * hq, (rank + 1) * hq)
        outs.append(out.reshape(B, hq, D)); lses.append(lse.reshape(B, hq))
    full_o = np.concatenate(outs, axis=1).reshape(B * Hq, D)
    full_l = np.concatenate(lses, axis=1).reshape(B * Hq)
    assert_close(full_o, full_l, ref_o, ref_l, f"head shards, world {world}")


def test_prompt_shards_through_the_kernels_cover_every_sample():
    cfg = wl.PsaConfig("ps", 5, 6, 8, 2, 128, (100, 1500), (0, 200), permute_pages=True, seed=3)
    w = wl.make_workload(cfg, poison=True)
    Hq = w["num_q_heads"]
    ref_o, ref_l, _ = oracle.attend(w)
    covered = 0
    for rank in range(3):
        sub = shard_workload(w, rank, 3)
        s0, s1 = sub["sample_range"]
        assert s0 == covered
        covered = s1
        if s1 > s0:
            out, lse, _ = run_gpu(sub, "f32")
            assert_close(out, lse, ref_o[s0 * Hq:s1 * Hq], ref_l[s0 * Hq:s1 * Hq], f"prompt shard {rank}")
    assert covered == int(np.sum(w["n_samples"]))
