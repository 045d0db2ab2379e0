"""World-size-2 run of the multi-rank plumbing on CPU (gloo): prompts are partitioned across
ranks, each rank works on its shard alone (the oracle stands in for the GPU here), and the
gathered rows equal the unsharded result.  Timing is reduced with a max over ranks."""
import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, tmpdir):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import oracle
    import psa_workloads as wl
    from paper_2502_02534_b200.sharding import max_over_ranks, shard_workload
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    cfg = wl.PsaConfig("mr", 5, 3, 4, 2, 16, (4, 60), (0, 40), page_size=16, permute_pages=True, seed=9)
    w = wl.make_workload(cfg, poison=True)
    sub = shard_workload(w, rank, world)
    out, lse, _ = oracle.attend(sub, n_threads=1)
    s0, s1 = sub["sample_range"]
    np.savez(os.path.join(tmpdir, f"r{rank}.npz"), out=out, lse=lse, s0=s0, s1=s1)
    slow = max_over_ranks([10.0 + rank, 5.0 - rank])
    assert slow == [10.0 + world - 1, 5.0]
    dist.barrier()
    dist.destroy_process_group()


def test_prompt_sharding_over_two_gloo_ranks(tmp_path):
    import torch.multiprocessing as mp
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    sys.path.insert(0, ROOT)
    import oracle
    import psa_workloads as wl
    cfg = wl.PsaConfig("mr", 5, 3, 4, 2, 16, (4, 60), (0, 40), page_size=16, permute_pages=True, seed=9)
    w = wl.make_workload(cfg, poison=True)
    ref_o, ref_l, _ = oracle.attend(w)
    Hq = 4
    covered = 0
    for r in range(2):
        z = np.load(tmp_path / f"r{r}.npz")
        s0, s1 = int(z["s0"]), int(z["s1"])
        assert s0 == covered
        covered = s1
        assert np.array_equal(z["out"], ref_o[s0 * Hq:s1 * Hq]) and np.array_equal(z["lse"], ref_l[s0 * Hq:s1 * Hq])
    assert covered == int(np.sum(w["n_samples"]))


def _head_worker(rank, world, port, tmpdir):
    sys.path.insert(0, ROOT)
    import torch
    import torch.distributed as dist
    import oracle
    import psa_workloads as wl
    from paper_2502_02534_b200.sharding import gather_heads, shard_heads
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    cfg = wl.PsaConfig("hs", 2, 5, 8, 4, 16, (30, 90), (0, 50), page_size=16, permute_pages=True, seed=4)
    w = wl.make_workload(cfg, poison=True)
    sub = shard_heads(w, rank, world)
    B, hq, D = 10, sub["num_q_heads"], 16
    out, lse, _ = oracle.attend(sub, n_threads=1)                       # the oracle stands in for the GPU step of this rank
    full_o, full_l = gather_heads(torch.from_numpy(out.reshape(B, hq, D)), torch.from_numpy(lse.reshape(B, hq)))
    np.savez(os.path.join(tmpdir, f"h{rank}.npz"), out=full_o.numpy(), lse=full_l.numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_kv_head_sharding_and_its_all_gather_over_two_gloo_ranks(tmp_path):
    """Each rank attends with half of the KV heads (and their query heads); one all-gather along the head axis gives
    every rank the unsharded result, bit for bit."""
    import torch.multiprocessing as mp
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_head_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    sys.path.insert(0, ROOT)
    import oracle
    import psa_workloads as wl
    cfg = wl.PsaConfig("hs", 2, 5, 8, 4, 16, (30, 90), (0, 50), page_size=16, permute_pages=True, seed=4)
    w = wl.make_workload(cfg, poison=True)
    ref_o, ref_l, _ = oracle.attend(w)
    for r in range(2):
        z = np.load(tmp_path / f"h{r}.npz")
        assert np.array_equal(z["out"].reshape(-1, 16), ref_o) and np.array_equal(z["lse"].reshape(-1), ref_l)


def test_partition_is_contiguous_complete_and_balanced():
    from paper_2502_02534_b200.sharding import partition_prompts
    rng = np.random.default_rng(0)
    for world in (1, 2, 3, 8):
        P = 16
        L = rng.integers(1024, 32768, P); N = np.full(P, 16); S = rng.integers(0, 4096, P * 16)
        parts = partition_prompts(L, N, S, world)
        assert parts[0][0] == 0 and parts[-1][1] == P
        assert all(parts[i][1] == parts[i + 1][0] for i in range(world - 1))
        cost = [L[a:b].sum() + S[a * 16:b * 16].sum() for a, b in parts]
        if world <= 3:
            assert max(cost) <= 1.6 * sum(cost) / world


def test_rank_launcher_starts_the_ranks_bench_asks_for(tmp_path):
    """`bench.py --gpus 2`, started as a plain python process, must run as two ranks and report n_gpus 2: the decision
    (`needs_launcher`) and the launcher itself, with a small gloo program standing in for the GPU step."""
    import json
    import subprocess
    sys.path.insert(0, ROOT)
    import bench
    from paper_2502_02534_b200.launch import rank_environment, spawn_ranks
    assert bench.needs_launcher(2, {}) and bench.needs_launcher(8, {"PATH": "/bin"})
    assert not bench.needs_launcher(1, {}) and not bench.needs_launcher(2, {"WORLD_SIZE": "2"})
    env = rank_environment(1, 2, 29512, {"KEEP": "1"})
    assert env["RANK"] == "1" and env["LOCAL_RANK"] == "1" and env["WORLD_SIZE"] == "2" and env["MASTER_ADDR"] == "127.0.0.1"
    assert env["MASTER_PORT"] == "29512" and env["KEEP"] == "1"
    child = os.path.join(ROOT, "tests", "rank_child.py")
    out_path = tmp_path / "rank0.out"
    with open(out_path, "w") as f:
        rc = spawn_ranks(2, [sys.executable, child, "--gpus", "2"], stdout=f, timeout_s=120)
    assert rc == 0
    lines = [ln for ln in open(out_path).read().splitlines() if ln.startswith("{")]
    assert len(lines) == 1                       # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["sum"] == 3.0 and line["max_ms"] == 11.0 and line["argv"] == ["--gpus", "2"]
    # a rank that fails ends the run with its exit code, and the other rank does not linger
    rc = spawn_ranks(2, [sys.executable, "-c", "import os, sys, time; sys.exit(7) if os.environ['RANK'] == '1' else time.sleep(60)"],
                     timeout_s=30)
    assert rc == 7
