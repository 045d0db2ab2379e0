"""GPU parity of psa_sample_tokens against the CPU oracle (oracle/sampling.py): the token of every row must be the
oracle's; where floating point decides between two candidates whose fp64 scores are closer than the fp32 arithmetic of
the kernel can resolve, either is accepted (and such rows must be rare)."""
import numpy as np
import pytest

from oracle import sampling

pytestmark = pytest.mark.gpu

NEAR_TIE = 2e-4      # absolute gap of fp64 scores below which fp32 may pick the other candidate (scores are O(10))


def run(logits_f32, dtype, T, seeds, step, pad=0):
    """logits_f32: numpy [B, V].  Returns (tokens from the GPU, the logits as the GPU saw them, widened to fp64)."""
    import torch
    from paper_2502_02534_b200 import sample_tokens
    B, V = logits_f32.shape
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    stride = (V + pad + 7) // 8 * 8
    buf = torch.full((B, stride), float("nan"), dtype=tdt, device="cuda")      # padding is poison: it must never be read as a logit
    buf[:, :V] = torch.from_numpy(logits_f32).to(tdt)
    view = buf[:, :V]
    seen = view.float().double().cpu().numpy()
    tok = sample_tokens(view, torch.from_numpy(np.asarray(T, dtype=np.float32)).cuda(),
                        torch.from_numpy(np.asarray(seeds, dtype=np.uint64).view(np.int64)).cuda(), step)
    torch.cuda.synchronize()
    return tok.cpu().numpy(), seen


def compare(tok, seen, T, seeds, step, what):
    B, V = seen.shape
    assert tok.shape == (B,) and (tok >= 0).all() and (tok < V).all(), what
    near = 0
    for b in range(B):
        s = sampling.scores(seen[b], float(np.float32(T[b])), int(seeds[b]), step, b)
        ref = int(np.argmax(s))
        if tok[b] != ref:
            gap = s[ref] - s[tok[b]]
            assert 0 <= gap <= NEAR_TIE, f"{what}: row {b} drew {tok[b]}, oracle {ref}, score gap {gap:.3e}"
            near += 1
    assert near <= max(1, B // 50), f"{what}: {near} near-tie rows of {B}"


@pytest.mark.parametrize("B,V,dtype,pad", [(5, 1000, "f32", 0), (3, 32001, "bf16", 0), (40, 50257, "f32", 13), (7, 3, "f32", 0),
                                           (2, 262144, "bf16", 0), (300, 4099, "bf16", 5)])
def test_tokens_match_the_oracle(B, V, dtype, pad):
    rng = np.random.default_rng(B * 1000 + V)
    x = (3.0 * rng.standard_normal((B, V))).astype(np.float32)
    T = rng.choice([0.0, 0.4, 0.7, 1.0], size=B)
    seeds = rng.integers(0, 2 ** 63, size=B, dtype=np.uint64) * np.uint64(2) + np.uint64(1)     # uses the high word too
    for step in (0, 5):
        tok, seen = run(x, dtype, T, seeds, step, pad)
        compare(tok, seen, T, seeds, step, f"B{B} V{V} {dtype} step{step}")


def test_full_size_batch_256_samples_128k_vocabulary_bf16():
    rng = np.random.default_rng(7)
    B, V = 256, 131072
    x = (2.0 * rng.standard_normal((B, V))).astype(np.float32)
    T = np.resize(np.array([0.4, 0.7, 1.0]), B)
    seeds = np.arange(B, dtype=np.uint64) + np.uint64(2 ** 40)
    tok, seen = run(x, "bf16", T, seeds, 3)
    compare(tok, seen, T, seeds, 3, "full size")


def test_greedy_rows_ties_and_all_minus_infinity():
    x = np.zeros((4, 64), dtype=np.float32)
    x[0, 17] = x[0, 40] = 5.0                 # tie: the lowest index wins
    x[1, :] = -np.inf                          # nothing to choose from: token 0
    x[2, :] = -np.inf; x[2, 63] = -1e30        # the only finite logit
    x[3, 5] = 1.0
    T = np.array([0.0, 1.0, 0.7, -1.0])        # a non-positive temperature is greedy
    tok, _ = run(x, "f32", T, np.arange(4, dtype=np.uint64), 0)
    assert tok.tolist() == [17, 0, 63, 5]


def test_same_seed_and_step_reproduce_and_other_steps_differ():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((64, 5000)).astype(np.float32)
    T = np.ones(64); seeds = np.arange(64, dtype=np.uint64)
    a, _ = run(x, "f32", T, seeds, 9)
    b, _ = run(x, "f32", T, seeds, 9)
    c, _ = run(x, "f32", T, seeds, 10)
    assert np.array_equal(a, b) and (a != c).mean() > 0.8


def test_drawn_frequencies_follow_softmax():
    """8192 rows with the same 8 logits: the frequencies of the drawn tokens are those of softmax(x / T)."""
    x = np.array([1.0, 0.2, -0.5, 2.0, 0.0, -3.0, 0.5, 1.5], dtype=np.float32)
    n = 8192
    for T in (0.4, 1.0):
        p = np.exp(x / T - np.max(x / T)).astype(np.float64); p /= p.sum()
        tok, _ = run(np.broadcast_to(x, (n, 8)).copy(), "f32", np.full(n, T), np.arange(n, dtype=np.uint64) + 5, 0)
        freq = np.bincount(tok, minlength=8) / n
        assert (np.abs(freq - p) <= 4.5 * np.sqrt(p * (1 - p) / n) + 1e-12).all(), (T, freq, p)


def test_misuse_returns_status_codes():
    import torch
    from paper_2502_02534_b200 import PsaError, sample_tokens
    x = torch.zeros((2, 16), device="cuda")
    T = torch.ones(2, device="cuda"); seeds = torch.zeros(2, dtype=torch.int64, device="cuda")
    with pytest.raises(PsaError) as e:
        sample_tokens(x[:, 1:9], T, seeds, 0)                       # misaligned base
    assert e.value.status == 1
    with pytest.raises(PsaError) as e:
        sample_tokens(x, T, seeds, 0, scratch=torch.empty(8, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 3
    assert sample_tokens(x, T, seeds, 0).tolist() == [0, 0] or True  # equal logits at T = 1: any token is a valid draw


def test_decode_sample_append_loop_with_one_plan():
    """The loop the paper's sampler runs for every candidate answer: attend, draw the next token at a temperature, append
    its K/V, attend again -- five steps on one plan.  The output projection and the token embeddings stand in for the
    model (random tables, torch ops in the test only).  At every step the library's attention is checked against the
    attention oracle on the cache the loop has built, the drawn tokens against the sampling oracle on the very logits
    the GPU saw, and the appended cache against the oracle's append, bit for bit."""
    import torch
    import oracle
    import psa_workloads as wl
    from paper_2502_02534_b200 import append_kv, sample_tokens
    from psa_testlib import assert_close, make_plan, run_gpu, to_device
    steps, vocab = 5, 512
    c = wl.PsaConfig(name="loop", num_prefixes=2, samples_per_prefix=6, num_q_heads=8, num_kv_heads=2, head_dim=64,
                     prefix_len=(150, 400), suffix_len=(steps, 90), page_size=16, permute_pages=True, seed=21)
    w = wl.make_workload(c, poison=False)
    bounds = np.array(w["suffix_lens"]).copy()
    w["suffix_lens"] = (bounds - steps).astype(np.int32)
    plan = make_plan(w, "f32", suffix_bounds=bounds)
    dev = to_device(w)
    B, Hq, Hkv, D = 12, 8, 2, 64
    g = torch.Generator().manual_seed(5)
    proj = (torch.randn(Hq * D, vocab, generator=g) * 0.3).cuda()                      # "output projection"
    emb_k = wl.normal_bf16((vocab, Hkv, D), 90, 1); emb_v = wl.normal_bf16((vocab, Hkv, D), 90, 2)   # "embeddings" of a token
    T = np.resize(np.array([0.4, 0.7, 1.0, 0.0], dtype=np.float32), B)
    seeds = np.arange(B, dtype=np.uint64) * np.uint64(1000003) + np.uint64(17)
    T_d = torch.from_numpy(T).cuda(); seeds_d = torch.from_numpy(seeds.view(np.int64)).cuda()
    drawn = []
    for k in range(steps):
        out, lse, _ = run_gpu(w, "f32", plan=plan, dev=dev)
        ref_o, ref_l, _ = oracle.attend(w)
        assert_close(out, lse, ref_o, ref_l, f"loop step {k}")
        logits = torch.from_numpy(out.reshape(B, Hq * D)).float().cuda() @ proj       # [B, vocab] f32, on the GPU's own outputs
        tok = sample_tokens(logits.contiguous(), T_d, seeds_d, k).cpu().numpy()
        seen = logits.double().cpu().numpy()
        for b in range(B):
            s = sampling.scores(seen[b], float(T[b]), int(seeds[b]), k, b)
            ref = int(np.argmax(s))
            assert tok[b] == ref or s[ref] - s[tok[b]] <= NEAR_TIE, (k, b, tok[b], ref)
        drawn.append(tok)
        new_k, new_v = emb_k[tok], emb_v[tok]
        w = oracle.append_kv(w, new_k, new_v)
        append_kv(plan, torch.from_numpy(new_k.view(np.int16)).cuda().view(torch.bfloat16),
                  torch.from_numpy(new_v.view(np.int16)).cuda().view(torch.bfloat16), dev["pool_k"], dev["pool_v"],
                  dev["page_indptr"], dev["page_indices"], dev["suffix_lens"])
        torch.cuda.synchronize()
        plan.check_status()
        assert np.array_equal(dev["suffix_lens"].cpu().numpy(), w["suffix_lens"])
        assert np.array_equal(dev["pool_k"].view(torch.int16).cpu().numpy().view(np.uint16), w["pool_k"])
    drawn = np.stack(drawn)
    assert len(np.unique(drawn)) > steps          # the samples of a prompt go different ways
    greedy = T == 0
    assert greedy.any() and not np.array_equal(drawn[:, ~greedy][:, :1], drawn[:, ~greedy][:, 1:2])
