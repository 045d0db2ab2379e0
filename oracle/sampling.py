"""TEST INFRASTRUCTURE ONLY: CPU oracle for drawing the next token of every sample at a temperature.

The paper samples every candidate answer at temperature T in {0.4, 0.7, 1.0} with a seed per run (appendix
"Experiment details").  Drawing token i with probability softmax(logits / T)_i is done here by the Gumbel-max
identity: argmax_i (logits_i / T + g_i) with g_i = -ln(-ln u_i), u_i independent uniforms on (0, 1), has exactly that
distribution; T = 0 means greedy decoding (argmax of the logits).  The uniforms come from the counter-based generator
Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC'11), written out from its
published definition, so that a (seed, step, row, vocabulary index) names one number on every machine:

    counter = (index // 4, step, row, 0),  key = (seed low word, seed high word),
    u = ((x >> 9) + 0.5) * 2^-23  for the word x = output[index % 4].   (23 bits: what an fp32 mantissa holds exactly)

Everything after the generator is fp64.  Ties go to the lowest index.
"""
from __future__ import annotations

import numpy as np

_M0, _M1 = np.uint64(0xD2511F53), np.uint64(0xCD9E8D57)
_W0, _W1 = np.uint32(0x9E3779B9), np.uint32(0xBB67AE85)


def philox4x32_10(counter, key):
    """counter: 4 arrays of uint32 (same shape), key: 2 arrays / scalars of uint32.  Returns 4 uint32 arrays."""
    c0, c1, c2, c3 = (np.asarray(c, dtype=np.uint32) for c in counter)
    k0, k1 = (np.asarray(k, dtype=np.uint32) for k in key)
    mask = np.uint64(0xFFFFFFFF)
    with np.errstate(over="ignore"):
        for _ in range(10):
            p0 = _M0 * c0.astype(np.uint64)
            p1 = _M1 * c2.astype(np.uint64)
            hi0, lo0 = (p0 >> np.uint64(32)).astype(np.uint32), (p0 & mask).astype(np.uint32)
            hi1, lo1 = (p1 >> np.uint64(32)).astype(np.uint32), (p1 & mask).astype(np.uint32)
            c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
            k0 = (k0 + _W0).astype(np.uint32)
            k1 = (k1 + _W1).astype(np.uint32)
    return c0, c1, c2, c3


def uniforms(seed: int, step: int, row: int, vocab: int) -> np.ndarray:
    """u[i] for i < vocab, fp64 in (0, 1)."""
    idx = np.arange(vocab, dtype=np.uint64)
    blk = (idx // np.uint64(4)).astype(np.uint32)
    z = np.zeros_like(blk)
    words = philox4x32_10((blk, z + np.uint32(step & 0xFFFFFFFF), z + np.uint32(row & 0xFFFFFFFF), z),
                          (np.uint32(seed & 0xFFFFFFFF), np.uint32((seed >> 32) & 0xFFFFFFFF)))
    x = np.choose((idx % np.uint64(4)).astype(np.int64), [words[0], words[1], words[2], words[3]])
    return ((x >> np.uint32(9)).astype(np.float64) + 0.5) * 2.0 ** -23


def scores(logits_row: np.ndarray, temperature: float, seed: int, step: int, row: int) -> np.ndarray:
    """The perturbed scores whose argmax is the sampled token (the logits themselves when T = 0)."""
    x = np.asarray(logits_row, dtype=np.float64)
    if temperature == 0.0:
        return x
    g = -np.log(-np.log(uniforms(seed, step, row, len(x))))
    return x / float(temperature) + g


def sample_tokens(logits: np.ndarray, temperature, seeds, step: int) -> np.ndarray:
    """logits [B, V] (any float dtype, widened exactly), temperature [B], seeds [B] (uint64) -> tokens [B] int32."""
    B = logits.shape[0]
    out = np.empty(B, dtype=np.int32)
    for b in range(B):
        out[b] = int(np.argmax(scores(logits[b], float(temperature[b]), int(seeds[b]), step, b)))   # first maximum
    return out
