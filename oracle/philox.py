"""TEST INFRASTRUCTURE — CPU oracle, not part of the product path.

Philox4x32-10 counter-based generator (Salmon, Moraes, Dror, Shaw: "Parallel random
numbers: as easy as 1, 2, 3", SC'11), written from its published definition in plain
numpy, and the random streams of one SpecDiff round built on it.

The paper only says "r ~ U(0,1)" (Algorithm 1) and "standard decoding methods"
(Section "SpecDiff: Formulation"); the counter layout below is this library's own
convention so that the CPU oracle and the GPU kernels can be compared draw for draw.

    key      = 64-bit seed           (k0 = low word, k1 = high word)
    counter  = (c0, c1, c2, c3)
        c0 = v >> 2 for per-vocabulary streams (v = vocabulary index), else 0
        c1 = slot index j (0-based position inside the draft; gamma for the bonus draw)
        c2 = round index r
        c3 = purpose << 24 | step k << 16 | sequence index b
    lane     = v & 3 for per-vocabulary streams, else 0
    uniform  = ((word >> 9) + 0.5) * 2**-23     -- strictly inside (0, 1), exact in fp32 (24 bits)
    gumbel   = -log(-log(uniform))
"""
from __future__ import annotations

import numpy as np

M0 = np.uint64(0xD2511F53)
M1 = np.uint64(0xCD9E8D57)
W0 = 0x9E3779B9
W1 = 0xBB67AE85
MASK32 = np.uint64(0xFFFFFFFF)

# purposes of the method's random streams
UNMASK, DRAFT, ACCEPT, RESID, BONUS = 1, 2, 3, 4, 5


def philox4x32_10(counter, key):
    """counter: integer array [..., 4]; key: (k0, k1).  Returns uint32 array [..., 4]."""
    c = np.asarray(counter, dtype=np.uint64) & MASK32
    c0, c1, c2, c3 = (c[..., i].copy() for i in range(4))
    k0 = int(key[0]) & 0xFFFFFFFF
    k1 = int(key[1]) & 0xFFFFFFFF
    for _ in range(10):
        p0 = M0 * c0  # 32x32 -> 64 bit products, exact in uint64
        p1 = M1 * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & MASK32
        hi1, lo1 = p1 >> np.uint64(32), p1 & MASK32
        n0 = hi1 ^ c1 ^ np.uint64(k0)
        n2 = hi0 ^ c3 ^ np.uint64(k1)
        c0, c1, c2, c3 = n0, lo1, n2, lo0
        k0 = (k0 + W0) & 0xFFFFFFFF
        k1 = (k1 + W1) & 0xFFFFFFFF
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def split_seed(seed: int):
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    return seed & 0xFFFFFFFF, seed >> 32


def word_to_uniform(w):
    """((w >> 9) + 0.5) / 2^23 as float64: an odd multiple of 2^-24 below 1, so the value has at
    most 24 significant bits and is exactly representable in fp32."""
    return ((np.asarray(w, dtype=np.uint32) >> np.uint32(9)).astype(np.float64) + 0.5) * (2.0 ** -23)


def _c3(purpose: int, k: int, b: int) -> int:
    assert 0 <= purpose < 256 and 0 <= k < 256 and 0 <= b < 65536
    return (purpose << 24) | (k << 16) | b


def scalar_uniform(seed: int, purpose: int, rnd: int, k: int, j: int, b: int) -> float:
    """One uniform for (purpose, round, step, slot, sequence): word 0 of counter (0, j, r, c3)."""
    out = philox4x32_10(np.array([0, j, rnd, _c3(purpose, k, b)], dtype=np.uint64), split_seed(seed))
    return float(word_to_uniform(out[0]))


def vocab_uniforms(seed: int, purpose: int, rnd: int, k: int, j: int, b: int, vocab: int) -> np.ndarray:
    """Uniforms u[v], v = 0..vocab-1: word (v & 3) of counter (v >> 2, j, r, c3)."""
    nblk = (vocab + 3) // 4
    ctr = np.empty((nblk, 4), dtype=np.uint64)
    ctr[:, 0] = np.arange(nblk, dtype=np.uint64)
    ctr[:, 1] = j
    ctr[:, 2] = rnd
    ctr[:, 3] = _c3(purpose, k, b)
    words = philox4x32_10(ctr, split_seed(seed)).reshape(-1)[:vocab]
    return word_to_uniform(words)


def vocab_gumbels(seed: int, purpose: int, rnd: int, k: int, j: int, b: int, vocab: int) -> np.ndarray:
    u = vocab_uniforms(seed, purpose, rnd, k, j, b, vocab)
    return -np.log(-np.log(u))
