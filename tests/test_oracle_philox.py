"""Pins for the oracle's Philox4x32-10 and the uniforms / Gumbels built on it."""
import os

import numpy as np
from scipy import stats

from oracle import philox as px

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def test_known_answer_vectors():
    n = 0
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        out = px.philox4x32_10(np.array(w[:4], dtype=np.uint64), (w[4], w[5]))
        assert [int(x) for x in out] == w[6:], line
        n += 1
    assert n == 3


def test_vectorised_equals_scalar_calls():
    rng = np.random.default_rng(0)
    ctr = rng.integers(0, 2 ** 32, size=(64, 4), dtype=np.uint64)
    key = (0x12345678, 0x9ABCDEF0)
    batch = px.philox4x32_10(ctr, key)
    for i in range(64):
        assert np.array_equal(batch[i], px.philox4x32_10(ctr[i], key))


def test_uniform_is_open_interval_and_fp32_exact():
    w = np.array([0, 511, 512, 0xFFFFFFFF, 0x80000000], dtype=np.uint32)
    u = px.word_to_uniform(w)
    assert u[0] == 2.0 ** -24 and u[1] == u[0] and u[2] == 3 * 2.0 ** -24
    assert u[3] == 1.0 - 2.0 ** -24
    assert np.all(u > 0.0) and np.all(u < 1.0)
    assert np.array_equal(u.astype(np.float32).astype(np.float64), u)  # representable in fp32


def test_counter_layout():
    seed = 0xDEADBEEFCAFEF00D
    k0, k1 = px.split_seed(seed)
    assert (k0, k1) == (0xCAFEF00D, 0xDEADBEEF)
    # scalar stream: word 0 of counter (0, j, r, purpose<<24 | k<<16 | b)
    u = px.scalar_uniform(seed, px.ACCEPT, rnd=5, k=0, j=7, b=3)
    w = px.philox4x32_10(np.array([0, 7, 5, (px.ACCEPT << 24) | 3], dtype=np.uint64), (k0, k1))
    assert u == float(px.word_to_uniform(w[0]))
    # vocabulary stream: element v is word v&3 of counter (v>>2, ...)
    uv = px.vocab_uniforms(seed, px.DRAFT, rnd=2, k=0, j=1, b=0, vocab=11)
    assert uv.shape == (11,)
    w = px.philox4x32_10(np.array([2, 1, 2, px.DRAFT << 24], dtype=np.uint64), (k0, k1))
    assert uv[9] == float(px.word_to_uniform(w[1]))
    # distinct purposes / rounds / slots / sequences give distinct streams
    base = px.vocab_uniforms(seed, px.DRAFT, 2, 0, 1, 0, 64)
    for alt in [(px.RESID, 2, 0, 1, 0), (px.DRAFT, 3, 0, 1, 0), (px.DRAFT, 2, 0, 2, 0), (px.DRAFT, 2, 0, 1, 1),
                (px.DRAFT, 2, 1, 1, 0)]:
        assert not np.array_equal(base, px.vocab_uniforms(seed, *alt, 64))


def test_uniform_and_gumbel_distributions():
    u = px.vocab_uniforms(99, px.DRAFT, 0, 0, 0, 0, 200_000)
    assert stats.kstest(u, "uniform").pvalue > 1e-3
    g = px.vocab_gumbels(99, px.BONUS, 1, 0, 0, 0, 200_000)
    assert stats.kstest(g, "gumbel_r").pvalue > 1e-3
    # successive words are uncorrelated
    assert abs(np.corrcoef(u[:-1], u[1:])[0, 1]) < 0.01
