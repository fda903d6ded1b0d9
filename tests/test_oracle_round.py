"""Pins for the oracle's whole round: the unmasking schedule, losslessness where it holds
exactly (first emitted token for any T; every prefix for T = 1, by brute force on a tiny
vocabulary), greedy SpecDiff == greedy autoregressive decoding, drafter cost = T evaluations."""
import itertools

import numpy as np
from scipy import stats

import synth
from oracle import specdiff as sd
from oracle import transformer as tf
from oracle.transformer import Model


def _tiny_pair(V=4, d=16, seed=3, std=0.5):
    sp = synth.ModelShape(V, 1, d, 2, 16, True)
    sq = synth.ModelShape(V, 1, d, 2, 16, False)
    return (Model(sp, synth.model_weights(sp, seed, "fp32", std=std, bias_std=0.1)),
            Model(sq, synth.model_weights(sq, seed + 1, "fp32", std=std, bias_std=0.1)))


def _softmax(z):
    e = np.exp(z - z.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


def test_unmask_schedule_uniform_reveal_step():
    """Reveal probability 1/k at step k => each slot's reveal step is uniform on {1..T};
    nothing stays masked after k = 1; every slot is written exactly once."""
    gamma, T, V, N = 8, 4, 4, 700
    logits = np.zeros((gamma, V))
    hist = np.zeros(T)
    for rnd in range(N):
        st = sd.DraftState.fresh(gamma, V)
        total = 0
        for k in range(T, 0, -1):
            before = st.slots.copy()
            total += sd.unmask_sample_step(st, logits, k, 1.0, 17, rnd, 0)
            kept = before != V
            assert np.array_equal(st.slots[kept], before[kept])     # revealed slots never change
        assert total == gamma and np.all(st.slots != V) and np.all(st.reveal_step >= 1)
        for k in st.reveal_step:
            hist[k - 1] += 1
    assert stats.chisquare(hist, np.full(T, N * gamma / T)).pvalue > 1e-3


def test_round_structure_and_drafter_evaluation_count(monkeypatch):
    mp, mq = _tiny_pair(V=6)
    calls = []
    real = sd.drafter_slot_logits
    monkeypatch.setattr(sd, "drafter_slot_logits", lambda m, c, s: (calls.append(s.copy()), real(m, c, s))[1])
    gamma, T = 5, 3
    for rnd in range(6):
        calls.clear()
        tr = sd.specdiff_round(mp, mq, [1, 2, 3], gamma, T, 1.0, 1.0, 9, rnd, keep=True)
        assert len(calls) == T                                   # cost is T drafter evaluations
        assert np.all(calls[0] == 6)                             # first evaluation sees only [MASK]
        assert 1 <= len(tr.emitted) <= gamma + 1
        assert tr.emitted[:-1] == [int(x) for x in tr.draft.slots[: tr.acc.n]]
        assert tr.lam.shape == (gamma + 1, 6)
        # stored q rows are the logits of the step that revealed the slot
        for j in range(gamma):
            step = T - int(tr.draft.reveal_step[j])
            assert np.array_equal(tr.draft.qrows[j], tr.step_logits[step][j])
            assert abs(tr.draft.logq[j] - sd.log_softmax(tr.draft.qrows[j])[tr.draft.slots[j]]) < 1e-12


def test_first_emitted_token_follows_target_for_any_T():
    mp, mq = _tiny_pair(V=5, seed=11, std=0.25)
    ctx = np.array([0, 3, 1])
    p1 = _softmax(mp.logits(ctx, [2])[0])
    N = 2500
    counts = np.zeros(5)
    for rnd in range(N):
        tr = sd.specdiff_round(mp, mq, ctx, 3, 3, 1.0, 1.0, 123, rnd)
        counts[tr.emitted[0]] += 1
    assert p1.min() > 0.02 and p1.max() > 0.3          # a non-trivial target
    assert stats.chisquare(counts, p1 * N).pvalue > 1e-3


def test_T1_round_prefix_law_by_brute_force():
    """T = 1, V = 4, gamma = 2.  For every prefix y_{1:k}:
    P(at least k tokens emitted and they equal y) = prod_{j<k} min(p_j, q_j)(y_j) * p_k(y_k | y_<k),
    with p from the target forward on ctx ∘ y_<j and q_j from the single all-[MASK] drafter forward."""
    V, gamma, N = 4, 2, 5000
    mp, mq = _tiny_pair(V=V, seed=21, std=0.4)
    ctx = np.array([2, 0, 1])
    q = _softmax(tf.drafter_slot_logits(mq, ctx, np.full(gamma, V)))            # [gamma, V]

    def p_next(prefix):
        ids = np.concatenate([ctx, np.array(prefix, dtype=np.int64)])
        return _softmax(mp.logits(ids, [len(ids) - 1])[0])

    law = {}
    for k in range(1, gamma + 2):
        for y in itertools.product(range(V), repeat=k):
            pr = 1.0
            for j in range(k - 1):
                pr *= min(p_next(y[:j])[y[j]], q[j][y[j]])
            law[y] = pr * p_next(y[: k - 1])[y[k - 1]]
    counts = {y: 0 for y in law}
    for rnd in range(N):
        em = tuple(sd.specdiff_round(mp, mq, ctx, gamma, 1, 1.0, 1.0, 77, rnd).emitted)
        for k in range(1, len(em) + 1):
            counts[em[:k]] += 1
    for k in range(1, gamma + 2):
        ys = [y for y in law if len(y) == k]
        exp = np.array([law[y] for y in ys]) * N
        obs = np.array([counts[y] for y in ys], dtype=float)
        rest_e, rest_o = N - exp.sum(), N - obs.sum()
        if rest_e > 1e-9:
            exp, obs = np.append(exp, rest_e), np.append(obs, rest_o)
        keep = exp > 5
        assert keep.sum() >= 4
        assert stats.chisquare(obs[keep] + 0.0, exp[keep] * obs[keep].sum() / exp[keep].sum()).pvalue > 1e-3
        assert abs(obs[keep].sum() - exp[keep].sum()) < 5 * np.sqrt(N)
    # k = 1 marginal is exactly the target distribution
    assert abs(sum(law[(v,)] for v in range(V)) - 1.0) < 1e-12


def test_greedy_specdiff_equals_greedy_autoregressive():
    wl = synth.WORKLOADS["tiny_fp32"]
    mp = Model(wl.target, synth.model_weights(wl.target, wl.weight_seed, "fp32"))
    mq = Model(wl.drafter, synth.model_weights(wl.drafter, wl.weight_seed, "fp32"))
    prompt = synth.prompt_ids(wl.target.vocab, 1, wl.prompt_len, wl.prompt_seed)[0]
    n_new = 14
    ids, traces = sd.generate(mp, mq, prompt, wl.gamma, wl.T, n_new, 0.0, 0.0, wl.philox_seed)
    ref = sd.autoregressive_greedy(mp, prompt, n_new)
    assert np.array_equal(ids, ref)
    assert len(ids) == wl.prompt_len + n_new               # truncated to max_new
    assert sum(len(t.emitted) for t in traces) == n_new


def test_generate_bookkeeping_stochastic():
    mp, mq = _tiny_pair(V=6, seed=31)
    ids, traces = sd.generate(mp, mq, [1, 2], 3, 2, 7, 1.0, 1.0, 5)
    assert len(ids) == 9
    pos = 2
    for r, tr in enumerate(traces):
        assert tr.ctx_len == pos
        assert list(ids[pos: pos + len(tr.emitted)]) == tr.emitted
        pos += len(tr.emitted)
    # same seed -> same output; another seed -> (almost surely) another
    ids2, _ = sd.generate(mp, mq, [1, 2], 3, 2, 7, 1.0, 1.0, 5)
    assert np.array_equal(ids, ids2)


def test_autoregressive_sampling_is_a_round_with_an_empty_draft():
    mp, mq = _tiny_pair(V=5, seed=41, std=0.25)
    ctx = np.array([1, 4, 2])
    p1 = _softmax(mp.logits(ctx, [2])[0])
    N = 2500
    counts = np.zeros(5)
    for rnd in range(N):
        counts[sd.autoregressive_sample(mp, ctx, 1, 1.0, 9, first_round=rnd)[-1]] += 1
    assert stats.chisquare(counts, p1 * N).pvalue > 1e-3          # the draw follows the target distribution
    # greedy limit: identical to arg-max decoding
    assert np.array_equal(sd.autoregressive_sample(mp, ctx, 6, 0.0, 9), sd.autoregressive_greedy(mp, ctx, 6))
    # the draw is the bonus stream at slot 0 of the round
    from oracle import philox as px
    lam = mp.logits(ctx, [2])[0]
    g = px.vocab_gumbels(9, px.BONUS, 7, 0, 0, 0, 5)
    assert sd.autoregressive_sample(mp, ctx, 1, 1.0, 9, first_round=7)[-1] == int(np.argmax(lam + g))
