"""Pins for the oracle's acceptance / resampling stage against what the paper and
speculative sampling fix: alpha = sum_x min(p, q) (Corollary in the appendix), the output
law equals the target distribution ("directly match the sampling output", Introduction),
and the accepted-length law behind Eq. 2."""
import math

import numpy as np
from scipy import stats

import synth
from oracle import philox as px
from oracle import specdiff as sd


def _softmax(z):
    z = np.asarray(z, dtype=np.float64)
    e = np.exp(z - z.max())
    return e / e.sum()


def test_logsumexp_textbook():
    rng = np.random.default_rng(1)
    z = rng.normal(size=1000) * 3
    naive = math.log(sum(math.exp(v) for v in z))
    assert abs(sd.logsumexp(z) - naive) < 1e-12
    assert abs(sd.logsumexp(z + 500.0) - (naive + 500.0)) < 1e-9      # shift invariance, no overflow
    assert abs(np.exp(sd.log_softmax(z)).sum() - 1.0) < 1e-12
    assert sd.logsumexp(np.array([-1e4, -1e4])) == -1e4 + math.log(2.0)


def test_argmax_with_gap():
    i, gap = sd.argmax_with_gap(np.array([1.0, 5.0, 5.0, 2.0]))
    assert i == 1 and gap == 0.0          # lowest index wins a tie
    i, gap = sd.argmax_with_gap(np.array([1.0, 5.0, 4.5]))
    assert i == 1 and gap == 0.5


def _one_row(lam, ell, x, rnd, seed=7, tau_p=1.0, tau_q=1.0, keep=False):
    """gamma = 1 acceptance of draft x; second target row is a fixed bonus row."""
    V = len(lam)
    lam2 = np.stack([lam, np.zeros(V)])
    qrow = np.asarray(ell, dtype=np.float64) / (tau_q if tau_q > 0 else 1.0)
    logq = sd.log_softmax(qrow)[x] if tau_q > 0 else 0.0
    return sd.accept_resample(lam2, qrow[None], np.array([logq]), np.array([x]), tau_p, tau_q, seed, rnd, 0,
                              keep_scores=keep)


def test_accept_probability_and_output_law_by_enumeration():
    """Exact, vocab <= 8: sum_x q(x) min(1, p/q) = sum min(p,q); sum max(0,p-q) = 1 - alpha;
    and P(out = y) = p(y) for every y."""
    rng = np.random.default_rng(2)
    for V in (2, 5, 8):
        for _ in range(4):
            lam, ell = rng.normal(size=V) * 1.5, rng.normal(size=V) * 1.5
            p, q = _softmax(lam), _softmax(ell)
            alpha = np.minimum(p, q).sum()
            assert abs(np.maximum(0, p - q).sum() - (1 - alpha)) < 1e-12
            assert abs(0.5 * np.abs(p - q).sum() - (1 - alpha)) < 1e-12       # D_LK = TV
            out_law = np.zeros(V)
            acc_prob = 0.0
            for x in range(V):
                res = _one_row(lam, ell, x, rnd=0)
                assert abs(res.ratio[0] - min(1.0, p[x] / q[x])) < 1e-12
                assert abs(res.sum_min[0] - alpha) < 1e-12
                acc_prob += q[x] * res.ratio[0]
                out_law[x] += q[x] * res.ratio[0]
                if res.ratio[0] < 1.0:
                    # find a round whose uniform rejects, and read the residual weights it used
                    for rnd in range(400):
                        rj = _one_row(lam, ell, x, rnd, keep=True)
                        if rj.n == 0:
                            break
                    assert rj.n == 0
                    g = px.vocab_gumbels(7, px.RESID, rnd, 0, 0, 0, V)
                    w = np.exp(rj.final_scores - g)
                    resid = w / w.sum()
                    out_law += q[x] * (1 - res.ratio[0]) * resid
            assert abs(acc_prob - alpha) < 1e-12
            assert np.abs(out_law - p).max() < 1e-12


def test_accept_decision_is_u_le_ratio_and_left_to_right():
    rng = np.random.default_rng(3)
    V, gamma = 6, 5
    lam = rng.normal(size=(gamma + 1, V))
    ell = rng.normal(size=(gamma, V))
    logq_all = np.stack([sd.log_softmax(r) for r in ell])
    seen = set()
    for rnd in range(300):
        x = rng.integers(0, V, size=gamma)
        logq = logq_all[np.arange(gamma), x]
        r = sd.accept_resample(lam, ell, logq, x, 1.0, 1.0, 11, rnd, 2)
        ok = r.u <= r.ratio
        n = gamma if ok.all() else int(np.argmin(ok))
        assert r.n == n and 0 <= r.t < V
        for j in range(gamma):
            assert r.u[j] == px.scalar_uniform(11, px.ACCEPT, rnd, 0, j, 2)
        if n < gamma:  # the resampled token can never be one with p <= q at the rejected row
            p, q = _softmax(lam[n]), _softmax(ell[n])
            assert p[r.t] > q[r.t]
        seen.add(n)
    assert len(seen) >= 4


def test_output_law_chi_square_philox_driven():
    """x ~ q by the oracle's own Gumbel draw, then accept/resample: the emitted token ~ p."""
    V, N = 8, 12000
    rng = np.random.default_rng(4)
    lam, ell = rng.normal(size=V) * 1.2, rng.normal(size=V) * 1.2
    p, q = _softmax(lam), _softmax(ell)
    counts = np.zeros(V)
    draft_counts = np.zeros(V)
    n_acc = 0
    for rnd in range(N):
        st = sd.DraftState.fresh(1, V)
        sd.unmask_sample_step(st, ell[None], 1, 1.0, 5, rnd, 0)
        x = int(st.slots[0])
        draft_counts[x] += 1
        lam2 = np.stack([lam, lam])
        r = sd.accept_resample(lam2, st.qrows, st.logq, st.slots, 1.0, 1.0, 5, rnd, 0)
        n_acc += r.n
        counts[x if r.n == 1 else r.t] += 1
    assert stats.chisquare(draft_counts, q * N).pvalue > 1e-3      # Gumbel-max draws follow softmax
    assert stats.chisquare(counts, p * N).pvalue > 1e-3            # lossless
    alpha = np.minimum(p, q).sum()
    assert abs(n_acc / N - alpha) < 4 * math.sqrt(alpha * (1 - alpha) / N)


def test_gumbel_draw_shift_invariant():
    V = 8
    ell = np.random.default_rng(5).normal(size=V)
    for rnd in range(20):
        a, b = sd.DraftState.fresh(1, V), sd.DraftState.fresh(1, V)
        sd.unmask_sample_step(a, ell[None], 1, 1.0, 1, rnd, 0)
        sd.unmask_sample_step(b, ell[None] + 3.25, 1, 1.0, 1, rnd, 0)
        assert a.slots[0] == b.slots[0] and abs(a.logq[0] - b.logq[0]) < 1e-12


def test_accepted_length_law_eq2():
    """Rows with constant alpha: P(n = k) = alpha^k (1 - alpha), P(n = gamma) = alpha^gamma,
    mean emitted = (1 - alpha^(gamma+1)) / (1 - alpha)   (Eq. 2)."""
    V, gamma, N = 4, 6, 3000
    p = np.array([0.55, 0.25, 0.15, 0.05])
    q = np.array([0.25, 0.55, 0.05, 0.15])
    alpha = np.minimum(p, q).sum()  # 0.6
    lam = np.tile(np.log(p), (gamma + 1, 1))
    ell = np.tile(np.log(q), (gamma, 1))
    rng = np.random.default_rng(6)
    hist = np.zeros(gamma + 1)
    for rnd in range(N):
        x = rng.choice(V, size=gamma, p=q)
        r = sd.accept_resample(lam, ell, np.log(q)[x], x, 1.0, 1.0, 21, rnd, 0)
        hist[r.n] += 1
    expect = np.array([alpha ** k * (1 - alpha) for k in range(gamma)] + [alpha ** gamma]) * N
    assert stats.chisquare(hist, expect).pvalue > 1e-3
    mean_emitted = (hist * (np.arange(gamma + 1) + 1)).sum() / N
    assert abs(mean_emitted - sd.expected_tokens_per_draft(alpha, gamma)) < 0.12
    assert abs(sd.expected_tokens_per_draft(0.5, 1) - 1.5) < 1e-15
    assert abs(sd.expected_tokens_per_second(0.5, 1, 2, 1.0, 1.0) - 0.5) < 1e-15


def test_greedy_rule_is_argmax_match():
    rng = np.random.default_rng(8)
    V, gamma = 7, 4
    lam = rng.normal(size=(gamma + 1, V))
    top = lam.argmax(axis=1)
    drafts = top[:gamma].copy()
    drafts[2] = (drafts[2] + 1) % V
    r = sd.accept_resample(lam, np.zeros((gamma, V)), np.zeros(gamma), drafts, 0.0, 0.0, 1, 0, 0)
    assert r.n == 2 and r.t == top[2]
    r = sd.accept_resample(lam, np.zeros((gamma, V)), np.zeros(gamma), top[:gamma], 0.0, 0.0, 1, 0, 0)
    assert r.n == gamma and r.t == top[gamma]


def test_degenerate_p_equals_q_falls_back_to_p():
    V = 5
    z = np.random.default_rng(9).normal(size=V)
    # force the rejection branch by an impossible logq (claims q(x) = 1 while p(x) < 1)
    r = sd.accept_resample(np.stack([z, z]), z[None], np.array([0.0]), np.array([int(np.argmin(z))]),
                           1.0, 1.0, 3, 0, 0, keep_scores=True)
    if r.n == 0:
        g = px.vocab_gumbels(3, px.RESID, 0, 0, 0, 0, V)
        w = np.exp(r.final_scores - g)
        assert np.allclose(w / w.sum(), _softmax(z), atol=1e-12)


def test_microbench_generator_overlap_closed_form_and_acceptance():
    """Large-vocab inputs: mean sum_x min(p,q) matches 2 Phi(-sigma / sqrt 2) within 0.01 and the
    empirical acceptance frequency sits inside its binomial interval."""
    rows, gamma, V = 3, 8, 50257
    for si, sigma in ((1, 0.30), (3, 0.70)):
        case = synth.accept_case(rows, gamma, V, sigma, seed=31 + si)
        tested = accepted = 0
        sm = []
        for r in range(rows):
            lq = case.logits_q[r].astype(np.float64)
            logq = np.array([sd.log_softmax(lq[j])[case.draft_ids[r, j]] for j in range(gamma)])
            res = sd.accept_resample(case.logits_p[r], lq, logq, case.draft_ids[r], 1.0, 1.0, 77, 0, r)
            sm += list(res.sum_min)
            tested += gamma
            accepted += int((res.u <= res.ratio).sum())
            assert 0 <= res.t < V
        alpha = float(np.mean(sm))
        assert abs(alpha - 2 * stats.norm.cdf(-sigma / math.sqrt(2))) < 0.01
        assert abs(accepted / tested - alpha) < 4 * math.sqrt(alpha * (1 - alpha) / tested)
