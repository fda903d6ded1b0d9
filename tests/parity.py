"""Helpers of the GPU parity tests: run the oracle's sampling / acceptance stage on given logits
and compare another implementation's decisions with it, setting aside (and counting) the draws
that fp32 arithmetic cannot decide."""
from __future__ import annotations

import numpy as np

from oracle import philox as px
from oracle import specdiff as sd

U_BAND = 1e-5        # |u - ratio| below this: the accept decision is a logged near-tie
GAP_BAND = 1e-4      # Gumbel top-2 gap below this: the draw is a logged near-tie
FP32_LOGP_ERR = 4e-6  # absolute error allowed on a log-probability computed in fp32


def draw_ambiguous(g: np.ndarray, logp: np.ndarray, p: np.ndarray, q: np.ndarray, resid: bool):
    """Which band, if any, excuses an fp32 evaluation of the final Gumbel arg-max that picks another index than fp64
    does: None (the draw is decidable), "gap" (top-2 gap of the scores below GAP_BAND) or "cancellation" (residual
    draw only: a runner-up whose score reaches the winner's once p - q is given its cancellation error of about
    delta * (p + q))."""
    if not resid:
        score = logp + g
        win = int(np.argmax(score))
        rest = np.delete(score, win)
        return "gap" if rest.max() >= score[win] - GAP_BAND else None
    w = p - q
    slack = FP32_LOGP_ERR * (p + q)
    if not np.any(w > 0):
        return "cancellation"
    with np.errstate(divide="ignore"):
        score = np.where(w > 0, np.log(np.maximum(w, 1e-300)) + g, -np.inf)
        upper = np.where(w + slack > 0, np.log(np.maximum(w + slack, 1e-300)) + g, -np.inf)
    win = int(np.argmax(score))
    rest = score.copy()
    rest[win] = -np.inf
    if rest.max() >= score[win] - GAP_BAND:
        return "gap"
    lower_win = np.log(max(w[win] - slack[win], 1e-300)) + g[win]
    upper[win] = -np.inf
    return "cancellation" if upper.max() >= lower_win - GAP_BAND else None


def accepted_lengths_within_band(u: np.ndarray, ratio: np.ndarray):
    """Every accepted length that follows from the tests u_j <= ratio_j when each test inside the band
    |u - ratio| < U_BAND may go either way: {n: tuple of the rows whose decision differs from the fp64 one}."""
    gamma = len(u)
    acc = u <= ratio
    near = [j for j in range(gamma) if abs(u[j] - ratio[j]) < U_BAND][:12]
    out = {}
    for mask in range(1 << len(near)):
        a = acc.copy()
        flipped = tuple(j for i, j in enumerate(near) if (mask >> i) & 1)
        for j in flipped:
            a[j] = not a[j]
        n = 0
        while n < gamma and a[n]:
            n += 1
        # only flips at rows the scan reaches matter; keep the smallest explanation
        used = tuple(j for j in flipped if j <= n)
        if n not in out or len(used) < len(out[n]):
            out[n] = used
    return out


def check_accept(lam, qrows, logq, draft_ids, tau_p, tau_q, seed, rnd, b, got_n, got_t, got_prob, log):
    """Compare one sequence's acceptance outcome with the oracle run on the same logits.
    lam [gamma+1, V], qrows [gamma, V] (already divided by tau_q), logq [gamma] (as stored by the
    implementation, or None to take the oracle's own).  Where fp32 cannot decide, every valid outcome is
    worked out and the implementation's must be one of them: the accepted length must follow from the tests
    with the near-tie decisions taken either way, and the extra token is checked FOR THAT LENGTH.  Appends
    (event, band, ...) records to `log` for every decision that needed a band.  Returns the oracle result."""
    gamma = qrows.shape[0]
    lam = np.asarray(lam, np.float64)
    qrows = np.asarray(qrows, np.float64)
    if logq is None:
        if tau_q > 0:
            logq = np.array([sd.log_softmax(qrows[j])[draft_ids[j]] for j in range(gamma)])
        else:
            logq = np.zeros(gamma)
    res = sd.accept_resample(lam, qrows, np.asarray(logq, np.float64), draft_ids, tau_p, tau_q, seed, rnd, b,
                             keep_scores=True)
    assert np.abs(np.asarray(got_prob, np.float64) - res.ratio).max() < 1e-5, (got_prob, res.ratio)
    valid = accepted_lengths_within_band(res.u, res.ratio)
    assert got_n in valid, (got_n, res.n, sorted(valid), res.u, res.ratio)
    for j in valid[got_n]:
        log.append(("accept", "u", rnd, b, int(j), float(res.u[j]), float(res.ratio[j]), int(got_n), int(res.n)))
    # the extra token that belongs to the implementation's accepted length
    t_ref, gap, _ = (res.t, res.final_gap, None) if got_n == res.n else \
        sd.extra_token(lam, qrows, draft_ids, got_n, tau_p, tau_q, seed, rnd, b)
    if got_t != t_ref:
        band = None
        if tau_p > 0:
            resid = got_n < gamma
            V = lam.shape[1]
            logp = sd.log_softmax(lam[got_n] / tau_p)
            p = np.exp(logp)
            q = sd.q_probs(qrows[got_n], int(draft_ids[got_n]), tau_q) if resid else np.zeros_like(p)
            g = px.vocab_gumbels(seed, px.RESID if resid else px.BONUS, rnd, 0, got_n, b, V)
            band = draw_ambiguous(g, logp, p, q, resid)
        assert band is not None, (got_t, t_ref, gap)
        log.append(("draw", band, rnd, b, int(got_n), int(got_t), int(t_ref), float(gap)))
    return res


def kinds(log):
    """Number of log records per (event, band)."""
    out = {}
    for rec in log:
        out[(rec[0], rec[1])] = out.get((rec[0], rec[1]), 0) + 1
    return out


def assert_few(log, u=1, gap=2, cancellation=1):
    """A test may meet a few undecidable draws, counted by the band that excused them."""
    k = kinds(log)
    n_u = sum(v for (e, band), v in k.items() if band == "u")
    n_gap = sum(v for (e, band), v in k.items() if band == "gap")
    n_c = sum(v for (e, band), v in k.items() if band == "cancellation")
    assert n_u <= u and n_gap <= gap and n_c <= cancellation, k


def check_unmask_step(st: "sd.DraftState", step_logits, k, tau_q, seed, rnd, b, got_slots, got_logq, got_reveal,
                      got_qrows, log):
    """Advance the oracle draft state `st` by denoising step k on `step_logits` [gamma, V] and compare with
    the implementation's state after the same step."""
    V = st.vocab
    sd.unmask_sample_step(st, np.asarray(step_logits, np.float64), k, tau_q, seed, rnd, b)
    for j in range(st.gamma):
        if st.reveal_step[j] != k:
            continue
        assert got_reveal[j] == k, (j, k, got_reveal)
        if st.gumbel_gap[j] < GAP_BAND and got_slots[j] != st.slots[j]:
            log.append(("draft", "gap", rnd, b, j, int(got_slots[j]), int(st.slots[j]), float(st.gumbel_gap[j])))
            # follow the implementation so that later steps see the same state
            x = int(got_slots[j])
            st.slots[j] = x
            st.logq[j] = st.qrows[j][x] - sd.logsumexp(st.qrows[j]) if tau_q > 0 else 0.0
        else:
            assert got_slots[j] == st.slots[j], (j, got_slots[j], st.slots[j], st.gumbel_gap[j])
        assert abs(got_logq[j] - st.logq[j]) < 1e-5, (j, got_logq[j], st.logq[j])
        if got_qrows is not None:
            assert np.abs(np.asarray(got_qrows[j], np.float64) - st.qrows[j]).max() < 1e-5
    # the reveal pattern (which slots are still masked) is integer work: bit-exact
    assert np.array_equal(np.asarray(got_slots) == V, st.slots == V)
    assert np.array_equal(np.asarray(got_reveal), st.reveal_step)
