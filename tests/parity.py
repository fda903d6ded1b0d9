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


def draw_ambiguous(g: np.ndarray, logp: np.ndarray, p: np.ndarray, q: np.ndarray, resid: bool) -> bool:
    """True if an fp32 evaluation of the final Gumbel arg-max could pick another index than fp64 does.
    Bonus draw: scores logp + g, each known to about FP32_LOGP_ERR.  Residual draw: scores
    log(p - q) + g where p - q carries an absolute error of about delta * (p + q) from cancellation."""
    if not resid:
        score = logp + g
        win = int(np.argmax(score))
        rest = np.delete(score, win)
        return bool(rest.max() >= score[win] - GAP_BAND)
    w = p - q
    slack = FP32_LOGP_ERR * (p + q)
    if not np.any(w > 0):
        return True
    with np.errstate(divide="ignore"):
        score = np.where(w > 0, np.log(np.maximum(w, 1e-300)) + g, -np.inf)
        upper = np.where(w + slack > 0, np.log(np.maximum(w + slack, 1e-300)) + g, -np.inf)
    win = int(np.argmax(score))
    lower_win = np.log(max(w[win] - slack[win], 1e-300)) + g[win]
    upper[win] = -np.inf
    return bool(upper.max() >= lower_win - GAP_BAND)


def check_accept(lam, qrows, logq, draft_ids, tau_p, tau_q, seed, rnd, b, got_n, got_t, got_prob, log):
    """Compare one sequence's acceptance outcome with the oracle run on the same logits.
    lam [gamma+1, V], qrows [gamma, V] (already divided by tau_q), logq [gamma] (as stored by the
    implementation, or None to take the oracle's own).  Appends near-tie records to `log`.
    Returns the oracle result."""
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
    near = np.abs(res.u - res.ratio) < U_BAND
    # walk left to right: decisions must agree until the first undecidable row
    n_ok = True
    for j in range(gamma):
        if near[j] and j <= min(res.n, got_n):
            log.append(("accept-near-tie", rnd, b, j, float(res.u[j]), float(res.ratio[j]), int(got_n), int(res.n)))
            n_ok = False
            break
        if j >= res.n:
            break
    if n_ok:
        assert got_n == res.n, (got_n, res.n, res.u, res.ratio)
    if got_n == res.n:
        if tau_p > 0:
            resid = res.n < gamma
            V = lam.shape[1]
            logp = sd.log_softmax(lam[res.n] / tau_p)
            p = np.exp(logp)
            q = sd.q_probs(qrows[res.n], int(draft_ids[res.n]), tau_q) if resid else np.zeros_like(p)
            g = px.vocab_gumbels(seed, px.RESID if resid else px.BONUS, rnd, 0, res.n, b, V)
            amb = draw_ambiguous(g, logp, p, q, resid)
        else:
            amb = False
        if amb and got_t != res.t:
            log.append(("draw-near-tie", rnd, b, int(res.n), int(got_t), int(res.t), float(res.final_gap)))
        else:
            assert got_t == res.t, (got_t, res.t, res.final_gap)
    return res


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
            log.append(("draft-near-tie", rnd, b, j, int(got_slots[j]), int(st.slots[j]), float(st.gumbel_gap[j])))
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
