"""The comparison helpers of the GPU parity tests, checked on the CPU with the oracle standing in for "the other
implementation": an exact copy of the oracle's outcome passes without a log record, a wrong outcome fails, and where
fp32 cannot decide (|u - p/q| inside the band) both outcomes pass, each checked against the extra token that belongs
to ITS accepted length, and each logged under the band that excused it."""
import numpy as np
import pytest

from oracle import philox as px
from oracle import specdiff as sd
from tests import parity

SEED, RND, B = 17, 3, 2


def _case(V=6, gamma=4, tie_at=None):
    """Logits whose acceptance ratio at row `tie_at` equals that row's accept uniform (to rounding)."""
    rng = np.random.default_rng(5)
    lam = rng.standard_normal((gamma + 1, V))
    qrows = rng.standard_normal((gamma, V))
    drafts = rng.integers(0, V, size=gamma)
    # make every row before the tie an accept (p(x) >= q(x)): give the draft token a large target logit
    for j in range(gamma):
        lam[j, drafts[j]] += 8.0
    if tie_at is not None:
        j, x = tie_at, int(drafts[tie_at])
        u = px.scalar_uniform(SEED, px.ACCEPT, RND, 0, j, B)
        qx = np.exp(sd.log_softmax(qrows[j]))[x]
        px_target = u * qx                      # want p(x) = u q(x)  =>  ratio = u
        others = np.delete(np.arange(V), x)
        rest = np.exp(sd.log_softmax(lam[j, others]))
        lam[j, others] = np.log(rest * (1.0 - px_target))
        lam[j, x] = np.log(px_target)
    return lam, qrows, drafts


def _oracle(lam, qrows, drafts):
    logq = np.array([sd.log_softmax(qrows[j])[drafts[j]] for j in range(len(drafts))])
    return sd.accept_resample(lam, qrows, logq, drafts, 1.0, 1.0, SEED, RND, B), logq


def test_exact_copy_passes_and_wrong_outcomes_fail():
    lam, qrows, drafts = _case()
    res, logq = _oracle(lam, qrows, drafts)
    log = []
    parity.check_accept(lam, qrows, logq, drafts, 1.0, 1.0, SEED, RND, B, res.n, res.t, res.ratio, log)
    assert log == []
    with pytest.raises(AssertionError):          # an accepted length no reading of the tests allows
        parity.check_accept(lam, qrows, logq, drafts, 1.0, 1.0, SEED, RND, B, (res.n + 1) % (len(drafts) + 1), res.t,
                            res.ratio, [])
    with pytest.raises(AssertionError):          # right length, wrong extra token, no band to excuse it
        parity.check_accept(lam, qrows, logq, drafts, 1.0, 1.0, SEED, RND, B, res.n, (res.t + 1) % lam.shape[1],
                            res.ratio, [])
    with pytest.raises(AssertionError):          # acceptance probability off by more than 1e-5
        parity.check_accept(lam, qrows, logq, drafts, 1.0, 1.0, SEED, RND, B, res.n, res.t, res.ratio + 1e-4, [])


def test_near_tie_admits_both_lengths_each_with_its_own_extra_token():
    tie = 2
    lam, qrows, drafts = _case(tie_at=tie)
    res, logq = _oracle(lam, qrows, drafts)
    assert abs(res.u[tie] - res.ratio[tie]) < 1e-12
    valid = parity.accepted_lengths_within_band(res.u, res.ratio)
    assert len(valid) == 2 and res.n in valid and tie in valid
    other_n = [n for n in valid if n != res.n][0]
    t_other = sd.extra_token(lam, qrows, drafts, other_n, 1.0, 1.0, SEED, RND, B)[0]
    # the oracle's own outcome: no band needed
    log = []
    parity.check_accept(lam, qrows, logq, drafts, 1.0, 1.0, SEED, RND, B, res.n, res.t, res.ratio, log)
    assert log == []
    # the flipped decision: allowed, logged under the u band, and checked against the token of THAT length
    log = []
    parity.check_accept(lam, qrows, logq, drafts, 1.0, 1.0, SEED, RND, B, other_n, t_other, res.ratio, log)
    assert [r[:2] for r in log] == [("accept", "u")] and log[0][4] == tie
    assert parity.kinds(log) == {("accept", "u"): 1}
    parity.assert_few(log)
    # the flipped length with the token of the oracle's length is an error unless both happen to coincide
    if t_other != res.t:
        with pytest.raises(AssertionError):
            parity.check_accept(lam, qrows, logq, drafts, 1.0, 1.0, SEED, RND, B, other_n, res.t, res.ratio, [])
    # a length that no flip explains stays an error
    bad = [n for n in range(len(drafts) + 1) if n not in valid][0]
    with pytest.raises(AssertionError):
        parity.check_accept(lam, qrows, logq, drafts, 1.0, 1.0, SEED, RND, B, bad, res.t, res.ratio, [])


def test_extra_token_function_is_what_the_round_uses():
    lam, qrows, drafts = _case(V=9, gamma=3)
    res, _ = _oracle(lam, qrows, drafts)
    t, gap, _ = sd.extra_token(lam, qrows, drafts, res.n, 1.0, 1.0, SEED, RND, B)
    assert (t, gap) == (res.t, res.final_gap)
    # n = gamma is the bonus draw from the last target row alone: the q rows do not matter
    t_b = sd.extra_token(lam, qrows, drafts, 3, 1.0, 1.0, SEED, RND, B)[0]
    t_b2 = sd.extra_token(lam, qrows + 1.0, drafts, 3, 1.0, 1.0, SEED, RND, B)[0]
    assert t_b == t_b2 == int(np.argmax(lam[3] + px.vocab_gumbels(SEED, px.BONUS, RND, 0, 3, B, 9)))


def test_too_many_band_records_fail():
    with pytest.raises(AssertionError):
        parity.assert_few([("accept", "u")] * 2)
    with pytest.raises(AssertionError):
        parity.assert_few([("draw", "cancellation")] * 2)
    parity.assert_few([("draft", "gap"), ("draw", "gap"), ("accept", "u"), ("draw", "cancellation")])
