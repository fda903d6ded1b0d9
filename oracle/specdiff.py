"""TEST INFRASTRUCTURE — CPU oracle, not part of the product path.

One draft–verify–accept round of Speculative Diffusion Decoding (Algorithm 1 of the
paper), taken step by step in the paper's order, in fp64 numpy.  A round is a randomised
procedure, so the oracle follows the algorithm (it has no closed-form result) and is
driven by explicit Philox streams (`oracle/philox.py`) so that another implementation
can be compared with it draw for draw.

Readings of the paper taken here (the paper is silent or garbled on each):
  * Algorithm 1's initial state "q^T ~ N(0, sigma_T I)" is continuous-diffusion notation;
    for a *masked* discrete model (Section "SpecDiff: Formulation") the initial state is
    all gamma slots = [MASK].
  * The reverse update is not given.  Used here: ancestral masked-diffusion sampling on a
    uniform time grid t_k = k/T with mask probability t, i.e. at step k (k = T..1) a
    still-masked slot is revealed with probability (t_k - t_{k-1})/t_k = 1/k by sampling
    the network's categorical for that slot; revealed slots never change again.
  * The drafter takes tokens only (no time-step input).
  * q_j in the acceptance ratio is the distribution slot j's token was actually drawn
    from: the logits of the step that revealed it, kept from then on (Section "SpecDiff: Formulation").
  * gamma+1 target rows: row j is the distribution after context ∘ draft[0:j].
  * "r > p/q  => reject" is evaluated as: accept iff u <= min(1, p/q), in log space.
  * "if n < i + gamma" in Algorithm 1 means n < gamma.
  * norm(max(0, p - q)) with an all-zero numerator (p == q up to rounding) falls back to p.
  * "t ~ p'" and "x ~ q" are Gumbel-max draws keyed per vocabulary entry.
  * temperature tau divides the logits; tau = 0 is greedy decoding (the setting of every
    result the paper reports).
  * the last round's emission is truncated to `max_new`.
  * Section "Sequence initialization" names standard speculative decoding for the start of a sequence (the
    evaluation: its first 100 tokens) and nothing more.  Taken here: whole speculative-decoding rounds with an autoregressive
    drafter run while fewer than `n_init` tokens have been generated; the round that crosses `n_init` is kept
    whole; the rounds share one round counter (and so one random stream layout) with the diffusion rounds.
MDLM-faithfulness of the unmasking rule: parity unpinned (MDLM's sampler is not available).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

from . import philox as px
from .transformer import Model, drafter_slot_logits, target_verify_logits


def logsumexp(z: np.ndarray) -> float:
    m = float(np.max(z))
    return m + float(np.log(np.sum(np.exp(z - m))))


def log_softmax(z: np.ndarray) -> np.ndarray:
    return z - logsumexp(z)


def argmax_with_gap(score: np.ndarray):
    """Index of the maximum (lowest index on ties) and the gap to the runner-up."""
    i = int(np.argmax(score))
    if score.shape[0] == 1:
        return i, float("inf")
    rest = np.delete(score, i)
    return i, float(score[i] - np.max(rest))


# ----------------------------------------------------------------------------------
# drafting: T denoising evaluations (Algorithm 1, first loop, and "x ~ q^0")
# ----------------------------------------------------------------------------------

@dataclass
class DraftState:
    gamma: int
    vocab: int
    slots: np.ndarray            # int64 [gamma]; MASK == vocab
    qrows: np.ndarray            # fp64 [gamma, V]: logits / tau_q of the revealing step (tau_q == 0: raw logits)
    logq: np.ndarray             # fp64 [gamma]: log q_j(draft_j)
    reveal_step: np.ndarray      # int [gamma]: k at which slot j was revealed (0 = still masked)
    gumbel_gap: np.ndarray       # fp64 [gamma]: top-2 gap of the revealing draw (diagnostic)
    unmask_u: List[np.ndarray] = field(default_factory=list)  # per step: uniforms of the reveal test (nan = not tested)

    @staticmethod
    def fresh(gamma: int, vocab: int) -> "DraftState":
        return DraftState(gamma, vocab, np.full(gamma, vocab, np.int64), np.zeros((gamma, vocab)),
                          np.zeros(gamma), np.zeros(gamma, np.int64), np.full(gamma, np.inf))


def unmask_sample_step(st: DraftState, step_logits: np.ndarray, k: int, tau_q: float,
                       seed: int, rnd: int, b: int) -> int:
    """Denoising step k on the logits of this step's drafter evaluation [gamma, V].
    Returns the number of slots revealed."""
    V = st.vocab
    revealed = 0
    us = np.full(st.gamma, np.nan)
    for j in range(st.gamma):
        if st.slots[j] != V:
            continue
        u = px.scalar_uniform(seed, px.UNMASK, rnd, k, j, b)
        us[j] = u
        if not (u < 1.0 / k):
            continue
        row = np.asarray(step_logits[j], dtype=np.float64)
        if tau_q > 0.0:
            z = row / tau_q
            g = px.vocab_gumbels(seed, px.DRAFT, rnd, 0, j, b, V)
            x, gap = argmax_with_gap(z + g)
            st.qrows[j] = z
            st.logq[j] = z[x] - logsumexp(z)
        else:  # greedy: q is the point mass at the arg-max
            x, gap = argmax_with_gap(row)
            st.qrows[j] = row
            st.logq[j] = 0.0
        st.slots[j] = x
        st.reveal_step[j] = k
        st.gumbel_gap[j] = gap
        revealed += 1
    st.unmask_u.append(us)
    return revealed


def draft(model_q: Model, ctx_ids: np.ndarray, gamma: int, T: int, tau_q: float,
          seed: int, rnd: int, b: int, keep_step_logits: bool = False):
    st = DraftState.fresh(gamma, model_q.shape.vocab)
    step_logits = []
    for k in range(T, 0, -1):
        lg = drafter_slot_logits(model_q, ctx_ids, st.slots)
        if keep_step_logits:
            step_logits.append(lg)
        unmask_sample_step(st, lg, k, tau_q, seed, rnd, b)
    assert np.all(st.slots != st.vocab)  # step k = 1 reveals with probability 1
    return st, step_logits


def sps_draft(model_a: Model, ctx_ids: np.ndarray, gamma: int, tau_q: float, seed: int, rnd: int, b: int,
              keep_step_logits: bool = False):
    """Drafting of standard speculative decoding (Section "Preliminaries and Settings", paragraph "Speculative
    decoding"): an autoregressive drafter M_q produces x_{i+1..i+gamma} one token per evaluation,
    x_{i+j} ~ q_{i+j}(. | x_{1:i+j-1}), and every q row is stored for the acceptance test.  The draw of slot j uses
    the same keyed Gumbel stream as the diffusion drafter's draw of slot j."""
    V = model_a.shape.vocab
    st = DraftState.fresh(gamma, V)
    ids = [int(x) for x in ctx_ids]
    step_logits = []
    for j in range(gamma):
        row = model_a.logits(np.array(ids), [len(ids) - 1])[0]
        if keep_step_logits:
            step_logits.append(row)
        if tau_q > 0.0:
            z = row / tau_q
            x, gap = argmax_with_gap(z + px.vocab_gumbels(seed, px.DRAFT, rnd, 0, j, b, V))
            st.qrows[j] = z
            st.logq[j] = z[x] - logsumexp(z)
        else:
            x, gap = argmax_with_gap(row)
            st.qrows[j] = row
            st.logq[j] = 0.0
        st.slots[j] = x
        st.reveal_step[j] = gamma - j          # bookkeeping only: evaluation j + 1 of gamma wrote this slot
        st.gumbel_gap[j] = gap
        ids.append(int(x))
    return st, step_logits


# ----------------------------------------------------------------------------------
# acceptance and the extra token (Algorithm 1, from the acceptance block to the return statement)
# ----------------------------------------------------------------------------------

def q_probs(qrow: np.ndarray, draft_id: int, tau_q: float) -> np.ndarray:
    if tau_q > 0.0:
        return np.exp(log_softmax(qrow))
    p = np.zeros_like(qrow)
    p[draft_id] = 1.0
    return p


def p_probs(lam_row: np.ndarray, tau_p: float) -> np.ndarray:
    if tau_p > 0.0:
        return np.exp(log_softmax(lam_row / tau_p))
    p = np.zeros_like(lam_row, dtype=np.float64)
    p[int(np.argmax(lam_row))] = 1.0
    return p


@dataclass
class AcceptResult:
    n: int                       # number of accepted draft tokens
    t: int                       # the extra token (from the adjusted or the plain target distribution)
    ratio: np.ndarray            # fp64 [gamma]: min(1, p_j(x_j)/q_j(x_j)) for every row (also past n)
    u: np.ndarray                # fp64 [gamma]: the accept uniforms
    logp: np.ndarray             # fp64 [gamma]
    sum_min: np.ndarray          # fp64 [gamma]: sum_x min(p_j, q_j)
    final_gap: float             # top-2 gap of the final Gumbel draw (diagnostic)
    final_scores: Optional[np.ndarray] = None


def accept_resample(lam: np.ndarray, qrows: np.ndarray, logq: np.ndarray, draft_ids: np.ndarray,
                    tau_p: float, tau_q: float, seed: int, rnd: int, b: int,
                    keep_scores: bool = False) -> AcceptResult:
    """lam: target logits [gamma+1, V]; qrows: stored draft rows [gamma, V] (already / tau_q);
    logq[j] = log q_j(draft_j)."""
    gamma, V = qrows.shape
    lam = np.asarray(lam, dtype=np.float64)
    ratio = np.zeros(gamma)
    us = np.zeros(gamma)
    logp = np.zeros(gamma)
    sum_min = np.zeros(gamma)
    for j in range(gamma):
        x = int(draft_ids[j])
        if tau_p > 0.0:
            z = lam[j] / tau_p
            logp[j] = z[x] - logsumexp(z)
            ratio[j] = np.exp(min(0.0, logp[j] - logq[j]))
        else:
            hit = x == int(np.argmax(lam[j]))
            logp[j] = 0.0 if hit else -np.inf
            ratio[j] = 1.0 if hit else 0.0
        us[j] = px.scalar_uniform(seed, px.ACCEPT, rnd, 0, j, b)
        sum_min[j] = np.minimum(p_probs(lam[j], tau_p), q_probs(qrows[j], x, tau_q)).sum()
    n = 0
    while n < gamma and us[n] <= ratio[n]:
        n += 1
    t, gap, score = extra_token(lam, qrows, draft_ids, n, tau_p, tau_q, seed, rnd, b)
    return AcceptResult(n, t, ratio, us, logp, sum_min, gap, score if keep_scores else None)


def extra_token(lam: np.ndarray, qrows: np.ndarray, draft_ids: np.ndarray, n: int, tau_p: float, tau_q: float,
                seed: int, rnd: int, b: int):
    """The token that follows n accepted drafts (Algorithm 1, the block that adjusts the distribution): for
    n < gamma a draw from norm(max(0, p_n - q_n)), for n == gamma a draw from p_gamma.
    Returns (token, top-2 gap of the Gumbel scores, scores)."""
    gamma, V = qrows.shape
    lam = np.asarray(lam, dtype=np.float64)
    if n < gamma:
        p = p_probs(lam[n], tau_p)
        q = q_probs(qrows[n], int(draft_ids[n]), tau_q)
        w = np.maximum(0.0, p - q)
        if not np.any(w > 0.0):
            w = p
        if tau_p > 0.0:
            with np.errstate(divide="ignore"):
                score = np.log(w) + px.vocab_gumbels(seed, px.RESID, rnd, 0, n, b, V)
        else:
            score = np.where(w > 0.0, 0.0, -np.inf)
    else:
        if tau_p > 0.0:
            score = lam[gamma] / tau_p + px.vocab_gumbels(seed, px.BONUS, rnd, 0, gamma, b, V)
        else:
            score = lam[gamma]
    t, gap = argmax_with_gap(score)
    return t, gap, score


# ----------------------------------------------------------------------------------
# whole round and generation loop
# ----------------------------------------------------------------------------------

@dataclass
class RoundTrace:
    ctx_len: int
    draft: DraftState
    acc: AcceptResult
    emitted: List[int]
    lam: Optional[np.ndarray] = None
    step_logits: Optional[list] = None


def specdiff_round(model_p: Model, model_q: Model, ctx_ids, gamma: int, T: int,
                   tau_p: float, tau_q: float, seed: int, rnd: int, b: int = 0,
                   keep: bool = False) -> RoundTrace:
    ctx_ids = np.asarray(ctx_ids, dtype=np.int64)
    st, step_logits = draft(model_q, ctx_ids, gamma, T, tau_q, seed, rnd, b, keep_step_logits=keep)
    lam = target_verify_logits(model_p, ctx_ids, st.slots)
    acc = accept_resample(lam, st.qrows, st.logq, st.slots, tau_p, tau_q, seed, rnd, b)
    emitted = [int(x) for x in st.slots[: acc.n]] + [acc.t]
    return RoundTrace(len(ctx_ids), st, acc, emitted, lam if keep else None, step_logits if keep else None)


def sps_round(model_p: Model, model_a: Model, ctx_ids, gamma: int, tau_p: float, tau_q: float, seed: int, rnd: int,
              b: int = 0, keep: bool = False) -> RoundTrace:
    """One round of standard speculative decoding: autoregressive drafting, then the same verification,
    acceptance and extra-token steps as Algorithm 1 (which differs from it only in how the draft is made)."""
    ctx_ids = np.asarray(ctx_ids, dtype=np.int64)
    st, step_logits = sps_draft(model_a, ctx_ids, gamma, tau_q, seed, rnd, b, keep_step_logits=keep)
    lam = target_verify_logits(model_p, ctx_ids, st.slots)
    acc = accept_resample(lam, st.qrows, st.logq, st.slots, tau_p, tau_q, seed, rnd, b)
    emitted = [int(x) for x in st.slots[: acc.n]] + [acc.t]
    return RoundTrace(len(ctx_ids), st, acc, emitted, lam if keep else None, step_logits if keep else None)


def generate_with_sps_init(model_p: Model, model_q: Model, model_a: Model, prompt, gamma: int, T: int, gamma_sps: int,
                           n_init: int, max_new: int, tau_p: float = 1.0, tau_q: float = 1.0, seed: int = 0,
                           b: int = 0, keep: bool = False):
    """Section "Sequence initialization": speculative-decoding rounds (drafter model_a, gamma_sps tokens per draft)
    while fewer than n_init tokens exist, SpecDiff rounds (drafter model_q) after that.
    Returns (all ids, list of RoundTrace, number of speculative-decoding rounds)."""
    ids = [int(x) for x in prompt]
    P = len(ids)
    traces = []
    rnd = 0
    n_sps = 0
    while len(ids) - P < max_new:
        if len(ids) - P < n_init:
            tr = sps_round(model_p, model_a, np.array(ids), gamma_sps, tau_p, tau_q, seed, rnd, b, keep)
            n_sps += 1
        else:
            tr = specdiff_round(model_p, model_q, np.array(ids), gamma, T, tau_p, tau_q, seed, rnd, b, keep)
        tr.emitted = tr.emitted[: max_new - (len(ids) - P)]
        ids += tr.emitted
        traces.append(tr)
        rnd += 1
    return np.array(ids, dtype=np.int64), traces, n_sps


def generate(model_p: Model, model_q: Model, prompt, gamma: int, T: int, max_new: int,
             tau_p: float = 1.0, tau_q: float = 1.0, seed: int = 0, b: int = 0,
             max_rounds: Optional[int] = None, keep: bool = False):
    """Repeat rounds until `max_new` tokens (Section "Preliminaries": produce the next n tokens).
    Returns (all ids, list of RoundTrace)."""
    ids = [int(x) for x in prompt]
    P = len(ids)
    traces = []
    rnd = 0
    while len(ids) - P < max_new and (max_rounds is None or rnd < max_rounds):
        tr = specdiff_round(model_p, model_q, np.array(ids), gamma, T, tau_p, tau_q, seed, rnd, b, keep)
        room = max_new - (len(ids) - P)
        tr.emitted = tr.emitted[:room]
        ids += tr.emitted
        traces.append(tr)
        rnd += 1
    return np.array(ids, dtype=np.int64), traces


def autoregressive_greedy(model_p: Model, prompt, n_new: int) -> np.ndarray:
    """Plain greedy decoding of the target, one token per forward (the baseline of Table 1)."""
    ids = [int(x) for x in prompt]
    for _ in range(n_new):
        lg = model_p.logits(np.array(ids), [len(ids) - 1])[0]
        ids.append(int(np.argmax(lg)))
    return np.array(ids, dtype=np.int64)


def autoregressive_sample(model_p: Model, prompt, n_new: int, tau_p: float, seed: int, b: int = 0,
                          first_round: int = 0) -> np.ndarray:
    """Standard generation (Section "Preliminaries": x_{i+1} ~ p(. | x_{1:i}), one token per evaluation of M_p),
    written as rounds of Algorithm 1 with an empty draft: nothing is tested and the returned token is the draw
    from p, so it shares the round counter and the random stream of the speculative rounds."""
    ids = [int(x) for x in prompt]
    V = model_p.shape.vocab
    for r in range(n_new):
        lam = model_p.logits(np.array(ids), [len(ids) - 1])
        res = accept_resample(lam, np.zeros((0, V)), np.zeros(0), np.zeros(0, np.int64), tau_p, tau_p, seed,
                              first_round + r, b)
        assert res.n == 0
        ids.append(res.t)
    return np.array(ids, dtype=np.int64)


# ----------------------------------------------------------------------------------
# closed forms the paper states (Appendix "Drafter Convergence Analysis")
# ----------------------------------------------------------------------------------

def expected_tokens_per_draft(alpha: float, gamma: int) -> float:
    """Eq. 2: E(#tokens) = (1 - alpha^(gamma+1)) / (1 - alpha)."""
    return (1.0 - alpha ** (gamma + 1)) / (1.0 - alpha) if alpha < 1.0 else gamma + 1.0


def expected_tokens_per_second(alpha: float, gamma: int, T: int, c1: float, c2: float) -> float:
    """Eq. 3: E(#tokens / second) = E(#tokens) / (T c1 + c2)."""
    return expected_tokens_per_draft(alpha, gamma) / (T * c1 + c2)
