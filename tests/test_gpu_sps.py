"""GPU parity of the speculative-decoding warm start (autoregressive drafter, sdd_sps_attach / sdd_sps_step) against
the oracle's sps_round, and of a generation that starts with such rounds and continues with SpecDiff rounds.

Per round the oracle starts from the library's token state.  The drafter's row of evaluation j must match the
oracle's logits for context + the library's first j drafts within the logit tolerance; every draw, the acceptance
and the commit are then recomputed by the oracle on the library's rows and must be identical (near-ties logged)."""
import numpy as np
import pytest

import synth
from oracle import philox as px
from oracle import specdiff as sd
from oracle.transformer import Model, target_verify_logits
from tests import parity, roundcheck

pytestmark = pytest.mark.gpu


def _models(wl, **wkw):
    import paper_2408_05636_b200 as sdd
    mp, mq, dp, dq = roundcheck.build_pair(wl, **wkw)
    wa = synth.model_weights(wl.ar_drafter, wl.ar_weight_seed, wl.dtype, **wkw)
    return mp, mq, Model(wl.ar_drafter, wa), dp, dq, sdd.DeviceModel(wl.ar_drafter, wa, synth.tensor_names(wl.ar_drafter), wl.dtype)


def check_sps_rounds(sess, mp, ma, wl, gamma_sps, n_rounds, tau_p, tau_q, tol, first_round=0):
    import paper_2408_05636_b200 as sdd
    B, G, V = sess.batch, gamma_sps, sess.V
    log, stats = [], {"max_q_err": 0.0, "max_p_err": 0.0, "emitted": []}
    for r in range(n_rounds):
        rnd = first_round + r
        toks = sess.tap_numpy(sdd.TAP_TOKENS).reshape(B, sess.tok_stride)
        clen = sess.tap_numpy(sdd.TAP_CTX_LEN)
        n_em = sess.tap_numpy(sdd.TAP_N_EMITTED)
        sess.sdd_sps_step(G)
        # the round's buffers are laid out with its own draft length
        qrows = sess.tap_numpy(sdd.TAP_Q_LOGITS)[: B * G * V].reshape(B, G, V)
        slots = sess.tap_numpy(sdd.TAP_DRAFT_IDS)[: B * G].reshape(B, G)
        logq = sess.tap_numpy(sdd.TAP_LOGQ)[: B * G].reshape(B, G)
        lam = sess.tap_numpy(sdd.TAP_LOGITS_P)[: B * (G + 1) * V].reshape(B, G + 1, V)
        prob = sess.tap_numpy(sdd.TAP_ACCEPT_PROB)[: B * G].reshape(B, G)
        n_acc = sess.tap_numpy(sdd.TAP_N_ACCEPT)
        extra = sess.tap_numpy(sdd.TAP_EXTRA_TOKEN)
        toks2 = sess.tap_numpy(sdd.TAP_TOKENS).reshape(B, sess.tok_stride)
        clen2 = sess.tap_numpy(sdd.TAP_CTX_LEN)
        out_ids = sess.sps_ids.cpu().numpy()
        n_out = sess.n_out.cpu().numpy()
        for b in range(B):
            ctx = toks[b, : clen[b]].astype(np.int64)
            for j in range(G):
                ids = np.concatenate([ctx, slots[b, :j].astype(np.int64)])
                ref = ma.logits(ids, [len(ids) - 1])[0] / (tau_q if tau_q > 0 else 1.0)
                err = float(np.abs(qrows[b, j] - ref).max())
                stats["max_q_err"] = max(stats["max_q_err"], err)
                assert err < tol, f"drafter logits round {rnd} evaluation {j} seq {b}: {err}"
                z = qrows[b, j].astype(np.float64)
                if tau_q > 0:
                    x, gap = sd.argmax_with_gap(z + px.vocab_gumbels(wl.philox_seed, px.DRAFT, rnd, 0, j, b, V))
                    want_logq = z[slots[b, j]] - sd.logsumexp(z)
                else:
                    x, gap = sd.argmax_with_gap(z)
                    want_logq = 0.0
                if x != slots[b, j]:
                    assert gap < parity.GAP_BAND, (rnd, b, j, x, slots[b, j], gap)
                    log.append(("draft", "gap", rnd, b, j, int(slots[b, j]), int(x), float(gap)))
                assert abs(logq[b, j] - want_logq) < 1e-5
            ref = target_verify_logits(mp, ctx, slots[b].astype(np.int64))
            err = float(np.abs(lam[b] - ref).max())
            stats["max_p_err"] = max(stats["max_p_err"], err)
            assert err < tol, f"target logits round {rnd} seq {b}: {err}"
            parity.check_accept(lam[b], qrows[b], logq[b], slots[b], tau_p, tau_q, wl.philox_seed, rnd, b, int(n_acc[b]),
                                int(extra[b]), prob[b], log)
            n, t = int(n_acc[b]), int(extra[b])
            emit = max(0, min(n + 1, sess.max_new - int(n_em[b])))
            want = ([int(x) for x in slots[b, :n]] + [t])[:emit]
            assert clen2[b] == clen[b] + emit and n_out[b] == emit
            assert list(toks2[b, clen[b]: clen2[b]]) == want
            assert list(out_ids[b, :emit]) == want and np.all(out_ids[b, emit:] == -1)
            stats["emitted"].append(emit)
    return log, stats


def test_sps_rounds_fp32_then_specdiff_rounds():
    import paper_2408_05636_b200 as sdd
    wl = synth.scaled_workload(synth.WORKLOADS["tiny_fp32"], batch=2, max_new=60)
    mp, mq, ma, dp, dq, da = _models(wl, bias_std=0.02, perturb_ln=True)
    prompts = synth.prompt_ids(wl.target.vocab, wl.batch, wl.prompt_len, wl.prompt_seed)
    plen = [wl.prompt_len, wl.prompt_len - 7]
    sess = sdd.Session(dp, dq, prompts, plen, wl.gamma, wl.T, wl.max_new, 1.0, 1.0, wl.philox_seed)
    sess.sdd_sps_attach(da)
    log, st = check_sps_rounds(sess, mp, ma, wl, 4, 5, 1.0, 1.0, 1e-4)
    assert st["max_q_err"] < 1e-4 and st["max_p_err"] < 1e-4
    assert len(set(st["emitted"])) >= 3                    # short and long acceptances both occurred
    assert 5 in st["emitted"]                              # a fully accepted draft: the next round feeds two new tokens
    # a different draft length in the same session, then the hand-over to SpecDiff rounds
    log2, _ = check_sps_rounds(sess, mp, ma, wl, 3, 2, 1.0, 1.0, 1e-4, first_round=5)
    log3, _ = roundcheck.check_rounds(sess, mp, mq, wl, 2, 1.0, 1.0, 1e-4, first_round=7)
    parity.assert_few(log + log2 + log3)
    # once another kind of round has run the drafter's cache has gaps: the call is refused
    with pytest.raises(sdd.SddError) as e:
        sess.sdd_sps_step(4)
    assert e.value.status == sdd.SDD_E_STATE
    sess.close()


def test_sps_greedy_equals_autoregressive_greedy():
    import paper_2408_05636_b200 as sdd
    wl = synth.scaled_workload(synth.WORKLOADS["tiny_fp32"], max_new=24)
    mp, mq, ma, dp, dq, da = _models(wl)
    prompt = synth.prompt_ids(wl.target.vocab, 1, wl.prompt_len, wl.prompt_seed)
    sess = sdd.Session(dp, dq, prompt, [wl.prompt_len], wl.gamma, wl.T, wl.max_new, 0.0, 0.0, wl.philox_seed)
    sess.sdd_sps_attach(da)
    while sess.tap_numpy(sdd.TAP_N_EMITTED)[0] < 10:       # warm start: the first 10 tokens
        sess.sdd_sps_step(4)
    toks, clen = sess.generate()
    ref = sd.autoregressive_greedy(mp, prompt[0], wl.max_new)
    assert clen[0] == wl.prompt_len + wl.max_new
    assert np.array_equal(toks[0, : clen[0]], ref)
    sess.close()


def test_sps_rounds_bf16():
    import paper_2408_05636_b200 as sdd
    wl = synth.scaled_workload(synth.WORKLOADS["small_bf16"], prompt_len=150, max_new=40)
    mp, mq, ma, dp, dq, da = _models(wl)
    prompt = synth.prompt_ids(wl.target.vocab, 1, wl.prompt_len, wl.prompt_seed)
    sess = sdd.Session(dp, dq, prompt, [wl.prompt_len], wl.gamma, wl.T, wl.max_new, 1.0, 1.0, wl.philox_seed)
    sess.sdd_sps_attach(da)
    log, st = check_sps_rounds(sess, mp, ma, wl, 5, 3, 1.0, 1.0, 2e-2)
    parity.assert_few(log)
    sess.close()


def test_sps_call_order_and_argument_errors():
    import paper_2408_05636_b200 as sdd
    wl = synth.WORKLOADS["tiny_fp32"]
    mp, mq, ma, dp, dq, da = _models(wl)
    prompt = synth.prompt_ids(wl.target.vocab, 1, wl.prompt_len, wl.prompt_seed)
    sess = sdd.Session(dp, dq, prompt, [wl.prompt_len], wl.gamma, wl.T, wl.max_new, 1.0, 1.0, wl.philox_seed)
    with pytest.raises(sdd.SddError) as e:                 # no drafter attached
        sess.sdd_sps_step(2)
    assert e.value.status == sdd.SDD_E_STATE
    sess.sdd_sps_attach(da)
    with pytest.raises(sdd.SddError) as e:                 # longer than the context's draft capacity
        sess.sdd_sps_step(wl.gamma + 1)
    assert e.value.status == sdd.SDD_E_ARG
    with pytest.raises(sdd.SddError) as e:                 # attached twice
        sess.sdd_sps_attach(da)
    assert e.value.status == sdd.SDD_E_STATE
    sess.sdd_sps_step(2)
    sess.sdd_sync_status()
    sess.close()
    # a one-token prompt cannot be warm-started (the first evaluation feeds two positions)
    s2 = sdd.Session(dp, dq, prompt, [1], wl.gamma, wl.T, wl.max_new, 1.0, 1.0, wl.philox_seed)
    with pytest.raises(sdd.SddError) as e:
        s2.sdd_sps_attach(da)
    assert e.value.status == sdd.SDD_E_ARG
    # the diffusion drafter (not causal) is not an autoregressive drafter
    with pytest.raises(sdd.SddError):
        s2.sdd_sps_attach(dq)
    s2.close()
