"""Stage-by-stage parity of whole SpecDiff rounds: the CUDA library against the oracle.

For every checked round the oracle starts from the library's own token state.  Network outputs
(drafter logits of every denoising evaluation, target logits) are compared within a tolerance;
the sampling / acceptance stage of the oracle is then run on the library's logits, where integer
results (reveal pattern, draft ids, accepted length, extra token, committed tokens) must be
identical except for draws flagged as fp32 near-ties, which are logged."""
from __future__ import annotations

import numpy as np

import synth
from oracle import philox as px
from oracle import specdiff as sd
from oracle.transformer import Model, drafter_slot_logits, target_verify_logits
from tests import parity


def build_pair(wl, **wkw):
    """Oracle models and device models of a workload from the same seeded weights."""
    import paper_2408_05636_b200 as sdd
    wp = synth.model_weights(wl.target, wl.weight_seed, wl.dtype, **wkw)
    wq = synth.model_weights(wl.drafter, wl.weight_seed, wl.dtype, **wkw)
    mp, mq = Model(wl.target, wp), Model(wl.drafter, wq)
    dp = sdd.DeviceModel(wl.target, wp, synth.tensor_names(wl.target), wl.dtype)
    dq = sdd.DeviceModel(wl.drafter, wq, synth.tensor_names(wl.drafter), wl.dtype)
    return mp, mq, dp, dq


def check_rounds(sess, mp, mq, wl, n_rounds, tau_p, tau_q, tol, seqs=None, first_round=0, check_networks=True):
    """Runs n_rounds on the session, checking each stage.  Returns (near-tie log, stats dict)."""
    import paper_2408_05636_b200 as sdd
    B, G, T, V = sess.batch, sess.gamma, sess.T, sess.V
    seqs = list(range(B)) if seqs is None else list(seqs)
    log = []
    stats = {"max_q_err": 0.0, "max_p_err": 0.0, "emitted": [], "accepted": 0, "tested": 0, "sum_min": []}
    for r in range(n_rounds):
        rnd = first_round + r
        toks = sess.tap_numpy(sdd.TAP_TOKENS).reshape(B, sess.tok_stride)
        clen = sess.tap_numpy(sdd.TAP_CTX_LEN)
        n_em = sess.tap_numpy(sdd.TAP_N_EMITTED)
        sess.sdd_draft_begin()
        states = {b: sd.DraftState.fresh(G, V) for b in seqs}
        for k in range(T, 0, -1):
            sess.sdd_draft_step()
            step = sess.tap_numpy(sdd.TAP_STEP_LOGITS).reshape(B, G, V)
            slots = sess.tap_numpy(sdd.TAP_DRAFT_IDS).reshape(B, G)
            logq = sess.tap_numpy(sdd.TAP_LOGQ).reshape(B, G)
            reveal = sess.tap_numpy(sdd.TAP_REVEAL_STEP).reshape(B, G)
            qrows = sess.tap_numpy(sdd.TAP_Q_LOGITS).reshape(B, G, V)
            for b in seqs:
                st = states[b]
                if check_networks:
                    ref = drafter_slot_logits(mq, toks[b, : clen[b]], st.slots)
                    err = float(np.abs(step[b] - ref).max())
                    stats["max_q_err"] = max(stats["max_q_err"], err)
                    assert err < tol, f"drafter logits round {rnd} step {k} seq {b}: {err}"
                parity.check_unmask_step(st, step[b], k, tau_q, wl.philox_seed, rnd, b, slots[b], logq[b], reveal[b],
                                         qrows[b], log)
        sess.sdd_verify_accept()
        lam = sess.tap_numpy(sdd.TAP_LOGITS_P).reshape(B, G + 1, V)
        qrows = sess.tap_numpy(sdd.TAP_Q_LOGITS).reshape(B, G, V)
        logq = sess.tap_numpy(sdd.TAP_LOGQ).reshape(B, G)
        n_acc = sess.tap_numpy(sdd.TAP_N_ACCEPT)
        extra = sess.tap_numpy(sdd.TAP_EXTRA_TOKEN)
        prob = sess.tap_numpy(sdd.TAP_ACCEPT_PROB).reshape(B, G)
        toks2 = sess.tap_numpy(sdd.TAP_TOKENS).reshape(B, sess.tok_stride)
        clen2 = sess.tap_numpy(sdd.TAP_CTX_LEN)
        out_ids = sess.out_ids.cpu().numpy()
        n_out = sess.n_out.cpu().numpy()
        for b in seqs:
            st = states[b]
            assert np.all(st.slots != V)
            if check_networks:
                ref = target_verify_logits(mp, toks[b, : clen[b]], st.slots)
                err = float(np.abs(lam[b] - ref).max())
                stats["max_p_err"] = max(stats["max_p_err"], err)
                assert err < tol, f"target logits round {rnd} seq {b}: {err}"
            res = parity.check_accept(lam[b], qrows[b], logq[b], st.slots, tau_p, tau_q, wl.philox_seed, rnd, b,
                                      int(n_acc[b]), int(extra[b]), prob[b], log)
            # commit: exactly the library's own (n, t), truncated to max_new
            n, t = int(n_acc[b]), int(extra[b])
            emit = max(0, min(n + 1, sess.max_new - int(n_em[b])))
            want = ([int(x) for x in st.slots[:n]] + [t])[:emit]
            assert clen2[b] == clen[b] + emit and n_out[b] == emit
            assert list(toks2[b, clen[b]: clen2[b]]) == want
            assert list(out_ids[b, :emit]) == want and np.all(out_ids[b, emit:] == -1)
            assert np.array_equal(toks2[b, : clen[b]], toks[b, : clen[b]])
            stats["emitted"].append(emit)
            tested = res.n + 1 if res.n < G else G
            stats["tested"] += tested
            stats["accepted"] += res.n
            stats["sum_min"] += list(res.sum_min[:tested])
    return log, stats


def check_whole_rounds(sess, mp, mq, wl, n_rounds, tol, seqs, n_sampled_steps=2, first_round=0):
    """Rounds through sdd_step (one graph launch per round: the benchmark's launch configuration), checked on what a
    finished round leaves behind.  The state of the slots at denoising step k follows from the reveal steps (a slot
    revealed at a step > k already had its final id, the others were [MASK]), so the stored q rows of the slots
    revealed at `n_sampled_steps` steps per round are compared with the oracle's drafter evaluation of that state,
    together with their draws and reveal tests; target logits, acceptance, extra token and commit are checked in full
    for the sequences `seqs`.  Returns (near-tie log, worst drafter error, worst target error)."""
    import paper_2408_05636_b200 as sdd
    B, G, T, V = sess.batch, sess.gamma, sess.T, sess.V
    log = []
    worst_q = worst_p = 0.0
    for r in range(n_rounds):
        rnd = first_round + r
        toks = sess.tap_numpy(sdd.TAP_TOKENS).reshape(B, sess.tok_stride)
        clen = sess.tap_numpy(sdd.TAP_CTX_LEN)
        sess.sdd_step()
        slots_all = sess.tap_numpy(sdd.TAP_DRAFT_IDS).reshape(B, G).astype(np.int64)
        reveal_all = sess.tap_numpy(sdd.TAP_REVEAL_STEP).reshape(B, G)
        logq_all = sess.tap_numpy(sdd.TAP_LOGQ).reshape(B, G)
        n_acc_all = sess.tap_numpy(sdd.TAP_N_ACCEPT)
        extra_all = sess.tap_numpy(sdd.TAP_EXTRA_TOKEN)
        prob_all = sess.tap_numpy(sdd.TAP_ACCEPT_PROB).reshape(B, G)
        toks2 = sess.tap_numpy(sdd.TAP_TOKENS).reshape(B, sess.tok_stride)
        clen2 = sess.tap_numpy(sdd.TAP_CTX_LEN)
        out_ids = sess.out_ids.cpu().numpy()
        q_dev = sess.sdd_tap(sdd.TAP_Q_LOGITS).view(B, G, V)
        p_dev = sess.sdd_tap(sdd.TAP_LOGITS_P).view(B, G + 1, V)
        for b in seqs:
            ctx = toks[b, : clen[b]].astype(np.int64)
            slots, reveal, logq = slots_all[b], reveal_all[b], logq_all[b]
            qrows = q_dev[b].cpu().numpy()
            lam = p_dev[b].cpu().numpy()
            assert np.all(slots != V) and np.all((reveal >= 1) & (reveal <= T))
            steps = sorted(set(int(k) for k in reveal), reverse=True)
            picks = [steps[(i * len(steps)) // n_sampled_steps] for i in range(min(n_sampled_steps, len(steps)))]
            for k in picks:
                state = np.where(reveal > k, slots, V)
                ref = drafter_slot_logits(mq, ctx, state)
                for j in np.nonzero(reveal == k)[0]:
                    z = qrows[j].astype(np.float64)
                    worst_q = max(worst_q, float(np.abs(z - ref[j]).max()))
                    x, gap = sd.argmax_with_gap(z + px.vocab_gumbels(wl.philox_seed, px.DRAFT, rnd, 0, int(j), b, V))
                    if x != slots[j]:
                        assert gap < parity.GAP_BAND
                        log.append(("draft", "gap", rnd, b, int(j), int(slots[j]), int(x), float(gap)))
                    assert abs(logq[j] - (z[slots[j]] - sd.logsumexp(z))) < 1e-5
                    # the reveal test of this slot: failed at every step before k, passed at k
                    for kk in range(T, k - 1, -1):
                        u = px.scalar_uniform(wl.philox_seed, px.UNMASK, rnd, kk, int(j), b)
                        assert (u < 1.0 / kk) == (kk == k)
            ref_p = target_verify_logits(mp, ctx, slots)
            worst_p = max(worst_p, float(np.abs(lam - ref_p).max()))
            n_acc, extra = int(n_acc_all[b]), int(extra_all[b])
            parity.check_accept(lam, qrows, logq, slots, 1.0, 1.0, wl.philox_seed, rnd, b, n_acc, extra, prob_all[b], log)
            want = [int(x) for x in slots[:n_acc]] + [extra]
            assert clen2[b] == clen[b] + n_acc + 1 and list(toks2[b, clen[b]: clen2[b]]) == want
            assert list(out_ids[b, : n_acc + 1]) == want
        assert worst_q < tol and worst_p < tol, (worst_q, worst_p)
    return log, worst_q, worst_p
