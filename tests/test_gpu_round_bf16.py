"""GPU parity of whole rounds on the bf16 configurations (bf16 tolerance 2e-2 on logits).
The oracle uses the same bf16-rounded weights in fp64 arithmetic."""
import numpy as np
import pytest

import synth
from tests import roundcheck

pytestmark = pytest.mark.gpu
TOL = 2e-2


def test_small_bf16_two_rounds():
    import paper_2408_05636_b200 as sdd
    wl = synth.WORKLOADS["small_bf16"]
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 1, wl.prompt_len, wl.prompt_seed)
    s = sdd.Session(dp, dq, prompts, [wl.prompt_len], wl.gamma, wl.T, wl.max_new, 1.0, 1.0, wl.philox_seed)
    log, stats = roundcheck.check_rounds(s, mp, mq, wl, 2, 1.0, 1.0, TOL)
    print("near-ties:", log, "max logit err q/p:", stats["max_q_err"], stats["max_p_err"],
          "alpha:", stats["accepted"] / max(1, stats["tested"]), "mean sum-min:", float(np.mean(stats["sum_min"])))
    assert len(log) <= 2
    s.close()


def test_small_bf16_whole_rounds_as_the_benchmark_runs_them():
    """The headline configuration through sdd_step, i.e. in the launch configuration the benchmark times (one CUDA
    graph per round, programmatic dependent launches, skipped evaluations, key-split attention): three rounds, checked
    on what a finished round leaves behind.  The state of the slots at denoising step k follows from the reveal steps
    (a slot revealed at a step > k already had its final id, the others were [MASK]), so the stored q rows of the
    slots revealed at two sampled steps per round are compared with the oracle's drafter evaluation of that state;
    the target logits, the acceptance, the extra token and the commit are checked in full."""
    import paper_2408_05636_b200 as sdd
    from oracle import philox as px
    from oracle import specdiff as sd
    from oracle.transformer import drafter_slot_logits, target_verify_logits
    from tests import parity
    wl = synth.WORKLOADS["small_bf16"]
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 1, wl.prompt_len, wl.prompt_seed)
    s = sdd.Session(dp, dq, prompts, [wl.prompt_len], wl.gamma, wl.T, wl.max_new, 1.0, 1.0, wl.philox_seed)
    G, V = wl.gamma, wl.target.vocab
    log = []
    worst_q = worst_p = 0.0
    for rnd in range(3):
        toks = s.tap_numpy(sdd.TAP_TOKENS).reshape(1, s.tok_stride)[0]
        c = int(s.tap_numpy(sdd.TAP_CTX_LEN)[0])
        ctx = toks[:c].astype(np.int64)
        s.sdd_step()
        slots = s.tap_numpy(sdd.TAP_DRAFT_IDS).reshape(1, G)[0].astype(np.int64)
        reveal = s.tap_numpy(sdd.TAP_REVEAL_STEP).reshape(1, G)[0]
        qrows = s.tap_numpy(sdd.TAP_Q_LOGITS).reshape(1, G, V)[0]
        logq = s.tap_numpy(sdd.TAP_LOGQ).reshape(1, G)[0]
        lam = s.tap_numpy(sdd.TAP_LOGITS_P).reshape(1, G + 1, V)[0]
        n_acc = int(s.tap_numpy(sdd.TAP_N_ACCEPT)[0])
        extra = int(s.tap_numpy(sdd.TAP_EXTRA_TOKEN)[0])
        prob = s.tap_numpy(sdd.TAP_ACCEPT_PROB).reshape(1, G)[0]
        assert np.all(slots != V) and np.all((reveal >= 1) & (reveal <= wl.T))
        steps = sorted(set(int(k) for k in reveal), reverse=True)
        for k in (steps[0], steps[len(steps) // 2]):             # the first revealing step and a later one
            state = np.where(reveal > k, slots, V)
            ref = drafter_slot_logits(mq, ctx, state)
            for j in np.nonzero(reveal == k)[0]:
                z = qrows[j].astype(np.float64)
                worst_q = max(worst_q, float(np.abs(z - ref[j]).max()))
                x, gap = sd.argmax_with_gap(z + px.vocab_gumbels(wl.philox_seed, px.DRAFT, rnd, 0, int(j), 0, V))
                if x != slots[j]:
                    assert gap < parity.GAP_BAND
                    log.append(("draft-near-tie", rnd, int(j), int(slots[j]), int(x), float(gap)))
                assert abs(logq[j] - (z[slots[j]] - sd.logsumexp(z))) < 1e-5
                # the reveal test of this slot: passed at step k, failed at every earlier step k' > k
                for kk in range(wl.T, k - 1, -1):
                    u = px.scalar_uniform(wl.philox_seed, px.UNMASK, rnd, kk, int(j), 0)
                    assert (u < 1.0 / kk) == (kk == k)
        ref_p = target_verify_logits(mp, ctx, slots)
        worst_p = max(worst_p, float(np.abs(lam - ref_p).max()))
        parity.check_accept(lam, qrows, logq, slots, 1.0, 1.0, wl.philox_seed, rnd, 0, n_acc, extra, prob, log)
        toks2 = s.tap_numpy(sdd.TAP_TOKENS).reshape(1, s.tok_stride)[0]
        c2 = int(s.tap_numpy(sdd.TAP_CTX_LEN)[0])
        want = [int(x) for x in slots[:n_acc]] + [extra]
        assert c2 == c + n_acc + 1 and list(toks2[c:c2]) == want
        assert list(s.out_ids.cpu().numpy()[0, : n_acc + 1]) == want
    print("near-ties:", log, "max logit err q/p:", worst_q, worst_p)
    assert worst_q < TOL and worst_p < TOL and len(log) <= 2
    s.close()


def test_small_bf16_ragged_batch():
    """Three sequences of different lengths on the GPT-2-small-shaped pair (the batch layout of the serving
    configuration at a size the oracle can follow); two rounds, T = 3."""
    import paper_2408_05636_b200 as sdd
    wl = synth.scaled_workload(synth.WORKLOADS["small_bf16"], batch=3, T=3)
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 3, 200, wl.prompt_seed)
    plen = [200, 90, 131]
    s = sdd.Session(dp, dq, prompts, plen, wl.gamma, 3, 40, 1.0, 1.0, wl.philox_seed)
    log, stats = roundcheck.check_rounds(s, mp, mq, wl, 2, 1.0, 1.0, TOL)
    print("near-ties:", log, "max logit err q/p:", stats["max_q_err"], stats["max_p_err"])
    assert len(log) <= 2
    s.close()


def test_small_bf16_ragged_batch_slot_row_pruning(monkeypatch):
    """The same batch with the drafter's last block restricted to the slot rows (what large forwards do)."""
    import paper_2408_05636_b200 as sdd
    monkeypatch.setenv("SDD_SLOT_PRUNE", "1")
    wl = synth.scaled_workload(synth.WORKLOADS["small_bf16"], batch=3, T=3)
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 3, 200, wl.prompt_seed)
    s = sdd.Session(dp, dq, prompts, [200, 90, 131], wl.gamma, 3, 40, 1.0, 1.0, wl.philox_seed)
    log, stats = roundcheck.check_rounds(s, mp, mq, wl, 1, 1.0, 1.0, TOL)
    print("near-ties:", log, "max logit err q/p:", stats["max_q_err"], stats["max_p_err"])
    assert len(log) <= 2
    s.close()


@pytest.mark.parametrize("pairs", ["1", "2"])
def test_small_bf16_batch12_sampled_sequences(pairs, monkeypatch):
    """Twelve sequences: the drafter forward has 4608 rows, which is where the large-forward code paths start (the
    persistent GEMM with its fused-QKV tiles, V^T tiles stored by TMA, vector LayerNorm, slot-row pruning chosen by
    size).  One round with T = 2; three of the twelve sequences are followed by the oracle.  pairs = 2: the GEMMs that
    are eligible run on CTA pairs although the forward is smaller than the size rule asks (fused-QKV, GELU and
    residual epilogues of the pair kernel inside a round)."""
    import paper_2408_05636_b200 as sdd
    monkeypatch.setenv("SDD_GEMM_PAIR", pairs)
    wl = synth.scaled_workload(synth.WORKLOADS["small_bf16"], batch=12, T=2)
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 12, 260, wl.prompt_seed)
    plen = [260, 131, 250, 199, 260, 77, 240, 258, 129, 260, 200, 255]
    s = sdd.Session(dp, dq, prompts, plen, wl.gamma, 2, 40, 1.0, 1.0, wl.philox_seed)
    log, stats = roundcheck.check_rounds(s, mp, mq, wl, 1, 1.0, 1.0, TOL, seqs=[0, 5, 11])
    print("near-ties:", log, "max logit err q/p:", stats["max_q_err"], stats["max_p_err"])
    assert len(log) <= 2
    s.close()


def test_xl_bf16_one_round_reduced_T():
    """GPT-2-XL-shaped target (48L d1600 h25) with the 24L d1024 drafter, prompt 512, gamma 32; one round with
    T = 2 denoising evaluations (the oracle needs about 3 TFLOP in fp64 for this round)."""
    import paper_2408_05636_b200 as sdd
    wl = synth.scaled_workload(synth.WORKLOADS["xl_bf16"], T=2)
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 1, wl.prompt_len, wl.prompt_seed)
    s = sdd.Session(dp, dq, prompts, [wl.prompt_len], wl.gamma, 2, wl.max_new, 1.0, 1.0, wl.philox_seed)
    log, stats = roundcheck.check_rounds(s, mp, mq, wl, 1, 1.0, 1.0, TOL)
    print("near-ties:", log, "max logit err q/p:", stats["max_q_err"], stats["max_p_err"])
    assert len(log) <= 2
    s.close()


def test_small_bf16_greedy_round():
    """Temperature 0 (the setting of every result the paper reports): draft = arg-max, accept iff it equals the
    target's arg-max, extra token = target arg-max; checked stage by stage on the library's own logits."""
    import paper_2408_05636_b200 as sdd
    wl = synth.scaled_workload(synth.WORKLOADS["small_bf16"], T=2)
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 1, 64, wl.prompt_seed)
    s = sdd.Session(dp, dq, prompts, [64], wl.gamma, 2, 40, 0.0, 0.0, wl.philox_seed)
    log, stats = roundcheck.check_rounds(s, mp, mq, wl, 2, 0.0, 0.0, TOL)
    assert not log
    s.close()
