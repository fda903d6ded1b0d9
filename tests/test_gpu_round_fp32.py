"""GPU parity of whole rounds on the tiny fp32 configuration (fp32 tolerance 1e-4 on logits)."""
import numpy as np
import pytest

import synth
from oracle import specdiff as sd
from tests import parity, roundcheck

pytestmark = pytest.mark.gpu
TOL = 1e-4


def _session(wl, dp, dq, prompts, plen, max_new, tau=1.0, gamma=None, T=None):
    import paper_2408_05636_b200 as sdd
    return sdd.Session(dp, dq, prompts, plen, gamma or wl.gamma, T or wl.T, max_new, tau, tau, wl.philox_seed)


def test_stage_parity_four_rounds():
    wl = synth.WORKLOADS["tiny_fp32"]
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 1, wl.prompt_len, wl.prompt_seed)
    s = _session(wl, dp, dq, prompts, [wl.prompt_len], wl.max_new)
    log, stats = roundcheck.check_rounds(s, mp, mq, wl, 4, 1.0, 1.0, TOL)
    print("near-ties:", log, "max logit err q/p:", stats["max_q_err"], stats["max_p_err"])
    parity.assert_few(log)
    s.close()


def test_end_to_end_four_rounds_no_teacher_forcing():
    import paper_2408_05636_b200 as sdd
    wl = synth.WORKLOADS["tiny_fp32"]
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 1, wl.prompt_len, wl.prompt_seed)
    s = _session(wl, dp, dq, prompts, [wl.prompt_len], wl.max_new)
    for _ in range(4):
        s.sdd_step()
    s.sdd_sync_status()
    toks = s.tap_numpy(sdd.TAP_TOKENS).reshape(1, -1)[0]
    c = int(s.tap_numpy(sdd.TAP_CTX_LEN)[0])
    ids, traces = sd.generate(mp, mq, prompts[0], wl.gamma, wl.T, wl.max_new, 1.0, 1.0, wl.philox_seed, max_rounds=4)
    assert c == len(ids)
    assert np.array_equal(toks[:c], ids)
    rounds, launches = s.sdd_counters()
    assert rounds == 4 and launches > 0
    s.close()


def test_ragged_batch_with_truncation_and_perturbed_weights():
    """Three sequences of different prompt lengths; biases and LayerNorm parameters non-trivial so that a
    dropped bias or gain shows; max_new small so that sequences finish in different rounds."""
    wl = synth.scaled_workload(synth.WORKLOADS["tiny_fp32"], batch=3)
    mp, mq, dp, dq = roundcheck.build_pair(wl, bias_std=0.05, perturb_ln=True)
    prompts = synth.prompt_ids(wl.target.vocab, 3, 40, wl.prompt_seed)
    plen = [40, 7, 1]
    s = _session(wl, dp, dq, prompts, plen, max_new=9, gamma=5, T=3)
    log, stats = roundcheck.check_rounds(s, mp, mq, wl, 5, 1.0, 1.0, TOL)
    parity.assert_few(log)
    assert list(s.tap_numpy(__import__("paper_2408_05636_b200").TAP_N_EMITTED)) == [9, 9, 9]
    assert stats["emitted"][-3:] != [6, 6, 6]
    s.close()


def test_slot_row_pruning_of_the_last_drafter_block(monkeypatch):
    """Forced on (it is chosen by size otherwise): after the drafter's last attention only the slot rows go through
    the rest of the block.  Same stage-by-stage parity as the full forward, ragged batch, non-trivial biases."""
    monkeypatch.setenv("SDD_SLOT_PRUNE", "1")
    wl = synth.scaled_workload(synth.WORKLOADS["tiny_fp32"], batch=3)
    mp, mq, dp, dq = roundcheck.build_pair(wl, bias_std=0.05, perturb_ln=True)
    prompts = synth.prompt_ids(wl.target.vocab, 3, 40, wl.prompt_seed)
    s = _session(wl, dp, dq, prompts, [40, 7, 1], max_new=9, gamma=5, T=3)
    log, stats = roundcheck.check_rounds(s, mp, mq, wl, 3, 1.0, 1.0, TOL)
    parity.assert_few(log)
    assert stats["max_q_err"] < TOL
    s.close()


def test_reset_equals_fresh_context():
    """sdd_reset starts a new generation in the same context (graphs and workspace kept): the tokens must be those of
    a fresh context on the same prompts, also after a generation that left longer sequences in the caches."""
    import paper_2408_05636_b200 as sdd
    wl = synth.scaled_workload(synth.WORKLOADS["tiny_fp32"], batch=2)
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    p1 = synth.prompt_ids(wl.target.vocab, 2, 40, wl.prompt_seed)
    p2 = synth.prompt_ids(wl.target.vocab, 2, 40, wl.prompt_seed + 1)
    s = _session(wl, dp, dq, p1, [40, 33], max_new=20, gamma=5, T=3)
    s.generate()
    with pytest.raises(sdd.SddError):                      # not in the middle of a round
        s.sdd_draft_begin()
        s.sdd_reset(p2, [12, 25])
    for _ in range(3):
        s.sdd_draft_step()
    s.sdd_verify_accept()
    s.sdd_reset(p2, [12, 25])
    toks_a, len_a = s.generate()
    rounds_a, _ = s.sdd_counters()
    s.close()
    f = _session(wl, dp, dq, p2, [12, 25], max_new=20, gamma=5, T=3)
    toks_b, len_b = f.generate()
    rounds_b, _ = f.sdd_counters()
    f.close()
    assert np.array_equal(len_a, len_b) and rounds_a == rounds_b
    for b in range(2):
        assert np.array_equal(toks_a[b, : len_a[b]], toks_b[b, : len_b[b]])


def test_greedy_equals_autoregressive_greedy():
    import paper_2408_05636_b200 as sdd
    wl = synth.WORKLOADS["tiny_fp32"]
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 1, wl.prompt_len, wl.prompt_seed)
    n_new = 20
    s = _session(wl, dp, dq, prompts, [wl.prompt_len], n_new, tau=0.0)
    toks, clen = s.generate()
    assert clen[0] == wl.prompt_len + n_new
    ref = sd.autoregressive_greedy(mp, prompts[0], n_new)
    assert np.array_equal(toks[0, : clen[0]], ref)
    s.close()


def test_temperature_and_T1():
    wl = synth.scaled_workload(synth.WORKLOADS["tiny_fp32"], T=1)
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 1, 12, wl.prompt_seed)
    import paper_2408_05636_b200 as sdd
    s = sdd.Session(dp, dq, prompts, [12], 6, 1, 30, 0.8, 1.5, wl.philox_seed)
    log, stats = roundcheck.check_rounds(s, mp, mq, wl, 3, 0.8, 1.5, TOL)
    parity.assert_few(log)
    s.close()


def test_call_order_and_argument_errors():
    import paper_2408_05636_b200 as sdd
    wl = synth.WORKLOADS["tiny_fp32"]
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 1, wl.prompt_len, wl.prompt_seed)
    s = _session(wl, dp, dq, prompts, [wl.prompt_len], wl.max_new)
    with pytest.raises(sdd.SddError) as e:
        s.sdd_verify_accept()                      # no draft yet
    assert e.value.status == sdd.SDD_E_STATE
    s.sdd_draft()
    with pytest.raises(sdd.SddError) as e:
        s.sdd_draft_step()                         # more than T steps
    assert e.value.status == sdd.SDD_E_STATE
    s.sdd_verify_accept()
    s.sdd_sync_status()
    s.close()
    with pytest.raises(sdd.SddError) as e:         # prompt + max_new + gamma beyond the position table
        _session(wl, dp, dq, prompts, [wl.prompt_len], 200)
    assert e.value.status == sdd.SDD_E_CTX_FULL
    with pytest.raises(sdd.SddError) as e:         # swapped models
        sdd.Session(dq, dp, prompts, [wl.prompt_len], 8, 4, 10)
    assert e.value.status == sdd.SDD_E_ARG


def test_cache_skip_changes_nothing(monkeypatch):
    """A denoising step that reveals nothing leaves the drafter's input unchanged, so the next evaluation is skipped
    and its logits are reused ("ddpm cache").  Tokens must be identical with the skip switched off."""
    import paper_2408_05636_b200 as sdd
    wl = synth.WORKLOADS["tiny_fp32"]
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 2, wl.prompt_len, wl.prompt_seed)
    outs = []
    for flag in ("1", "0"):
        monkeypatch.setenv("SDD_CACHE_SKIP", flag)
        # T much larger than gamma: most steps reveal nothing
        s = sdd.Session(dp, dq, prompts, [wl.prompt_len, 20], 4, 12, 24, 1.0, 1.0, wl.philox_seed)
        toks, clen = s.generate()
        outs.append((toks.copy(), clen.copy()))
        s.close()
    assert np.array_equal(outs[0][1], outs[1][1]) and np.array_equal(outs[0][0], outs[1][0])
    assert outs[0][1].min() > wl.prompt_len - 13


def test_autoregressive_steps_match_oracle_and_mix_with_rounds():
    """sdd_ar_step = a round with an empty draft: tokens must equal the oracle's, also when interleaved with
    speculative rounds (shared round counter and KV cache)."""
    import paper_2408_05636_b200 as sdd
    wl = synth.WORKLOADS["tiny_fp32"]
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 2, wl.prompt_len, wl.prompt_seed)
    plen = [wl.prompt_len, 9]
    s = sdd.Session(dp, dq, prompts, plen, wl.gamma, wl.T, 60, 1.0, 1.0, wl.philox_seed)
    for _ in range(5):
        s.sdd_ar_step()
    s.sdd_sync_status()
    toks = s.tap_numpy(sdd.TAP_TOKENS).reshape(2, -1)
    clen = s.tap_numpy(sdd.TAP_CTX_LEN)
    for b in range(2):
        ref = sd.autoregressive_sample(mp, prompts[b, : plen[b]], 5, 1.0, wl.philox_seed, b=b)
        assert clen[b] == plen[b] + 5 and np.array_equal(toks[b, : clen[b]], ref)
    assert list(s.ar_ids.cpu().numpy()) == [int(toks[b, clen[b] - 1]) for b in range(2)]
    # speculative rounds continue from there (rounds 5, 6), then one more plain token (round 7)
    log, stats = roundcheck.check_rounds(s, mp, mq, wl, 2, 1.0, 1.0, TOL, first_round=5)
    parity.assert_few(log)
    before = s.tap_numpy(sdd.TAP_CTX_LEN).copy()
    toks_before = s.tap_numpy(sdd.TAP_TOKENS).reshape(2, -1).copy()
    s.sdd_ar_step()
    s.sdd_sync_status()
    toks = s.tap_numpy(sdd.TAP_TOKENS).reshape(2, -1)
    for b in range(2):
        ref = sd.autoregressive_sample(mp, toks_before[b, : before[b]], 1, 1.0, wl.philox_seed, b=b, first_round=7)
        assert toks[b, before[b]] == ref[-1]
    s.close()


def test_prompt_id_outside_the_vocabulary_is_reported_not_used():
    """The host cannot see the prompt ids (they are device memory), so the embedding kernels check them: an id that is
    no row of the table becomes a zero embedding, the round completes, and sdd_sync_status reports SDD_E_INDEX."""
    import paper_2408_05636_b200 as sdd
    wl = synth.WORKLOADS["tiny_fp32"]
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 1, 12, wl.prompt_seed)
    prompts[0, 5] = wl.target.vocab + 7
    s = sdd.Session.__new__(sdd.Session)
    with pytest.raises(sdd.SddError) as e:
        s.__init__(dp, dq, prompts, [12], 4, 2, 8, 1.0, 1.0, wl.philox_seed)
        s.sdd_step()
        s.sdd_sync_status()
    assert e.value.status == sdd.SDD_E_INDEX
    s.close()
