"""GPU parity of whole rounds on the bf16 configurations (bf16 tolerance 2e-2 on logits).
The oracle uses the same bf16-rounded weights in fp64 arithmetic."""
import numpy as np
import pytest

import synth
from tests import parity, roundcheck

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
    parity.assert_few(log)
    s.close()


def test_small_bf16_whole_rounds_as_the_benchmark_runs_them():
    """The headline configuration through sdd_step, i.e. in the launch configuration the benchmark times (one CUDA
    graph per round, programmatic dependent launches, skipped evaluations, key-split attention): three rounds, checked
    on what a finished round leaves behind (roundcheck.check_whole_rounds)."""
    import paper_2408_05636_b200 as sdd
    wl = synth.WORKLOADS["small_bf16"]
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 1, wl.prompt_len, wl.prompt_seed)
    s = sdd.Session(dp, dq, prompts, [wl.prompt_len], wl.gamma, wl.T, wl.max_new, 1.0, 1.0, wl.philox_seed)
    log, worst_q, worst_p = roundcheck.check_whole_rounds(s, mp, mq, wl, 3, TOL, seqs=[0])
    print("near-ties:", log, "max logit err q/p:", worst_q, worst_p)
    parity.assert_few(log)
    s.close()


def test_xl_bf16_b16_one_round_sampled_sequence():
    """The serving configuration at full size (48-layer d1600 target, 24-layer d1024 drafter, 16 sequences with
    1024-token prompts, gamma 16, T 8), one round through sdd_step as the benchmark runs it: CTA-pair GEMMs,
    persistent GEMMs, slot-row pruning.  One sequence of the sixteen is followed by the oracle: one sampled drafter
    state, the target logits, the acceptance and the commit."""
    import paper_2408_05636_b200 as sdd
    wl = synth.WORKLOADS["xl_bf16_b16"]
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, wl.batch, wl.prompt_len, wl.prompt_seed)
    s = sdd.Session(dp, dq, prompts, [wl.prompt_len] * wl.batch, wl.gamma, wl.T, wl.max_new, 1.0, 1.0, wl.philox_seed)
    log, worst_q, worst_p = roundcheck.check_whole_rounds(s, mp, mq, wl, 1, TOL, seqs=[9], n_sampled_steps=1)
    print("near-ties:", log, "max logit err q/p:", worst_q, worst_p)
    parity.assert_few(log)
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
    parity.assert_few(log)
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
    parity.assert_few(log)
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
    parity.assert_few(log)
    s.close()


@pytest.mark.parametrize("gamma,T", [(64, 32), (32, 16)])
def test_small_bf16_sweep_corner_whole_rounds(gamma, T):
    """The serving sweep's largest draft length and step count (gamma 64, T 32) and its middle point, on the
    GPT-2-small-shaped pair with two sequences of different lengths: two rounds through sdd_step.  65 (33) target rows
    per sequence, 64 (32) slot rows per LM head, many evaluations that reveal nothing (skipped), reveal steps spread
    over 1..T.  Both sequences are followed by the oracle on two sampled denoising states per round."""
    import paper_2408_05636_b200 as sdd
    wl = synth.scaled_workload(synth.WORKLOADS["small_bf16"], batch=2, gamma=gamma, T=T)
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 2, 300, wl.prompt_seed)
    s = sdd.Session(dp, dq, prompts, [300, 171], gamma, T, 4 * (gamma + 1), 1.0, 1.0, wl.philox_seed)
    log, worst_q, worst_p = roundcheck.check_whole_rounds(s, mp, mq, wl, 2, TOL, seqs=[0, 1])
    print("near-ties:", log, "max logit err q/p:", worst_q, worst_p)
    parity.assert_few(log)
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
    parity.assert_few(log)
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


def test_xl_bf16_whole_round_at_its_own_T():
    """The GPT-2-XL-shaped configuration exactly as the benchmark runs it (prompt 512, gamma 32, T = 16, batch 1,
    rounds through sdd_step: graph replay, dependent launches, skipped evaluations): one round, checked on what it
    leaves behind.  The oracle evaluates the drafter at one sampled denoising state and the target once."""
    import paper_2408_05636_b200 as sdd
    wl = synth.WORKLOADS["xl_bf16"]
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 1, wl.prompt_len, wl.prompt_seed)
    s = sdd.Session(dp, dq, prompts, [wl.prompt_len], wl.gamma, wl.T, wl.max_new, 1.0, 1.0, wl.philox_seed)
    log, worst_q, worst_p = roundcheck.check_whole_rounds(s, mp, mq, wl, 1, TOL, seqs=[0], n_sampled_steps=1)
    ev = s.tap_numpy(sdd.TAP_EVALS)
    print("near-ties:", log, "max logit err q/p:", worst_q, worst_p, "evaluations run / skipped:", ev)
    assert int(ev[0]) + int(ev[1]) == wl.T and int(ev[0]) >= 1
    parity.assert_few(log)
    s.close()


def test_xl_bf16_whole_round_late_in_generation():
    """The same configuration where a generation of the benchmark ends: 1000 tokens of context, so the drafter runs on
    1152 padded rows (nine query tiles x 16 heads of pipelined attention with nine key tiles each, GEMM grids of more
    than one wave) and the target attends over eight cached key tiles.  One round through sdd_step."""
    import paper_2408_05636_b200 as sdd
    wl = synth.scaled_workload(synth.WORKLOADS["xl_bf16"], prompt_len=1000, max_new=64)
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 1, wl.prompt_len, wl.prompt_seed)
    s = sdd.Session(dp, dq, prompts, [wl.prompt_len], wl.gamma, wl.T, wl.max_new, 1.0, 1.0, wl.philox_seed)
    log, worst_q, worst_p = roundcheck.check_whole_rounds(s, mp, mq, wl, 1, TOL, seqs=[0], n_sampled_steps=1)
    print("near-ties:", log, "max logit err q/p:", worst_q, worst_p)
    parity.assert_few(log)
    s.close()


def test_xl_bf16_b16_sweep_corner_gamma64_T32():
    """The serving sweep's largest corner at full size: 16 sequences of 1024 tokens on the XL pair, gamma 64, T 32
    (pair GEMMs, slot-row pruning and 65 target rows per sequence in one round), through sdd_step.  One sequence of
    the sixteen is followed by the oracle: one sampled drafter state, target logits, acceptance, commit."""
    import paper_2408_05636_b200 as sdd
    wl = synth.scaled_workload(synth.WORKLOADS["xl_bf16_b16"], gamma=64, T=32)
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, wl.batch, wl.prompt_len, wl.prompt_seed)
    s = sdd.Session(dp, dq, prompts, [wl.prompt_len] * wl.batch, wl.gamma, wl.T, wl.max_new, 1.0, 1.0, wl.philox_seed)
    log, worst_q, worst_p = roundcheck.check_whole_rounds(s, mp, mq, wl, 1, TOL, seqs=[5], n_sampled_steps=1)
    print("near-ties:", log, "max logit err q/p:", worst_q, worst_p)
    parity.assert_few(log)
    s.close()


def test_tiny_bf16_rounds_every_stage():
    """The smallest tensor-core pair (2 layers, d 128, two heads of 64; the smoke check's second leg): four rounds,
    every stage against the oracle."""
    import paper_2408_05636_b200 as sdd
    wl = synth.WORKLOADS["tiny_bf16"]
    mp, mq, dp, dq = roundcheck.build_pair(wl, bias_std=0.05, perturb_ln=True)
    prompts = synth.prompt_ids(wl.target.vocab, 1, wl.prompt_len, wl.prompt_seed)
    s = sdd.Session(dp, dq, prompts, [wl.prompt_len], wl.gamma, wl.T, wl.max_new, 1.0, 1.0, wl.philox_seed)
    log, stats = roundcheck.check_rounds(s, mp, mq, wl, 4, 1.0, 1.0, TOL)
    print("near-ties:", log, "max logit err q/p:", stats["max_q_err"], stats["max_p_err"])
    parity.assert_few(log)
    s.close()


def test_small_bf16_batch8_greedy_round():
    """Temperature 0 with 136 target rows: the LM head then runs in the token-major orientation on the persistent kernel,
    whose epilogue hands the acceptance step each row's arg-max (statistics fused into the LM head).  One round, T = 2,
    two of the eight sequences followed by the oracle."""
    import paper_2408_05636_b200 as sdd
    wl = synth.scaled_workload(synth.WORKLOADS["small_bf16"], batch=8, T=2)
    mp, mq, dp, dq = roundcheck.build_pair(wl)
    prompts = synth.prompt_ids(wl.target.vocab, 8, 150, wl.prompt_seed)
    plen = [150, 64, 131, 77, 150, 99, 140, 128]
    s = sdd.Session(dp, dq, prompts, plen, wl.gamma, 2, 40, 0.0, 0.0, wl.philox_seed)
    log, stats = roundcheck.check_rounds(s, mp, mq, wl, 1, 0.0, 0.0, TOL, seqs=[0, 7])
    assert not log
    s.close()
