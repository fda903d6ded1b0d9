"""GPU parity of the stand-alone acceptance entry point (sdd_accept_logits) with the oracle."""
import numpy as np
import pytest
import torch

import synth
from tests import parity

pytestmark = pytest.mark.gpu


def _run_case(case, tau_p, tau_q, seed, rnd):
    import paper_2408_05636_b200 as sdd
    dev = "cuda:0"
    lp = torch.from_numpy(case.logits_p).to(dev)
    lq = torch.from_numpy(case.logits_q).to(dev)
    ids = torch.from_numpy(case.draft_ids).to(dev)
    n, out, prob = sdd.sdd_accept_logits(lp, lq, ids, tau_p, tau_q, seed, rnd)
    torch.cuda.synchronize()
    n, out, prob = n.cpu().numpy(), out.cpu().numpy(), prob.cpu().numpy()
    rows, gamma = case.draft_ids.shape
    log = []
    for r in range(rows):
        qrows = case.logits_q[r].astype(np.float64) / (tau_q if tau_q > 0 else 1.0)
        res = parity.check_accept(case.logits_p[r], qrows, None, case.draft_ids[r], tau_p, tau_q, seed, rnd, r,
                                  int(n[r]), int(out[r, n[r]]), prob[r], log)
        if int(n[r]) == res.n:
            assert list(out[r, : n[r]]) == list(case.draft_ids[r, : n[r]])
            assert np.all(out[r, n[r] + 1:] == -1)
    return log, n


@pytest.mark.parametrize("V,gamma,rows", [(2, 1, 3), (8, 3, 16), (5, 7, 9), (1000, 5, 7), (8191, 4, 3), (8193, 2, 5)])
def test_small_vocab_cases(V, gamma, rows):
    for sigma in (0.3, 1.0):
        case = synth.accept_case(rows, gamma, V, sigma, seed=100 + V)
        log, n = _run_case(case, 1.0, 1.0, seed=99, rnd=3)
        parity.assert_few(log)


def test_temperatures_and_rounds():
    case = synth.accept_case(6, 6, 777, 0.8, seed=5)
    for tau_p, tau_q, rnd in ((0.7, 1.3, 0), (2.0, 0.5, 11), (1.0, 1.0, 4_000_000_000)):
        _run_case(case, tau_p, tau_q, seed=(1 << 40) + 17, rnd=rnd)


def test_greedy_mode():
    case = synth.accept_case(8, 6, 3001, 0.5, seed=6, draw_drafts=False)
    # make half of the drafts equal to the target arg-max so that acceptance actually happens
    top = case.logits_p[:, :-1].argmax(-1).astype(np.int32)
    case.draft_ids[:, :3] = top[:, :3]
    log, n = _run_case(case, 0.0, 0.0, seed=1, rnd=0)
    assert not log and n.min() >= 3


def test_paper_vocab_ragged_tail_and_all_overlap_levels():
    rows, gamma, V = 4, 8, 50257
    total_log = []
    ns = []
    for si, sigma in enumerate(synth.MICRO_SIGMAS):
        case = synth.accept_case(rows, gamma, V, sigma, seed=31 + si)
        log, n = _run_case(case, 1.0, 1.0, seed=31, rnd=si)
        total_log += log
        ns.append(n.mean())
    print("near-ties logged:", total_log)
    parity.assert_few(total_log)
    assert ns[0] > ns[-1]          # more overlap, longer accepted prefixes


def test_argument_errors():
    import paper_2408_05636_b200 as sdd
    case = synth.accept_case(2, 2, 16, 0.5, seed=1)
    lp, lq = torch.from_numpy(case.logits_p).cuda(), torch.from_numpy(case.logits_q).cuda()
    ids = torch.from_numpy(case.draft_ids).cuda()
    with pytest.raises(sdd.SddError) as e:
        sdd.sdd_accept_logits(lp, lq, ids, 1.0, 0.0, 0, 0)      # mixed greedy / stochastic
    assert e.value.status == sdd.SDD_E_ARG
    assert sdd.sdd_accept_scratch_bytes(0, 1, 1) == 0


def test_extreme_shapes():
    """Largest supported draft length (gamma = 256 fills the decision stage's thread block), a single row with a
    single draft, and a vocabulary of two."""
    for rows, gamma, V in ((2, 256, 40), (1, 1, 2), (3, 200, 129)):
        case = synth.accept_case(rows, gamma, V, 0.4, seed=rows + gamma)
        log, n = _run_case(case, 1.0, 1.0, seed=5, rnd=1)
        parity.assert_few(log)
    import paper_2408_05636_b200 as sdd
    case = synth.accept_case(1, 2, 16, 0.5, seed=1)
    lp, lq = torch.from_numpy(case.logits_p).cuda(), torch.from_numpy(case.logits_q).cuda()
    ids = torch.from_numpy(case.draft_ids).cuda()
    L = sdd.lib()
    out = torch.zeros(8, dtype=torch.int32, device="cuda")
    prob = torch.zeros(8, device="cuda")
    scratch = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    # gamma beyond the supported maximum is refused before anything is launched
    assert L.sdd_accept_logits(lp.data_ptr(), lq.data_ptr(), ids.data_ptr(), 1, 257, 16, 1.0, 1.0, 0, 0, out.data_ptr(),
                               out.data_ptr(), prob.data_ptr(), scratch.data_ptr(), None) == sdd.SDD_E_ARG


def test_microbenchmark_shape_64_rows_gamma_32():
    """The acceptance microbenchmark's own case (64 rows x gamma 32 x V 50257 fp32 logits, 0.84 GB; the inputs that
    bench.py times, from the same generator call), every row compared with the oracle."""
    case = synth.accept_case(64, 32, 50257, 0.5, seed=31)
    log, n = _run_case(case, 1.0, 1.0, seed=31, rnd=7)
    print("near-ties logged:", log, "mean accepted:", float(n.mean()))
    parity.assert_few(log, u=1, gap=2, cancellation=2)
    assert n.min() >= 0 and n.max() <= 32


@pytest.mark.parametrize("gamma", [8, 128])
def test_microbenchmark_sweep_ends(gamma):
    """Both ends of the draft-length sweep (gamma 8 and 128) at the paper's vocabulary, built from the gamma-32 case
    by the re-indexing that bench.py uses for its sweep; 8 rows."""
    base = synth.accept_case(8, 32, 50257, 0.3, seed=32)
    case = synth.resize_accept_case(base, gamma)
    assert case.logits_p.shape == (8, gamma + 1, 50257) and case.draft_ids.shape == (8, gamma)
    log, n = _run_case(case, 1.0, 1.0, seed=32, rnd=gamma)
    print("near-ties logged:", log, "mean accepted:", float(n.mean()))
    parity.assert_few(log)


def test_draft_id_outside_the_vocabulary_is_refused_not_used():
    """A draft id that is no valid column is never used as an index: that sequence reports n_accept = -1 and an
    all -1 output row; the other sequences are unaffected."""
    import paper_2408_05636_b200 as sdd
    case = synth.accept_case(3, 4, 300, 0.5, seed=9)
    good_log, good_n = _run_case(case, 1.0, 1.0, seed=3, rnd=2)
    ids = case.draft_ids.copy()
    ids[1, 2] = 300                      # == V: one past the last column
    lp, lq = torch.from_numpy(case.logits_p).cuda(), torch.from_numpy(case.logits_q).cuda()
    n, out, prob = sdd.sdd_accept_logits(lp, lq, torch.from_numpy(ids).cuda(), 1.0, 1.0, 3, 2)
    torch.cuda.synchronize()
    n, out = n.cpu().numpy(), out.cpu().numpy()
    assert n[1] == -1 and np.all(out[1] == -1)
    assert n[0] == good_n[0] and n[2] == good_n[2]
