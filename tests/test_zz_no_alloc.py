"""The allocation-free acceptance entry point (sdd_accept_logits_static) against the regular one.

Some users of the library run where device allocation is not available to them: an inference server
that carved up all GPU memory at start-up, a latency-critical loop that may not enter the allocator,
or a host framework that passes in its own tensors.  For them the library keeps the scratch of the
acceptance step in a fixed device array.  This file checks, through the C ABI, that the variant gives
the regular entry point's results on two calls in a row (the second call meets the first call's
left-overs in the shared array), and that it refuses sizes beyond the fixed array.  It is named to be
collected last, so a run that stops at the first failure has already run everything else."""
import numpy as np
import pytest
import torch

import synth

pytestmark = pytest.mark.gpu


def _outputs(rows, gamma, dev):
    return (torch.full((rows,), -7, dtype=torch.int32, device=dev),
            torch.full((rows, gamma + 1), -7, dtype=torch.int32, device=dev),
            torch.full((rows, gamma), -7.0, dtype=torch.float32, device=dev))


def test_static_scratch_variant_matches_regular_entry_point_twice():
    import paper_2408_05636_b200 as sdd
    dev = "cuda:0"
    # two different problems, the second one smaller so that stale entries of the first stay in the array
    for call, (rows, gamma, V, sigma, rnd) in enumerate(((5, 6, 50257, 0.5, 3), (3, 4, 9001, 0.9, 4))):
        case = synth.accept_case(rows, gamma, V, sigma, seed=70 + call)
        lp = torch.from_numpy(case.logits_p).to(dev)
        lq = torch.from_numpy(case.logits_q).to(dev)
        ids = torch.from_numpy(case.draft_ids).to(dev)
        n_ref, out_ref, prob_ref = sdd.sdd_accept_logits(lp, lq, ids, 1.0, 1.0, 123, rnd)
        n, out, prob = _outputs(rows, gamma, dev)
        sdd.sdd_accept_logits_static(lp, lq, ids, n, out, prob, 1.0, 1.0, 123, rnd)
        torch.cuda.synchronize()
        assert torch.equal(n, n_ref) and torch.equal(out, out_ref)             # integer results: identical
        assert float((prob - prob_ref).abs().max()) < 1e-5                      # the tests' probability tolerance
        assert int(n.min()) >= 0 and int(n.max()) <= gamma


def test_static_scratch_variant_greedy_and_allocates_nothing():
    """Temperature 0 (arg-max statistics in the scratch instead of soft-max sums), and the point of the entry point:
    a call leaves the device's free memory and torch's own allocation count where they were."""
    import paper_2408_05636_b200 as sdd
    dev = "cuda:0"
    rows, gamma, V = 4, 5, 3001
    case = synth.accept_case(rows, gamma, V, 0.5, seed=72, draw_drafts=False)
    top = case.logits_p[:, :-1].argmax(-1).astype(np.int32)
    case.draft_ids[:, :2] = top[:, :2]                    # two accepted tokens per row
    lp = torch.from_numpy(case.logits_p).to(dev)
    lq = torch.from_numpy(case.logits_q).to(dev)
    ids = torch.from_numpy(case.draft_ids).to(dev)
    n_ref, out_ref, prob_ref = sdd.sdd_accept_logits(lp, lq, ids, 0.0, 0.0, 5, 1)
    n, out, prob = _outputs(rows, gamma, dev)
    sdd.sdd_accept_logits_static(lp, lq, ids, n, out, prob, 0.0, 0.0, 5, 1)     # first call: address look-up done
    torch.cuda.synchronize()
    free0, alloc0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
    sdd.sdd_accept_logits_static(lp, lq, ids, n, out, prob, 0.0, 0.0, 5, 1)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == alloc0
    assert torch.equal(n, n_ref) and torch.equal(out, out_ref) and torch.equal(prob, prob_ref)
    assert int(n.min()) >= 2
    with pytest.raises(AssertionError):                   # the binding refuses tensors of another element type
        sdd.sdd_accept_logits_static(lp.to(torch.bfloat16), lq, ids, n, out, prob, 0.0, 0.0, 5, 1)


def test_static_scratch_variant_rejects_oversize_problem():
    import paper_2408_05636_b200 as sdd
    dev = "cuda:0"
    rows, gamma, V = 4000, 8, 50257                     # 4000 * 17 * 7 * 8 bytes = 3.8 MB > 2 MiB of fixed scratch
    assert rows * (2 * gamma + 1) * 7 * 8 > sdd.ACCEPT_STATIC_SCRATCH_BYTES
    lp = torch.zeros(1, device=dev).expand(rows, gamma + 1, V)      # never read: the call must fail before any launch
    lq = torch.zeros(1, device=dev).expand(rows, gamma, V)
    ids = torch.zeros(rows, gamma, dtype=torch.int32, device=dev)
    n, out, prob = _outputs(rows, gamma, dev)
    L = sdd.lib()
    st = torch.cuda.current_stream().cuda_stream
    status = L.sdd_accept_logits_static(lp.data_ptr(), lq.data_ptr(), ids.data_ptr(), rows, gamma, V, 1.0, 1.0, 0, 0,
                                        n.data_ptr(), out.data_ptr(), prob.data_ptr(), st)
    assert status == sdd.SDD_E_WORKSPACE
    assert b"workspace" in L.sdd_strerror(status)
    torch.cuda.synchronize()
    assert int(n[0]) == -7                                            # nothing ran
