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
