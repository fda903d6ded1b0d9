"""The bounded device-side waits of the tensor-core kernels, made to run out once: a one-CTA kernel with the GEMM
kernels' role layout whose consumer waits on a barrier that nothing arrives on.  Nothing faults or hangs: the wait
gives up after its limit (about a millisecond here), the status word says so, and the device goes on working."""
import pytest
import torch

pytestmark = pytest.mark.gpu


def test_wait_runs_out_sets_status_and_leaves_the_device_usable():
    import paper_2408_05636_b200 as sdd
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    sdd.sdd_debug_wait_timeout(2_000_000, status)        # about 1 ms of SM clocks
    t1.record()
    torch.cuda.synchronize()
    assert int(status.item()) == 1                       # DEV_TIMEOUT
    assert 0.2 < t0.elapsed_time(t1) < 200.0             # it waited for its limit, and not much longer
    assert b"wait" in sdd.lib().sdd_strerror(sdd.SDD_E_TIMEOUT)
    # the next ordinary tensor-core GEMM on the same device is correct (TMEM was freed, the context is intact)
    g = torch.Generator(device="cuda").manual_seed(1)
    A = torch.randn(256, 512, device="cuda", generator=g).to(torch.bfloat16)
    W = (torch.randn(384, 512, device="cuda", generator=g) * 0.05).to(torch.bfloat16)
    out = torch.zeros(256, 384, device="cuda", dtype=torch.bfloat16)
    st2 = torch.zeros(1, dtype=torch.int32, device="cuda")
    sdd.sdd_debug_gemm_bf16(A, W, None, 256, 0, out, 0, True, st2)
    torch.cuda.synchronize()
    ref = A.float() @ W.float().t()
    assert int(st2.item()) == 0
    assert float((out.float() - ref).abs().max()) < 0.05 * float(ref.abs().max())


def test_argument_errors():
    import paper_2408_05636_b200 as sdd
    L = sdd.lib()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert L.sdd_debug_wait_timeout(0, status.data_ptr(), None) == sdd.SDD_E_ARG
    assert L.sdd_debug_wait_timeout(1000, None, None) == sdd.SDD_E_ARG
