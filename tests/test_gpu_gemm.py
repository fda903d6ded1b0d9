"""The bf16 tensor-core GEMM (tcgen05 / TMEM / TMA) against a plain fp32 matmul of the same bf16 inputs:
all tile widths, both orientations (normal and swapped for few rows), ragged M / N, every epilogue."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _ref(A, W, bias, M, epi, out0):
    acc = A[:M].float() @ W.float().t()
    if bias is not None:
        acc = acc + bias
    if epi == 0:
        return acc
    if epi == 1:
        return torch.nn.functional.gelu(acc, approximate="tanh")
    if epi == 2:
        return out0 + acc
    return acc


CASES = [
    # M, N, K, n_tile
    (128, 128, 64, 128), (128, 256, 128, 256), (300, 200, 192, 64), (257, 96, 768, 32), (384, 2304, 768, 0),
    (400, 768, 3072, 0), (130, 50257, 128, 128),
    # many tiles: the persistent kernel with two TMEM accumulators (ragged M and N)
    (8200, 2000, 192, 0), (5000, 4096, 1024, 0),
    # CTA pairs (n_tile 512): 256 x 256 tiles computed by two SMs, one tile / several tiles per pair / long K
    (256, 256, 64, 512), (512, 768, 192, 512), (1024, 512, 1024, 512), (4864, 1024, 320, 512),
    # swapped orientation: M <= 64 rows
    (1, 128, 64, 0), (17, 768, 3072, 0), (17, 2304, 768, 0), (33, 1600, 1600, 0), (64, 777, 256, 0), (17, 50257, 768, 0),
]


@pytest.mark.parametrize("M,N,K,n_tile", CASES)
def test_tc_gemm_matches_fp32_matmul(M, N, K, n_tile):
    import paper_2408_05636_b200 as sdd
    g = torch.Generator(device="cuda").manual_seed(M * 7 + N)
    cap = M + 37
    A = torch.randn(cap, K, device="cuda", generator=g).to(torch.bfloat16)
    W = (torch.randn(N, K, device="cuda", generator=g) * 0.05).to(torch.bfloat16)
    bias = torch.randn(N, device="cuda", generator=g)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    epis = (0, 1, 2, 3) if N < 10000 else (3,)
    for epi in epis:
        for b in (bias, None):
            # fp32 outputs: a row stride that is not a multiple of 4 takes the hand-written epilogue, a multiple of 4
            # the TMA add-reduce (the CTA-pair cases use the latter)
            ldcs = [N + (8 if epi in (0, 1) else (4 if n_tile == 512 else 3))]
            if epi == 2 and M <= 64:
                ldcs.append(N + 4)      # swapped orientation: the residual tile leaves by TMA add-reduce as well
            for ldc in ldcs:
                if epi in (0, 1):
                    out = torch.full((M, ldc), 7.0, device="cuda", dtype=torch.bfloat16)
                else:
                    out = torch.randn(M, ldc, device="cuda", generator=g)
                out0 = out[:, :N].float().clone()
                pad0 = out[:, N:].float().clone()
                sdd.sdd_debug_gemm_bf16(A, W, b, M, epi, out, n_tile, True, status)
                torch.cuda.synchronize()
                assert int(status.item()) == 0
                ref = _ref(A, W, b, M, epi, out0)
                got = out[:, :N].float()
                tol = 2e-2 if epi in (0, 1) else 2e-3      # bf16 output rounding / fp32 accumulation order
                err = (got - ref).abs().max().item()
                scale = ref.abs().max().item()
                assert err <= tol * max(1.0, scale), (epi, ldc, err, scale)
                assert torch.equal(out[:, N:].float(), pad0)   # nothing written past column N


def test_simt_and_tc_agree():
    import paper_2408_05636_b200 as sdd
    g = torch.Generator(device="cuda").manual_seed(3)
    A = torch.randn(200, 256, device="cuda", generator=g).to(torch.bfloat16)
    W = (torch.randn(300, 256, device="cuda", generator=g) * 0.05).to(torch.bfloat16)
    o1 = torch.zeros(200, 300, device="cuda")
    o2 = torch.zeros(200, 300, device="cuda")
    sdd.sdd_debug_gemm_bf16(A, W, None, 200, 3, o1, 0, True)
    sdd.sdd_debug_gemm_bf16(A, W, None, 200, 3, o2, 0, False)
    torch.cuda.synchronize()
    assert (o1 - o2).abs().max().item() < 1e-3


@pytest.mark.parametrize("M,N,K", [(17, 768, 3072), (33, 3072, 768), (300, 512, 256), (1000, 1024, 512)])
def test_hi_lo_activation_pairs(M, N, K):
    """A given as hi + lo bf16 halves: the product must match the fp32 matmul of the un-split activations far more
    closely than a single bf16 rounding allows; the GELU epilogue's (out, out_lo) pair likewise."""
    import paper_2408_05636_b200 as sdd
    g = torch.Generator(device="cuda").manual_seed(M + N)
    x = torch.randn(M + 5, K, device="cuda", generator=g)
    hi = x.to(torch.bfloat16)
    lo = (x - hi.float()).to(torch.bfloat16)
    W = (torch.randn(N, K, device="cuda", generator=g) * 0.05).to(torch.bfloat16)
    bias = torch.randn(N, device="cuda", generator=g)
    ref = x[:M] @ W.float().t() + bias
    out = torch.zeros(M, N, device="cuda")
    sdd.sdd_debug_gemm_bf16(hi, W, bias, M, 3, out, 0, True, None, None, lo)
    single = torch.zeros(M, N, device="cuda")
    sdd.sdd_debug_gemm_bf16(hi, W, bias, M, 3, single)
    torch.cuda.synchronize()
    err_pair = (out - ref).abs().max().item()
    err_single = (single - ref).abs().max().item()
    assert err_pair < 2e-4 * max(1.0, ref.abs().max().item()) and err_pair < err_single / 20
    # GELU epilogue writing a hi/lo pair
    o_hi = torch.zeros(M, N, device="cuda", dtype=torch.bfloat16)
    o_lo = torch.zeros(M, N, device="cuda", dtype=torch.bfloat16)
    sdd.sdd_debug_gemm_bf16(hi, W, bias, M, 1, o_hi, 0, True, None, None, lo, o_lo)
    torch.cuda.synchronize()
    gref = torch.nn.functional.gelu(ref, approximate="tanh")
    pair = o_hi.float() + o_lo.float()
    assert (pair - gref).abs().max().item() < 2e-3 * max(1.0, gref.abs().max().item())     # hardware tanh ~ 2^-11
    assert (pair - gref).abs().max().item() <= (o_hi.float() - gref).abs().max().item()
