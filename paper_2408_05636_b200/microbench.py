"""Stand-alone timing of the library's kernels through the C ABI (CUDA events, back-to-back launches).

    python -m paper_2408_05636_b200.microbench gemm  --m 8192 --n 4096 --k 4096 [--epilogue 0] [--n-tile 0]
    python -m paper_2408_05636_b200.microbench attn  --heads 16 --len 1024 [--batch 1]
    python -m paper_2408_05636_b200.microbench attn-verify --heads 25 --len 1000 --rows 33 [--batch 1]
    python -m paper_2408_05636_b200.microbench accept --rows 64 --gamma 32 [--vocab 50257]

Each prints one JSON line with the time per launch and the achieved rate.  `--iters` launches are timed
after `--warmup`; inputs are seeded random tensors created on the device (bench.py times the acceptance step on the
host-generated cases of synth.accept_case instead, see accept_case_timed).
"""
from __future__ import annotations

import argparse
import json

import torch

import paper_2408_05636_b200 as sdd


def time_launches(fn, iters: int, warmup: int, stream) -> float:
    """Milliseconds per call of fn(), timed with CUDA events on `stream`."""
    with torch.cuda.stream(stream):
        for _ in range(warmup):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        stream.synchronize()
        e0.record(stream)
        for _ in range(iters):
            fn()
        e1.record(stream)
        stream.synchronize()
    return e0.elapsed_time(e1) / iters


def gemm(m, n, k, epilogue=0, n_tile=0, iters=50, warmup=5, seed=0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    A = torch.randn(m, k, device="cuda", generator=g).to(torch.bfloat16)
    W = (torch.randn(n, k, device="cuda", generator=g) * 0.02).to(torch.bfloat16)
    bias = torch.zeros(n, device="cuda")
    out = torch.zeros(m, n, device="cuda", dtype=torch.bfloat16 if epilogue in (0, 1) else torch.float32)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    st = torch.cuda.Stream()
    ms = time_launches(lambda: sdd.sdd_debug_gemm_bf16(A, W, bias, m, epilogue, out, n_tile, True, status, st),
                       iters, warmup, st)
    assert int(status.item()) == 0
    flops = 2.0 * m * n * k
    nbytes = 2.0 * (m * k + n * k) + out.element_size() * m * n
    return {"kernel": "gemm_tc", "m": m, "n": n, "k": k, "epilogue": epilogue, "n_tile": n_tile, "us": ms * 1e3,
            "tflops": flops / (ms * 1e-3) / 1e12, "gbs": nbytes / (ms * 1e-3) / 1e9}


def attn(heads, length, batch=1, gamma=16, iters=50, warmup=5, seed=0):
    d = heads * 64
    lcap = (length + 127) // 128 * 128
    g = torch.Generator(device="cuda").manual_seed(seed)
    qkv = torch.randn(batch * lcap, 3 * d, device="cuda", generator=g).to(torch.bfloat16)
    vt = torch.randn(batch * d, lcap, device="cuda", generator=g).to(torch.bfloat16)
    out = torch.zeros(batch * lcap, d, device="cuda", dtype=torch.bfloat16)
    ctx = torch.full((batch,), length - gamma, dtype=torch.int32, device="cuda")
    st = torch.cuda.Stream()
    ms = time_launches(lambda: sdd.sdd_debug_attention_bf16(qkv, 0, qkv, d, lcap, vt, out, ctx, batch, heads, gamma, 0,
                                                            lcap, None, st), iters, warmup, st)
    flops = 4.0 * batch * length * length * d
    return {"kernel": "attn_tc", "heads": heads, "len": length, "batch": batch, "us": ms * 1e3,
            "tflops": flops / (ms * 1e-3) / 1e12}


def attn_target(heads, ctx_len, rows=33, batch=1, n_ctx=2048, iters=50, warmup=5, seed=0):
    """Verification-mode attention: `rows` new query rows per sequence over a cache of ctx_len - 1 keys plus themselves."""
    d = heads * 64
    g = torch.Generator(device="cuda").manual_seed(seed)
    qkv = torch.randn(batch * rows + 200, 3 * d, device="cuda", generator=g).to(torch.bfloat16)
    kc = torch.randn(batch * n_ctx, d, device="cuda", generator=g).to(torch.bfloat16)
    vt = torch.randn(batch * d, n_ctx, device="cuda", generator=g).to(torch.bfloat16)
    out = torch.zeros(batch * rows, d, device="cuda", dtype=torch.bfloat16)
    ctx = torch.full((batch,), ctx_len, dtype=torch.int32, device="cuda")
    st = torch.cuda.Stream()
    ms = time_launches(lambda: sdd.sdd_debug_attention_bf16(qkv, 0, kc, 0, n_ctx, vt, out, ctx, batch, heads, rows - 1, 1,
                                                            rows, None, st), iters, warmup, st)
    nbytes = batch * (2.0 * (ctx_len - 1 + rows) * d * 2 + 2.0 * rows * d * 2)
    return {"kernel": "attn_tc_verify", "heads": heads, "ctx_len": ctx_len, "rows": rows, "batch": batch, "us": ms * 1e3,
            "gbs": nbytes / (ms * 1e-3) / 1e9}


def accept(rows, gamma, vocab=50257, sigma=0.5, iters=20, warmup=3, seed=31):
    g = torch.Generator(device="cuda").manual_seed(seed)
    c = torch.randn(rows, gamma + 1, vocab, device="cuda", generator=g)
    lp = (c + sigma * torch.randn(rows, gamma + 1, vocab, device="cuda", generator=g)).contiguous()
    lq = (c[:, :gamma] + sigma * torch.randn(rows, gamma, vocab, device="cuda", generator=g)).contiguous()
    del c
    ids = torch.distributions.Categorical(logits=lq).sample().to(torch.int32).contiguous()
    scratch = torch.empty(sdd.sdd_accept_scratch_bytes(rows, gamma, vocab), dtype=torch.uint8, device="cuda")
    st = torch.cuda.Stream()
    res = {}

    def call():
        res["n"] = sdd.sdd_accept_logits(lp, lq, ids, 1.0, 1.0, seed, 7, scratch, st)[0]

    ms = time_launches(call, iters, warmup, st)
    nbytes = rows * (2 * gamma + 1) * vocab * 4.0
    return {"kernel": "accept", "rows": rows, "gamma": gamma, "vocab": vocab, "us": ms * 1e3,
            "gbs": nbytes / (ms * 1e-3) / 1e9, "bytes": nbytes, "mean_accepted": float(res["n"].float().mean().item())}


def accept_case_timed(base, gamma, iters=20, warmup=3, seed=31, rnd=7):
    """Times sdd_accept_logits on a seeded case of the input generator (synth.AcceptCase: host arrays), re-indexed to
    draft length `gamma` with the generator's own row index (synth.accept_row_index), so that the timed inputs are
    exactly the ones the parity tests replay through the oracle."""
    import synth
    rows, g0 = base.draft_ids.shape
    vocab = base.logits_p.shape[2]
    p_idx, q_idx = synth.accept_row_index(g0, gamma)
    lp0 = torch.from_numpy(base.logits_p).cuda()
    lq0 = torch.from_numpy(base.logits_q).cuda()
    ids0 = torch.from_numpy(base.draft_ids).cuda()
    lp = lp0[:, torch.from_numpy(p_idx).cuda()].contiguous()
    del lp0
    lq = lq0[:, torch.from_numpy(q_idx).cuda()].contiguous()
    del lq0
    ids = ids0[:, torch.from_numpy(q_idx).cuda()].contiguous()
    scratch = torch.empty(sdd.sdd_accept_scratch_bytes(rows, gamma, vocab), dtype=torch.uint8, device="cuda")
    st = torch.cuda.Stream()
    res = {}

    def call():
        res["n"] = sdd.sdd_accept_logits(lp, lq, ids, 1.0, 1.0, seed, rnd, scratch, st)[0]

    ms = time_launches(call, iters, warmup, st)
    nbytes = rows * (2 * gamma + 1) * vocab * 4.0
    return {"kernel": "accept", "rows": rows, "gamma": gamma, "vocab": vocab, "us": ms * 1e3,
            "gbs": nbytes / (ms * 1e-3) / 1e9, "bytes": nbytes, "mean_accepted": float(res["n"].float().mean().item())}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("kernel", choices=["gemm", "attn", "attn-verify", "accept"])
    ap.add_argument("--m", type=int, default=8192)
    ap.add_argument("--n", type=int, default=4096)
    ap.add_argument("--k", type=int, default=4096)
    ap.add_argument("--epilogue", type=int, default=0)
    ap.add_argument("--n-tile", type=int, default=0)
    ap.add_argument("--heads", type=int, default=16)
    ap.add_argument("--len", type=int, default=1024)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--rows", type=int, default=64)
    ap.add_argument("--gamma", type=int, default=32)
    ap.add_argument("--vocab", type=int, default=50257)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    a = ap.parse_args()
    if a.kernel == "gemm":
        r = gemm(a.m, a.n, a.k, a.epilogue, a.n_tile, a.iters, a.warmup)
    elif a.kernel == "attn":
        r = attn(a.heads, a.len, a.batch, iters=a.iters, warmup=a.warmup)
    elif a.kernel == "attn-verify":
        r = attn_target(a.heads, a.len, a.rows, a.batch, iters=a.iters, warmup=a.warmup)
    else:
        r = accept(a.rows, a.gamma, a.vocab, iters=a.iters, warmup=a.warmup)
    print(json.dumps(r))


if __name__ == "__main__":
    main()
