"""The bf16 tensor-core attention kernel against torch's scaled_dot_product_attention on the same bf16
inputs (fp32 maths): drafter mode (no mask, ragged lengths, several key tiles) and the two target modes."""
import pytest
import torch
import torch.nn.functional as F

pytestmark = pytest.mark.gpu


def _ref(q, k, v, causal_from=None):
    """q [Lq, H, 64], k, v [Lk, H, 64] (float); causal_from: position of query row 0 (None = no mask)."""
    qh, kh, vh = (t.float().transpose(0, 1) for t in (q, k, v))
    mask = None
    if causal_from is not None:
        pos = causal_from + torch.arange(q.shape[0], device=q.device)[:, None]
        mask = torch.arange(k.shape[0], device=q.device)[None, :] <= pos
    o = F.scaled_dot_product_attention(qh[None], kh[None], vh[None], attn_mask=mask)[0]
    return o.transpose(0, 1)


# the fourth case: many CTAs (several waves), sequences whose last key tile is full or ragged; the last two: grids of at
# most one CTA per SM with long chains of key tiles (the pipelined variant: 8, 9 and 7 tiles per CTA)
@pytest.mark.parametrize("H,lens,gamma,lcap", [(2, [100], 16, 128), (3, [250, 37, 511], 16, 640), (12, [300], 32, 384),
                                                (16, [700, 130, 250, 1000, 496, 129], 16, 1024),
                                                (4, [1000, 1100], 32, 1152), (16, [850], 32, 896)])
def test_drafter_mode(H, lens, gamma, lcap):
    import paper_2408_05636_b200 as sdd
    B, d = len(lens), H * 64
    g = torch.Generator(device="cuda").manual_seed(sum(lens))
    qkv = torch.randn(B * lcap, 3 * d, device="cuda", generator=g).to(torch.bfloat16)
    vt_ld = lcap + 128
    vt = torch.zeros(B * d, vt_ld, device="cuda", dtype=torch.bfloat16)
    for b in range(B):
        vt[b * d:(b + 1) * d, :lcap] = qkv[b * lcap:(b + 1) * lcap, 2 * d:].t()
    out = torch.full((B * lcap, d), 9.0, device="cuda", dtype=torch.bfloat16)
    ctx = torch.tensor(lens, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sdd.sdd_debug_attention_bf16(qkv, 0, qkv, d, lcap, vt, out, ctx, B, H, gamma, 0, lcap, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for b, c in enumerate(lens):
        L = c + gamma
        rows = qkv[b * lcap: b * lcap + L]
        ref = _ref(rows[:, :d].reshape(L, H, 64), rows[:, d:2 * d].reshape(L, H, 64), rows[:, 2 * d:].reshape(L, H, 64))
        got = out[b * lcap: b * lcap + L].float().reshape(L, H, 64)
        assert (got - ref).abs().max().item() < 2e-2
        assert torch.all(out[b * lcap + L: (b + 1) * lcap] == 9.0)      # padding rows untouched


@pytest.mark.parametrize("mode,lens,rows", [(1, [40, 300], 17), (1, [1, 129], 33), (2, [200, 50], 199), (2, [2], 1),
                                            (1, [1000, 650], 33), (2, [1100], 1099)])
def test_target_modes(mode, lens, rows):
    import paper_2408_05636_b200 as sdd
    H, n_ctx, gamma = 4, (512 if max(lens) + rows <= 512 else 1280), rows - 1
    B, d = len(lens), H * 64
    g = torch.Generator(device="cuda").manual_seed(17 * mode + rows)
    qkv = torch.randn(B * rows + 200, 3 * d, device="cuda", generator=g).to(torch.bfloat16)
    kc = torch.randn(B * n_ctx, d, device="cuda", generator=g).to(torch.bfloat16)
    v = torch.randn(B, n_ctx, d, device="cuda", generator=g).to(torch.bfloat16)
    vt = v.transpose(1, 2).contiguous().reshape(B * d, n_ctx)
    out = torch.full((B * rows, d), 9.0, device="cuda", dtype=torch.bfloat16)
    ctx = torch.tensor(lens, dtype=torch.int32, device="cuda")
    sdd.sdd_debug_attention_bf16(qkv, 0, kc, 0, n_ctx, vt, out, ctx, B, H, gamma, mode, rows)
    torch.cuda.synchronize()
    for b, c in enumerate(lens):
        nq = rows if mode == 1 else max(0, c - 1)
        start = c - 1 if mode == 1 else 0
        if nq == 0:
            continue
        nk = start + nq
        q = qkv[b * rows: b * rows + nq, :d].reshape(nq, H, 64)
        k = kc[b * n_ctx: b * n_ctx + nk].reshape(nk, H, 64)
        vv = v[b, :nk].reshape(nk, H, 64)
        ref = _ref(q, k, vv, causal_from=start)
        got = out[b * rows: b * rows + nq].float().reshape(nq, H, 64)
        assert (got - ref).abs().max().item() < 2e-2
