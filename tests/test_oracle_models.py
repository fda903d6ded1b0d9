"""Pins for the oracle's two transformer forwards: a library cross-check (torch CPU fp64
ops), causality / non-causality, permutation equivariance and trivial-weight cases."""
import numpy as np
import torch
import torch.nn.functional as F

import synth
from oracle.transformer import Model, drafter_slot_logits, gelu_tanh, layer_norm, target_verify_logits


def _shape(causal, V=37, L=2, d=24, h=3, n_ctx=20):
    return synth.ModelShape(V, L, d, h, n_ctx, causal)


def _model(causal, seed=5, **kw):
    s = _shape(causal, **kw)
    return Model(s, synth.model_weights(s, seed, "fp32", std=0.35, bias_std=0.2, perturb_ln=True))


def _torch_forward(m: Model, ids):
    """The same network from torch's own library routines (fp64)."""
    s = m.shape
    t = {k: torch.from_numpy(v.astype(np.float64)) for k, v in m.t.items()}
    ids = torch.as_tensor(np.asarray(ids), dtype=torch.long)
    L = ids.numel()
    h = F.embedding(ids, t["wte"]) + t["wpe"][:L]
    for l in range(s.n_layer):
        p = f"l{l}."
        x = F.layer_norm(h, (s.d_model,), t[p + "ln1_g"], t[p + "ln1_b"], 1e-5)
        qkv = F.linear(x, t[p + "w_qkv"], t[p + "b_qkv"])
        q, k, v = [a.reshape(L, s.n_head, s.d_head).transpose(0, 1) for a in qkv.split(s.d_model, dim=-1)]
        a = F.scaled_dot_product_attention(q[None], k[None], v[None], is_causal=s.causal)[0]
        a = a.transpose(0, 1).reshape(L, s.d_model)
        h = h + F.linear(a, t[p + "w_o"], t[p + "b_o"])
        x = F.layer_norm(h, (s.d_model,), t[p + "ln2_g"], t[p + "ln2_b"], 1e-5)
        h = h + F.linear(F.gelu(F.linear(x, t[p + "w_fc1"], t[p + "b_fc1"]), approximate="tanh"),
                         t[p + "w_fc2"], t[p + "b_fc2"])
    hf = F.layer_norm(h, (s.d_model,), t["lnf_g"], t["lnf_b"], 1e-5)
    return (hf @ t["wte"][: s.vocab].T).numpy()


def test_blocks_against_torch_library_ops():
    x = np.random.default_rng(0).normal(size=(5, 24))
    g, b = np.random.default_rng(1).normal(size=(2, 24))
    ref = F.layer_norm(torch.from_numpy(x), (24,), torch.from_numpy(g), torch.from_numpy(b), 1e-5).numpy()
    assert np.abs(layer_norm(x, g, b) - ref).max() < 1e-12
    assert np.abs(gelu_tanh(x) - F.gelu(torch.from_numpy(x), approximate="tanh").numpy()).max() < 1e-12


def test_full_forward_against_torch_library_ops():
    rng = np.random.default_rng(2)
    for causal in (True, False):
        m = _model(causal)
        ids = rng.integers(0, m.shape.emb_rows, size=13)
        if not causal:
            ids[-3:] = m.shape.vocab  # [MASK] rows use the extra embedding row
        got = m.logits(ids, np.arange(13))
        ref = _torch_forward(m, ids)
        assert got.shape == (13, m.shape.vocab)
        assert np.abs(got - ref).max() < 1e-10


def test_target_rows_are_causal_and_match_growing_prefix():
    m = _model(True)
    rng = np.random.default_rng(3)
    ctx = rng.integers(0, 37, size=6)
    dr = rng.integers(0, 37, size=4)
    lam = target_verify_logits(m, ctx, dr)
    assert lam.shape == (5, 37)
    for j in range(5):  # row j = next-token logits after ctx ∘ dr[:j], computed on its own
        ids = np.concatenate([ctx, dr[:j]])
        alone = m.logits(ids, [len(ids) - 1])[0]
        assert np.abs(lam[j] - alone).max() < 1e-11
    dr2 = dr.copy()
    dr2[2] = (dr2[2] + 1) % 37
    lam2 = target_verify_logits(m, ctx, dr2)
    assert np.array_equal(lam2[:3], lam[:3])           # rows before the change are untouched
    assert np.abs(lam2[3] - lam[3]).max() > 1e-6       # rows from the change on move


def test_drafter_is_bidirectional_and_position_equivariant():
    m = _model(False)
    V = m.shape.vocab
    rng = np.random.default_rng(4)
    ctx = rng.integers(0, V, size=6)
    slots = np.array([V, int(rng.integers(0, V)), V])
    base = drafter_slot_logits(m, ctx, slots)
    assert base.shape == (3, V)
    # non-causality witness: a later slot changes an earlier slot's logits, and so does the context
    s2 = slots.copy()
    s2[2] = 3
    assert np.abs(drafter_slot_logits(m, ctx, s2)[0] - base[0]).max() > 1e-6
    c2 = ctx.copy()
    c2[0] = (c2[0] + 1) % V
    assert np.abs(drafter_slot_logits(m, c2, slots) - base).max() > 1e-6
    # permuting tokens together with their position rows permutes nothing the slots can see
    perm = rng.permutation(6)
    t2 = dict(m.t)
    wpe = m.t["wpe"].copy()
    wpe[:6] = m.t["wpe"][:6][perm]
    t2["wpe"] = wpe
    got = drafter_slot_logits(Model(m.shape, t2), ctx[perm], slots)
    assert np.abs(got - base).max() < 1e-10


def test_trivial_weights():
    s = _shape(False)
    w = synth.model_weights(s, 1, "fp32")
    for k in w:
        if not k.endswith("_g"):
            w[k] = np.zeros_like(w[k])
    lg = drafter_slot_logits(Model(s, w), np.array([1, 2, 3]), np.array([s.vocab, s.vocab]))
    assert np.array_equal(lg, np.zeros((2, s.vocab)))   # zero weights: uniform distribution
    # default generator: N(0, 0.02) matrices, zero biases, unit gains; bf16 variant is bf16-exact
    s = _shape(True)
    w32, w16 = synth.model_weights(s, 9, "fp32"), synth.model_weights(s, 9, "bf16")
    assert abs(float(w32["wte"].std()) - 0.02) < 0.004 and not w32["l0.b_qkv"].any() and (w32["lnf_g"] == 1).all()
    assert np.array_equal(torch.from_numpy(w32["wte"]).to(torch.bfloat16).float().numpy(), w16["wte"])
    assert np.array_equal(synth.model_weights(s, 9, "fp32")["l1.w_fc2"], w32["l1.w_fc2"])  # deterministic
