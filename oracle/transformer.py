"""TEST INFRASTRUCTURE — CPU oracle, not part of the product path.

Plain fp64 numpy forward pass of the two networks of a SpecDiff round (Algorithm 1):
the autoregressive target M_p (causal attention) and the masked-diffusion drafter M_q
(no attention mask at all: every position of context ∘ draft slots sees every other).

The paper names its models (GPT-2 XL, GPT-Neo, MDLM; Section "Experimental Setup") but
does not define an architecture, so both networks here are GPT-2-shaped:

    h_0   = wte[ids] + wpe[0..L-1]
    h     = h + Attn(LN1(h)) ; h = h + MLP(LN2(h))          (pre-LayerNorm, eps 1e-5)
    Attn  = softmax(Q K^T / sqrt(d_head) [+ causal mask]) V, fused QKV with bias, output proj
    MLP   = W2 gelu_tanh(W1 x + b1) + b2,  width 4 d
    out   = LN_f(h) @ wte[:V]^T                                (LM head tied to the embedding)

The drafter's [MASK] token is id V (one extra embedding row, no logit) and it takes no
time-step input.  MDLM-faithfulness of this architecture: parity unpinned (the MDLM code
and weights are not available); it is this library's definition.

Every reduction is a plain numpy fp64 sum or matmul; there is no blocking or caching.
"""
from __future__ import annotations

from typing import Dict

import numpy as np

LN_EPS = 1e-5


def layer_norm(x: np.ndarray, g: np.ndarray, b: np.ndarray) -> np.ndarray:
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + LN_EPS) * g + b


def gelu_tanh(x: np.ndarray) -> np.ndarray:
    return 0.5 * x * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (x + 0.044715 * x ** 3)))


def softmax_rows(z: np.ndarray) -> np.ndarray:
    z = z - z.max(axis=-1, keepdims=True)
    e = np.exp(z)
    return e / e.sum(axis=-1, keepdims=True)


class Model:
    """Weights (fp32 arrays from the input generator) + shape; all maths in fp64."""

    def __init__(self, shape, tensors: Dict[str, np.ndarray]):
        self.shape = shape
        self.t = tensors

    def w(self, name: str) -> np.ndarray:
        return self.t[name].astype(np.float64)

    # ------------------------------------------------------------------
    def hidden(self, ids: np.ndarray) -> np.ndarray:
        """ids: int [L] (values in [0, emb_rows)).  Returns LN_f(h_last) as fp64 [L, d]."""
        s = self.shape
        ids = np.asarray(ids, dtype=np.int64)
        L = ids.shape[0]
        assert L <= s.n_ctx, "sequence longer than the position table"
        assert ids.min() >= 0 and ids.max() < s.emb_rows
        d, H, dh = s.d_model, s.n_head, s.d_head
        h = self.t["wte"][ids].astype(np.float64) + self.t["wpe"][:L].astype(np.float64)
        if s.causal:
            allowed = np.tril(np.ones((L, L), dtype=bool))
        for l in range(s.n_layer):
            p = f"l{l}."
            x = layer_norm(h, self.w(p + "ln1_g"), self.w(p + "ln1_b"))
            qkv = x @ self.w(p + "w_qkv").T + self.w(p + "b_qkv")
            q, k, v = qkv[:, :d], qkv[:, d:2 * d], qkv[:, 2 * d:]
            att = np.empty((L, d), dtype=np.float64)
            for hd in range(H):
                sl = slice(hd * dh, (hd + 1) * dh)
                sc = (q[:, sl] @ k[:, sl].T) / np.sqrt(dh)
                if s.causal:
                    sc = np.where(allowed, sc, -np.inf)
                att[:, sl] = softmax_rows(sc) @ v[:, sl]
            h = h + att @ self.w(p + "w_o").T + self.w(p + "b_o")
            x = layer_norm(h, self.w(p + "ln2_g"), self.w(p + "ln2_b"))
            a = gelu_tanh(x @ self.w(p + "w_fc1").T + self.w(p + "b_fc1"))
            h = h + a @ self.w(p + "w_fc2").T + self.w(p + "b_fc2")
        return layer_norm(h, self.w("lnf_g"), self.w("lnf_b"))

    def logits(self, ids: np.ndarray, rows) -> np.ndarray:
        """Logits over the V real tokens at the given row positions: fp64 [len(rows), V]."""
        hf = self.hidden(ids)[np.asarray(rows, dtype=np.int64)]
        return hf @ self.t["wte"][: self.shape.vocab].astype(np.float64).T


def drafter_slot_logits(model_q: Model, ctx_ids: np.ndarray, slot_ids: np.ndarray) -> np.ndarray:
    """One denoising evaluation M_q([x_{0:i}] ∘ [slots]) (Algorithm 1, the loop body):
    logits of the gamma slot positions, fp64 [gamma, V]."""
    c, g = len(ctx_ids), len(slot_ids)
    ids = np.concatenate([np.asarray(ctx_ids, np.int64), np.asarray(slot_ids, np.int64)])
    return model_q.logits(ids, np.arange(c, c + g))


def target_verify_logits(model_p: Model, ctx_ids: np.ndarray, draft_ids: np.ndarray) -> np.ndarray:
    """The gamma+1 target distributions of Algorithm 1 (its parallel evaluation of M_p), as logits:
    row j is the next-token logits after x_{0:c-1} ∘ draft[0:j], j = 0..gamma; fp64 [gamma+1, V].
    Written as the plain definition: one causal forward over all c+gamma tokens."""
    c, g = len(ctx_ids), len(draft_ids)
    ids = np.concatenate([np.asarray(ctx_ids, np.int64), np.asarray(draft_ids, np.int64)])
    return model_p.logits(ids, np.arange(c - 1, c + g))
