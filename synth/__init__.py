"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests.

This module only *generates data*: random-init transformer weights, random prompts,
and correlated logit pairs for the accept-kernel microbenchmark.  It holds none of
the decoding method's arithmetic (no softmax of the method, no acceptance rule, no
Philox streams of the method) and imports neither the oracle nor the CUDA binding.

All generators are pure functions of their seeds (numpy PCG64 streams), so the two
sides see byte-identical inputs.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List

import numpy as np

# ----------------------------------------------------------------------------------
# model shapes
# ----------------------------------------------------------------------------------


@dataclass(frozen=True)
class ModelShape:
    """GPT-2-shaped transformer; `causal=False` is the masked-diffusion drafter."""

    vocab: int
    n_layer: int
    d_model: int
    n_head: int
    n_ctx: int
    causal: bool

    @property
    def d_head(self) -> int:
        return self.d_model // self.n_head

    @property
    def emb_rows(self) -> int:
        # the drafter owns one extra embedding row, the [MASK] token, with id == vocab
        return self.vocab + (0 if self.causal else 1)


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str  # "fp32" or "bf16"
    target: ModelShape
    drafter: ModelShape
    prompt_len: int
    gamma: int
    T: int
    batch: int
    max_new: int
    weight_seed: int
    prompt_seed: int
    philox_seed: int

    @property
    def ar_drafter(self) -> ModelShape:
        """Autoregressive drafter of the speculative-decoding warm start: the diffusion drafter's size, causal."""
        d = self.drafter
        return ModelShape(d.vocab, d.n_layer, d.d_model, d.n_head, d.n_ctx, True)

    @property
    def ar_weight_seed(self) -> int:
        return self.weight_seed + 500


def _wl(name, dtype, V, tl, td, th, ql, qd, qh, n_ctx, prompt, gamma, T, batch, max_new, seeds):
    return Workload(
        name, dtype,
        ModelShape(V, tl, td, th, n_ctx, True),
        ModelShape(V, ql, qd, qh, n_ctx, False),
        prompt, gamma, T, batch, max_new, *seeds)


WORKLOADS: Dict[str, Workload] = {
    # tiny fp32 case the oracle finishes in well under a second per round
    "tiny_fp32": _wl("tiny_fp32", "fp32", 512, 2, 256, 4, 2, 128, 4, 128, 32, 8, 4, 1, 36, (1, 2, 3)),
    # the smallest pair that runs on the bf16 tensor-core path (d_head must be 64 there): two layers, two heads
    "tiny_bf16": _wl("tiny_bf16", "bf16", 512, 2, 128, 2, 2, 128, 2, 128, 32, 8, 2, 1, 36, (5, 6, 7)),
    # GPT-2-small-shaped pair (the paper's 110M-class drafter size), 256 new tokens
    "small_bf16": _wl("small_bf16", "bf16", 50257, 12, 768, 12, 12, 768, 12, 1024, 256, 16, 8, 1, 256, (11, 12, 13)),
    # GPT-2-XL-shaped target with a 24-layer d=1024 drafter
    "xl_bf16": _wl("xl_bf16", "bf16", 50257, 48, 1600, 25, 24, 1024, 16, 2048, 512, 32, 16, 1, 512, (21, 22, 23)),
    # serving sweep shape (gamma / T are swept by the caller)
    "xl_bf16_b16": _wl("xl_bf16_b16", "bf16", 50257, 48, 1600, 25, 24, 1024, 16, 2048, 1024, 16, 8, 16, 512, (41, 42, 43)),
}


def scaled_workload(base: Workload, **kw) -> Workload:
    """Copy of `base` with some fields replaced (used for reduced parity cases)."""
    d = dict(base.__dict__)
    d.update(kw)
    return Workload(**d)


# ----------------------------------------------------------------------------------
# weights
# ----------------------------------------------------------------------------------

# Fixed tensor order of one model.  Linear weights are stored [out_features, in_features]
# row-major (y = x @ W.T + b); the LM head is tied to the first `vocab` rows of `wte`.
PER_LAYER = ("ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o",
             "ln2_g", "ln2_b", "w_fc1", "b_fc1", "w_fc2", "b_fc2")


def tensor_names(shape: ModelShape) -> List[str]:
    names = ["wte", "wpe"]
    for l in range(shape.n_layer):
        names += [f"l{l}.{n}" for n in PER_LAYER]
    names += ["lnf_g", "lnf_b"]
    return names


def tensor_shape(shape: ModelShape, name: str):
    d = shape.d_model
    base = name.split(".")[-1]
    return {
        "wte": (shape.emb_rows, d), "wpe": (shape.n_ctx, d),
        "ln1_g": (d,), "ln1_b": (d,), "ln2_g": (d,), "ln2_b": (d,), "lnf_g": (d,), "lnf_b": (d,),
        "w_qkv": (3 * d, d), "b_qkv": (3 * d,), "w_o": (d, d), "b_o": (d,),
        "w_fc1": (4 * d, d), "b_fc1": (4 * d,), "w_fc2": (d, 4 * d), "b_fc2": (d,),
    }[base]


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); result kept as fp32."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return rounded.view(np.float32)


def model_weights(shape: ModelShape, seed: int, dtype: str, *, std: float = 0.02,
                  bias_std: float = 0.0, perturb_ln: bool = False) -> Dict[str, np.ndarray]:
    """Random-init weights: matrices and embeddings ~ N(0, std^2), LayerNorm gain 1 / bias 0,
    linear biases 0 (or N(0, bias_std^2) so that tests can see a dropped bias).

    With dtype == "bf16" the matrix/embedding values are rounded to bf16 once (returned as
    fp32 arrays holding bf16-representable values) so that both sides use identical numbers.
    """
    out: Dict[str, np.ndarray] = {}
    tag = 1 if shape.causal else 2
    for idx, name in enumerate(tensor_names(shape)):
        shp = tensor_shape(shape, name)
        base = name.split(".")[-1]
        rng = np.random.default_rng([seed, tag, idx])
        if base in ("ln1_g", "ln2_g", "lnf_g"):
            t = np.ones(shp, np.float32)
            if perturb_ln:
                t += 0.1 * rng.standard_normal(shp, dtype=np.float32)
        elif base in ("ln1_b", "ln2_b", "lnf_b"):
            t = np.zeros(shp, np.float32)
            if perturb_ln:
                t += 0.1 * rng.standard_normal(shp, dtype=np.float32)
        elif base.startswith("b_"):
            t = (bias_std * rng.standard_normal(shp, dtype=np.float32)).astype(np.float32)
        else:
            t = (std * rng.standard_normal(shp, dtype=np.float32)).astype(np.float32)
            if dtype == "bf16":
                t = round_to_bf16(t)
        out[name] = t
    return out


def prompt_ids(vocab: int, batch: int, length: int, seed: int) -> np.ndarray:
    """Uniform-random prompt token ids, int32 [batch, length]."""
    rng = np.random.default_rng([seed, 7])
    return rng.integers(0, vocab, size=(batch, length), dtype=np.int32)


# ----------------------------------------------------------------------------------
# accept-kernel microbenchmark inputs
# ----------------------------------------------------------------------------------

# sigma of the private Gaussian component <-> overlap sum_x min(p, q) for large vocab
MICRO_SIGMAS = (0.178, 0.30, 0.50, 0.70, 0.954)


@dataclass
class AcceptCase:
    logits_p: np.ndarray  # fp32 [rows, gamma + 1, V]
    logits_q: np.ndarray  # fp32 [rows, gamma, V]
    draft_ids: np.ndarray  # int32 [rows, gamma]
    sigma: float
    meta: dict = field(default_factory=dict)


def accept_case(rows: int, gamma: int, vocab: int, sigma: float, seed: int,
                *, draw_drafts: bool = True) -> AcceptCase:
    """Target / draft logits with a shared Gaussian component: lambda = c + sigma*a,
    l = c + sigma*b with a, b, c iid N(0,1).  Draft ids are drawn from softmax(l) with a
    plain inverse-CDF draw of this module's own generator (they are *inputs* of the
    acceptance step, so they come from here and not from either implementation)."""
    rng = np.random.default_rng([seed, 31])
    c = rng.standard_normal((rows, gamma + 1, vocab), dtype=np.float32)
    lp = c + np.float32(sigma) * rng.standard_normal((rows, gamma + 1, vocab), dtype=np.float32)
    lq = c[:, :gamma] + np.float32(sigma) * rng.standard_normal((rows, gamma, vocab), dtype=np.float32)
    del c
    ids = np.zeros((rows, gamma), np.int32)
    if draw_drafts:
        u = rng.random((rows, gamma))
        for r in range(rows):
            z = lq[r].astype(np.float64)
            z -= z.max(axis=-1, keepdims=True)
            cdf = np.cumsum(np.exp(z), axis=-1)
            cdf /= cdf[:, -1:]
            for j in range(gamma):
                ids[r, j] = min(int(np.searchsorted(cdf[j], u[r, j], side="right")), vocab - 1)
    else:
        ids[:] = rng.integers(0, vocab, size=(rows, gamma), dtype=np.int32)
    return AcceptCase(np.ascontiguousarray(lp), np.ascontiguousarray(lq), ids, float(sigma))


def accept_row_index(gamma_base: int, gamma: int):
    """Row indices that turn a case of draft length gamma_base into one of length gamma by cutting or repeating
    rows: target row j and draft row j of the new case are rows j % gamma_base of the old one (so a target row stays
    paired with the draft row it shares its common component with), the last target row (the one that follows a fully
    accepted draft) stays the last.  Returns (target row index [gamma + 1], draft row index [gamma])."""
    q_idx = np.arange(gamma, dtype=np.int64) % gamma_base
    p_idx = np.concatenate([q_idx, np.array([gamma_base], dtype=np.int64)])
    return p_idx, q_idx


def resize_accept_case(case: AcceptCase, gamma: int) -> AcceptCase:
    """The same rows with another draft length (see accept_row_index); pure re-indexing of `case`."""
    p_idx, q_idx = accept_row_index(case.draft_ids.shape[1], gamma)
    return AcceptCase(np.ascontiguousarray(case.logits_p[:, p_idx]), np.ascontiguousarray(case.logits_q[:, q_idx]),
                      np.ascontiguousarray(case.draft_ids[:, q_idx]), case.sigma, dict(case.meta))
