"""Python binding of the SpecDiff CUDA library (libsdd.so, built from csrc/ for sm_100a).

Argument marshalling only: every step of a draft–verify–accept round runs in the library's
CUDA kernels.  torch is used for device memory and streams.  The functions carry the same
names as the C ABI in include/sdd.h; `Session` is a thin convenience wrapper around them.

There is no CPU path: importing this package without a built libsdd.so raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsdd.so")

SDD_OK = 0
SDD_E_ARG, SDD_E_SHAPE, SDD_E_WORKSPACE, SDD_E_CTX_FULL = -1, -2, -3, -4
SDD_E_CUDA, SDD_E_TIMEOUT, SDD_E_UNIMPL, SDD_E_STATE, SDD_E_INDEX = -5, -6, -7, -8, -9
SDD_FP32, SDD_BF16 = 0, 1

(TAP_TOKENS, TAP_CTX_LEN, TAP_DRAFT_IDS, TAP_STEP_LOGITS, TAP_Q_LOGITS, TAP_LOGQ, TAP_REVEAL_STEP,
 TAP_LOGITS_P, TAP_ACCEPT_PROB, TAP_N_ACCEPT, TAP_EXTRA_TOKEN, TAP_N_EMITTED, TAP_STATUS, TAP_EVALS) = range(14)

PROF_NAMES = ["gemm_drafter", "gemm_target", "head_drafter", "head_target", "attn_drafter", "attn_target",
              "layernorm", "glue", "sample", "row_stats", "accept", "commit"]

EXPORTS = [
    "sdd_workspace_bytes", "sdd_create", "sdd_reset", "sdd_draft_begin", "sdd_draft_step", "sdd_draft",
    "sdd_verify_accept", "sdd_step", "sdd_ar_step", "sdd_sps_workspace_bytes", "sdd_sps_attach", "sdd_sps_step",
    "sdd_progress", "sdd_accept_scratch_bytes", "sdd_accept_logits",
    "sdd_accept_logits_static", "sdd_debug_gemm_bf16", "sdd_debug_attention_bf16", "sdd_debug_wait_timeout",
    "sdd_tap", "sdd_counters", "sdd_profile_begin", "sdd_profile_end", "sdd_sync_status", "sdd_destroy", "sdd_strerror", "sdd_last_cuda_error",
]


class SddError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().sdd_strerror(status).decode()
        cuda = lib().sdd_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} ({status})" + (f" [{cuda}]" if status == SDD_E_CUDA and cuda else ""))


class sdd_model(C.Structure):
    _fields_ = [("vocab", C.c_int32), ("n_layer", C.c_int32), ("d_model", C.c_int32), ("n_head", C.c_int32),
                ("n_ctx", C.c_int32), ("causal", C.c_int32), ("dtype", C.c_int32),
                ("tensors", C.POINTER(C.c_void_p)), ("n_tensors", C.c_int32)]


class sdd_params(C.Structure):
    _fields_ = [("gamma", C.c_int32), ("T", C.c_int32), ("batch", C.c_int32), ("max_new", C.c_int32),
                ("temp_p", C.c_float), ("temp_q", C.c_float), ("seed", C.c_uint64), ("stream", C.c_void_p)]


_lib = None


def lib() -> C.CDLL:
    """The loaded library; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2408_05636_b200.build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i32, u64, f32 = C.c_void_p, C.c_int32, C.c_uint64, C.c_float
        L.sdd_workspace_bytes.argtypes = [C.POINTER(sdd_model), C.POINTER(sdd_model), C.POINTER(sdd_params), C.POINTER(u64)]
        L.sdd_create.argtypes = [C.POINTER(sdd_model), C.POINTER(sdd_model), C.POINTER(sdd_params), vp, i32,
                                 C.POINTER(i32), vp, u64, C.POINTER(vp)]
        L.sdd_reset.argtypes = [vp, vp, i32, C.POINTER(i32)]
        for n in ("sdd_draft_begin", "sdd_draft_step", "sdd_draft", "sdd_sync_status"):
            getattr(L, n).argtypes = [vp]
        L.sdd_verify_accept.argtypes = [vp, vp, vp]
        L.sdd_step.argtypes = [vp, vp, vp]
        L.sdd_ar_step.argtypes = [vp, vp, vp]
        L.sdd_sps_workspace_bytes.argtypes = [C.POINTER(sdd_model), C.POINTER(sdd_params), C.POINTER(u64)]
        L.sdd_sps_attach.argtypes = [vp, C.POINTER(sdd_model), vp, u64]
        L.sdd_sps_step.argtypes = [vp, i32, vp, vp]
        L.sdd_progress.argtypes = [vp, C.POINTER(u64), C.POINTER(i32)]
        L.sdd_accept_scratch_bytes.argtypes = [i32, i32, i32]
        L.sdd_accept_scratch_bytes.restype = u64
        L.sdd_accept_logits.argtypes = [vp, vp, vp, i32, i32, i32, f32, f32, u64, u64, vp, vp, vp, vp, vp]
        L.sdd_accept_logits_static.argtypes = [vp, vp, vp, i32, i32, i32, f32, f32, u64, u64, vp, vp, vp, vp]
        L.sdd_debug_gemm_bf16.argtypes = [vp, C.c_int64, vp, vp, i32, i32, i32, i32, vp, i32, i32, i32, vp, vp, vp, vp]
        L.sdd_debug_attention_bf16.argtypes = [vp, C.c_int64, i32, i32, vp, C.c_int64, i32, i32, i32, vp, i32, vp, i32, vp,
                                               i32, i32, i32, i32, i32, vp, vp]
        L.sdd_debug_wait_timeout.argtypes = [C.c_int64, vp, vp]
        L.sdd_tap.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(u64)]
        L.sdd_counters.argtypes = [vp, C.POINTER(u64), C.POINTER(u64)]
        L.sdd_profile_begin.argtypes = [vp]
        L.sdd_profile_end.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(u64), i32]
        L.sdd_destroy.argtypes = [vp]
        L.sdd_destroy.restype = None
        L.sdd_strerror.argtypes = [i32]
        L.sdd_strerror.restype = C.c_char_p
        L.sdd_last_cuda_error.argtypes = []
        L.sdd_last_cuda_error.restype = C.c_char_p
        for n in EXPORTS:
            if getattr(L, n).restype is C.c_int:
                getattr(L, n).restype = i32
        _lib = L
    return _lib


def _check(status: int, where: str):
    if status != SDD_OK:
        raise SddError(status, where)


def _torch():
    import torch
    return torch


# ----------------------------------------------------------------------------------------------
# models on the device
# ----------------------------------------------------------------------------------------------
class DeviceModel:
    """One transformer's weights uploaded to the GPU in the library's tensor order."""

    def __init__(self, shape, tensors: Dict[str, np.ndarray], names: Sequence[str], dtype: str, device="cuda:0"):
        torch = _torch()
        self.shape = shape
        self.dtype = SDD_BF16 if dtype == "bf16" else SDD_FP32
        self.keep = []
        ptrs = (C.c_void_p * len(names))()
        for i, n in enumerate(names):
            t = torch.from_numpy(np.ascontiguousarray(tensors[n]))
            is_matrix = t.dim() == 2
            t = t.to(device=device, dtype=torch.bfloat16 if (is_matrix and self.dtype == SDD_BF16) else torch.float32)
            self.keep.append(t)
            ptrs[i] = t.data_ptr()
        self.ptrs = ptrs
        self.c = sdd_model(shape.vocab, shape.n_layer, shape.d_model, shape.n_head, shape.n_ctx,
                           1 if shape.causal else 0, self.dtype, C.cast(ptrs, C.POINTER(C.c_void_p)), len(names))


# ----------------------------------------------------------------------------------------------
# C ABI, same names
# ----------------------------------------------------------------------------------------------
def sdd_workspace_bytes(target: DeviceModel, drafter: DeviceModel, params: sdd_params) -> int:
    out = C.c_uint64(0)
    _check(lib().sdd_workspace_bytes(C.byref(target.c), C.byref(drafter.c), C.byref(params), C.byref(out)),
           "sdd_workspace_bytes")
    return int(out.value)


def sdd_accept_scratch_bytes(rows: int, gamma: int, V: int) -> int:
    return int(lib().sdd_accept_scratch_bytes(rows, gamma, V))


def sdd_accept_logits(logits_p, logits_q, draft_ids, temp_p: float, temp_q: float, seed: int, rnd: int,
                      scratch=None, stream=None):
    """logits_p [rows, gamma+1, V] fp32, logits_q [rows, gamma, V] fp32, draft_ids [rows, gamma] int32, all CUDA
    tensors.  Returns (n_accept [rows], out_ids [rows, gamma+1], accept_prob [rows, gamma])."""
    torch = _torch()
    rows, g1, V = logits_p.shape
    gamma = g1 - 1
    assert logits_q.shape == (rows, gamma, V) and draft_ids.shape == (rows, gamma)
    assert logits_p.is_contiguous() and logits_q.is_contiguous() and draft_ids.is_contiguous()
    assert logits_p.dtype == torch.float32 and logits_q.dtype == torch.float32 and draft_ids.dtype == torch.int32
    dev = logits_p.device
    n_accept = torch.empty(rows, dtype=torch.int32, device=dev)
    out_ids = torch.empty(rows, gamma + 1, dtype=torch.int32, device=dev)
    prob = torch.empty(rows, gamma, dtype=torch.float32, device=dev)
    if scratch is None:
        scratch = torch.empty(sdd_accept_scratch_bytes(rows, gamma, V), dtype=torch.uint8, device=dev)
    st = stream if stream is not None else torch.cuda.current_stream(dev)
    _check(lib().sdd_accept_logits(logits_p.data_ptr(), logits_q.data_ptr(), draft_ids.data_ptr(), rows, gamma, V,
                                   float(temp_p), float(temp_q), int(seed), int(rnd), n_accept.data_ptr(),
                                   out_ids.data_ptr(), prob.data_ptr(), scratch.data_ptr(), st.cuda_stream),
           "sdd_accept_logits")
    return n_accept, out_ids, prob


ACCEPT_STATIC_SCRATCH_BYTES = 2 << 20


def sdd_accept_logits_static(logits_p, logits_q, draft_ids, n_accept, out_ids, accept_prob, temp_p: float,
                             temp_q: float, seed: int, rnd: int, stream=None):
    """sdd_accept_logits for callers that must not allocate on the device: the scratch is a fixed array inside
    the library, and this wrapper allocates nothing either -- inputs AND outputs are the caller's CUDA tensors
    (n_accept [rows] int32, out_ids [rows, gamma+1] int32, accept_prob [rows, gamma] fp32).  Problems whose
    statistics do not fit ACCEPT_STATIC_SCRATCH_BYTES raise SddError(SDD_E_WORKSPACE).  Calls that may overlap on
    the GPU share the scratch and race; make the first call on a device outside stream capture."""
    torch = _torch()
    rows, g1, V = logits_p.shape
    gamma = g1 - 1
    assert logits_q.shape == (rows, gamma, V) and draft_ids.shape == (rows, gamma)
    assert n_accept.shape == (rows,) and out_ids.shape == (rows, gamma + 1) and accept_prob.shape == (rows, gamma)
    for t in (logits_p, logits_q, draft_ids, n_accept, out_ids, accept_prob):
        assert t.is_cuda and t.is_contiguous()
    assert logits_p.dtype == torch.float32 and logits_q.dtype == torch.float32 and accept_prob.dtype == torch.float32
    assert draft_ids.dtype == torch.int32 and n_accept.dtype == torch.int32 and out_ids.dtype == torch.int32
    st = stream if stream is not None else torch.cuda.current_stream(logits_p.device)
    _check(lib().sdd_accept_logits_static(logits_p.data_ptr(), logits_q.data_ptr(), draft_ids.data_ptr(), rows, gamma,
                                          V, float(temp_p), float(temp_q), int(seed), int(rnd), n_accept.data_ptr(),
                                          out_ids.data_ptr(), accept_prob.data_ptr(), st.cuda_stream),
           "sdd_accept_logits_static")


def sdd_debug_gemm_bf16(A, W, bias, M: int, epilogue: int, out, n_tile: int = 0, use_tensor_cores: bool = True,
                        status=None, stream=None, A_lo=None, out_lo=None):
    """out = epilogue((A[:M] + A_lo[:M]) @ W.T + bias) with the library's bf16 GEMM; A [cap, K], W [N, K] bf16 CUDA
    tensors; out_lo (bf16 epilogues) receives the rounding remainder of out."""
    torch = _torch()
    cap, K = A.shape
    N = W.shape[0]
    st = stream if stream is not None else torch.cuda.current_stream(A.device)
    _check(lib().sdd_debug_gemm_bf16(A.data_ptr(), cap, W.data_ptr(), bias.data_ptr() if bias is not None else None, M, N,
                                     K, epilogue, out.data_ptr(), out.stride(0), n_tile, 1 if use_tensor_cores else 0,
                                     status.data_ptr() if status is not None else None, st.cuda_stream,
                                     A_lo.data_ptr() if A_lo is not None else None,
                                     out_lo.data_ptr() if out_lo is not None else None),
           "sdd_debug_gemm_bf16")


def sdd_debug_attention_bf16(q, q_col0, k, k_col0, k_rows_per_seq, vt, out, ctx_len, batch, n_head, gamma, mode,
                             q_rows_per_seq, status=None, stream=None):
    """The library's tensor-core attention on caller tensors (see include/sdd.h for the layouts)."""
    torch = _torch()
    st = stream if stream is not None else torch.cuda.current_stream(q.device)
    _check(lib().sdd_debug_attention_bf16(q.data_ptr(), q.shape[0], q.stride(0), q_col0, k.data_ptr(), k.shape[0],
                                          k.stride(0), k_col0, k_rows_per_seq, vt.data_ptr(), vt.stride(0),
                                          out.data_ptr(), out.stride(0), ctx_len.data_ptr(), batch, n_head, gamma, mode,
                                          q_rows_per_seq, status.data_ptr() if status is not None else None,
                                          st.cuda_stream), "sdd_debug_attention_bf16")


def sdd_debug_wait_timeout(limit_cycles: int, status, stream=None):
    """Runs the library's one-CTA probe whose bounded waits run out after `limit_cycles` SM clocks; `status` (int32
    CUDA tensor holding 0) then holds 1."""
    torch = _torch()
    st = stream if stream is not None else torch.cuda.current_stream(status.device)
    _check(lib().sdd_debug_wait_timeout(int(limit_cycles), status.data_ptr(), st.cuda_stream), "sdd_debug_wait_timeout")


_TAP_DTYPES = {TAP_STEP_LOGITS: "f", TAP_Q_LOGITS: "f", TAP_LOGQ: "f", TAP_LOGITS_P: "f", TAP_ACCEPT_PROB: "f"}


class Session:
    """One generation: owns the workspace tensor and the sdd_ctx handle."""

    def __init__(self, target: DeviceModel, drafter: DeviceModel, prompts: np.ndarray, prompt_len: Sequence[int],
                 gamma: int, T: int, max_new: int, temp_p: float = 1.0, temp_q: float = 1.0, seed: int = 0,
                 device="cuda:0", stream=None):
        torch = _torch()
        self.torch = torch
        self.device = torch.device(device)
        # a stream of its own by default: the library replays whole rounds as CUDA graphs, which the legacy
        # default stream cannot capture.  Results are read after sdd_sync_status(), or on this stream.
        self.stream = stream if stream is not None else torch.cuda.Stream(self.device)
        prompts = np.ascontiguousarray(prompts, dtype=np.int32)
        self.batch, self.prompt_stride = prompts.shape
        self.gamma, self.T, self.max_new, self.V = gamma, T, max_new, target.shape.vocab
        self.tok_stride = min(target.shape.n_ctx, drafter.shape.n_ctx)
        self.params = sdd_params(gamma, T, self.batch, max_new, temp_p, temp_q, seed, self.stream.cuda_stream)
        self.target, self.drafter = target, drafter
        nbytes = sdd_workspace_bytes(target, drafter, self.params)
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        self.prompts_dev = torch.from_numpy(prompts).to(self.device)
        plen = (C.c_int32 * self.batch)(*[int(x) for x in prompt_len])
        h = C.c_void_p(0)
        _check(lib().sdd_create(C.byref(target.c), C.byref(drafter.c), C.byref(self.params), self.prompts_dev.data_ptr(),
                                self.prompt_stride, plen, self.workspace.data_ptr(), nbytes, C.byref(h)), "sdd_create")
        self.h = h
        self.out_ids = torch.empty(self.batch, gamma + 1, dtype=torch.int32, device=self.device)
        self.n_out = torch.empty(self.batch, dtype=torch.int32, device=self.device)

    def sdd_reset(self, prompts: np.ndarray, prompt_len: Sequence[int]):
        """New prompts, same context (graphs, workspace and models are kept)."""
        prompts = np.ascontiguousarray(prompts, dtype=np.int32)
        assert prompts.shape[0] == self.batch
        self.prompts_dev = self.torch.from_numpy(prompts).to(self.device)
        plen = (C.c_int32 * self.batch)(*[int(x) for x in prompt_len])
        _check(lib().sdd_reset(self.h, self.prompts_dev.data_ptr(), prompts.shape[1], plen), "sdd_reset")

    # --- the C ABI calls --------------------------------------------------------------------
    def sdd_draft_begin(self): _check(lib().sdd_draft_begin(self.h), "sdd_draft_begin")
    def sdd_draft_step(self): _check(lib().sdd_draft_step(self.h), "sdd_draft_step")
    def sdd_draft(self): _check(lib().sdd_draft(self.h), "sdd_draft")

    def sdd_verify_accept(self):
        _check(lib().sdd_verify_accept(self.h, self.out_ids.data_ptr(), self.n_out.data_ptr()), "sdd_verify_accept")

    def sdd_step(self, out_ids=None, n_out=None):
        """One round.  out_ids [batch, gamma + 1] / n_out [batch] int32: where the emitted ids go (default: the
        session's device tensors).  Page-locked host tensors work too (the commit kernel then writes the ids
        straight into host memory; they are complete once sdd_progress() counts the round)."""
        o = self.out_ids if out_ids is None else out_ids
        n = self.n_out if n_out is None else n_out
        _check(lib().sdd_step(self.h, o.data_ptr(), n.data_ptr()), "sdd_step")

    def sdd_ar_step(self):
        """One plain autoregressive token per sequence (emitted ids in self.ar_ids [batch])."""
        if not hasattr(self, "ar_ids"):
            self.ar_ids = self.torch.empty(self.batch, dtype=self.torch.int32, device=self.device)
        _check(lib().sdd_ar_step(self.h, self.ar_ids.data_ptr(), self.n_out.data_ptr()), "sdd_ar_step")

    def sdd_sps_attach(self, ar_drafter: DeviceModel):
        """Attach the autoregressive drafter of the speculative-decoding warm start (right after construction)."""
        n = C.c_uint64(0)
        _check(lib().sdd_sps_workspace_bytes(C.byref(ar_drafter.c), C.byref(self.params), C.byref(n)), "sdd_sps_workspace_bytes")
        self.ar_drafter = ar_drafter
        self.ar_workspace = self.torch.empty(int(n.value), dtype=self.torch.uint8, device=self.device)
        _check(lib().sdd_sps_attach(self.h, C.byref(ar_drafter.c), self.ar_workspace.data_ptr(), int(n.value)), "sdd_sps_attach")

    def sdd_sps_step(self, gamma_sps: int):
        """One speculative-decoding round with the attached drafter (emitted ids in self.out_ids[:, :gamma_sps + 1])."""
        if getattr(self, "sps_ids", None) is None or self.sps_ids.shape[1] != gamma_sps + 1:
            self.sps_ids = self.torch.empty(self.batch, gamma_sps + 1, dtype=self.torch.int32, device=self.device)
        _check(lib().sdd_sps_step(self.h, gamma_sps, self.sps_ids.data_ptr(), self.n_out.data_ptr()), "sdd_sps_step")

    def sdd_sync_status(self): _check(lib().sdd_sync_status(self.h), "sdd_sync_status")

    def sdd_progress(self):
        r, e = C.c_uint64(0), C.c_int32(0)
        _check(lib().sdd_progress(self.h, C.byref(r), C.byref(e)), "sdd_progress")
        return int(r.value), int(e.value)

    def sdd_counters(self):
        r, k = C.c_uint64(0), C.c_uint64(0)
        _check(lib().sdd_counters(self.h, C.byref(r), C.byref(k)), "sdd_counters")
        return int(r.value), int(k.value)

    def sdd_profile_begin(self): _check(lib().sdd_profile_begin(self.h), "sdd_profile_begin")

    def sdd_profile_end(self):
        """{category name: (milliseconds, launches)} since sdd_profile_begin."""
        ms = (C.c_double * len(PROF_NAMES))()
        n = (C.c_uint64 * len(PROF_NAMES))()
        _check(lib().sdd_profile_end(self.h, ms, n, len(PROF_NAMES)), "sdd_profile_end")
        return {name: (float(ms[i]), int(n[i])) for i, name in enumerate(PROF_NAMES)}

    def sdd_tap(self, what: int):
        """Device view of a workspace buffer as a flat torch tensor (no copy)."""
        torch = self.torch
        p, n = C.c_void_p(0), C.c_uint64(0)
        _check(lib().sdd_tap(self.h, what, C.byref(p), C.byref(n)), "sdd_tap")
        off = p.value - self.workspace.data_ptr()
        raw = self.workspace[off: off + n.value]
        return raw.view(torch.float32 if what in _TAP_DTYPES else torch.int32)

    def tap_numpy(self, what: int) -> np.ndarray:
        self.sdd_sync_status()
        return self.sdd_tap(what).cpu().numpy()

    def generate(self):
        """Run rounds until every sequence has max_new tokens; returns the token matrix [batch, tok_stride]
        and the context lengths (host)."""
        while True:
            self.sdd_step()
            _, emitted = self.sdd_progress()
            if emitted >= self.max_new:
                break
        self.sdd_sync_status()
        toks = self.sdd_tap(TAP_TOKENS).view(self.batch, self.tok_stride).cpu().numpy()
        return toks, self.sdd_tap(TAP_CTX_LEN).cpu().numpy()

    def close(self):
        if getattr(self, "h", None) is not None and self.h.value:
            lib().sdd_destroy(self.h)
            self.h = C.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
