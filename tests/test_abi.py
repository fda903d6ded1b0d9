"""The C-ABI library loads and exports every function that include/sdd.h declares (no compute calls)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "sdd.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(sdd_[a-z0-9_]+)\s*\(", src)))


def test_header_symbols_are_exported_and_bound():
    import paper_2408_05636_b200 as sdd
    names = _declared()
    assert "sdd_create" in names and "sdd_draft" in names and "sdd_verify_accept" in names and "sdd_step" in names
    L = sdd.lib()
    for n in names:
        assert hasattr(L, n), n
    assert sorted(sdd.EXPORTS) == names


def test_host_only_calls():
    import paper_2408_05636_b200 as sdd
    L = sdd.lib()
    assert L.sdd_strerror(0) == b"ok"
    assert b"argument" in L.sdd_strerror(sdd.SDD_E_ARG)
    assert L.sdd_accept_scratch_bytes(64, 32, 50257) == 64 * 65 * 7 * 8
    out = ctypes.c_uint64(0)
    assert L.sdd_workspace_bytes(None, None, None, ctypes.byref(out)) == sdd.SDD_E_ARG
    assert L.sdd_draft(None) == sdd.SDD_E_ARG and L.sdd_step(None, None, None) == sdd.SDD_E_ARG
    assert L.sdd_accept_logits(None, None, None, 1, 1, 8, 1.0, 1.0, 0, 0, None, None, None, None, None) == sdd.SDD_E_ARG


def test_workspace_size_model(tmp_path):
    """sdd_workspace_bytes is a host computation: check it against the documented buffer list."""
    import numpy as np
    import synth
    import paper_2408_05636_b200 as sdd
    wl = synth.WORKLOADS["tiny_fp32"]
    fake = np.zeros(64, dtype=np.uint8)
    addr = fake.ctypes.data & ~15

    def model(shape):
        n = 2 + 12 * shape.n_layer + 2
        ptrs = (ctypes.c_void_p * n)(*([addr + 16] * n))
        m = sdd.sdd_model(shape.vocab, shape.n_layer, shape.d_model, shape.n_head, shape.n_ctx,
                          1 if shape.causal else 0, sdd.SDD_FP32, ctypes.cast(ptrs, ctypes.POINTER(ctypes.c_void_p)), n)
        m._keep = ptrs
        return m

    mp, mq = model(wl.target), model(wl.drafter)
    prm = sdd.sdd_params(wl.gamma, wl.T, 1, wl.max_new, 1.0, 1.0, 1, None)
    out = ctypes.c_uint64(0)
    assert sdd.lib().sdd_workspace_bytes(ctypes.byref(mp), ctypes.byref(mq), ctypes.byref(prm), ctypes.byref(out)) == 0
    V, G = wl.target.vocab, wl.gamma
    logits = (2 * G + (G + 1)) * V * 4
    kv = wl.target.n_layer * wl.target.n_ctx * 2 * wl.target.d_model * 4
    assert out.value > logits + kv and out.value < 4 * (logits + kv) + (64 << 20)
    prm.gamma = 0
    assert sdd.lib().sdd_workspace_bytes(ctypes.byref(mp), ctypes.byref(mq), ctypes.byref(prm), ctypes.byref(out)) == sdd.SDD_E_ARG
