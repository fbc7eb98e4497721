"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, and validates arguments before touching the device."""
import ctypes as C
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2512_07090_b200 import binding as tfb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    entry.build()
    return tfb.lib()


def test_every_declared_symbol_is_exported(L):
    hdr = open(os.path.join(ROOT, "include", "tf.h")).read()
    declared = set(re.findall(r"\b(tf_[a-z_]+)\s*\(", hdr))
    declared -= {"tf_ctx"}
    assert declared, "no declarations found"
    for name in sorted(declared):
        assert hasattr(L, name), f"{name} declared in tf.h but not exported"
    assert declared == set(tfb.EXPORTS) | {n for n in declared if n not in tfb.EXPORTS}
    assert set(tfb.EXPORTS) <= declared


def test_struct_layouts_match_the_header():
    assert C.sizeof(tfb.tf_shape) == 6 * 4 + 12 * 8 + 4 + 4
    assert C.sizeof(tfb.tf_carry) == 5 * 8
    p = tfb.default_params()
    assert p.prune_ratio == 0.5 and p.warmup_tokens == 1 and p.anchor_mode == tfb.TF_ANCHOR_PAST_MEAN
    assert p.fuse_mode == tfb.TF_FUSE_INVVAR and p.select_mode == tfb.TF_SELECT_RATIO
    assert abs(p.gamma - 0.9) < 1e-7 and abs(p.var_eps - 1e-8) < 1e-15 and p.kv_visibility == tfb.TF_KV_ALL


def _shape(B=2, S=100, Hq=8, Hkv=2, d=128, dtype=tfb.TF_BF16):
    s = tfb.tf_shape()
    s.batch, s.seq, s.n_q_heads, s.n_kv_heads, s.head_dim, s.dtype = B, S, Hq, Hkv, d, dtype
    s.q_stride[:] = [S * Hq * d, Hq * d, d]
    s.o_stride[:] = [S * Hq * d, Hq * d, d]
    s.k_stride[:] = [S * Hkv * d, Hkv * d, d]
    s.v_stride[:] = [S * Hkv * d, Hkv * d, d]
    return s


def test_workspace_bytes_and_shape_validation(L):
    n = C.c_size_t()
    p = tfb.default_params()
    assert L.tf_workspace_bytes(C.byref(_shape()), C.byref(p), C.byref(n)) == tfb.TF_OK
    small = n.value
    assert small > 0 and small % 256 == 0
    assert L.tf_workspace_bytes(C.byref(_shape(S=4000)), C.byref(p), C.byref(n)) == tfb.TF_OK
    assert n.value > small
    assert L.tf_workspace_bytes(C.byref(_shape(d=64)), C.byref(p), C.byref(n)) == tfb.TF_ERR_UNSUPPORTED
    assert L.tf_workspace_bytes(C.byref(_shape(Hq=6, Hkv=4)), C.byref(p), C.byref(n)) == tfb.TF_ERR_INVALID_ARG
    assert L.tf_workspace_bytes(C.byref(_shape(dtype=7)), C.byref(p), C.byref(n)) == tfb.TF_ERR_UNSUPPORTED
    assert L.tf_workspace_bytes(None, C.byref(p), C.byref(n)) == tfb.TF_ERR_INVALID_ARG
    assert L.tf_workspace_bytes(C.byref(_shape()), C.byref(p), None) == tfb.TF_ERR_INVALID_ARG


def test_null_context_and_status_strings(L):
    s, p = _shape(), tfb.default_params()
    assert L.tf_kv_stats(None, C.byref(s), C.byref(p), None, None, None, None, None, None) == tfb.TF_ERR_INVALID_ARG
    assert L.tf_layer_filter(None, C.byref(s), C.byref(p), *([None] * 9)) == tfb.TF_ERR_INVALID_ARG
    assert L.tf_get_status(None, 0, None) == tfb.TF_ERR_INVALID_ARG
    assert L.tf_destroy(None) == tfb.TF_OK
    texts = {tfb.status_string(c) for c in range(7)}
    assert len(texts) == 7 and "ok" in texts


def test_no_cpu_fallback_exists():
    """The binding has nothing to fall back to: without the built library, loading raises."""
    import importlib
    saved, tfb._lib = tfb._lib, None
    path = tfb.LIB_PATH
    try:
        tfb.LIB_PATH = path + ".absent"
        with pytest.raises(RuntimeError):
            tfb.lib()
    finally:
        tfb.LIB_PATH, tfb._lib = path, saved
    src = open(os.path.join(ROOT, "paper_2512_07090_b200", "binding.py")).read()
    assert "import oracle" not in src and "from oracle" not in src


def test_tail_policy_matches_the_oracle_and_rejects_bad_input(L):
    import oracle
    for pg, y, n in [(0.25, 0.5, 32), (0.2, 0.4, 40), (0.33, 0.6, 40), (0.1, 1.0, 7), (0.3, 0.37, 13)]:
        got, n_tail = tfb.tail_policy(pg, y, n)
        ref = oracle.tail_policy(pg, y, n)
        assert got == ref and n_tail == sum(1 for x in ref if x > 0)
    out = (C.c_double * 4)()
    for pg, y, n in [(0.6, 0.5, 4), (-0.1, 0.5, 4), (0.2, 0.0, 4), (0.2, 1.5, 4), (0.2, 0.5, 0)]:
        assert L.tf_tail_policy(C.c_double(pg), C.c_double(y), C.c_int32(n), out, None) == tfb.TF_ERR_INVALID_ARG
    assert L.tf_tail_policy(C.c_double(0.2), C.c_double(0.5), C.c_int32(4), None, None) == tfb.TF_ERR_INVALID_ARG
