"""ctypes binding of the C-ABI library declared in ``include/tf.h``.

Argument marshalling only: every step of the layer runs in the CUDA kernels of
``libtokenfilter.so``.  torch supplies device memory and the current stream.
There is no fallback -- if the library is missing, loading raises.

Tensors are token-major ``[B, S, H, 128]`` (any strides whose last dim is dense).
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtokenfilter.so")

TF_OK, TF_ERR_INVALID_ARG, TF_ERR_UNSUPPORTED, TF_ERR_WORKSPACE, TF_ERR_CUDA, TF_ERR_TIMEOUT, TF_ERR_NAN_SCORE = range(7)
TF_F32, TF_BF16 = 0, 1
TF_ANCHOR_PAST_MEAN, TF_ANCHOR_INCL_MEAN, TF_ANCHOR_EMA = 0, 1, 2
TF_FUSE_INVVAR, TF_FUSE_EQ2_LITERAL, TF_FUSE_KEY_ONLY, TF_FUSE_VALUE_ONLY, TF_FUSE_MEAN = 0, 1, 2, 3, 4
TF_SELECT_RATIO, TF_SELECT_THRESHOLD = 0, 1
TF_KV_ALL, TF_KV_RETAINED = 0, 1
TF_STATIC_SCRATCH_BYTES = 8 << 20
(TF_KERNEL_NONE, TF_KERNEL_SCAN_PLAIN, TF_KERNEL_SCAN_GRAM_TILE, TF_KERNEL_SCAN_GRAM_PERSISTENT) = range(4)
TF_KERNEL_ATTN_SIMT, TF_KERNEL_ATTN_TC_SHARED, TF_KERNEL_ATTN_TC_SPLIT, TF_KERNEL_ATTN_TC_SINGLE = 10, 11, 12, 13
TF_KERNEL_ATTN_TC_HEAD_PAIR, TF_KERNEL_ATTN_TC_HEAD_QUAD = 14, 15

EXPORTS = ("tf_default_params", "tf_create", "tf_destroy", "tf_workspace_bytes", "tf_set_workspace",
           "tf_kv_stats", "tf_kv_stats_static", "tf_score_fuse", "tf_select", "tf_pruned_attention", "tf_layer_filter",
           "tf_layer_filter_host", "tf_get_status", "tf_clear_status", "tf_set_attention_path",
           "tf_status_string", "tf_tail_policy", "tf_decode_step", "tf_set_scan_path", "tf_last_kernels",
           "tf_set_wait_limits", "tf_wait_selftest", "tf_score_select", "tf_set_select_path")


class tf_shape(C.Structure):
    _fields_ = [("batch", C.c_int32), ("seq", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("dtype", C.c_int32),
                ("q_stride", C.c_int64 * 3), ("k_stride", C.c_int64 * 3),
                ("v_stride", C.c_int64 * 3), ("o_stride", C.c_int64 * 3),
                ("window", C.c_int32), ("softmax_scale", C.c_float)]


class tf_filter_params(C.Structure):
    _fields_ = [("prune_ratio", C.c_double), ("warmup_tokens", C.c_int32),
                ("eligible", C.c_void_p), ("anchor_mode", C.c_int32), ("gamma", C.c_float),
                ("fuse_mode", C.c_int32), ("var_eps", C.c_float), ("select_mode", C.c_int32),
                ("threshold", C.c_void_p), ("kv_visibility", C.c_int32)]


class tf_carry(C.Structure):
    _fields_ = [("sum_k_in", C.c_void_p), ("sum_v_in", C.c_void_p), ("count_in", C.c_void_p),
                ("sum_k_out", C.c_void_p), ("sum_v_out", C.c_void_p)]


class tf_decode_state(C.Structure):
    _fields_ = [("sum_k", C.c_void_p), ("sum_v", C.c_void_p), ("count", C.c_void_p),
                ("tau", C.c_void_p), ("steps", C.c_void_p), ("skips", C.c_void_p)]


class TokenFilterError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {status_string(code)} (tf_status {code})")
        self.code = code


_lib = None


def lib() -> C.CDLL:
    """Load the CUDA library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with __graft_entry__.build() "
                               "(python -m paper_2512_07090_b200.build); there is no CPU fallback")
        L = C.CDLL(LIB_PATH)
        for name in EXPORTS:
            getattr(L, name).restype = C.c_int
        L.tf_default_params.restype = None
        L.tf_status_string.restype = C.c_char_p
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().tf_status_string(C.c_int(code)).decode()


def _check(code: int, what: str) -> None:
    if code != TF_OK:
        raise TokenFilterError(code, what)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def default_params(**kw) -> tf_filter_params:
    p = tf_filter_params()
    lib().tf_default_params(C.byref(p))
    for k, v in kw.items():
        if k in ("eligible", "threshold"):
            v = None if v is None else v.data_ptr()
        setattr(p, k, v)
    return p


def make_shape(Q: Optional[torch.Tensor], K: torch.Tensor, V: torch.Tensor, O: Optional[torch.Tensor] = None,
               window: int = 0, softmax_scale: float = 0.0, n_q_heads: Optional[int] = None) -> tf_shape:
    """Describe ``[B,S,H,128]`` tensors (element strides of batch, token, head)."""
    B, S, Hkv, d = K.shape
    s = tf_shape()
    s.batch, s.seq, s.n_kv_heads, s.head_dim = B, S, Hkv, d
    s.n_q_heads = Q.shape[2] if Q is not None else (n_q_heads or Hkv)
    s.dtype = {torch.float32: TF_F32, torch.bfloat16: TF_BF16}[K.dtype]
    for name, t in (("q_stride", Q), ("k_stride", K), ("v_stride", V), ("o_stride", O if O is not None else Q)):
        if t is None:
            t = K
        assert t.stride(3) == 1, "head_dim must be contiguous"
        getattr(s, name)[:] = [t.stride(0), t.stride(1), t.stride(2)]
    s.window, s.softmax_scale = int(window), float(softmax_scale)
    return s


def tail_policy(p_global: float, tail_fraction: float, n_layers: int):
    """Per-layer pruning ratios of the tail-focused policy (host helper); returns (ratios, n_tail)."""
    out = (C.c_double * n_layers)()
    n_tail = C.c_int32()
    _check(lib().tf_tail_policy(C.c_double(p_global), C.c_double(tail_fraction), C.c_int32(n_layers), out,
                                C.byref(n_tail)), "tf_tail_policy")
    return list(out), int(n_tail.value)


class DecodeState:
    """Device tensors of the decode-step state and the struct that points at them."""

    def __init__(self, B: int, Hkv: int, device, tau0: float = 0.0):
        self.sum_k = torch.zeros(B, Hkv, 128, device=device)
        self.sum_v = torch.zeros(B, Hkv, 128, device=device)
        self.count = torch.zeros(B, dtype=torch.int64, device=device)
        self.tau = torch.full((B,), float(tau0), device=device)
        self.steps = torch.zeros(B, dtype=torch.int64, device=device)
        self.skips = torch.zeros(B, dtype=torch.int64, device=device)
        self.struct = tf_decode_state(*(t.data_ptr() for t in (self.sum_k, self.sum_v, self.count, self.tau,
                                                               self.steps, self.skips)))


class Context:
    """Owns a tf_ctx and (optionally) a torch-allocated workspace bound to it."""

    def __init__(self, device: int = 0):
        self._h = C.c_void_p()
        _check(lib().tf_create(C.byref(self._h), C.c_int(device)), "tf_create")
        self.device = device
        self._ws = None

    def close(self):
        if self._h:
            lib().tf_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- workspace -----------------------------------------------------------------------------
    def workspace_bytes(self, shape: tf_shape, params: tf_filter_params) -> int:
        n = C.c_size_t()
        _check(lib().tf_workspace_bytes(C.byref(shape), C.byref(params), C.byref(n)), "tf_workspace_bytes")
        return int(n.value)

    def set_workspace(self, buf: Optional[torch.Tensor]) -> None:
        self._ws = buf
        _check(lib().tf_set_workspace(self._h, _ptr(buf), C.c_size_t(0 if buf is None else buf.numel() * buf.element_size())),
               "tf_set_workspace")

    def ensure_workspace(self, shape: tf_shape, params: tf_filter_params) -> None:
        need = self.workspace_bytes(shape, params)
        if self._ws is None or self._ws.numel() < need:
            self.set_workspace(torch.empty(need, dtype=torch.uint8, device=f"cuda:{self.device}"))

    # ---- the five entry points -----------------------------------------------------------------
    def tf_kv_stats(self, shape, params, K, V, sim_k, sim_v, carry: Optional[tf_carry] = None):
        _check(lib().tf_kv_stats(self._h, C.byref(shape), C.byref(params), _ptr(K), _ptr(V), _ptr(sim_k),
                                 _ptr(sim_v), None if carry is None else C.byref(carry), _stream()), "tf_kv_stats")

    def tf_kv_stats_static(self, shape, params, K, V, sim_k, sim_v, carry: Optional[tf_carry] = None):
        """tf_kv_stats on the library's built-in scratch array: no workspace, nothing allocated."""
        _check(lib().tf_kv_stats_static(self._h, C.byref(shape), C.byref(params), _ptr(K), _ptr(V), _ptr(sim_k),
                                        _ptr(sim_v), None if carry is None else C.byref(carry), _stream()),
               "tf_kv_stats_static")

    def tf_score_fuse(self, shape, params, sim_k, sim_v, score):
        _check(lib().tf_score_fuse(self._h, C.byref(shape), C.byref(params), _ptr(sim_k), _ptr(sim_v),
                                   _ptr(score), _stream()), "tf_score_fuse")

    def tf_select(self, shape, params, score, keep_mask, kept_idx, n_kept, theta=None):
        _check(lib().tf_select(self._h, C.byref(shape), C.byref(params), _ptr(score), _ptr(keep_mask),
                               _ptr(kept_idx), _ptr(n_kept), _ptr(theta), _stream()), "tf_select")

    def tf_score_select(self, shape, params, sim_k, sim_v, score, keep_mask, kept_idx, n_kept, theta=None):
        _check(lib().tf_score_select(self._h, C.byref(shape), C.byref(params), _ptr(sim_k), _ptr(sim_v), _ptr(score),
                                     _ptr(keep_mask), _ptr(kept_idx), _ptr(n_kept), _ptr(theta), _stream()), "tf_score_select")

    def tf_pruned_attention(self, shape, params, Q, K, V, kept_idx, n_kept, O):
        _check(lib().tf_pruned_attention(self._h, C.byref(shape), C.byref(params), _ptr(Q), _ptr(K), _ptr(V),
                                         _ptr(kept_idx), _ptr(n_kept), _ptr(O), _stream()), "tf_pruned_attention")

    def tf_layer_filter(self, shape, params, Q, K, V, O, score=None, keep_mask=None, kept_idx=None, n_kept=None):
        _check(lib().tf_layer_filter(self._h, C.byref(shape), C.byref(params), _ptr(Q), _ptr(K), _ptr(V), _ptr(O),
                                     _ptr(score), _ptr(keep_mask), _ptr(kept_idx), _ptr(n_kept), _stream()),
               "tf_layer_filter")

    def tf_decode_step(self, shape, params, eta, q_new, K_cache, V_cache, pos, state: "DecodeState", O_new,
                       score=None, skip=None, alg1_sign=False):
        _check(lib().tf_decode_step(self._h, C.byref(shape), C.byref(params), C.c_float(eta),
                                    C.c_int32(1 if alg1_sign else 0), _ptr(q_new), _ptr(K_cache), _ptr(V_cache),
                                    _ptr(pos), C.byref(state.struct), _ptr(O_new), _ptr(score), _ptr(skip), _stream()),
               "tf_decode_step")

    def tf_layer_filter_host(self, shape, params, Q, K, V, O, score=None, keep_mask=None, kept_idx=None, n_kept=None):
        """Host tensors in, host tensors out (copies inside the call; returns after the stream is idle)."""
        _check(lib().tf_layer_filter_host(self._h, C.byref(shape), C.byref(params), _ptr(Q), _ptr(K), _ptr(V),
                                          _ptr(O), _ptr(score), _ptr(keep_mask), _ptr(kept_idx), _ptr(n_kept),
                                          _stream()), "tf_layer_filter_host")

    # ---- status --------------------------------------------------------------------------------
    def tf_get_status(self, sync: bool = True):
        det = (C.c_int64 * 4)()
        code = lib().tf_get_status(self._h, C.c_int(1 if sync else 0), det)
        return code, dict(code=det[0], where=det[1], nan_count=det[2], launches=det[3])

    def tf_clear_status(self):
        _check(lib().tf_clear_status(self._h), "tf_clear_status")

    def tf_set_attention_path(self, path):
        """0 / False: CUDA-core kernel; 1 / True: tensor-core kernel (form chosen by size); 2: shared form; 3: split form;
        4: single form (one Q tile and one softmax group per CTA, two CTAs per SM); 5 / 6: two / four query heads of one
        KV group per CTA (grouped-query shapes)."""
        _check(lib().tf_set_attention_path(self._h, C.c_int(int(path))), "tf_set_attention_path")

    def tf_set_select_path(self, path: int):
        """0: choose; 1: selection by one CTA per sequence (fusion as its own launch); 2: fusion + selection by a cluster per sequence."""
        _check(lib().tf_set_select_path(self._h, C.c_int(int(path))), "tf_set_select_path")

    def tf_set_scan_path(self, path: int):
        """0: choose; 1: plain CUDA-core similarity scan; 2: Gram-matrix scan on the tensor cores (bf16 sums), one tile per CTA; 3: the same, persistent."""
        _check(lib().tf_set_scan_path(self._h, C.c_int(int(path))), "tf_set_scan_path")

    def tf_last_kernels(self):
        """(kernel of the latest similarity scan, kernel of the latest attention) as TF_KERNEL_* ids."""
        out = (C.c_int32 * 2)()
        _check(lib().tf_last_kernels(self._h, out), "tf_last_kernels")
        return int(out[0]), int(out[1])

    def tf_set_wait_limits(self, max_polls: int = -1, wait_cycles: int = -1):
        """Limits of the kernels' bounded waits (negative: the default, about a second)."""
        _check(lib().tf_set_wait_limits(self._h, C.c_int64(int(max_polls)), C.c_int64(int(wait_cycles))),
               "tf_set_wait_limits")

    def tf_wait_selftest(self):
        """Make bounded waits run out on purpose (conditions nothing ever fulfils); tf_get_status then says TF_ERR_TIMEOUT."""
        _check(lib().tf_wait_selftest(self._h, _stream()), "tf_wait_selftest")

    @property
    def launches(self) -> int:
        return self.tf_get_status(sync=False)[1]["launches"]
