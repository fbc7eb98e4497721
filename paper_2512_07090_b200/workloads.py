"""Seeded synthetic workloads shaped like the paper's LLaMA-2 / LLaMA-3 / Mistral runs.

This module only manufactures inputs (Q, K, V tensors and token ids).  It holds
none of the Token Filtering arithmetic and is the one module that both the CUDA
path's tests/benchmark and the CPU oracle's tests draw inputs from.  Nothing in
here comes from a dataset: the paper's evaluation suites are replaced by random
token ids with controlled repetition, pushed through a random-init decoder
stack of the right shape (Section 4.1 lists the model families).

All tensors are token-major ``[B, S, H, d]``.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, Iterator, List, Optional, Sequence, Tuple

import torch
import torch.nn.functional as F

BASE_SEED = 20251207


# ----------------------------------------------------------------------------------------------
# direct Q/K/V generator (config 1 and the reduced-size parity cases)
# ----------------------------------------------------------------------------------------------
def duplicate_qkv(B: int, S: int, Hq: int, Hkv: int, d: int = 128, dup_frac: float = 0.25,
                  noise: float = 0.05, seed: int = BASE_SEED, dtype=torch.float32
                  ) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """Q, K, V ~ N(0,1); a fraction ``dup_frac`` of positions (never position 0)
    are copies of a uniformly chosen earlier token plus N(0, noise^2), applied to
    Q, K and V alike in increasing position order (so copies of copies occur)."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    q = torch.randn(B, S, Hq, d, generator=g, dtype=torch.float32)
    k = torch.randn(B, S, Hkv, d, generator=g, dtype=torch.float32)
    v = torch.randn(B, S, Hkv, d, generator=g, dtype=torch.float32)
    n_dup = int(round(dup_frac * S)) if S > 1 else 0
    n_dup = min(n_dup, max(S - 1, 0))
    for b in range(B):
        if n_dup == 0:
            break
        pos = (torch.randperm(S - 1, generator=g)[:n_dup] + 1).sort().values.tolist()
        for t in pos:
            j = int(torch.randint(0, t, (1,), generator=g))
            q[b, t] = q[b, j] + noise * torch.randn(Hq, d, generator=g)
            k[b, t] = k[b, j] + noise * torch.randn(Hkv, d, generator=g)
            v[b, t] = v[b, j] + noise * torch.randn(Hkv, d, generator=g)
    return q.to(dtype), k.to(dtype), v.to(dtype)


# ----------------------------------------------------------------------------------------------
# token-id recipes
# ----------------------------------------------------------------------------------------------
def ids_with_repeats(B: int, S: int, vocab: int, frac: float, seed: int) -> torch.Tensor:
    """Uniform ids; ``frac`` of positions repeat the id at a uniformly chosen earlier position."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    ids = torch.randint(0, vocab, (B, S), generator=g)
    for b in range(B):
        n = int(frac * S)
        pos = (torch.randperm(S - 1, generator=g)[:n] + 1).sort().values
        src = (torch.rand(n, generator=g) * pos.double()).long()
        for t, j in zip(pos.tolist(), src.tolist()):
            ids[b, t] = ids[b, j]
    return ids


def ids_zipf(B: int, S: int, vocab: int, a: float, seed: int) -> torch.Tensor:
    """Ids whose rank follows Zipf(a) over 1..vocab, through a seeded rank->id permutation."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    w = torch.arange(1, vocab + 1, dtype=torch.float64).pow(-a)
    ranks = torch.multinomial(w / w.sum(), B * S, replacement=True, generator=g)
    perm = torch.randperm(vocab, generator=g)
    return perm[ranks].reshape(B, S)


def ids_with_copied_spans(B: int, S: int, vocab: int, frac: float, seed: int,
                          span_lo: int = 16, span_hi: int = 256, redraw: float = 0.05) -> torch.Tensor:
    """Uniform ids; then spans (length uniform in [span_lo, span_hi]) covering about ``frac`` of
    the positions are overwritten by a copy of an earlier span, 5% of the copied ids re-drawn."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    ids = torch.randint(0, vocab, (B, S), generator=g)
    for b in range(B):
        covered, guard = 0, 0
        while covered < frac * S and guard < 100000:
            guard += 1
            L = int(torch.randint(span_lo, span_hi + 1, (1,), generator=g))
            if S < 2 * L + 1:
                L = max(1, S // 4)
            dst = int(torch.randint(L, S - L + 1, (1,), generator=g))
            src = int(torch.randint(0, dst - L + 1, (1,), generator=g))
            seg = ids[b, src:src + L].clone()
            flip = torch.rand(L, generator=g) < redraw
            seg[flip] = torch.randint(0, vocab, (int(flip.sum()),), generator=g)
            ids[b, dst:dst + L] = seg
            covered += L
    return ids


# ----------------------------------------------------------------------------------------------
# random-init decoder stack: produces the per-layer Q, K, V the filter layer sees
# ----------------------------------------------------------------------------------------------
@dataclass
class StackShape:
    name: str
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    n_layers: int
    rope_theta: float
    vocab: int
    window: int = 0
    rms_eps: float = 1e-5


def _rope(x: torch.Tensor, theta: float) -> torch.Tensor:
    """Rotary embedding (rotate-half form) over ``[B,S,H,d]``, positions 0..S-1."""
    B, S, H, d = x.shape
    inv = 1.0 / (theta ** (torch.arange(0, d, 2, device=x.device, dtype=torch.float32) / d))
    ang = torch.arange(S, device=x.device, dtype=torch.float32)[:, None] * inv[None, :]
    cos = torch.cat([ang.cos(), ang.cos()], -1)[None, :, None, :]
    sin = torch.cat([ang.sin(), ang.sin()], -1)[None, :, None, :]
    xf = x.float()
    rot = torch.cat([-xf[..., d // 2:], xf[..., : d // 2]], -1)
    return (xf * cos + rot * sin).to(x.dtype)


def _rms(x: torch.Tensor, eps: float) -> torch.Tensor:
    xf = x.float()
    return (xf * torch.rsqrt(xf.pow(2).mean(-1, keepdim=True) + eps)).to(x.dtype)


def _dense_attention(q, k, v, window: int) -> torch.Tensor:
    """Unpruned causal attention of the generator stack (torch SDPA); [B,S,H,d] in and out."""
    B, S, Hq, d = q.shape
    g = Hq // k.shape[2]
    qt = q.transpose(1, 2)
    kt = k.repeat_interleave(g, dim=2).transpose(1, 2)
    vt = v.repeat_interleave(g, dim=2).transpose(1, 2)
    if window <= 0 or window >= S:
        o = F.scaled_dot_product_attention(qt, kt, vt, is_causal=True)
    else:
        o = torch.empty_like(qt)
        blk = window
        for s0 in range(0, S, blk):
            s1 = min(S, s0 + blk)
            k0 = max(0, s0 - window + 1)
            qi = torch.arange(s0, s1, device=q.device)[:, None]
            kj = torch.arange(k0, s1, device=q.device)[None, :]
            mask = (kj <= qi) & (kj > qi - window)
            o[:, :, s0:s1] = F.scaled_dot_product_attention(qt[:, :, s0:s1], kt[:, :, k0:s1],
                                                            vt[:, :, k0:s1], attn_mask=mask)
    return o.transpose(1, 2)


class DecoderStack:
    """Random-init pre-norm decoder (RMSNorm, RoPE on Q and K, SwiGLU).  Weights are N(0, 0.02^2),
    drawn layer by layer from the seed and never stored, so 13B-shaped stacks fit anywhere."""

    def __init__(self, shape: StackShape, seed: int, device="cpu", dtype=torch.bfloat16):
        self.shape, self.seed, self.device, self.dtype = shape, seed, torch.device(device), dtype

    def _w(self, g, rows, cols):
        return (torch.randn(rows, cols, generator=g, device=self.device, dtype=torch.float32) * 0.02
                ).to(self.dtype)

    @torch.no_grad()
    def layer_qkv(self, ids: torch.Tensor, layers: Sequence[int]) -> Iterator[Tuple[int, torch.Tensor, torch.Tensor, torch.Tensor]]:
        """Yield (layer, Q, K, V) for the requested layers, in order.  Q/K are post-RoPE."""
        sh = self.shape
        want = sorted(set(int(l) for l in layers))
        g = torch.Generator(device=self.device).manual_seed(self.seed)
        emb = self._w(g, sh.vocab, sh.hidden)
        x = emb[ids.to(self.device)]
        del emb
        B, S = ids.shape
        for l in range(max(want) + 1):
            gl = torch.Generator(device=self.device).manual_seed(self.seed + 1000 + l)
            wq = self._w(gl, sh.hidden, sh.n_q_heads * sh.head_dim)
            wk = self._w(gl, sh.hidden, sh.n_kv_heads * sh.head_dim)
            wv = self._w(gl, sh.hidden, sh.n_kv_heads * sh.head_dim)
            h = _rms(x, sh.rms_eps)
            q = _rope((h @ wq).view(B, S, sh.n_q_heads, sh.head_dim), sh.rope_theta)
            k = _rope((h @ wk).view(B, S, sh.n_kv_heads, sh.head_dim), sh.rope_theta)
            v = (h @ wv).view(B, S, sh.n_kv_heads, sh.head_dim)
            del wq, wk, wv
            if l in want:
                yield l, q.contiguous(), k.contiguous(), v.contiguous()
            if l == max(want):
                return
            wo = self._w(gl, sh.n_q_heads * sh.head_dim, sh.hidden)
            x = x + _dense_attention(q, k, v, sh.window).reshape(B, S, -1) @ wo
            del wo, q, k, v
            w1 = self._w(gl, sh.hidden, sh.ffn)
            w3 = self._w(gl, sh.hidden, sh.ffn)
            w2 = self._w(gl, sh.ffn, sh.hidden)
            h = _rms(x, sh.rms_eps)
            x = x + (F.silu(h @ w1) * (h @ w3)) @ w2
            del w1, w2, w3


# ----------------------------------------------------------------------------------------------
# the five named configurations
# ----------------------------------------------------------------------------------------------
@dataclass
class Workload:
    name: str
    batch: int
    seq: int
    dtype: torch.dtype
    prune_ratios: Tuple[float, ...]
    stack: Optional[StackShape]
    ids: str = ""                       # which id recipe
    window: int = 0
    seed: int = BASE_SEED
    note: str = ""

    @property
    def n_q_heads(self):
        return self.stack.n_q_heads if self.stack else 32

    @property
    def n_kv_heads(self):
        return self.stack.n_kv_heads if self.stack else 32

    def make_ids(self, batch: Optional[int] = None, seq: Optional[int] = None) -> torch.Tensor:
        B, S, vocab = batch or self.batch, seq or self.seq, self.stack.vocab
        if self.ids == "repeat30":
            return ids_with_repeats(B, S, vocab, 0.30, self.seed)
        if self.ids == "zipf1.1":
            return ids_zipf(B, S, vocab, 1.1, self.seed)
        if self.ids == "spans40":
            return ids_with_copied_spans(B, S, vocab, 0.40, self.seed)
        raise ValueError(self.ids)

    def layer_qkv(self, layers: Sequence[int], device="cpu", batch=None, seq=None):
        """Yield (layer, Q, K, V) for this workload (config 1 has a single 'layer' 0)."""
        if self.stack is None:
            q, k, v = duplicate_qkv(batch or self.batch, seq or self.seq, 32, 32, 128, 0.25, 0.05,
                                    self.seed, self.dtype)
            yield 0, q.to(device), k.to(device), v.to(device)
            return
        ids = self.make_ids(batch, seq)
        yield from DecoderStack(self.stack, self.seed, device, self.dtype).layer_qkv(ids, layers)


_L2_7B = StackShape("llama2-7b", 4096, 32, 32, 128, 11008, 32, 1e4, 32000)
_L2_13B = StackShape("llama2-13b", 5120, 40, 40, 128, 13824, 40, 1e4, 32000)
_L3_8B = StackShape("llama3-8b", 4096, 32, 8, 128, 14336, 32, 5e5, 128256)
_MISTRAL = StackShape("mistral-7b", 4096, 32, 8, 128, 14336, 32, 1e4, 32000, window=4096)

WORKLOADS: Dict[str, Workload] = {
    "c1": Workload("c1", 1, 128, torch.float32, (0.5,), None, seed=BASE_SEED + 1,
                   note="single layer, LLaMA-2-7B head shape, fp32, 25% near-duplicate tokens"),
    "c2": Workload("c2", 1, 2048, torch.bfloat16, (0.0, 0.25, 0.5), _L2_7B, "repeat30",
                   seed=BASE_SEED + 2),
    "c3": Workload("c3", 4, 4096, torch.bfloat16, (0.5,), _L2_13B, "zipf1.1", seed=BASE_SEED + 3),
    "c4": Workload("c4", 2, 8192, torch.bfloat16, (0.3, 0.5, 0.7), _L3_8B, "zipf1.1",
                   seed=BASE_SEED + 4),
    "c5": Workload("c5", 8, 16384, torch.bfloat16, (0.5,), _MISTRAL, "spans40", window=4096,
                   seed=BASE_SEED + 5),
}
