"""fp64 forward pass of the shared drafter M_q on one drafting input (one batch row).

TEST INFRASTRUCTURE ONLY.

The paper's drafters are small LLaMA-style decoders (Sec. 3.1 "small public LLaMA
models"); all m drafting inputs share these parameters and are decoded as one
batch (Sec. 4.1 "Ensemble learning via Batched Inference", Algorithm 1 step 5).
This file is the textbook pre-norm decoder, one row at a time, a whole chunk of
positions per call with a causal mask:

    x = E[token]                         (or a supplied embedding row)
    per layer:  a = RMSNorm(x) g1;  q,k,v = a Wq^T, a Wk^T, a Wv^T;  RoPE(q,k) at the
                row's own positions;  append k,v to the row's cache;
                o = softmax(q K^T / sqrt(hd)) V  (grouped-query: H/Hkv query heads per KV head);
                x += o Wo^T;  b = RMSNorm(x) g2;  x += (SiLU(b Wg^T) * (b Wu^T)) Wd^T
    logits = RMSNorm(x) gf  W_lm^T

All sums are float64.  For a bf16 drafter ("fp32 accumulate over bf16 inputs")
every matmul input (a, q, k, v, o, b, the gated product, the final normed state)
is rounded to bf16, round-to-nearest-even, exactly where marked `rb`; for an fp32
drafter `rb` is the identity.  RoPE rotates pairs (i, i + hd/2) by pos * theta^(-2i/hd).
"""
from __future__ import annotations

from typing import Dict, List, Optional

import numpy as np


def round_bf16(x: np.ndarray) -> np.ndarray:
    """float64 -> float32 (nearest) -> bf16 (nearest, ties to even) -> float64."""
    x32 = np.ascontiguousarray(x, dtype=np.float32)
    b = x32.view(np.uint32)
    r = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32).astype(np.float64)


class RowCache:
    """K and V of one row: [L][Hkv][positions][hd], `length` valid positions, at most `capacity`.

    Storage only: the arrays hold the positions in use (they grow as the row grows) instead of the whole
    capacity, and the values of a bf16 drafter - bf16 numbers, which float32 holds exactly - are kept
    as float32; every product and sum that reads them is taken in float64 as before."""

    def __init__(self, n_layers: int, n_kv_heads: int, head_dim: int, capacity: int, dtype=np.float64):
        self.shape = (n_layers, n_kv_heads, head_dim)
        self.capacity = capacity
        self.dtype = dtype
        self.k = np.zeros((n_layers, n_kv_heads, 0, head_dim), dtype)
        self.v = np.zeros((n_layers, n_kv_heads, 0, head_dim), dtype)
        self.length = 0

    def reserve(self, n: int) -> None:
        """Make room for positions [0, n)."""
        if n > self.capacity:
            raise ValueError("row cache capacity exceeded")
        have = self.k.shape[2]
        if n <= have:
            return
        room = min(self.capacity, max(n, have + have // 2 + 16))
        L, Hkv, hd = self.shape
        for name in ("k", "v"):
            old = getattr(self, name)
            new = np.zeros((L, Hkv, room, hd), self.dtype)
            new[:, :, :have] = old
            setattr(self, name, new)

    def load(self, k: np.ndarray, v: np.ndarray) -> None:
        n = k.shape[2]
        self.reserve(n)
        self.k[:, :, :n] = k
        self.v[:, :, :n] = v
        self.length = n


class OracleDrafter:
    def __init__(self, cfg, weights: Dict[str, object]):
        self.cfg = cfg
        self.bf16 = cfg.dtype == "bf16"
        f64 = lambda a: np.asarray(a, np.float64)
        self.embed = f64(weights["embed"])
        self.lm_head = f64(weights["lm_head"])
        self.final_norm = f64(weights["final_norm"])
        self.layers = []
        for l in range(cfg.n_layers):
            self.layers.append({k: f64(weights[k][l]) for k in
                                ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "norm1", "norm2")})
        hd = cfg.head_dim
        self.inv_freq = cfg.rope_theta ** (-2.0 * np.arange(hd // 2) / hd)

    def rb(self, x: np.ndarray) -> np.ndarray:
        return round_bf16(x) if self.bf16 else x

    def new_cache(self, capacity: int) -> RowCache:
        c = self.cfg
        return RowCache(c.n_layers, c.n_kv_heads, c.head_dim, capacity, np.float32 if self.bf16 else np.float64)

    def rmsnorm(self, x: np.ndarray, g: np.ndarray) -> np.ndarray:
        ms = np.mean(x * x, axis=-1, keepdims=True)
        return x / np.sqrt(ms + self.cfg.rms_eps) * g

    def rope(self, x: np.ndarray, pos: np.ndarray) -> np.ndarray:
        """x [T][H][hd], pos [T]."""
        half = self.cfg.head_dim // 2
        ang = pos[:, None].astype(np.float64) * self.inv_freq[None, :]       # [T][half]
        c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
        x1, x2 = x[..., :half], x[..., half:]
        return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)

    def embed_tokens(self, tokens) -> np.ndarray:
        return self.embed[np.asarray(tokens, np.int64)]

    def forward(self, cache: RowCache, x: np.ndarray, want_logits: bool = True) -> Optional[np.ndarray]:
        """Run T new positions [T][d] of one row, append their K,V, return logits [T][V]."""
        c = self.cfg
        T = x.shape[0]
        H, Hkv, hd = c.n_heads, c.n_kv_heads, c.head_dim
        grp = H // Hkv
        p0 = cache.length
        cache.reserve(p0 + T)
        pos = np.arange(p0, p0 + T)
        x = np.asarray(x, np.float64).copy()
        # causal mask: new position t sees cached [0, p0) and new [0, t]
        mask = np.arange(p0 + T)[None, :] <= pos[:, None]                  # [T][p0+T]
        for l, w in enumerate(self.layers):
            a = self.rb(self.rmsnorm(x, w["norm1"]))
            q = (a @ w["wq"].T).reshape(T, H, hd)
            k = (a @ w["wk"].T).reshape(T, Hkv, hd)
            v = (a @ w["wv"].T).reshape(T, Hkv, hd)
            q = self.rb(self.rope(q, pos))
            k = self.rb(self.rope(k, pos))
            v = self.rb(v)
            cache.k[l, :, p0:p0 + T] = k.transpose(1, 0, 2)
            cache.v[l, :, p0:p0 + T] = v.transpose(1, 0, 2)
            o = np.empty((T, H, hd))
            for h in range(H):
                K = cache.k[l, h // grp, :p0 + T]
                V = cache.v[l, h // grp, :p0 + T]
                s = (q[:, h, :] @ K.T) / np.sqrt(hd)
                s = np.where(mask, s, -np.inf)
                s = s - s.max(axis=-1, keepdims=True)
                e = np.exp(s)
                o[:, h, :] = (e / e.sum(axis=-1, keepdims=True)) @ V
            x = x + self.rb(o.reshape(T, H * hd)) @ w["wo"].T
            b = self.rb(self.rmsnorm(x, w["norm2"]))
            g = b @ w["w_gate"].T
            u = b @ w["w_up"].T
            x = x + self.rb(g / (1.0 + np.exp(-g)) * u) @ w["w_down"].T
        cache.length = p0 + T
        if not want_logits:
            return None
        xf = self.rb(self.rmsnorm(x, self.final_norm))
        return xf @ self.lm_head.T
