"""Seeded synthetic inputs for the TABED speculative-decoding round.

This module only *draws inputs*: drafter weights, prompt prefixes, synthetic
KV caches, sampling uniforms and the stand-in for the target model's logits.
It holds none of the method's arithmetic (no softmax, no ensemble, no
acceptance rule, no divergence) and is the single source of every random bit
handed identically to the CUDA path and to the CPU checker.

The five workloads mirror the shapes the paper evaluates on: a small
LLaMA-style drafter shared by m drafting inputs (multimodal prefix with 576
projected image tokens per image, text-only prefix, caption prefix), block
lengths gamma in {3,5,7} and observation windows h in {4,8,16} (Sec. 4.1,
App. B).  The paper's datasets and trained weights are replaced by seeded
random tensors of the same shapes.
"""
from __future__ import annotations

import dataclasses
import hashlib
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

MASTER_SEED = 0x7ABED

POLICY_STATIC = 0
POLICY_GRID_MT = 1
POLICY_SOFTMAX_INV_ERR = 2
POLICY_RANDOM = 3
POLICY_GRID_HARD = 4
POLICY_ADABOOST = 5

DIST_KL = 0
DIST_TVD = 1

MODE_SAMPLE = 0
MODE_GREEDY = 1


@dataclass(frozen=True)
class DrafterCfg:
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    d_ffn: int
    vocab: int
    dtype: str = "bf16"            # "fp32" or "bf16" (weights and KV)
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0

    @property
    def head_dim(self) -> int:
        return self.d_model // self.n_heads

    @property
    def n_params_layers(self) -> int:
        d, f = self.d_model, self.d_ffn
        kvd = self.n_kv_heads * self.head_dim
        return self.n_layers * (d * d + 2 * d * kvd + d * d + 3 * d * f)

    @property
    def n_params_head(self) -> int:
        return self.d_model * self.vocab


@dataclass(frozen=True)
class Workload:
    """One synthetic workload: a drafter, its drafting inputs and run lengths."""
    name: str
    config_id: int
    drafter: DrafterCfg
    n_inputs: int                  # paper's m: drafting inputs per request
    n_requests: int                # B
    gamma: int
    window_h: int                  # 0 = ALL
    rounds: int
    policy: int
    # prefix recipe per drafting input: list of (kind, length); kind in
    # {"embeds", "tokens", "noisy_embeds_of:<k>"}; empty when synthetic KV is used
    prefixes: Tuple[Tuple[Tuple[str, int], ...], ...] = ()
    # synthetic KV: (lo, hi) inclusive range of per-row cached lengths; lo==hi fixed
    synthetic_kv_len: Optional[Tuple[int, int]] = None
    kv_capacity: int = 0
    # target stand-in: logits = sum_k alpha_k * drafter_logits^(k) + sigma * N(0,1)
    alpha: Optional[Tuple[float, ...]] = None      # None -> per-request Dirichlet(1,..,1)
    sigma_schedule: Tuple[Tuple[int, float], ...] = ((0, 1.0),)  # (first round, sigma)
    distance: int = DIST_KL
    sample_mode: int = MODE_SAMPLE
    tau: float = 1.0
    tree_width: int = 1            # candidates per depth of the token tree (Sec. 5); 1 = a plain chain

    @property
    def n_target_rows(self) -> int:
        """Rows of target logits per request: the chain's gamma + 1 positions, then one leaf per sibling candidate."""
        return self.gamma + 1 + self.gamma * (self.tree_width - 1)

    @property
    def n_rows(self) -> int:
        return self.n_inputs * self.n_requests

    def sigma(self, rnd: int) -> float:
        s = self.sigma_schedule[0][1]
        for first, val in self.sigma_schedule:
            if rnd >= first:
                s = val
        return s

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


_LLAVA_SMALL = DrafterCfg(4, 768, 12, 12, 3072, 32000, "bf16")

WORKLOADS: Dict[str, Workload] = {}


def _register(w: Workload) -> Workload:
    WORKLOADS[w.name] = w
    return w


TINY = _register(Workload(
    name="tiny", config_id=1,
    drafter=DrafterCfg(2, 128, 4, 4, 512, 1024, "fp32"),
    n_inputs=2, n_requests=1, gamma=3, window_h=4, rounds=32,
    policy=POLICY_GRID_MT,
    prefixes=((("tokens", 64),), (("tokens", 16),)),
    kv_capacity=64 + 32 * 4 + 8,
    alpha=(1.0, 0.0), sigma_schedule=((0, 0.5),),
))

LLAVA_SMALL = _register(Workload(
    name="llava_small", config_id=2, drafter=_LLAVA_SMALL,
    n_inputs=3, n_requests=1, gamma=5, window_h=8, rounds=256,
    policy=POLICY_SOFTMAX_INV_ERR,
    prefixes=((("embeds", 576), ("tokens", 128)),
              (("tokens", 128),),
              (("tokens", 64), ("tokens", 128))),
    kv_capacity=704 + 256 * 6 + 8,
    alpha=(0.5, 0.3, 0.2), sigma_schedule=((0, 1.0),),
))

LARGE_VOCAB = _register(Workload(
    name="large_vocab", config_id=3,
    drafter=DrafterCfg(12, 896, 14, 2, 4864, 152064, "bf16"),
    n_inputs=4, n_requests=1, gamma=5, window_h=8, rounds=256,
    policy=POLICY_SOFTMAX_INV_ERR,
    prefixes=((("embeds", 1024), ("tokens", 128)),
              (("tokens", 128),),
              (("tokens", 64), ("tokens", 128)),
              (("noisy_embeds_of:0", 1024), ("tokens", 128))),
    kv_capacity=1152 + 256 * 6 + 8,
    alpha=(0.4, 0.3, 0.2, 0.1), sigma_schedule=((0, 1.0),),
))

LONG_CONTEXT = _register(Workload(
    name="long_context", config_id=4, drafter=_LLAVA_SMALL,
    n_inputs=3, n_requests=1, gamma=7, window_h=16, rounds=512,
    policy=POLICY_SOFTMAX_INV_ERR,
    synthetic_kv_len=(8192, 8192), kv_capacity=12288,
    alpha=(0.5, 0.3, 0.2), sigma_schedule=((0, 0.3), (256, 2.0)),
))

BATCHED_SERVING = _register(Workload(
    name="batched_serving", config_id=5, drafter=_LLAVA_SMALL,
    n_inputs=3, n_requests=32, gamma=5, window_h=8, rounds=1024,
    policy=POLICY_SOFTMAX_INV_ERR,
    synthetic_kv_len=(256, 4096), kv_capacity=4096 + 6 * 1024,
    alpha=None, sigma_schedule=((0, 1.0),),
))


# ---------------------------------------------------------------------------
# seeding
# ---------------------------------------------------------------------------

def substream(config_id: int, name: str, *idx: int) -> np.random.Generator:
    """Counter-based generator keyed by (master seed, config id, tensor name, indices)."""
    h = hashlib.sha256(f"{MASTER_SEED}:{config_id}:{name}:{idx}".encode()).digest()
    key = int.from_bytes(h[:16], "little")
    return np.random.Generator(np.random.Philox(key=key))


def to_bf16_grid(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16-representable value (ties to even).

    Used only to make synthetic *inputs* (weights, caches) exactly storable in
    bf16, so that both consumers start from identical bits.
    """
    x = np.ascontiguousarray(x, dtype=np.float32)
    b = x.view(np.uint32)
    r = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns of float32 values that already lie on the bf16 grid."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


# ---------------------------------------------------------------------------
# drafter weights
# ---------------------------------------------------------------------------

WEIGHT_NAMES_PER_LAYER = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")


def weight_shapes(cfg: DrafterCfg) -> Dict[str, Tuple[int, int]]:
    d, f, kvd = cfg.d_model, cfg.d_ffn, cfg.n_kv_heads * cfg.head_dim
    return {"wq": (d, d), "wk": (kvd, d), "wv": (kvd, d), "wo": (d, d),
            "w_gate": (f, d), "w_up": (f, d), "w_down": (d, f)}


def make_weights(wl: Workload) -> Dict[str, object]:
    """Drafter weights N(0, 0.02), [out][in] row-major, norm gains 1.

    Returns float32 arrays; for a bf16 drafter every value lies on the bf16 grid.
    Keys: embed [V][d], lm_head [V][d], final_norm [d], and per layer lists
    wq, wk, wv, wo, w_gate, w_up, w_down, norm1, norm2.
    """
    cfg = wl.drafter
    snap = to_bf16_grid if cfg.dtype == "bf16" else (lambda a: np.ascontiguousarray(a, np.float32))

    def normal(name, shape, *idx):
        g = substream(wl.config_id, "w:" + name, *idx)
        return snap(g.standard_normal(shape, dtype=np.float32) * np.float32(0.02))

    out: Dict[str, object] = {
        "embed": normal("embed", (cfg.vocab, cfg.d_model)),
        "lm_head": normal("lm_head", (cfg.vocab, cfg.d_model)),
        "final_norm": np.ones(cfg.d_model, np.float32),
        "norm1": [np.ones(cfg.d_model, np.float32) for _ in range(cfg.n_layers)],
        "norm2": [np.ones(cfg.d_model, np.float32) for _ in range(cfg.n_layers)],
    }
    shapes = weight_shapes(cfg)
    for nm in WEIGHT_NAMES_PER_LAYER:
        out[nm] = [normal(nm, shapes[nm], l) for l in range(cfg.n_layers)]
    return out


# ---------------------------------------------------------------------------
# prefixes / synthetic KV
# ---------------------------------------------------------------------------

@dataclass
class Segment:
    kind: str                      # "embeds" or "tokens"
    data: np.ndarray               # [len][d] float32  or  [len] int32


def make_prefixes(wl: Workload, request: int = 0) -> List[List[Segment]]:
    """Prompt prefix of each drafting input of one request (Algorithm 1's X = [x^(1..m)])."""
    cfg = wl.drafter
    rows: List[List[Segment]] = []
    first_embeds: Dict[int, np.ndarray] = {}
    for k, recipe in enumerate(wl.prefixes):
        segs: List[Segment] = []
        for s, (kind, length) in enumerate(recipe):
            g = substream(wl.config_id, "prefix", request, k, s)
            if kind == "embeds":
                e = g.standard_normal((length, cfg.d_model), dtype=np.float32)
                first_embeds.setdefault(k, e)
                segs.append(Segment("embeds", e))
            elif kind.startswith("noisy_embeds_of:"):
                src = int(kind.split(":")[1])
                base = first_embeds[src][:length]
                e = base + np.float32(0.5) * g.standard_normal(base.shape, dtype=np.float32)
                segs.append(Segment("embeds", e.astype(np.float32)))
            elif kind == "tokens":
                segs.append(Segment("tokens", g.integers(0, cfg.vocab, size=length, dtype=np.int32)))
            else:
                raise ValueError(kind)
        rows.append(segs)
    return rows


def synthetic_kv_lengths(wl: Workload) -> np.ndarray:
    """Cached length of every row [R], row index = request * n_inputs + input."""
    lo, hi = wl.synthetic_kv_len
    g = substream(wl.config_id, "kvlen")
    return g.integers(lo, hi + 1, size=wl.n_rows, dtype=np.int32)


def make_synthetic_kv(wl: Workload, row: int, length: int) -> Tuple[np.ndarray, np.ndarray]:
    """K and V of one row, [L][Hkv][length][hd] float32 on the bf16 grid, N(0, 0.5)."""
    cfg = wl.drafter
    shape = (cfg.n_layers, cfg.n_kv_heads, length, cfg.head_dim)
    g = substream(wl.config_id, "kv", row)
    k = g.standard_normal(shape, dtype=np.float32) * np.float32(0.5)
    v = g.standard_normal(shape, dtype=np.float32) * np.float32(0.5)
    if cfg.dtype == "bf16":
        k, v = to_bf16_grid(k), to_bf16_grid(v)
    return k, v


def initial_pending(wl: Workload) -> np.ndarray:
    """First token fed to the drafter for each request [B] (the last verified token)."""
    g = substream(wl.config_id, "pending")
    return g.integers(0, wl.drafter.vocab, size=wl.n_requests, dtype=np.int32)


# ---------------------------------------------------------------------------
# uniforms and target stand-in
# ---------------------------------------------------------------------------

def lattice_uniforms(g: np.random.Generator, shape) -> np.ndarray:
    """u = (k + 1/2) * 2^-23 with k uniform in [0, 2^23): exactly representable, inside (0,1)."""
    k = g.integers(0, 1 << 23, size=shape, dtype=np.int64)
    return ((k.astype(np.float64) + 0.5) * 2.0 ** -23).astype(np.float32)


def round_uniforms(wl: Workload, rnd: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """(u_draft [B][gamma], u_accept [B][gamma], u_resid [B]) of one round; with a token tree of width d the first two
    are [B][gamma][d] (one uniform per candidate)."""
    g = substream(wl.config_id, "uniforms", rnd)
    G, d = wl.gamma, wl.tree_width
    u = lattice_uniforms(g, (wl.n_requests, 2 * G * d + 1))
    shape = (wl.n_requests, G) if d == 1 else (wl.n_requests, G, d)
    return (np.ascontiguousarray(u[:, :G * d]).reshape(shape), np.ascontiguousarray(u[:, G * d:2 * G * d]).reshape(shape),
            np.ascontiguousarray(u[:, 2 * G * d]))


def policy_uniforms(wl: Workload, rnd: int) -> np.ndarray:
    """Uniforms of the Random weight policy for one round, [B][m], on the same lattice as the draws."""
    return lattice_uniforms(substream(wl.config_id, "policy_uniforms", rnd), (wl.n_requests, wl.n_inputs))


def request_alpha(wl: Workload) -> np.ndarray:
    """Mixing coefficients of the target stand-in, [B][n]."""
    if wl.alpha is not None:
        return np.tile(np.asarray(wl.alpha, np.float32), (wl.n_requests, 1))
    g = substream(wl.config_id, "alpha")
    return g.dirichlet(np.ones(wl.n_inputs), size=wl.n_requests).astype(np.float32)


def target_logits(wl: Workload, rnd: int, drafter_logits: np.ndarray) -> np.ndarray:
    """Stand-in for the target model M_p: [B][gamma+1][V] float32.

    drafter_logits is [gamma][B][n][V].  Position i < gamma is a fixed convex
    mix of the n drafter logit vectors of step i plus N(0, sigma) noise; the
    bonus position gamma reuses the mix of step gamma-1 with fresh noise (the
    drafter never runs on the last drafted token inside the round).
    """
    G, B, n, V = drafter_logits.shape
    assert (G, B, n) == (wl.gamma, wl.n_requests, wl.n_inputs)
    alpha = request_alpha(wl)                                   # [B][n]
    mix = np.einsum("gbnv,bn->bgv", drafter_logits.astype(np.float32), alpha).astype(np.float32)
    out = np.empty((B, G + 1, V), np.float32)
    out[:, :G] = mix
    out[:, G] = mix[:, G - 1]
    g = substream(wl.config_id, "target_noise", rnd)
    out += np.float32(wl.sigma(rnd)) * g.standard_normal(out.shape, dtype=np.float32)
    if wl.tree_width > 1:
        # leaves of the token tree: the target's distribution after sibling c of depth i stands in as the mix of the
        # next step (the last step's for the deepest leaves) plus fresh noise
        d = wl.tree_width
        leaves = np.repeat(mix[:, np.minimum(np.arange(G) + 1, G - 1)], d - 1, axis=1)      # [B][G (d-1)][V]
        g2 = substream(wl.config_id, "target_noise_leaves", rnd)
        leaves = leaves + np.float32(wl.sigma(rnd)) * g2.standard_normal(leaves.shape, dtype=np.float32)
        out = np.concatenate([out, leaves.astype(np.float32)], axis=1)
    return out


def logits_like_drafter(wl: Workload, rnd: int, scale: float = 0.55) -> np.ndarray:
    """Free-standing drafter-like logits [gamma][B][n][V] ~ N(0, scale) for stage tests.

    scale 0.55 ~ 0.02*sqrt(768): the spread a N(0,0.02) LM head gives unit-RMS hidden states.
    """
    g = substream(wl.config_id, "free_logits", rnd)
    shape = (wl.gamma, wl.n_requests, wl.n_inputs, wl.drafter.vocab)
    return (np.float32(scale) * g.standard_normal(shape, dtype=np.float32)).astype(np.float32)
