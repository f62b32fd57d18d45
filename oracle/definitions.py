"""Plain fp64 definitions of the quantities a TABED round is built from.

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import this
package; it exists so that tests (and the CPU-baseline leg of the benchmark)
can check the CUDA library against the paper's mathematics.

Every function is the textbook definition written out in float64 with no
blocking, fusion or reordering:

* softmax / weighted-average ensemble ........ Algorithm 1, steps 5-6
* KL divergence, total variation distance ... Sec. 4.1 (error e_t^j), TVD variant
* acceptance probability, residual law ...... Sec. 3, item 3
* emitted-token law of one SD position ...... Sec. 3 (distribution preserved)
* weight policies ........................... App. B "Weight Sampling Policy"
* expected walltime speedup ................. Eq. 1
"""
from __future__ import annotations

import numpy as np


def softmax(logits: np.ndarray) -> np.ndarray:
    """softmax over the last axis (temperature 1)."""
    x = np.asarray(logits, np.float64)
    x = x - x.max(axis=-1, keepdims=True)
    e = np.exp(x)
    return e / e.sum(axis=-1, keepdims=True)


def ensemble(qk: np.ndarray, w: np.ndarray) -> np.ndarray:
    """W-Avg: q = sum_k w_k q^(k).  qk [m][V], w [m]  (Algorithm 1, step 6)."""
    return np.tensordot(np.asarray(w, np.float64), np.asarray(qk, np.float64), axes=(0, 0))


def kl_divergence(p: np.ndarray, q: np.ndarray, q_floor: float = 0.0) -> float:
    """D_KL(p || q) in nats with 0 ln 0 = 0 (the summand of e_t^j, Sec. 4.1)."""
    p = np.asarray(p, np.float64)
    q = np.maximum(np.asarray(q, np.float64), q_floor)
    m = p > 0
    return float(np.sum(p[m] * (np.log(p[m]) - np.log(q[m]))))


def total_variation(p: np.ndarray, q: np.ndarray) -> float:
    """TVD = 1/2 sum |p - q| (Sec. 4.1, distance variant)."""
    return 0.5 * float(np.abs(np.asarray(p, np.float64) - np.asarray(q, np.float64)).sum())


def accept_probability(p_y: float, q_y: float) -> float:
    """min(1, p(y)/q(y))  (Sec. 3, item 3)."""
    return 1.0 if p_y >= q_y else p_y / q_y


def residual_distribution(p: np.ndarray, q: np.ndarray) -> np.ndarray:
    """norm(max(0, p - q))  (Sec. 3, item 3); falls back to p when p == q."""
    r = np.maximum(0.0, np.asarray(p, np.float64) - np.asarray(q, np.float64))
    s = r.sum()
    return r / s if s > 0 else np.asarray(p, np.float64).copy()


def emitted_law_one_position(p: np.ndarray, q: np.ndarray) -> np.ndarray:
    """Law of the token emitted at one position: draft y~q, accept w.p. min(1,p/q),
    otherwise redraw from the residual.  Sec. 3 states this equals p."""
    p = np.asarray(p, np.float64)
    q = np.asarray(q, np.float64)
    acc = np.minimum(p, q)                      # P(draft = v and accepted)
    reject_mass = 1.0 - acc.sum()
    return acc + reject_mass * residual_distribution(p, q)


def grid_candidates(n_grid: int = 10) -> np.ndarray:
    """Candidate weights w^j = [1 - j/n, j/n], j = 0..n  (App. B, two drafting methods)."""
    j = np.arange(n_grid + 1, dtype=np.float64)
    return np.stack([1.0 - j / n_grid, j / n_grid], axis=1)


def policy_softmax_inv_err(e: np.ndarray, tau: float = 1.0, e_floor: float = 1e-8) -> np.ndarray:
    """w = softmax([1/e^(1), ..., 1/e^(m)]; tau)  (App. B, more than two methods)."""
    s = 1.0 / np.maximum(np.asarray(e, np.float64), e_floor)
    return softmax(s / tau)


def policy_grid(p_window, qk_window, n_grid: int = 10):
    """argmin_j sum_{t'} KL(p_t' || q_t'^j) over the grid candidates (Algorithm 1, steps 2-3).

    p_window: list of [V]; qk_window: list of [2][V].  Returns (j*, w*, G[j])."""
    cands = grid_candidates(n_grid)
    G = np.zeros(len(cands))
    for p, qk in zip(p_window, qk_window):
        for j, w in enumerate(cands):
            G[j] += kl_divergence(p, ensemble(qk, w), q_floor=np.finfo(np.float32).tiny)
    j_star = int(np.argmin(G))
    return j_star, cands[j_star], G


def pool_image_tokens_2x2(x: np.ndarray, grid_h: int, grid_w: int) -> np.ndarray:
    """Pooled multimodal drafting input (Sec. 5, "Pooled Multimodal Drafting (P)"): the visual tokens keep their 2-D
    arrangement (row-major grid_h x grid_w, 24 x 24 = 576 in the paper's default) and every 2 x 2 block of tokens is
    replaced by its average, feature by feature: 576 -> 144 tokens.  x: [grid_h * grid_w][d]; returns
    [(grid_h / 2) * (grid_w / 2)][d] fp32 (the mean is taken in fp64 and rounded once)."""
    if grid_h % 2 or grid_w % 2 or x.shape[0] != grid_h * grid_w:
        raise ValueError("the token grid must have even sides and match the number of tokens")
    g = np.asarray(x, dtype=np.float64).reshape(grid_h, grid_w, -1)
    out = np.empty((grid_h // 2, grid_w // 2, g.shape[2]), dtype=np.float64)
    for i in range(grid_h // 2):
        for j in range(grid_w // 2):
            out[i, j] = (g[2 * i, 2 * j] + g[2 * i, 2 * j + 1] + g[2 * i + 1, 2 * j] + g[2 * i + 1, 2 * j + 1]) / 4.0
    return out.reshape(-1, g.shape[2]).astype(np.float32)


def expected_speedup(block_efficiency: float, gamma: int, latency_ratio: float) -> float:
    """Eq. 1: tau / (gamma * T_q/T_p + 1)."""
    return block_efficiency / (gamma * latency_ratio + 1.0)
