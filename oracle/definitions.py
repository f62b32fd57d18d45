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
* weight policies ........................... App. B "Weight Sampling Policy"; hard labels (Sec. 4.1); Random
                                              ablation (Sec. 5); TABED-AdaBoost (appendix)
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


def policy_random(u: np.ndarray) -> np.ndarray:
    """Non-negative, sum-to-one random weights (Sec. 5 "Effectiveness of Dynamic Weights", the Random ablation):
    a point drawn uniformly from the simplex, w_k = g_k / sum_j g_j with g_k = -ln u_k, u_k uniform in (0, 1)."""
    g = -np.log(np.asarray(u, np.float64))
    return g / g.sum()


def hard_label_matches(qk: np.ndarray, label: int, n_grid: int = 10) -> np.ndarray:
    """Hard-label score of every grid candidate at one verified position (Sec. 4.1, "utilizing hard labels"): 1 if the
    token the candidate's ensemble q^j = (1 - j/n) q^(1) + (j/n) q^(2) would emit (its most likely token, lowest id on
    ties) is the verified token, else 0.  qk [2][V].  Returns [n_grid + 1]."""
    return np.array([int(int(np.argmax(ensemble(qk, w))) == int(label)) for w in grid_candidates(n_grid)], np.int64)


def policy_grid_hard(label_window, qk_window, n_grid: int = 10):
    """argmax_j of the number of token matches over the window (lowest j on ties).  Returns (j*, w*, counts[j])."""
    counts = np.zeros(n_grid + 1, np.int64)
    for y, qk in zip(label_window, qk_window):
        counts += hard_label_matches(qk, y, n_grid)
    j_star = int(np.argmax(counts))
    return j_star, grid_candidates(n_grid)[j_star], counts


def policy_adaboost(errors: np.ndarray, n: int, vocab: int, c: float = 1.0) -> np.ndarray:
    """TABED-AdaBoost (App. "TABED-AdaBoost: A Theoretically Grounded Variant"): w_m = ln(1/eps_m - 1) + C ln(K - 1) with
    eps_m the error rate of drafting method m, here the smoothed fraction (errors_m + 1) / (n + 2) of the n verified
    positions of the window at which the method's most likely token was not the verified token; K the vocabulary
    size.  The ensemble needs non-negative weights that sum to one: negative values are cut at 0 and the rest is
    normalised (equal weights if nothing is left)."""
    eps = (np.asarray(errors, np.float64) + 1.0) / (n + 2.0)
    w = np.maximum(np.log(1.0 / eps - 1.0) + c * np.log(vocab - 1.0), 0.0)
    s = w.sum()
    return w / s if s > 0 else np.full(len(w), 1.0 / len(w))


# ---- token tree of width d (Sec. 5 "Verification: Integrating Token Tree") ---------------------------------
# Reading (the paper names the method and the widths 2 and 3, not the construction): at every depth of the block the
# drafter proposes d distinct candidate tokens, drawn from the ensembled q WITHOUT replacement; the first one (the
# primary) is the token the chain continues with, the others are leaves.  The target tries the candidates of a depth
# in order by recursive rejection sampling: candidate x is accepted with probability min(1, p'(x) / q'(x)); after a
# rejection p' <- norm(max(0, p' - q')) and q' <- q' restricted to the tokens not yet tried, renormalised (the law of
# the next candidate given the rejected ones); if every candidate is rejected the token is drawn from the last
# residual.  The emitted token follows the target law p exactly (checked by enumeration in the tests).

def tree_after_rejection(p: np.ndarray, q: np.ndarray, x: int):
    """(p', q') after candidate x has been rejected at a depth."""
    p = np.asarray(p, np.float64); q = np.asarray(q, np.float64)
    p2 = residual_distribution(p, q)
    q2 = q.copy(); q2[x] = 0.0
    s = q2.sum()
    return p2, (q2 / s if s > 0 else q2)


def tree_depth_outcomes(p: np.ndarray, q: np.ndarray, d: int):
    """Every outcome of one depth of a width-d tree with its probability: yields (prob, token, level) where level = c
    if candidate c was accepted (0 = the primary) and level = -1 for a token drawn from the last residual.
    Enumerates all ordered tuples of d distinct candidates (fewer if q runs out of support)."""
    p = np.asarray(p, np.float64); q = np.asarray(q, np.float64)
    out = []

    def rec(pp, qq, prob, c):
        if c == d or qq.sum() <= 0:
            for z, pz in enumerate(pp):
                if pz > 0:
                    out.append((prob * pz, z, -1))
            return
        for x in range(len(qq)):
            if qq[x] <= 0:
                continue
            acc = accept_probability(pp[x], qq[x])
            if acc > 0:
                out.append((prob * qq[x] * acc, x, c))
            if acc < 1:
                p2, q2 = tree_after_rejection(pp, qq, x)
                rec(p2, q2, prob * qq[x] * (1 - acc), c + 1)

    rec(p, q, 1.0, 0)
    return out


def tree_depth_emitted_law(p: np.ndarray, q: np.ndarray, d: int) -> np.ndarray:
    """Law of the token emitted at one depth of a width-d tree (equals p)."""
    law = np.zeros(len(p))
    for prob, tok, _ in tree_depth_outcomes(p, q, d):
        law[tok] += prob
    return law


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
