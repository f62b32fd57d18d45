"""Decision arithmetic of a TABED round in the kernel's precision (fp32 + exact integers).

TEST INFRASTRUCTURE ONLY (see oracle/definitions.py for the fp64 definitions
these functions are pinned to).

Token ids, accept counts and the weight argmax are integers decided by
floating point.  Two implementations agree on them bit for bit only if the
decision is a function of identical bits evaluated with operations whose
result does not depend on evaluation order.  This file states that function:

* every floating-point step is ONE correctly rounded IEEE-754 binary32
  operation (add, sub, mul, div, rint, int<->float conversion); no fused
  multiply-add, no library exp/log;
* every reduction over the vocabulary is either a max (order-free) or a sum
  of integers (order-free): probabilities are turned into integer masses
  m_v = trunc(q_v * 2^40) before they are summed.

What is computed follows the paper: softmax of logits, the weighted-average
ensemble q = sum_k w_k q^(k) and Sample(q) (Algorithm 1, steps 5-7); the
acceptance test min(1, p/q) and the residual norm(max(0, p-q)) (Sec. 3,
item 3); the deviation sum of KL(p || q) over the window and the two weight
policies (Sec. 4.1; App. B).
"""
from __future__ import annotations

import numpy as np

F = np.float32
U64 = np.uint64

MASS_BITS = 40                       # m_v = trunc(q_v * 2^40)
MASS_SCALE = F(2.0 ** MASS_BITS)
FLT_MIN = F(np.finfo(np.float32).tiny)

# ---- exp / log built from single correctly-rounded operations ---------------
_LOG2E = F(1.4426950408889634)
_LN2_HI = F(0.693359375)             # 355/512: products with small integers are exact
_LN2_LO = F(-2.12194440e-4)          # ln2 - LN2_HI
_EXP_C = [F(1.0 / f) for f in (1, 1, 2, 6, 24, 120, 720, 5040)]   # 1/i!, i = 0..7
_EXP_CUTOFF = F(-80.0)
_SQRT2 = F(1.41421356)
_LOG_K = [F(1.0), F(1.0 / 3.0), F(1.0 / 5.0), F(1.0 / 7.0), F(1.0 / 9.0)]


def xexp(x) -> np.ndarray:
    """exp(x) for x <= 0; exactly 0 below -80.

    n = rint(x*log2e); r = (x - n*LN2_HI) - n*LN2_LO; degree-7 Taylor polynomial of
    exp(r) evaluated by Horner with separate multiply and add; result scaled by 2^n.
    """
    x = np.asarray(x, F)
    n = np.rint(x * _LOG2E)
    r = x - n * _LN2_HI
    r = r - n * _LN2_LO
    p = np.full_like(r, _EXP_C[7])
    for c in _EXP_C[6::-1]:
        p = p * r
        p = p + c
    e = np.ldexp(p, n.astype(np.int32)).astype(F)
    return np.where(x < _EXP_CUTOFF, F(0), e)


def xlog(x) -> np.ndarray:
    """ln(x) for normal positive float32 x.

    x = m * 2^e with m in (sqrt2/2, sqrt2]; s = (m-1)/(m+1); ln m = 2 s (1 + s^2/3 + s^4/5 + s^6/7 + s^8/9);
    ln x = e*LN2_HI + (ln m + e*LN2_LO).
    """
    x = np.ascontiguousarray(x, F)
    bits = x.view(np.uint32)
    e = (bits >> np.uint32(23)).astype(np.int32) - 127
    m = ((bits & np.uint32(0x007FFFFF)) | np.uint32(0x3F800000)).view(F)
    big = m > _SQRT2
    m = np.where(big, m * F(0.5), m)
    e = e + big.astype(np.int32)
    s = (m - F(1)) / (m + F(1))
    z = s * s
    poly = np.full_like(z, _LOG_K[4])
    for c in _LOG_K[3::-1]:
        poly = poly * z
        poly = poly + c
    lnm = (s + s) * poly
    ef = e.astype(F)
    return ef * _LN2_HI + (lnm + ef * _LN2_LO)


# ---- softmax, ensemble, masses ----------------------------------------------

def masses(q) -> np.ndarray:
    """Integer masses m_v = trunc(q_v * 2^40) as uint64 (q >= 0)."""
    return (np.asarray(q, F) * MASS_SCALE).astype(U64)


def softmax_exact(logits) -> np.ndarray:
    """softmax over the last axis, fp32 [..., V] -> fp32 [..., V]  (Algorithm 1, step 5).

    e_v = xexp(x_v - max); S = float32(sum_v trunc(e_v * 2^40)) * 2^-40; out_v = e_v / S.
    """
    x = np.asarray(logits, F)
    mx = x.max(axis=-1, keepdims=True)
    e = xexp(x - mx)
    total = masses(e).sum(axis=-1, keepdims=True, dtype=U64)
    S = total.astype(F) * F(2.0 ** -MASS_BITS)
    return (e / S).astype(F)


def ensemble_exact(qk, w) -> np.ndarray:
    """q_v = ((w_0 q^(0)_v + w_1 q^(1)_v) + w_2 q^(2)_v) + ...  each product and sum rounded once.

    qk [m][V] fp32, w [m] fp32  (Algorithm 1, step 6)."""
    qk = np.asarray(qk, F)
    w = np.asarray(w, F)
    acc = w[0] * qk[0]
    for k in range(1, qk.shape[0]):
        acc = acc + w[k] * qk[k]
    return acc.astype(F)


def uniform_index(u) -> int:
    """k_u of u = (k_u + 1/2) * 2^-23."""
    return int(np.floor(np.float64(u) * 2.0 ** 23))


def draw(mass: np.ndarray, u) -> int:
    """Inverse-CDF draw in ascending token id on integer masses (Algorithm 1, step 7).

    thr = ((2 k_u + 1) * T) >> 24 with T = sum m;  y = min{ v : sum_{v'<=v} m_v' > thr }.
    Requires T > 0."""
    mass = np.asarray(mass, U64)
    T = int(mass.sum(dtype=U64))
    assert T > 0
    thr = ((2 * uniform_index(u) + 1) * T) >> 24
    cdf = np.cumsum(mass, dtype=U64)
    return int(np.searchsorted(cdf, np.uint64(thr), side="right"))


def argmax_lowest(x) -> int:
    """argmax with the lowest index on ties (greedy decoding)."""
    return int(np.argmax(np.asarray(x)))


# ---- verification (Sec. 3, item 3) -------------------------------------------

def accept(p_y, q_y, u) -> bool:
    """Accept with probability min(1, p/q): p >= q, or u*q < p with the product rounded once."""
    p_y, q_y, u = F(p_y), F(q_y), F(u)
    return bool(p_y >= q_y) or bool(F(u * q_y) < p_y)


def residual_masses(p, q) -> np.ndarray:
    """Integer masses of max(0, p - q); the difference is one rounded fp32 subtraction."""
    r = np.maximum(F(0), np.asarray(p, F) - np.asarray(q, F))
    return masses(r)


# ---- deviation and weights (Sec. 4.1; App. B) ---------------------------------

def kl_fixed(p, q) -> int:
    """KL(p || q) as an exact integer: sum_v trunc(p_v * (ln p_v - ln max(q_v, FLT_MIN)) * 2^40)
    over p_v > 0; value = result * 2^-40."""
    p = np.asarray(p, F)
    q = np.maximum(np.asarray(q, F), FLT_MIN)
    lp = xlog(np.maximum(p, FLT_MIN))
    lq = xlog(q)
    t = p * (lp - lq)
    t = np.where(p > F(0), t, F(0))
    return int((t * MASS_SCALE).astype(np.int64).sum(dtype=np.int64))


def tvd_fixed(p, q) -> int:
    """2*TVD as an exact integer: sum_v trunc(|p_v - q_v| * 2^40); TVD = result * 2^-41."""
    d = np.abs(np.asarray(p, F) - np.asarray(q, F))
    return int((d * MASS_SCALE).astype(np.int64).sum(dtype=np.int64))


def fixed_to_float(total: int, distance_is_tvd: bool = False) -> np.float32:
    """float32(total) * 2^-40 (KL) or * 2^-41 (TVD); the int->float conversion rounds to nearest."""
    f = np.array(total, dtype=np.int64).astype(F)
    return F(f * F(2.0 ** -(MASS_BITS + (1 if distance_is_tvd else 0))))


def grid_weight(j: int, n_grid: int = 10) -> np.ndarray:
    """w^j = [1 - j/n, j/n] in fp32: c1 = j / n (one division), c0 = 1 - c1."""
    c1 = F(F(j) / F(n_grid))
    return np.array([F(F(1) - c1), c1], F)


def policy_static(m: int) -> np.ndarray:
    return np.full(m, F(1) / F(m), F)


def policy_softmax_inv_err(e, tau=1.0) -> np.ndarray:
    """w = softmax(1/e; tau): s_k = 1/max(e_k,1e-8); x_k = xexp((s_k - max s)/tau);
    w_k = x_k / (((x_0 + x_1) + x_2) + ...)."""
    e = np.asarray(e, F)
    s = F(1) / np.maximum(e, F(1e-8))
    d = (s - s.max()) / F(tau)
    x = xexp(d)
    tot = x[0]
    for k in range(1, len(x)):
        tot = F(tot + x[k])
    return (x / tot).astype(F)


def policy_random(u) -> np.ndarray:
    """Random non-negative sum-to-one weights from uniforms on the lattice: g_k = -xlog(u_k), w_k = g_k / (((g_0 + g_1)
    + g_2) + ...)."""
    g = -xlog(np.asarray(u, F))
    tot = g[0]
    for k in range(1, len(g)):
        tot = F(tot + g[k])
    return (g / tot).astype(F)


def grid_hard_matches(qk, label: int, n_grid: int = 10) -> np.ndarray:
    """Per grid candidate j: 1 if argmax_v of the fp32 ensemble c0 q^(0) + c1 q^(1) (lowest id on ties) is `label`."""
    return np.array([int(argmax_lowest(ensemble_exact(qk, grid_weight(j, n_grid))) == int(label)) for j in range(n_grid + 1)],
                    np.int64)


def drafter_errors(qk, label: int) -> np.ndarray:
    """Per drafting method k: 1 if argmax_v q^(k)_v (lowest id on ties) is NOT `label`."""
    return np.array([int(argmax_lowest(qk[k]) != int(label)) for k in range(len(qk))], np.int64)


def policy_adaboost(errors, n: int, vocab: int, c=1.0) -> np.ndarray:
    """w_k = max(0, xlog(1/eps_k - 1) + c * xlog(K - 1)) normalised; eps_k = (errors_k + 1) / (n + 2); every step one
    rounded fp32 operation, the sum taken in k order; equal weights if every value is cut to 0."""
    errors = np.asarray(errors, np.int64)
    eps = (errors.astype(F) + F(1)) / F(F(n) + F(2))
    a = F(1) / eps
    t = xlog(a - F(1)) + F(F(c) * xlog(np.array([F(vocab - 1)], F))[0])
    t = np.maximum(t, F(0)).astype(F)
    tot = t[0]
    for k in range(1, len(t)):
        tot = F(tot + t[k])
    if not tot > 0:
        return policy_static(len(t))
    return (t / tot).astype(F)


# ---- token tree of width d (Sec. 5 "Verification: Integrating Token Tree"; reading in oracle/definitions.py) ----

def draw_candidates(q, u, greedy: bool = False) -> np.ndarray:
    """d distinct candidate tokens of one depth, [d] int32 (-1 where q has no mass left): candidate c is drawn by the
    inverse-CDF rule from the masses of q with the earlier candidates' masses set to 0 (sampling without replacement),
    with uniform u[c]; greedy: the d most likely tokens in order (lowest id on ties)."""
    q = np.asarray(q, F)
    d = len(u)
    out = np.full(d, -1, np.int32)
    if greedy:
        left = q.astype(np.float64).copy()
        for c in range(min(d, len(q))):
            out[c] = int(np.argmax(left))
            left[out[c]] = -1.0
        return out
    m = masses(q).copy()
    for c in range(d):
        if int(m.sum(dtype=U64)) == 0:
            break
        out[c] = draw(m, u[c])
        m[out[c]] = 0
    return out


def tree_after_rejection(p, q, x: int):
    """(p', q', ok) after candidate x was rejected: r = max(0, p - q) (one rounded subtraction); p' = r / R with
    R = float(sum of masses of r) * 2^-40; q' = q / Qn with Qn = float(sum of masses of q minus the mass of q_x) * 2^-40
    and q'_x = 0.  ok is False when either sum of masses is 0 (nothing to refine: the caller stops trying candidates)."""
    p = np.asarray(p, F); q = np.asarray(q, F)
    r = np.maximum(F(0), p - q)
    MR = int(masses(r).sum(dtype=U64))
    mq = masses(q)
    MQ = int(mq.sum(dtype=U64)) - int(mq[x])
    if MR == 0 or MQ == 0:
        return r, q, False
    Rn = F(np.array(MR, dtype=U64).astype(F) * F(2.0 ** -MASS_BITS))
    Qn = F(np.array(MQ, dtype=U64).astype(F) * F(2.0 ** -MASS_BITS))
    p2 = (r / Rn).astype(F)
    q2 = (q / Qn).astype(F)
    q2[x] = F(0)
    return p2, q2, True
