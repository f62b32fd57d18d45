"""Pins for oracle/definitions.py and oracle/exact32.py (CPU only).

Each test checks the checker against something other than itself: a library
routine (numpy exp/log, scipy), a closed form, an invariant the paper states
(weights non-negative and summing to one; verification with q = p accepts
everything; the emitted token follows the target law), or brute-force
enumeration on tiny vocabularies.
"""
import itertools
import os

import numpy as np
import pytest
import scipy.special

from oracle import definitions as D
from oracle import exact32 as X

F = np.float32
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def lattice(k):
    return F((np.float64(k) + 0.5) * 2.0 ** -23)


# ---------------------------------------------------------------- definitions
def test_softmax_matches_scipy():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((4, 1000)) * 3
    np.testing.assert_allclose(D.softmax(x), scipy.special.softmax(x, axis=-1), rtol=1e-13)


def test_kl_closed_form_two_point():
    # KL(Bern(a) || Bern(b)) = a ln(a/b) + (1-a) ln((1-a)/(1-b))
    for a, b in [(0.3, 0.6), (0.9, 0.5), (0.5, 0.5), (0.01, 0.99)]:
        ref = a * np.log(a / b) + (1 - a) * np.log((1 - a) / (1 - b))
        assert abs(D.kl_divergence([a, 1 - a], [b, 1 - b]) - ref) < 1e-14
        assert abs(D.kl_divergence([a, 1 - a], [b, 1 - b]) - scipy.special.rel_entr([a, 1 - a], [b, 1 - b]).sum()) < 1e-14
    assert D.kl_divergence([1.0, 0.0], [0.5, 0.5]) == pytest.approx(np.log(2))  # 0 ln 0 = 0


def test_kl_direction_is_p_first():
    p, q = np.array([0.7, 0.2, 0.1]), np.array([0.2, 0.3, 0.5])
    assert D.kl_divergence(p, q) != pytest.approx(D.kl_divergence(q, p))
    assert D.kl_divergence(p, q) == pytest.approx(float(scipy.special.rel_entr(p, q).sum()))


def test_tvd_range_and_values():
    assert D.total_variation([1, 0], [0, 1]) == 1.0
    assert D.total_variation([0.5, 0.5], [0.5, 0.5]) == 0.0
    assert D.total_variation([0.7, 0.3], [0.4, 0.6]) == pytest.approx(0.3)


@pytest.mark.parametrize("V", [2, 3, 5, 8])
def test_emitted_law_equals_target_bruteforce(V):
    """Sec. 3: rejection sampling with residual resampling preserves the target law.
    Enumerate every (draft token, accept/reject, replacement) branch."""
    rng = np.random.default_rng(V)
    for trial in range(20):
        p = rng.dirichlet(np.ones(V) * 0.7)
        q = rng.dirichlet(np.ones(V) * 0.7)
        if trial == 0:
            q = p.copy()
        if trial == 1:
            p[0] = 0.0
            p /= p.sum()
        law = np.zeros(V)
        res = D.residual_distribution(p, q)
        for y in range(V):
            if q[y] == 0:
                continue
            acc = D.accept_probability(p[y], q[y])
            law[y] += q[y] * acc
            for z in range(V):
                law[z] += q[y] * (1 - acc) * res[z]
        np.testing.assert_allclose(law, p, atol=1e-12)
        np.testing.assert_allclose(D.emitted_law_one_position(p, q), p, atol=1e-12)


def test_two_position_block_law_bruteforce():
    """gamma = 2 with table-defined conditionals: the first emitted token follows p0 and, when the
    first draft is accepted, the second emitted token follows p1(.|y0)."""
    rng = np.random.default_rng(7)
    V = 3
    p0, q0 = rng.dirichlet(np.ones(V)), rng.dirichlet(np.ones(V))
    p1 = rng.dirichlet(np.ones(V), size=V)      # p1[y0]
    q1 = rng.dirichlet(np.ones(V), size=V)
    first = np.zeros(V)
    joint = np.zeros((V, V))                    # P(y0 accepted, second emitted = v)
    for y0 in range(V):
        a0 = D.accept_probability(p0[y0], q0[y0])
        first[y0] += q0[y0] * a0
        first += q0[y0] * (1 - a0) * D.residual_distribution(p0, q0)
        for y1 in range(V):
            a1 = D.accept_probability(p1[y0, y1], q1[y0, y1])
            joint[y0, y1] += q0[y0] * a0 * q1[y0, y1] * a1
            joint[y0] += q0[y0] * a0 * q1[y0, y1] * (1 - a1) * D.residual_distribution(p1[y0], q1[y0])
    np.testing.assert_allclose(first, p0, atol=1e-12)
    np.testing.assert_allclose(joint, np.minimum(p0, q0)[:, None] * p1, atol=1e-12)


def test_eq1_speedup_worked_example():
    """App. G.1 worked example of Eq. 1 (values in tests/golden/eq1_speedup.txt)."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "eq1_speedup.txt")) if not l.startswith("#")]
    for tau, gamma, ratio, printed in rows:
        assert round(D.expected_speedup(float(tau), int(gamma), float(ratio)), 2) == float(printed)


def test_policy_definitions_invariants():
    rng = np.random.default_rng(3)
    for m in (2, 3, 4, 8):
        e = rng.uniform(0.05, 3.0, size=m)
        w = D.policy_softmax_inv_err(e)
        assert np.all(w >= 0) and abs(w.sum() - 1) < 1e-12
        assert np.argmax(w) == np.argmin(e)
        perm = rng.permutation(m)
        np.testing.assert_allclose(D.policy_softmax_inv_err(e[perm]), w[perm], rtol=1e-12)
        np.testing.assert_allclose(D.policy_softmax_inv_err(np.full(m, 0.7)), 1.0 / m)
    c = D.grid_candidates(10)
    assert c.shape == (11, 2) and np.allclose(c.sum(1), 1) and np.all(c >= 0)
    assert tuple(c[0]) == (1.0, 0.0) and tuple(c[10]) == (0.0, 1.0)


def test_grid_policy_definition_convexity():
    rng = np.random.default_rng(5)
    V = 50
    ps = [rng.dirichlet(np.ones(V)) for _ in range(4)]
    qks = [rng.dirichlet(np.ones(V), size=2) for _ in range(4)]
    j, w, G = D.policy_grid(ps, qks)
    e0 = sum(D.kl_divergence(p, qk[0]) for p, qk in zip(ps, qks))
    e1 = sum(D.kl_divergence(p, qk[1]) for p, qk in zip(ps, qks))
    assert G[0] == pytest.approx(e0) and G[10] == pytest.approx(e1)
    assert G.min() <= min(e0, e1) + 1e-12                      # KL is convex in q
    assert np.all(np.diff(G, 2) >= -1e-12)                      # convex along the segment


# ---------------------------------------------------------------- exact32: exp / log / softmax
def test_xexp_against_numpy():
    rng = np.random.default_rng(0)
    x = -np.abs(rng.standard_normal(200000).astype(F)) * 12
    x[:5] = [0.0, -1e-30, -79.9, -80.5, -1000.0]
    e = X.xexp(x)
    ref = np.exp(x.astype(np.float64))
    ok = x >= -80
    assert np.max(np.abs(e[ok] - ref[ok]) / ref[ok]) < 3e-7
    assert np.all(e[~ok] == 0) and e[0] == 1.0
    assert np.all(np.diff(X.xexp(np.sort(x))) >= 0)             # monotone


def test_xlog_against_numpy():
    rng = np.random.default_rng(0)
    v = np.exp(rng.uniform(-87, 5, 200000)).astype(F)
    v[:4] = [1.0, np.finfo(F).tiny, 2.0, 0.5]
    l = X.xlog(v)
    ref = np.log(v.astype(np.float64))
    assert np.max(np.abs(l - ref) / np.maximum(np.abs(ref), 1.0)) < 3e-7
    assert l[0] == 0.0


def test_softmax_exact_against_definition():
    rng = np.random.default_rng(2)
    for V, scale in [(7, 1.0), (1024, 0.3), (32000, 0.55), (152064, 1.2)]:
        x = (rng.standard_normal((2, V)) * scale).astype(F)
        q = X.softmax_exact(x)
        ref = D.softmax(x)
        assert q.dtype == F
        assert np.max(np.abs(q - ref) / ref) < 1e-6
        assert np.all(np.abs(q.astype(np.float64).sum(-1) - 1) < 1e-6)
    # shift invariance is exact: adding a constant that keeps x - max unchanged bit for bit
    x = np.array([[0.5, -1.25, 3.0, 2.75]], F)
    assert np.array_equal(X.softmax_exact(x), X.softmax_exact(x + F(8.0)))
    # permutation equivariance is exact (order-free reductions)
    x = (rng.standard_normal(5000) * 2).astype(F)
    perm = rng.permutation(5000)
    assert np.array_equal(X.softmax_exact(x)[perm], X.softmax_exact(x[perm]))


# ---------------------------------------------------------------- exact32: ensemble
def test_ensemble_sums_to_one_and_reduces_to_single_drafting():
    rng = np.random.default_rng(4)
    qk = X.softmax_exact((rng.standard_normal((3, 4096))).astype(F))
    for w in ([0.2, 0.5, 0.3], [1 / 3, 1 / 3, 1 / 3], [1, 0, 0], [0, 0, 1]):
        w = np.asarray(w, F)
        q = X.ensemble_exact(qk, w)
        assert abs(q.astype(np.float64).sum() - float(w.astype(np.float64).sum())) < 1e-6
        assert np.max(np.abs(q - D.ensemble(qk, w))) < 1e-9
    # m = 1: bitwise the single drafter's distribution
    assert np.array_equal(X.ensemble_exact(qk[:1], np.array([1.0], F)), qk[0])
    # one-hot weights select a drafter bitwise
    assert np.array_equal(X.ensemble_exact(qk, np.array([0, 1, 0], F)), qk[1])
    # identical rows: the mix does not depend on w (up to rounding)
    same = np.stack([qk[0]] * 3)
    a = X.ensemble_exact(same, np.array([0.2, 0.5, 0.3], F))
    assert np.max(np.abs(a - qk[0]) / qk[0]) < 3e-7


# ---------------------------------------------------------------- exact32: draw
def test_draw_histogram_matches_masses():
    """Over an arithmetic progression of the u lattice every token's count is within 1 of its share."""
    rng = np.random.default_rng(6)
    for V in (2, 5, 16):
        q = rng.dirichlet(np.ones(V) * 0.5).astype(F)
        q[rng.integers(V)] = 0.0                                     # an unreachable token
        m = X.masses(q)
        T = int(m.sum())
        stride = 128
        ks = np.arange(0, 1 << 23, stride)
        toks = np.array([X.draw(m, lattice(k)) for k in ks])
        assert np.all(np.diff(toks) >= 0)                              # monotone in u
        counts = np.bincount(toks, minlength=V)
        expect = len(ks) * m.astype(np.float64) / T
        assert np.all(np.abs(counts - expect) <= 1.0 + 1e-9)
        assert np.all(counts[m == 0] == 0)
    # extremes of the lattice hit the first / last token with mass
    q = np.array([0.0, 0.25, 0.5, 0.25, 0.0], F)
    assert X.draw(X.masses(q), lattice(0)) == 1
    assert X.draw(X.masses(q), lattice((1 << 23) - 1)) == 3


def test_draw_bruteforce_small_integer_masses():
    """Independent brute force: expand masses into a list of token ids and index it."""
    rng = np.random.default_rng(8)
    for _ in range(20):
        m = rng.integers(0, 6, size=7).astype(np.uint64)
        if m.sum() == 0:
            m[3] = 2
        bag = np.repeat(np.arange(7), m.astype(np.int64))            # token of every unit of mass
        T = len(bag)
        for k in rng.integers(0, 1 << 23, size=50):
            pos = ((2 * int(k) + 1) * T) // (1 << 24)                # unit of mass under u
            assert X.draw(m, lattice(k)) == bag[pos]


def test_argmax_lowest_on_ties():
    assert X.argmax_lowest(np.array([0.1, 0.4, 0.4, 0.1], F)) == 1


# ---------------------------------------------------------------- exact32: verification
def test_accept_rule_extremes_and_frequency():
    ks = np.concatenate([[0, 1, (1 << 23) - 1], np.arange(5, 1 << 23, 4099)])
    for q_y in (F(0.3), F(1e-6), F(3.1e-5)):
        assert all(X.accept(q_y, q_y, lattice(k)) for k in ks)         # q = p accepts everything
        assert not any(X.accept(F(0), q_y, lattice(k)) for k in ks)    # p(y) = 0 never accepted
        assert all(X.accept(F(2) * q_y, q_y, lattice(k)) for k in ks)  # p > q always
    p_y, q_y = F(0.2), F(0.5)
    freq = np.mean([X.accept(p_y, q_y, lattice(k)) for k in ks])
    assert abs(freq - D.accept_probability(0.2, 0.5)) < 2e-3


@pytest.mark.parametrize("V", [2, 3, 5, 8])
def test_exact_round_preserves_target_law_by_lattice_enumeration(V):
    """Compose the three independent uniforms from 1-D lattice sweeps of the exact32 routines:
    P(y), P(accept | y), P(z | reject).  The emitted law must equal p to lattice resolution."""
    rng = np.random.default_rng(100 + V)
    N = 4096
    ks = (np.arange(N) * ((1 << 23) // N) + 17)
    for trial in range(3):
        lp = (rng.standard_normal(V) * 1.5).astype(F)
        lq = (rng.standard_normal((2, V)) * 1.5).astype(F)
        p = X.softmax_exact(lp)
        q = X.ensemble_exact(X.softmax_exact(lq), np.array([0.6, 0.4], F))
        mq, mr = X.masses(q), X.residual_masses(p, q)
        py = np.bincount([X.draw(mq, lattice(k)) for k in ks], minlength=V) / N
        pz = np.bincount([X.draw(mr, lattice(k)) for k in ks], minlength=V) / N
        law = np.zeros(V)
        for y in range(V):
            acc = np.mean([X.accept(p[y], q[y], lattice(k)) for k in ks])
            law[y] += py[y] * acc
            law += py[y] * (1 - acc) * pz
        assert np.max(np.abs(law - p.astype(np.float64))) < 4.0 * V / N


def test_residual_masses_nonnegative_and_zero_when_equal():
    rng = np.random.default_rng(9)
    p = X.softmax_exact(rng.standard_normal(100).astype(F))
    assert int(X.residual_masses(p, p).sum()) == 0
    q = X.softmax_exact(rng.standard_normal(100).astype(F))
    r = X.residual_masses(p, q).astype(np.float64) * 2.0 ** -40
    np.testing.assert_allclose(r / r.sum(), D.residual_distribution(p, q), atol=1e-9)


# ---------------------------------------------------------------- exact32: deviation and policies
def test_kl_fixed_against_definition():
    rng = np.random.default_rng(10)
    for V in (16, 1024, 32000):
        p = X.softmax_exact((rng.standard_normal(V) * 1.2).astype(F))
        q = X.softmax_exact((rng.standard_normal(V) * 0.6).astype(F))
        assert X.kl_fixed(p, p) == 0
        val = X.kl_fixed(p, q) * 2.0 ** -40
        assert val > 0
        assert abs(val - D.kl_divergence(p, q)) < 2e-6
        tv = X.tvd_fixed(p, q) * 2.0 ** -41
        assert 0 <= tv <= 1 and abs(tv - D.total_variation(p, q)) < 1e-6
    # zero handling: p_v = 0 contributes nothing; q_v = 0 is floored, not infinite
    p = np.array([0.5, 0.5, 0.0], F)
    q = np.array([0.5, 0.0, 0.5], F)
    ref = D.kl_divergence(p, q, q_floor=float(np.finfo(F).tiny))
    assert abs(X.kl_fixed(p, q) * 2.0 ** -40 - ref) < 1e-4 and np.isfinite(ref)
    # order-free: permuting the vocabulary gives the same integer
    perm = rng.permutation(1024)
    p = X.softmax_exact(rng.standard_normal(1024).astype(F))
    q = X.softmax_exact(rng.standard_normal(1024).astype(F))
    assert X.kl_fixed(p, q) == X.kl_fixed(p[perm], q[perm])


def test_policy_softmax_inv_err_exact_invariants():
    rng = np.random.default_rng(11)
    for m in (2, 3, 4, 8):
        e = rng.uniform(0.05, 3.0, size=m).astype(F)
        w = X.policy_softmax_inv_err(e)
        assert w.dtype == F and np.all(w >= 0) and abs(float(w.astype(np.float64).sum()) - 1) < 1e-6
        np.testing.assert_allclose(w, D.policy_softmax_inv_err(e), atol=1e-6)
        order = np.argsort(e)
        assert np.all(np.diff(w[order]) < 0)                            # smaller error, larger weight
        perm = rng.permutation(m)
        np.testing.assert_allclose(X.policy_softmax_inv_err(e[perm]), w[perm], atol=1e-7)
        eq = X.policy_softmax_inv_err(np.full(m, 0.7, F))
        assert np.all(eq == eq[0]) and abs(float(eq[0]) - 1.0 / m) < 1e-7
    # e -> 0 is clamped, not infinite
    w = X.policy_softmax_inv_err(np.array([0.0, 1.0], F))
    assert np.all(np.isfinite(w)) and w[0] == 1.0
    # temperature flattens
    e = np.array([0.2, 0.5, 1.0], F)
    assert X.policy_softmax_inv_err(e, tau=4.0).max() < X.policy_softmax_inv_err(e, tau=1.0).max()


def test_grid_weights_and_static():
    for j in range(11):
        w = X.grid_weight(j)
        assert w.dtype == F and np.all(w >= 0) and abs(float(w[0]) + float(w[1]) - 1) < 1e-7
        np.testing.assert_allclose(w, D.grid_candidates(10)[j], atol=1e-7)
    assert tuple(X.grid_weight(0)) == (1.0, 0.0) and tuple(X.grid_weight(10)) == (0.0, 1.0)
    for m in (1, 2, 3, 4):
        np.testing.assert_allclose(X.policy_static(m), 1.0 / m, rtol=1e-7)


# ---------------------------------------------------------------- token tree of width d
@pytest.mark.parametrize("V,d", [(2, 2), (3, 2), (3, 3), (5, 2), (5, 3)])
def test_tree_depth_emitted_law_equals_target_bruteforce(V, d):
    """Sec. 5 "Verification: Integrating Token Tree" must keep Sec. 3's guarantee: with d candidates per depth, drawn
    without replacement and tried by recursive rejection, the emitted token still follows the target law.  Every
    ordered candidate tuple and every accept / reject / replacement branch is enumerated."""
    rng = np.random.default_rng(40 + 10 * V + d)
    for trial in range(12):
        p = rng.dirichlet(np.ones(V) * 0.7)
        q = rng.dirichlet(np.ones(V) * 0.7)
        if trial == 0:
            q = p.copy()
        if trial == 1:
            p[0] = 0.0; p /= p.sum()
        if trial == 2:
            q[-1] = 0.0; q /= q.sum()                       # the drafter never proposes a token the target wants
        outs = D.tree_depth_outcomes(p, q, d)
        assert abs(sum(pr for pr, _, _ in outs) - 1.0) < 1e-12
        np.testing.assert_allclose(D.tree_depth_emitted_law(p, q, d), p, atol=1e-12)
        # more candidates can only raise the chance that a drafted token is accepted
        acc = [sum(pr for pr, _, lvl in D.tree_depth_outcomes(p, q, w) if lvl >= 0) for w in range(1, d + 1)]
        assert all(acc[i + 1] >= acc[i] - 1e-12 for i in range(len(acc) - 1))
        assert abs(acc[0] - np.minimum(p, q).sum()) < 1e-12        # width 1 is plain speculative sampling


def test_tree_two_depth_block_law_bruteforce():
    """Two depths, width 2 and 3, table-defined conditionals: the first emitted token follows p0 and, whenever a
    drafted token was accepted at depth 0 (primary or sibling), the second emitted token follows p1(. | first)."""
    rng = np.random.default_rng(77)
    V = 3
    for d in (2, 3):
        p0, q0 = rng.dirichlet(np.ones(V)), rng.dirichlet(np.ones(V))
        p1 = rng.dirichlet(np.ones(V), size=V); q1 = rng.dirichlet(np.ones(V), size=V)
        first = np.zeros(V); joint = np.zeros((V, V)); accepted = np.zeros(V)
        for prob, tok, lvl in D.tree_depth_outcomes(p0, q0, d):
            first[tok] += prob
            if lvl < 0:
                continue                                    # replacement: the round ends with one token
            accepted[tok] += prob
            # primary: depth 1 is another tree depth on (p1, q1)[tok]; sibling: a leaf, the next token comes from p1[tok]
            second = D.tree_depth_emitted_law(p1[tok], q1[tok], d) if lvl == 0 else p1[tok]
            joint[tok] += prob * second
        np.testing.assert_allclose(first, p0, atol=1e-12)
        np.testing.assert_allclose(joint, accepted[:, None] * p1, atol=1e-12)


def test_draw_candidates_without_replacement():
    rng = np.random.default_rng(78)
    q = X.softmax_exact((rng.standard_normal(6) * 1.2).astype(F))
    N = 2048
    ks = np.arange(N) * ((1 << 23) // N) + 5
    # distinct tokens; the second candidate follows q restricted to the others
    pair = np.zeros((6, 6))
    for k0 in ks[::32]:
        for k1 in ks[::32]:
            c = X.draw_candidates(q, np.array([lattice(k0), lattice(k1)], F))
            assert c[0] != c[1] and c[0] == X.draw(X.masses(q), lattice(k0))
            pair[c[0], c[1]] += 1
    pair /= pair.sum()
    qd = q.astype(np.float64)
    ref = qd[:, None] * qd[None, :] / (1.0 - qd[:, None])
    np.fill_diagonal(ref, 0.0)
    assert np.max(np.abs(pair - ref)) < 0.03
    # greedy: the d most likely tokens in order, lowest id on ties; more candidates than tokens -> -1
    assert list(X.draw_candidates(np.array([0.2, 0.5, 0.2, 0.1], F), np.zeros(3, F), greedy=True)) == [1, 0, 2]
    assert list(X.draw_candidates(np.array([0.5, 0.5], F), np.zeros(3, F), greedy=True)) == [0, 1, -1]
    # all mass on one token: there is no second candidate
    assert list(X.draw_candidates(np.array([0.0, 1.0, 0.0], F), np.array([lattice(3), lattice(9)], F))) == [1, -1]


@pytest.mark.parametrize("V", [3, 5])
def test_exact_tree_depth_preserves_target_law_by_lattice_enumeration(V):
    """Width 2 in the kernel's arithmetic, composed from 1-D lattice sweeps: P(x0), P(x1 | x0), the two acceptance
    probabilities and the replacement law after two rejections."""
    rng = np.random.default_rng(300 + V)
    N = 2048
    ks = (np.arange(N) * ((1 << 23) // N) + 11)
    for trial in range(2):
        p = X.softmax_exact((rng.standard_normal(V) * 1.3).astype(F))
        q = X.softmax_exact((rng.standard_normal(V) * 1.3).astype(F))
        mq = X.masses(q)
        px0 = np.bincount([X.draw(mq, lattice(k)) for k in ks], minlength=V) / N
        law = np.zeros(V)
        for x0 in range(V):
            if px0[x0] == 0:
                continue
            a0 = np.mean([X.accept(p[x0], q[x0], lattice(k)) for k in ks])
            law[x0] += px0[x0] * a0
            p2, q2, ok = X.tree_after_rejection(p, q, x0)
            np.testing.assert_allclose(p2, D.tree_after_rejection(p, q, x0)[0], atol=1e-6)
            np.testing.assert_allclose(q2, D.tree_after_rejection(p, q, x0)[1], atol=1e-6)
            assert ok and q2[x0] == 0
            m1 = mq.copy(); m1[x0] = 0
            px1 = np.bincount([X.draw(m1, lattice(k)) for k in ks], minlength=V) / N
            for x1 in range(V):
                if px1[x1] == 0:
                    continue
                a1 = np.mean([X.accept(p2[x1], q2[x1], lattice(k)) for k in ks])
                law[x1] += px0[x0] * (1 - a0) * px1[x1] * a1
                mr = X.residual_masses(p2, q2)
                if int(mr.sum()) == 0:
                    mr = X.masses(p2)
                pz = np.bincount([X.draw(mr, lattice(k)) for k in ks], minlength=V) / N
                law += px0[x0] * (1 - a0) * px1[x1] * (1 - a1) * pz
        assert np.max(np.abs(law - p.astype(np.float64))) < 8.0 * V / N
