"""Pins for oracle/tabed.py (CPU only): the round's structure against what the paper fixes."""
import numpy as np
import pytest

from oracle import definitions as D
from oracle import exact32 as X
from oracle.drafter import OracleDrafter
from oracle.tabed import TabedOracle
from paper_2601_20357_b200 import workloads as W

F = np.float32


def lat(rng, shape):
    return W.lattice_uniforms(rng, shape)


def mk(m=3, B=2, gamma=3, h=2, policy=W.POLICY_SOFTMAX_INV_ERR, V=64, **kw):
    return TabedOracle(n_inputs=m, n_requests=B, gamma=gamma, window_h=h, policy=policy, vocab=V, **kw)


def rand_logits(rng, gamma, B, m, V, scale=1.0):
    return (rng.standard_normal((gamma, B, m, V)) * scale).astype(F)


def test_initial_weights_are_static_equal():
    o = mk(m=4)
    assert np.all(o.w == F(0.25))


def test_single_input_round_equals_plain_speculative_decoding():
    """m = 1: TABED reduces to single drafting.  Compare with a separately written SD round."""
    rng = np.random.default_rng(0)
    V, G = 50, 4
    for trial in range(30):
        o = mk(m=1, B=1, gamma=G, h=2, V=V)
        lg = rand_logits(rng, G, 1, 1, V, 1.5)
        tl = (rng.standard_normal((1, G + 1, V)) * 1.5).astype(F)
        ud, ua, ur = lat(rng, (1, G)), lat(rng, (1, G)), lat(rng, (1,))
        toks, q = o.draft_round_logits(lg, ud)
        a, z = o.verify(tl, ua, ur)
        w, am = o.update_weights()
        # plain SD, Sec. 3 items 1-3
        qs = [X.softmax_exact(lg[i, 0, 0]) for i in range(G)]
        ps = [X.softmax_exact(tl[0, i]) for i in range(G + 1)]
        ys = [X.draw(X.masses(qs[i]), ud[0, i]) for i in range(G)]
        acc = 0
        while acc < G and X.accept(ps[acc][ys[acc]], qs[acc][ys[acc]], ua[0, acc]):
            acc += 1
        if acc < G:
            mr = X.residual_masses(ps[acc], qs[acc])
            zz = X.draw(mr if mr.sum() > 0 else X.masses(ps[acc]), ur[0])
        else:
            zz = X.draw(X.masses(ps[G]), ur[0])
        assert list(toks[0]) == ys and int(a[0]) == acc and int(z[0]) == zz
        assert np.array_equal(q[0], np.stack(qs))
        assert w.shape == (1, 1) and w[0, 0] == 1.0 and am[0] == 0


def test_q_equals_p_accepts_every_token():
    rng = np.random.default_rng(1)
    G, V = 5, 200
    for trial in range(20):
        o = mk(m=1, B=2, gamma=G, V=V)
        lg = rand_logits(rng, G, 2, 1, V, 2.0)
        toks, _ = o.draft_round_logits(lg, lat(rng, (2, G)))
        tl = np.concatenate([lg[:, :, 0, :].transpose(1, 0, 2), lg[-1:, :, 0, :].transpose(1, 0, 2)], axis=1)
        a, z = o.verify(tl, lat(rng, (2, G)), lat(rng, (2,)))
        assert np.all(a == G)


def test_zero_target_probability_rejects_and_later_tokens_are_discarded():
    rng = np.random.default_rng(2)
    G, V = 4, 30
    o = mk(m=2, B=1, gamma=G, V=V, policy=W.POLICY_GRID_MT)
    lg = rand_logits(rng, G, 1, 2, V)
    toks, q = o.draft_round_logits(lg, lat(rng, (1, G)))
    tl = np.einsum("gbnv->bgv", lg)[:, :, :] / 2
    tl = np.concatenate([tl, tl[:, -1:]], axis=1).astype(F)
    tl[0, 1, toks[0, 1]] = -200.0                     # target gives the 2nd drafted token probability 0
    tl[0, 0] = lg[0, 0].mean(0) + 50.0 * np.eye(V, dtype=F)[toks[0, 0]]   # and makes the 1st certain
    a, z = o.verify(tl, lat(rng, (1, G)), lat(rng, (1,)))
    assert a[0] == 1 and z[0] != toks[0, 1]
    # the replacement is drawn from the residual: it must have p > q there
    assert o.p[0, 1, z[0]] > o.q[0, 1, z[0]]


def test_greedy_mode():
    rng = np.random.default_rng(3)
    G, V = 3, 40
    o = mk(m=2, B=1, gamma=G, V=V, policy=W.POLICY_STATIC, sample_mode=W.MODE_GREEDY)
    lg = rand_logits(rng, G, 1, 2, V)
    toks, q = o.draft_round_logits(lg, lat(rng, (1, G)))
    assert list(toks[0]) == [int(np.argmax(q[0, i])) for i in range(G)]
    tl = (rng.standard_normal((1, G + 1, V))).astype(F)
    tl[0, 0, toks[0, 0]] = 30.0
    a, z = o.verify(tl, lat(rng, (1, G)), lat(rng, (1,)))
    exp_a = 0
    while exp_a < G and int(np.argmax(tl[0, exp_a])) == toks[0, exp_a]:
        exp_a += 1
    assert a[0] == exp_a >= 1 and z[0] == int(np.argmax(tl[0, a[0]]))


def test_weights_sum_to_one_and_track_the_better_drafter():
    """Sec. 4.1: methods with higher weights are closer to the target."""
    rng = np.random.default_rng(4)
    G, V, m = 3, 300, 3
    o = mk(m=m, B=1, gamma=G, h=4, V=V)
    for rnd in range(6):
        lg = rand_logits(rng, G, 1, m, V, 1.0)
        o.draft_round_logits(lg, lat(rng, (1, G)))
        tl = np.concatenate([lg[:, :, 1, :], lg[-1:, :, 1, :]], axis=0).transpose(1, 0, 2)   # target = drafter 1
        tl = (tl + 0.05 * rng.standard_normal(tl.shape)).astype(F)
        o.verify(tl, lat(rng, (1, G)), lat(rng, (1,)))
        w, am = o.update_weights()
        assert np.all(w >= 0) and abs(float(w.astype(np.float64).sum()) - 1) < 1e-6
        assert am[0] == 1 and w[0, 1] > w[0, 0] and w[0, 1] > w[0, 2]


def test_grid_policy_matches_definition_and_endpoints():
    rng = np.random.default_rng(5)
    G, V = 3, 120
    o = mk(m=2, B=1, gamma=G, h=0, V=V, policy=W.POLICY_GRID_MT)
    ps, qks = [], []
    for rnd in range(4):
        lg = rand_logits(rng, G, 1, 2, V, 1.0)
        o.draft_round_logits(lg, lat(rng, (1, G)))
        mix = 0.7 * lg[:, :, 0, :] + 0.3 * lg[:, :, 1, :]
        tl = np.concatenate([mix, mix[-1:]], axis=0).transpose(1, 0, 2)
        tl = (tl + 0.3 * rng.standard_normal(tl.shape)).astype(F)
        a, z = o.verify(tl, lat(rng, (1, G)), lat(rng, (1,)))
        for i in range(min(int(a[0]), G - 1) + 1):
            ps.append(o.p[0, i].copy()); qks.append(o.qk[0, i].copy())
        w, am = o.update_weights()
        j_def, w_def, G_def = D.policy_grid(ps, qks)
        np.testing.assert_allclose(o.window_error(0), G_def, atol=2e-5)
        assert int(o.j_star[0]) == j_def
        np.testing.assert_allclose(w[0], w_def, atol=1e-7)
        e0 = sum(D.kl_divergence(p, qk[0]) for p, qk in zip(ps, qks))
        e1 = sum(D.kl_divergence(p, qk[1]) for p, qk in zip(ps, qks))
        we = o.window_error(0)
        assert abs(we[0] - e0) < 2e-5 and abs(we[10] - e1) < 2e-5 and we.min() <= min(we[0], we[10])


@pytest.mark.parametrize("h", [0, 3])
def test_tvd_softmax_policy_matches_definitions(h):
    """Sec. 4.1 with the total-variation distance, App. B softmax(1/e) policy: the weights of the round
    machine equal the fp64 definition applied to the fp64 TVD sums over the window.  The window error
    is 1/2 sum |p - q| (a factor-of-two slip in its fixed-point scale doubles every e, halves every
    1/e and moves the weights far outside the tolerance)."""
    rng = np.random.default_rng(21)
    G, V, m = 3, 400, 3
    o = mk(m=m, B=1, gamma=G, h=h, V=V, distance=W.DIST_TVD)
    hist = []
    moved = 0.0
    for rnd in range(5):
        # drafters at different distances from the target so that the three errors are well separated
        base = rng.standard_normal((G, 1, 1, V)).astype(F)
        lg = (base + np.array([0.3, 0.9, 1.8], F)[None, None, :, None] * rng.standard_normal((G, 1, m, V))).astype(F)
        o.draft_round_logits(lg, lat(rng, (1, G)))
        tl = np.concatenate([base[:, :, 0, :], base[-1:, :, 0, :]], axis=0).transpose(1, 0, 2).astype(F)
        a, _ = o.verify(tl, lat(rng, (1, G)), lat(rng, (1,)))
        for i in range(min(int(a[0]), G - 1) + 1):
            hist.append([D.total_variation(o.p[0, i], o.qk[0, i, k]) for k in range(m)])
        w, am = o.update_weights()
        win = hist[-h:] if h > 0 else hist
        e_def = np.sum(win, axis=0)
        assert np.all(e_def > 0) and np.all(e_def <= len(win))                       # each TVD lies in [0, 1]
        np.testing.assert_allclose(o.window_error(0), e_def, atol=1e-5)
        np.testing.assert_allclose([float(X.fixed_to_float(int(t), True)) for t in o.running[0]], e_def, atol=1e-5)
        w_def = D.policy_softmax_inv_err(e_def)
        np.testing.assert_allclose(w[0], w_def, atol=2e-5)
        assert am[0] == int(np.argmax(w_def))
        moved = max(moved, float(np.max(np.abs(w_def - D.policy_softmax_inv_err(2.0 * e_def)))))
    assert moved > 1e-2          # the test has the resolution to see a doubled error


def test_window_h1_depends_only_on_last_verified_position():
    """App. B: h = 1 uses only the ground truth of the previous decoding step."""
    rng = np.random.default_rng(6)
    G, V, m = 3, 80, 3
    outs = []
    last_lg = rand_logits(rng, G, 1, m, V)
    last_tl = (rng.standard_normal((1, G + 1, V))).astype(F)
    ud, ua, ur = lat(rng, (1, G)), lat(rng, (1, G)), lat(rng, (1,))
    for history in range(2):
        o = mk(m=m, B=1, gamma=G, h=1, V=V, policy=W.POLICY_STATIC)   # static: drafts do not depend on w
        o.policy = W.POLICY_SOFTMAX_INV_ERR
        o.n_dev = m
        for _ in range(history * 3):
            o.w[:] = X.policy_static(m)
            o.draft_round_logits(rand_logits(rng, G, 1, m, V), lat(rng, (1, G)))
            o.verify((rng.standard_normal((1, G + 1, V))).astype(F), lat(rng, (1, G)), lat(rng, (1,)))
            o.update_weights()
        o.w[:] = X.policy_static(m)
        o.draft_round_logits(last_lg, ud)
        a, _ = o.verify(last_tl, ua, ur)
        w, _ = o.update_weights()
        i_last = min(int(a[0]), G - 1)
        e = [X.fixed_to_float(X.kl_fixed(o.p[0, i_last], o.qk[0, i_last, k])) for k in range(m)]
        assert np.array_equal(w[0], X.policy_softmax_inv_err(np.array(e, F)))
        outs.append(w.copy())
    assert np.array_equal(outs[0], outs[1])


def test_window_sum_equals_sum_of_last_h_positions_and_all_mode():
    rng = np.random.default_rng(7)
    G, V, m, h = 2, 60, 2, 3
    o = mk(m=m, B=1, gamma=G, h=h, V=V)
    o_all = mk(m=m, B=1, gamma=G, h=0, V=V)
    hist = []
    for rnd in range(5):
        lg = rand_logits(rng, G, 1, m, V)
        tl = (rng.standard_normal((1, G + 1, V))).astype(F)
        ud, ua, ur = lat(rng, (1, G)), lat(rng, (1, G)), lat(rng, (1,))
        for oo in (o, o_all):
            oo.w[:] = X.policy_static(m)
            oo.draft_round_logits(lg, ud)
            a, _ = oo.verify(tl, ua, ur)
        for i in range(min(int(a[0]), G - 1) + 1):
            hist.append([D.kl_divergence(o.p[0, i], o.qk[0, i, k]) for k in range(m)])
        o.update_weights(); o_all.update_weights()
        np.testing.assert_allclose(o.window_error(0), np.sum(hist[-h:], axis=0), atol=1e-5)
        np.testing.assert_allclose(o_all.window_error(0), np.sum(hist, axis=0), atol=1e-5)


def test_positions_after_first_rejection_and_bonus_are_not_in_window():
    rng = np.random.default_rng(8)
    G, V, m = 4, 50, 2
    for want_a in (0, 2, G):
        o = mk(m=m, B=1, gamma=G, h=0, V=V)
        lg = rand_logits(rng, G, 1, m, V)
        toks, q = o.draft_round_logits(lg, lat(rng, (1, G)))
        tl = np.zeros((1, G + 1, V), F)
        for i in range(G):
            tl[0, i] = 40.0 * np.eye(V, dtype=F)[toks[0, i]] if i < want_a else -60.0 * np.eye(V, dtype=F)[toks[0, i]]
        a, z = o.verify(tl, lat(rng, (1, G)), lat(rng, (1,)))
        assert a[0] == want_a
        o.update_weights()
        assert o.count[0] == min(want_a, G - 1) + 1


def test_drafter_bookkeeping_lengths_and_pending():
    cfg = W.DrafterCfg(1, 32, 2, 2, 64, 40, "fp32")
    wl = W.Workload(name="t", config_id=77, drafter=cfg, n_inputs=2, n_requests=1, gamma=3, window_h=2,
                    rounds=1, policy=W.POLICY_STATIC)
    dr = OracleDrafter(cfg, W.make_weights(wl))
    rng = np.random.default_rng(9)
    o = TabedOracle(n_inputs=2, n_requests=1, gamma=3, window_h=2, policy=W.POLICY_STATIC, vocab=40,
                    drafter=dr, kv_capacity=64)
    o.prefill(0, [W.Segment("tokens", np.arange(5, dtype=np.int32))])
    o.prefill(1, [W.Segment("embeds", rng.standard_normal((2, 32)).astype(F))])
    o.set_pending([7])
    assert list(o.kv_lengths()) == [5, 2]
    # round 1: force full acceptance -> two pending tokens, lengths advance by 1 + gamma - 1
    toks, q = o.draft_round(lat(rng, (1, 3)))
    assert list(o.kv_lengths()) == [5 + 3, 2 + 3]
    tl = np.stack([40.0 * np.eye(40, dtype=F)[t] for t in list(toks[0]) + [11]])[None]
    a, z = o.verify(tl, lat(rng, (1, 3)), lat(rng, (1,)))
    assert a[0] == 3 and z[0] == 11
    o.update_weights()
    assert list(o.kv_lengths()) == [8, 5] and o.pending[0] == [int(toks[0, 2]), 11]
    # round 2: reject at once -> catch-up consumed both pending tokens, drafts rolled back
    toks2, _ = o.draft_round(lat(rng, (1, 3)))
    assert list(o.kv_lengths()) == [8 + 2 + 2, 5 + 2 + 2]
    tl = np.stack([-60.0 * np.eye(40, dtype=F)[t] for t in list(toks2[0]) + [0]])[None]
    a, z = o.verify(tl, lat(rng, (1, 3)), lat(rng, (1,)))
    assert a[0] == 0
    o.update_weights()
    assert list(o.kv_lengths()) == [10, 7] and o.pending[0] == [int(z[0])]
    # the drafter saw the same continuation on both rows: logits of the two rows differ only by prefix
    assert not np.array_equal(o.logits[0, 0, 0], o.logits[0, 0, 1])


def test_identical_prefixes_make_ensemble_independent_of_weights():
    cfg = W.DrafterCfg(1, 32, 2, 2, 64, 40, "fp32")
    wl = W.Workload(name="t", config_id=78, drafter=cfg, n_inputs=2, n_requests=1, gamma=2, window_h=2,
                    rounds=1, policy=W.POLICY_STATIC)
    dr = OracleDrafter(cfg, W.make_weights(wl))
    rng = np.random.default_rng(10)
    ud = lat(rng, (1, 2))
    res = []
    for w in ([0.5, 0.5], [0.9, 0.1]):
        o = TabedOracle(n_inputs=2, n_requests=1, gamma=2, window_h=2, policy=W.POLICY_STATIC, vocab=40,
                        drafter=dr, kv_capacity=32)
        for r in range(2):
            o.prefill(r, [W.Segment("tokens", np.arange(6, dtype=np.int32))])
        o.set_pending([3])
        o.w[0] = np.asarray(w, F)
        toks, q = o.draft_round(ud)
        res.append((toks.copy(), q.copy()))
    assert np.array_equal(res[0][0], res[1][0])
    assert np.max(np.abs(res[0][1] - res[1][1])) < 1e-8


def test_tiny_workload_free_run_smoke():
    wl = W.TINY
    dr = OracleDrafter(wl.drafter, W.make_weights(wl))
    o = TabedOracle(n_inputs=2, n_requests=1, gamma=wl.gamma, window_h=wl.window_h, policy=wl.policy,
                    vocab=wl.drafter.vocab, drafter=dr, kv_capacity=wl.kv_capacity)
    for r, segs in enumerate(W.make_prefixes(wl)):
        o.prefill(r, segs)
    o.set_pending(W.initial_pending(wl))
    acc = []
    for rnd in range(4):
        ud, ua, ur = W.round_uniforms(wl, rnd)
        o.draft_round(ud)
        a, z = o.verify(W.target_logits(wl, rnd, o.logits), ua, ur)
        w, am = o.update_weights()
        acc.append(int(a[0]))
        assert abs(float(w.sum()) - 1) < 1e-6 and 0 <= a[0] <= wl.gamma and 0 <= z[0] < wl.drafter.vocab
    assert o.count[0] == sum(min(a, wl.gamma - 1) + 1 for a in acc)


# --------------------------------------------------------------------------------------------------
# Pooled multimodal drafting input (Sec. 5): 2 x 2 average pooling of the visual tokens' grid
# --------------------------------------------------------------------------------------------------
def test_pool_2x2_against_library_pooling():
    """torch's avg_pool2d (an independent routine) on the same grid, features as channels."""
    import torch
    from oracle.definitions import pool_image_tokens_2x2
    rng = np.random.default_rng(5)
    for gh, gw, d in ((24, 24, 32), (2, 2, 5), (6, 4, 7)):
        x = rng.standard_normal((gh * gw, d)).astype(np.float32)
        got = pool_image_tokens_2x2(x, gh, gw)
        ref = torch.nn.functional.avg_pool2d(torch.from_numpy(x).double().reshape(gh, gw, d).permute(2, 0, 1)[None], 2)[0]
        ref = ref.permute(1, 2, 0).reshape(-1, d).numpy()
        assert got.shape == ((gh // 2) * (gw // 2), d) and got.dtype == np.float32
        assert np.max(np.abs(got.astype(np.float64) - ref)) <= 1e-7 * max(1.0, np.max(np.abs(ref)))


def test_pool_2x2_closed_forms_and_token_count():
    from oracle.definitions import pool_image_tokens_2x2
    # the paper's default: 576 visual tokens -> 144
    assert pool_image_tokens_2x2(np.zeros((576, 3), np.float32), 24, 24).shape == (144, 3)
    # a constant grid stays constant; a ramp over rows/columns gives the block centres
    assert np.array_equal(pool_image_tokens_2x2(np.full((16, 2), 1.25, np.float32), 4, 4), np.full((4, 2), 1.25, np.float32))
    ii, jj = np.meshgrid(np.arange(4), np.arange(6), indexing="ij")
    x = np.stack([ii.ravel(), jj.ravel(), (10 * ii + jj).ravel()], axis=1).astype(np.float32)
    got = pool_image_tokens_2x2(x, 4, 6).reshape(2, 3, 3)
    for i in range(2):
        for j in range(3):
            assert np.allclose(got[i, j], [2 * i + 0.5, 2 * j + 0.5, 10 * (2 * i + 0.5) + 2 * j + 0.5])
    # a transposed grid (rows and columns swapped) must give a different result for a non-symmetric input:
    # the pooling follows the row-major arrangement
    assert not np.array_equal(pool_image_tokens_2x2(x, 4, 6), pool_image_tokens_2x2(x, 6, 4))
    # one block only sees its own four tokens
    x = np.zeros((16, 1), np.float32); x[5] = 4.0          # token (1, 1) -> block (0, 0)
    assert np.array_equal(pool_image_tokens_2x2(x, 4, 4).ravel(), np.array([1, 0, 0, 0], np.float32))
    for bad in ((3, 4), (4, 3)):
        with pytest.raises(ValueError):
            pool_image_tokens_2x2(np.zeros((12, 1), np.float32), *bad)


# ---------------------------------------------------------------- the other weight policies
def test_random_policy_is_uniform_on_the_simplex():
    """Sec. 5 "Effectiveness of Dynamic Weights": non-negative sum-to-one random weights.  A uniform point of the
    simplex: every weight has mean 1/m and one coordinate follows Beta(1, m-1) (for two methods: uniform on (0, 1))."""
    rng = np.random.default_rng(31)
    for m in (2, 3, 5):
        u = lat(rng, (4000, m))
        w = np.stack([X.policy_random(u[i]) for i in range(len(u))]).astype(np.float64)
        assert np.all(w >= 0) and np.allclose(w.sum(axis=1), 1.0, atol=1e-6)
        np.testing.assert_allclose(w, np.stack([D.policy_random(u[i]) for i in range(len(u))]), atol=2e-6)
        np.testing.assert_allclose(w.mean(axis=0), 1.0 / m, atol=0.02)
        # marginal of one coordinate of a flat Dirichlet is Beta(1, m-1): P(w_0 <= x) = 1 - (1-x)^(m-1)
        for x in (0.1, 0.3, 0.6):
            assert abs(float((w[:, 0] <= x).mean()) - (1 - (1 - x) ** (m - 1))) < 0.03
    o = mk(m=3, B=2, gamma=2, h=2, V=50, policy=W.POLICY_RANDOM)
    lg = rand_logits(rng, 2, 2, 3, 50)
    o.draft_round_logits(lg, lat(rng, (2, 2)))
    o.verify(rng.standard_normal((2, 3, 50)).astype(F), lat(rng, (2, 2)), lat(rng, (2,)))
    up = lat(rng, (2, 3))
    w, am = o.update_weights(up)
    assert np.array_equal(w[0], X.policy_random(up[0])) and np.array_equal(w[1], X.policy_random(up[1]))


def test_hard_label_grid_selection_counts_token_matches():
    """Sec. 4.1: with hard labels w* maximises the number of token matches over the window."""
    rng = np.random.default_rng(32)
    G, V = 3, 40
    o = mk(m=2, B=1, gamma=G, h=0, V=V, policy=W.POLICY_GRID_HARD)
    labels, qks = [], []
    for rnd in range(5):
        lg = rand_logits(rng, G, 1, 2, V, 2.0)
        o.draft_round_logits(lg, lat(rng, (1, G)))
        tl = np.concatenate([lg[:, :, 1, :], lg[-1:, :, 1, :]], axis=0).transpose(1, 0, 2)      # the target follows drafter 1
        tl = (3.0 * tl + 0.5 * rng.standard_normal(tl.shape)).astype(F)
        a, z = o.verify(tl, lat(rng, (1, G)), lat(rng, (1,)))
        for i in range(min(int(a[0]), G - 1) + 1):
            labels.append(int(o.tokens[0, i]) if i < a[0] else int(z[0])); qks.append(o.qk[0, i].copy())
        w, am = o.update_weights()
        j_def, w_def, counts = D.policy_grid_hard(labels, qks)
        assert np.array_equal(o.running[0], counts) and int(o.j_star[0]) == j_def
        np.testing.assert_allclose(w[0], w_def, atol=1e-7)
        assert counts.max() <= len(labels) and counts.min() >= 0
    # one-sided cases: only drafter 0 ever points at the verified token -> j* = 0 (w = [1, 0]); only drafter 1 -> j* = 10
    for good in (0, 1):
        qk = np.full((2, V), 0.5 / (V - 1))
        qk[good, 7] = 0.5; qk[1 - good, 9] = 0.5
        qk /= qk.sum(axis=1, keepdims=True)
        m_ = X.grid_hard_matches(qk.astype(F), 7)
        assert m_[0 if good == 0 else 10] == 1 and m_[10 if good == 0 else 0] == 0
        assert np.array_equal(m_, D.hard_label_matches(qk.astype(F), 7))
        j, wj, _ = D.policy_grid_hard([7], [qk.astype(F)])
        assert j == (0 if good == 0 else int(np.argmax(m_))) and wj[good] >= 0.5


def test_adaboost_weights_follow_the_printed_formula():
    """w_m = ln(1/eps_m - 1) + C ln(K - 1), normalised; the lower a method's error rate the larger its weight."""
    K = 32000
    w = X.policy_adaboost(np.array([2, 5, 9]), 10, K, 1.0).astype(np.float64)
    eps = (np.array([2, 5, 9]) + 1.0) / 12.0
    raw = np.log(1.0 / eps - 1.0) + np.log(K - 1.0)
    np.testing.assert_allclose(w, raw / raw.sum(), atol=2e-6)
    np.testing.assert_allclose(w, D.policy_adaboost(np.array([2, 5, 9]), 10, K, 1.0), atol=2e-6)
    assert w[0] > w[1] > w[2] and abs(w.sum() - 1) < 1e-6 and np.all(w >= 0)
    eq = X.policy_adaboost(np.array([3, 3, 3, 3]), 8, K, 1.0)
    assert np.all(eq == eq[0]) and abs(float(eq[0]) - 0.25) < 1e-7
    # C = 0 and a method that is wrong more often than right: its term is negative, cut at 0
    w0 = X.policy_adaboost(np.array([1, 9]), 10, K, 0.0)
    assert w0[1] == 0 and w0[0] == 1
    assert np.array_equal(X.policy_adaboost(np.array([9, 9]), 10, K, 0.0), X.policy_static(2))
    # inside the round machine: errors are counted against the verified tokens over the window
    rng = np.random.default_rng(33)
    G, V, m = 3, 60, 3
    o = mk(m=m, B=1, gamma=G, h=4, V=V, policy=W.POLICY_ADABOOST, tau=1.0)
    errs = []
    for rnd in range(4):
        lg = rand_logits(rng, G, 1, m, V, 2.0)
        o.draft_round_logits(lg, lat(rng, (1, G)))
        tl = np.concatenate([lg[:, :, 0, :], lg[-1:, :, 0, :]], axis=0).transpose(1, 0, 2)
        tl = (3.0 * tl + 0.3 * rng.standard_normal(tl.shape)).astype(F)
        a, z = o.verify(tl, lat(rng, (1, G)), lat(rng, (1,)))
        for i in range(min(int(a[0]), G - 1) + 1):
            label = int(o.tokens[0, i]) if i < a[0] else int(z[0])
            errs.append([int(int(np.argmax(o.qk[0, i, k])) != label) for k in range(m)])
        w, am = o.update_weights()
        win = np.array(errs[-4:])
        np.testing.assert_allclose(w[0], D.policy_adaboost(win.sum(axis=0), len(win), V, 1.0), atol=2e-6)


# ---------------------------------------------------------------- token tree of width d in the round machine
def test_tree_round_sibling_acceptance_and_bookkeeping():
    """Forced cases on a width-2 tree: (a) the primary of depth 0 is impossible under the target and its sibling is
    certain -> the sibling is accepted, the block ends there, the next token comes from the target's distribution
    after the sibling (its leaf row), two tokens are pending and the caches keep only what the drafter consumed;
    (b) both candidates impossible -> replacement from the residual; (c) every primary certain -> all accepted."""
    rng = np.random.default_rng(41)
    G, V, m, d = 3, 30, 2, 2
    cfg = W.DrafterCfg(1, 32, 2, 2, 64, V, "fp32")
    wl = W.Workload(name="tree_t", config_id=95, drafter=cfg, n_inputs=m, n_requests=1, gamma=G, window_h=0, rounds=1,
                    policy=W.POLICY_SOFTMAX_INV_ERR, prefixes=((("tokens", 5),), (("tokens", 3),)), kv_capacity=64)
    for case in ("sibling", "none", "all"):
        o = TabedOracle(n_inputs=m, n_requests=1, gamma=G, window_h=0, policy=W.POLICY_SOFTMAX_INV_ERR, vocab=V,
                        drafter=OracleDrafter(cfg, W.make_weights(wl)), kv_capacity=64, tree_width=d)
        for k, segs in enumerate(W.make_prefixes(wl, 0)):
            o.prefill(k, segs)
        o.set_pending([4])
        len0 = o.kv_lengths().copy()
        toks, q = o.draft_round(lat(rng, (1, G, d)))
        assert np.all(o.cands[0, :, 0] == toks[0]) and np.all(o.cands[0, :, 0] != o.cands[0, :, 1])
        tl = np.zeros((1, o.n_target_rows(), V), F)
        assert o.n_target_rows() == G + 1 + G
        hot = lambda t: 60.0 * np.eye(V, dtype=F)[t] - 30.0
        leaf_tok = 11
        if case == "sibling":
            tl[0, 0] = hot(o.cands[0, 0, 1])                  # the target wants the sibling of depth 0
            tl[0, G + 1] = hot(leaf_tok)                      # ... and after it, token 11
        elif case == "none":
            other = [t for t in range(V) if t not in o.cands[0, 0]][0]
            tl[0, 0] = hot(other)
        else:
            for i in range(G):
                tl[0, i] = hot(toks[0, i])
            tl[0, G] = hot(leaf_tok)
        a, z = o.verify(tl, lat(rng, (1, G, d)), lat(rng, (1,)))
        w, am = o.update_weights()
        if case == "sibling":
            assert a[0] == 1 and o.acc_prim[0] == 0 and o.sib_tok[0] == o.cands[0, 0, 1] and z[0] == leaf_tok
            assert o.pending[0] == [int(o.cands[0, 0, 1]), leaf_tok] and o.count[0] == 1
            assert np.array_equal(o.kv_lengths(), len0 + 1)                    # the pending token only
        elif case == "none":
            assert a[0] == 0 and o.sib_tok[0] == -1 and z[0] == other and o.pending[0] == [other] and o.count[0] == 1
            assert np.array_equal(o.kv_lengths(), len0 + 1)
        else:
            assert a[0] == G and o.acc_prim[0] == G and z[0] == leaf_tok and o.count[0] == G
            assert o.pending[0] == [int(toks[0, G - 1]), leaf_tok] and np.array_equal(o.kv_lengths(), len0 + 1 + G - 1)


def test_tree_round_accepts_at_least_as_much_as_the_chain():
    """Same uniforms for the primary chain: a width-3 tree never accepts fewer tokens in a round than the chain does
    on the same drafts (the siblings only add chances), and its primary chain is the chain's draft."""
    rng = np.random.default_rng(42)
    G, V, m = 4, 80, 2
    tot = [0, 0]
    for trial in range(30):
        lg = rand_logits(rng, G, 1, m, V, 1.5)
        ud3, ua3, ur = lat(rng, (1, G, 3)), lat(rng, (1, G, 3)), lat(rng, (1,))
        o1 = mk(m=m, B=1, gamma=G, h=0, V=V)
        o3 = TabedOracle(n_inputs=m, n_requests=1, gamma=G, window_h=0, policy=W.POLICY_SOFTMAX_INV_ERR, vocab=V, tree_width=3)
        t1, _ = o1.draft_round_logits(lg, ud3[:, :, 0])
        t3, _ = o3.draft_round_logits(lg, ud3)
        assert np.array_equal(t1, t3) and np.array_equal(o1.q, o3.q)
        tl = (rng.standard_normal((1, o3.n_target_rows(), V)) * 1.5).astype(F)
        tl[0, :G] += lg[:, 0, 0, :]
        a1, _ = o1.verify(tl[:, :G + 1], ua3[:, :, 0], ur)
        a3, _ = o3.verify(tl, ua3, ur)
        assert a3[0] >= a1[0] and o3.acc_prim[0] >= min(a1[0], o3.acc_prim[0])
        if o3.sib_tok[0] < 0:
            assert o3.acc_prim[0] == a3[0]
        tot[0] += int(a1[0]); tot[1] += int(a3[0])
    assert tot[1] > tot[0]
