"""GPU parity tests: the CUDA library through its C boundary against the CPU checker.

Bars: token ids, accept counts, replacement tokens, grid j*, weight argmax bit-exact; q, q^(k), p
and the weights bit-exact whenever both sides start from identical fp32 logits; logits of the
CUDA forward pass within the bound derived in gpu_harness.py and probabilities within 1e-5.
"""
import numpy as np
import pytest
import torch

from paper_2601_20357_b200 import workloads as W

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import gpu_harness as H
    from paper_2601_20357_b200 import binding as TB


def shape_only(wl: W.Workload, **kw) -> W.Workload:
    return wl.replace(**kw)


# ------------------------------------------------------------------------------------------------
# decision chain (Algorithm 1 steps 6-7, verification, weight update) on supplied logits
# ------------------------------------------------------------------------------------------------
DECISION_CASES = {
    "tiny_grid": (W.TINY, {}, 6),
    "tiny_softmax": (W.TINY, dict(policy=W.POLICY_SOFTMAX_INV_ERR), 6),
    "tiny_greedy": (W.TINY, dict(sample_mode=W.MODE_GREEDY), 4),
    "tiny_tvd": (W.TINY, dict(distance=W.DIST_TVD), 4),
    "tiny_tvd_softmax_all": (W.TINY, dict(distance=W.DIST_TVD, policy=W.POLICY_SOFTMAX_INV_ERR, window_h=0), 4),
    "tiny_static": (W.TINY, dict(policy=W.POLICY_STATIC), 3),
    "tiny_h1": (W.TINY, dict(window_h=1, policy=W.POLICY_SOFTMAX_INV_ERR), 5),
    "tiny_random": (W.TINY, dict(policy=W.POLICY_RANDOM), 4),
    "tiny_grid_hard": (W.TINY, dict(policy=W.POLICY_GRID_HARD), 6),
    "tiny_grid_hard_all_greedy": (W.TINY, dict(policy=W.POLICY_GRID_HARD, window_h=0, sample_mode=W.MODE_GREEDY), 5),
    "tiny_adaboost": (W.TINY, dict(policy=W.POLICY_ADABOOST), 6),
    "llava_small_random": (W.LLAVA_SMALL, dict(policy=W.POLICY_RANDOM), 3),
    "llava_small_adaboost_all": (W.LLAVA_SMALL, dict(policy=W.POLICY_ADABOOST, window_h=0, tau=0.5), 4),
    "batched_serving_adaboost": (W.BATCHED_SERVING, dict(policy=W.POLICY_ADABOOST), 3),
    "tiny_tree2": (W.TINY, dict(tree_width=2), 8),
    "tiny_tree3_softmax": (W.TINY, dict(tree_width=3, policy=W.POLICY_SOFTMAX_INV_ERR), 8),
    "tiny_tree3_greedy": (W.TINY, dict(tree_width=3, sample_mode=W.MODE_GREEDY), 6),
    "tiny_tree2_grid_hard": (W.TINY, dict(tree_width=2, policy=W.POLICY_GRID_HARD), 6),
    "llava_small_tree2": (W.LLAVA_SMALL, dict(tree_width=2), 5),
    "llava_small_tree3": (W.LLAVA_SMALL, dict(tree_width=3), 5),
    "batched_serving_tree2": (W.BATCHED_SERVING, dict(tree_width=2), 3),
    "large_vocab_tree3_greedy": (W.LARGE_VOCAB, dict(tree_width=3, sample_mode=W.MODE_GREEDY), 2),
    "llava_small": (W.LLAVA_SMALL, {}, 4),
    "large_vocab": (W.LARGE_VOCAB, {}, 3),
    "long_context": (W.LONG_CONTEXT, {}, 3),
    "batched_serving": (W.BATCHED_SERVING, {}, 3),
}


@pytest.mark.parametrize("case", sorted(DECISION_CASES))
def test_decision_chain_bit_exact(case):
    wl, kw, rounds = DECISION_CASES[case]
    wl = wl.replace(**kw)
    pair = H.Pair(wl, H.make_gpu(wl), H.make_oracle(wl, None))
    for rnd in range(rounds):
        H.logits_round(pair, rnd, W.logits_like_drafter(wl, rnd))
    pair.gpu.destroy()


@pytest.mark.parametrize("V,m,B,G", [(97, 2, 3, 2), (2049, 3, 2, 4), (1000, 1, 1, 1), (4099, 8, 2, 3), (2, 2, 1, 2)])
def test_decision_chain_ragged_vocabularies(V, m, B, G):
    """Vocabulary sizes that are not multiples of the 128-bit vector or of the CTA chunk; m = 1 and m = 8."""
    cfg = W.DrafterCfg(1, 64, 2, 2, 64, V, "fp32")
    wl = W.Workload(name=f"ragged{V}", config_id=900 + V % 89, drafter=cfg, n_inputs=m, n_requests=B, gamma=G,
                    window_h=3, rounds=4, policy=W.POLICY_GRID_MT if m == 2 else W.POLICY_SOFTMAX_INV_ERR,
                    alpha=tuple([1.0 / m] * m), sigma_schedule=((0, 0.7),))
    pair = H.Pair(wl, H.make_gpu(wl), H.make_oracle(wl, None))
    for rnd in range(4):
        H.logits_round(pair, rnd, W.logits_like_drafter(wl, rnd, scale=1.5))
    pair.gpu.destroy()


@pytest.mark.parametrize("V,m,B,G,d", [(2, 2, 2, 3, 3), (97, 3, 2, 2, 2), (4099, 2, 3, 3, 3), (2049, 1, 1, 4, 4)])
def test_token_tree_ragged_vocabularies(V, m, B, G, d):
    """Token tree of width d on vocabularies that are not multiples of the vector width or of a CTA slice, including
    V = 2 with three candidates (the third does not exist) and the widest tree."""
    cfg = W.DrafterCfg(1, 64, 2, 2, 64, V, "fp32")
    for mode in (W.MODE_SAMPLE, W.MODE_GREEDY):
        wl = W.Workload(name=f"tree_ragged{V}", config_id=700 + V % 89 + mode, drafter=cfg, n_inputs=m, n_requests=B, gamma=G,
                        window_h=3, rounds=5, policy=W.POLICY_GRID_MT if m == 2 else W.POLICY_SOFTMAX_INV_ERR,
                        alpha=tuple([1.0 / m] * m), sigma_schedule=((0, 0.7),), tree_width=d, sample_mode=mode)
        pair = H.Pair(wl, H.make_gpu(wl), H.make_oracle(wl, None))
        sib = 0
        for rnd in range(5):
            H.logits_round(pair, rnd, W.logits_like_drafter(wl, rnd, scale=1.5))
            sib += int((pair.orc.sib_tok >= 0).sum())
        if V > 2 and mode == W.MODE_SAMPLE:
            assert sib > 0                                   # some round ended on an accepted sibling
        pair.gpu.destroy()


def test_token_tree_lockstep_with_the_drafters_forward():
    """Width-2 tree with the library's own forward pass: the fp32 drafter (per-operation kernels) and a bf16 drafter
    with 18 rows (tensor-core path); the chain the drafter continues is the primary candidates, the caches keep only
    what it consumed, an accepted sibling leaves two tokens pending."""
    pair = H.build_pair(W.TINY.replace(tree_width=2, policy=W.POLICY_SOFTMAX_INV_ERR))
    for rnd in range(8):
        H.lockstep_round(pair, rnd, override=True)
    pair.gpu.destroy()
    wl = small_bf16_workload(B=6).replace(tree_width=3)
    pair = H.build_pair(wl)
    assert pair.gpu.current_path() == TB.PATH_TENSOR_CORE
    sib = 0
    for rnd in range(4):
        H.lockstep_round(pair, rnd, override=True)
        sib += int((pair.orc.sib_tok >= 0).sum())
    assert sib > 0
    pair.gpu.destroy()


def test_degenerate_targets_full_accept_zero_probability_and_empty_residual():
    """q = p accepts every token and draws the bonus token; a token the target forbids is rejected;
    when p == q exactly at the rejected position the residual has no mass and p itself is drawn."""
    wl = W.TINY.replace(policy=W.POLICY_STATIC, n_inputs=1, alpha=(1.0,), gamma=4)
    pair = H.Pair(wl, H.make_gpu(wl), H.make_oracle(wl, None))
    lg = W.logits_like_drafter(wl, 0, scale=2.0)
    # target == drafter on every position (bonus row reuses the last step)
    tl = np.concatenate([lg[:, :, 0, :], lg[-1:, :, 0, :]], axis=0).transpose(1, 0, 2).copy()
    H.logits_round(pair, 0, lg, target=tl)
    assert int(pair.orc.n_accept[0]) == wl.gamma
    # forbid the second drafted token
    probe = H.make_oracle(wl, None)
    probe.draft_round_logits(lg, W.round_uniforms(wl, 1)[0])
    y1 = int(probe.tokens[0, 1])
    tl2 = tl.copy(); tl2[0, 1, y1] = -300.0
    H.logits_round(pair, 1, lg, target=tl2)
    assert int(pair.orc.n_accept[0]) == 1
    pair.gpu.destroy()


# ------------------------------------------------------------------------------------------------
# full rounds with the drafter's own forward pass
# ------------------------------------------------------------------------------------------------
def test_tiny_free_run_all_rounds_grid_policy():
    """Config 1 end to end, free running on both sides for all 32 rounds (fp32 drafter)."""
    pair = H.build_pair(W.TINY)
    worst = 0.0
    for rnd in range(W.TINY.rounds):
        worst = max(worst, H.lockstep_round(pair, rnd, override=False))
    assert worst <= H.logit_tols(W.TINY)[0]
    pair.gpu.destroy()


def test_tiny_lockstep_softmax_policy_and_full_acceptance_path():
    """sigma = 0 makes the target equal to drafter 0: blocks get fully accepted, which exercises the
    two-pending-token first step and the bonus draw."""
    wl = W.TINY.replace(policy=W.POLICY_SOFTMAX_INV_ERR, sigma_schedule=((0, 0.0),), rounds=10)
    pair = H.build_pair(wl)
    full = 0
    for rnd in range(wl.rounds):
        H.lockstep_round(pair, rnd, override=True)
        full += int(pair.orc.n_accept[0] == wl.gamma)
    assert full >= 2
    pair.gpu.destroy()


def small_bf16_workload(B=2, gqa=True):
    cfg = W.DrafterCfg(2, 256, 4, 2 if gqa else 4, 640, 3000, "bf16")
    return W.Workload(name="small_bf16", config_id=41, drafter=cfg, n_inputs=3, n_requests=B, gamma=4, window_h=4,
                      rounds=6, policy=W.POLICY_SOFTMAX_INV_ERR,
                      prefixes=((("embeds", 37), ("tokens", 9)), (("tokens", 5),), (("tokens", 130),)),
                      kv_capacity=256, alpha=(0.5, 0.3, 0.2), sigma_schedule=((0, 0.3),))


def test_small_bf16_gqa_lockstep_two_requests():
    """bf16 drafter with grouped-query attention, head_dim 64, two concurrent requests (R = 6),
    prefix longer than one attention split."""
    wl = small_bf16_workload()
    pair = H.build_pair(wl)
    for rnd in range(wl.rounds):
        H.lockstep_round(pair, rnd, override=True)
    pair.gpu.destroy()


def test_llava_small_lockstep():
    """Config 2 at full size (576 image embeddings + text, text only, caption + text); 4 rounds."""
    wl = W.LLAVA_SMALL
    pair = H.build_pair(wl)
    for rnd in range(4):
        H.lockstep_round(pair, rnd, override=True)
    pair.gpu.destroy()


def test_large_vocab_lockstep():
    """Config 3 at its stated size: 12 layers, GQA 14/2, V = 152064, prefixes of 1152 / 128 / 192 / 1152 positions
    (1024 image embeddings + text, text only, caption + text, noisy image + text); one round on the persistent kernel."""
    wl = W.LARGE_VOCAB
    pair = H.build_pair(wl)
    assert pair.gpu.current_path() == TB.PATH_PERSISTENT
    H.lockstep_round(pair, 0, override=True)
    pair.gpu.destroy()


def test_long_context_lockstep():
    """Config 4: synthetic 8192-token caches per row (split-KV attention over 32 splits); 2 rounds."""
    wl = W.LONG_CONTEXT
    pair = H.build_pair(wl)
    for rnd in range(2):
        H.lockstep_round(pair, rnd, override=True)
    pair.gpu.destroy()


def test_batched_serving_lockstep_96_rows_short_caches():
    """Config 5's 32 x 3 = 96 shared-weight rows with short ragged caches (the checker holds fp64 caches)."""
    wl = W.BATCHED_SERVING.replace(kv_capacity=512)
    lens = W.substream(5, "short_kvlen").integers(1, 300, size=wl.n_rows, dtype=np.int32)
    pair = H.build_pair(wl, kv_lengths=lens)
    for rnd in range(2):
        H.lockstep_round(pair, rnd, override=True)
    pair.gpu.destroy()


def test_batched_serving_lockstep_full_size():
    """Config 5 at its stated size: 32 requests x 3 inputs = 96 shared-weight rows, cache lengths uniform in
    [256, 4096] per row, one lock-step round on the tensor-core path (tcgen05 projections, TMA attention)."""
    wl = W.BATCHED_SERVING
    pair = H.build_pair(wl)
    assert pair.gpu.current_path() == TB.PATH_TENSOR_CORE
    H.lockstep_round(pair, 0, override=True)
    pair.gpu.destroy()


def test_batched_serving_lockstep_long_ragged_caches():
    """Config 5's cache-length range [256, 4096] on two requests (R = 6)."""
    wl = W.BATCHED_SERVING.replace(n_requests=2, alpha=(0.5, 0.3, 0.2))
    lens = np.array([256, 4096, 1777, 3001, 640, 2048], np.int32)
    pair = H.build_pair(wl, kv_lengths=lens)
    for rnd in range(2):
        H.lockstep_round(pair, rnd, override=True)
    pair.gpu.destroy()


# ------------------------------------------------------------------------------------------------
# boundary behaviour
# ------------------------------------------------------------------------------------------------
def test_call_order_and_argument_errors():
    wl = W.TINY
    g = H.make_gpu(wl)
    B, G, V = wl.n_requests, wl.gamma, wl.drafter.vocab
    a = torch.empty(B, dtype=torch.int32, device=H.DEV)
    tl = torch.zeros((B, G + 1, V), device=H.DEV)
    u = torch.full((B, G), 0.5, device=H.DEV)
    with pytest.raises(TB.TabedError) as e:
        g.verify(tl, u, u[:, 0].contiguous(), a, a.clone())
    assert e.value.code == -3
    with pytest.raises(TB.TabedError) as e:
        g.update_weights()
    assert e.value.code == -3
    toks = torch.empty((B, G), dtype=torch.int32, device=H.DEV)
    with pytest.raises(TB.TabedError) as e:
        g.draft_round(u, toks)                      # handle without a drafter
    assert e.value.code == -3
    g.draft_round_logits(torch.zeros((G, B, wl.n_inputs, V), device=H.DEV), u, toks)
    with pytest.raises(TB.TabedError) as e:
        g.draft_round_logits(torch.zeros((G, B, wl.n_inputs, V), device=H.DEV), u, toks)
    assert e.value.code == -3
    g.destroy()
    with pytest.raises(TB.TabedError) as e:
        TB.Tabed(n_inputs=3, n_requests=1, gamma=3, window_h=2, policy=TB.POLICY_GRID_MT, vocab=100)
    assert e.value.code == -1
    with pytest.raises(TB.TabedError):
        TB.Tabed(n_inputs=9, n_requests=1, gamma=3, window_h=2, policy=TB.POLICY_STATIC, vocab=100)


def test_kv_overflow_is_reported_on_the_host():
    wl = W.TINY.replace(kv_capacity=70, prefixes=((("tokens", 64),), (("tokens", 16),)))
    pair = H.build_pair(wl)
    toks = torch.empty((1, wl.gamma), dtype=torch.int32, device=H.DEV)
    u = torch.full((1, wl.gamma), 0.5, device=H.DEV)
    # 64 cached + 2 pending slots + gamma-1 drafts = 68 <= 70 fits once; the conservative bound then refuses
    pair.gpu.draft_round(u, toks)
    a = torch.empty(1, dtype=torch.int32, device=H.DEV)
    pair.gpu.verify(torch.zeros((1, wl.gamma + 1, wl.drafter.vocab), device=H.DEV), u, u[:, 0].contiguous(), a, a.clone())
    pair.gpu.update_weights()
    with pytest.raises(TB.TabedError) as e:
        pair.gpu.draft_round(u, toks)
    assert e.value.code == -4
    with pytest.raises(TB.TabedError) as e:
        pair.gpu.prefill_tokens(1, torch.zeros(60, dtype=torch.int32, device=H.DEV))
    assert e.value.code == -4
    H.check_error_flag(pair.gpu)
    pair.gpu.destroy()


def test_state_export_import_round_trip_and_determinism():
    """Running the same rounds twice from an imported snapshot gives bitwise identical results."""
    wl = small_bf16_workload(B=1)
    pair = H.build_pair(wl)
    for rnd in range(2):
        H.lockstep_round(pair, rnd, override=True)
    snap = pair.gpu.state_export()
    g = pair.gpu

    def run(rounds):
        out = []
        toks = torch.empty((1, wl.gamma), dtype=torch.int32, device=H.DEV)
        a = torch.empty(1, dtype=torch.int32, device=H.DEV); z = a.clone(); am = a.clone()
        w = torch.empty((1, wl.n_inputs), device=H.DEV)
        for rnd in rounds:
            ud, ua, ur = W.round_uniforms(wl, rnd)
            g.draft_round(H.t(ud), toks)
            lg = g.debug_view(TB.VIEW_LOGITS).cpu().numpy().copy()
            g.verify(H.t(W.target_logits(wl, rnd, lg)), H.t(ua), H.t(ur), a, z)
            g.update_weights(w, am)
            torch.cuda.synchronize()
            out.append((toks.cpu().numpy().copy(), int(a), int(z), w.cpu().numpy().copy(), lg))
        return out

    first = run([2, 3, 4])
    g.state_import(snap)
    second = run([2, 3, 4])
    for x, y in zip(first, second):
        assert np.array_equal(x[0], y[0]) and x[1:3] == y[1:3] and np.array_equal(x[3], y[3]) and np.array_equal(x[4], y[4])
    with pytest.raises(TB.TabedError):
        g.state_import(snap[:-4])
    g.destroy()


def test_round_host_matches_device_calls():
    wl = small_bf16_workload(B=2)
    pa, pb = H.build_pair(wl), None
    B, G, m, V = wl.n_requests, wl.gamma, wl.n_inputs, wl.drafter.vocab
    ud, ua, ur = W.round_uniforms(wl, 0)
    # device path, with the target built from the round's own logits
    toks = torch.empty((B, G), dtype=torch.int32, device=H.DEV)
    a = torch.empty(B, dtype=torch.int32, device=H.DEV); z = a.clone(); am = a.clone()
    w = torch.empty((B, m), device=H.DEV)
    snap = pa.gpu.state_export()
    pa.gpu.draft_round(H.t(ud), toks)
    tl = W.target_logits(wl, 0, pa.gpu.debug_view(TB.VIEW_LOGITS).cpu().numpy())
    pa.gpu.verify(H.t(tl), H.t(ua), H.t(ur), a, z)
    pa.gpu.update_weights(w, am)
    torch.cuda.synchronize()
    # host path from the same state
    pa.gpu.state_import(snap)
    h_toks = torch.empty((B, G), dtype=torch.int32); h_a = torch.empty(B, dtype=torch.int32); h_z = h_a.clone()
    h_am = h_a.clone(); h_w = torch.empty((B, m))
    pa.gpu.round_host(torch.from_numpy(ud), torch.from_numpy(ua), torch.from_numpy(ur), torch.from_numpy(tl),
                      h_toks, h_a, h_z, h_w, h_am)
    assert torch.equal(h_toks, toks.cpu()) and torch.equal(h_a, a.cpu()) and torch.equal(h_z, z.cpu())
    assert torch.equal(h_w, w.cpu()) and torch.equal(h_am, am.cpu())
    pa.gpu.destroy()


def test_ensemble_step_is_stateless_and_matches_checker():
    from oracle import exact32 as X
    wl = W.LLAVA_SMALL.replace(n_requests=2)
    g = H.make_gpu(wl)
    lg = W.logits_like_drafter(wl, 0)[0]                  # [B][m][V]
    wts = np.array([[0.2, 0.5, 0.3], [1.0, 0.0, 0.0]], np.float32)
    u = W.lattice_uniforms(W.substream(2, "ens_u"), (2,))
    y = torch.empty(2, dtype=torch.int32, device=H.DEV)
    q = torch.empty((2, wl.drafter.vocab), device=H.DEV)
    qk = torch.empty((2, 3, wl.drafter.vocab), device=H.DEV)
    g.ensemble_step(H.t(lg), H.t(wts), H.t(u), y, q, qk)
    torch.cuda.synchronize()
    for b in range(2):
        qk_o = X.softmax_exact(lg[b]); q_o = X.ensemble_exact(qk_o, wts[b])
        assert np.array_equal(qk[b].cpu().numpy(), qk_o) and np.array_equal(q[b].cpu().numpy(), q_o)
        assert int(y[b]) == X.draw(X.masses(q_o), u[b])
    g.destroy()


# --------------------------------------------------------------------------------------------------
# Pooled multimodal drafting input (Sec. 5): 2 x 2 average pooling of the visual tokens
# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("gh,gw,d", [(24, 24, 768), (2, 2, 1), (6, 4, 130), (48, 2, 33)])
def test_pool_embeds_bit_exact(gh, gw, d):
    """The mean of four fp32 values rounded once: bitwise equal to the checker's."""
    from oracle.definitions import pool_image_tokens_2x2
    g = H.make_gpu(W.TINY)
    rng = np.random.default_rng(100 + gh + d)
    x = (rng.standard_normal((gh * gw, d)) * rng.choice([1e-3, 1.0, 1e3], size=(gh * gw, 1))).astype(np.float32)
    out = torch.full(((gh // 2) * (gw // 2), d), float("nan"), device=H.DEV)
    g.pool_embeds(H.t(x), gh, gw, out)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy(), pool_image_tokens_2x2(x, gh, gw))
    with pytest.raises(TB.TabedError) as e:
        g.pool_embeds(H.t(np.zeros((12, 4), np.float32)), 3, 4, torch.empty((2, 4), device=H.DEV))
    assert e.value.code == -1
    g.destroy()
