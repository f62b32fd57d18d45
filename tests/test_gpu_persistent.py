"""GPU parity tests of the persistent drafting-round kernel (TABED_PATH_PERSISTENT) through the C boundary.

Same bars as tests/test_gpu_parity.py: with the checker's fp32 logits handed to the ensemble
(lock step), tokens, accept counts, replacement tokens, weights and window sums are bit-exact and
q, q^(k), p are bitwise equal; the kernel's own forward pass is compared at every step (logits within
the bf16 bound, probabilities within 1e-5).  The cases here are chosen for what is special in the
persistent kernel: tiles cut into 1, 2, 4 or 8 sub-units, the ragged last LM-head tile, grouped-query attention with
head sizes 32/64/128, several attention splits merged by the last CTA to finish, two pending tokens
fed in one weight pass (positions produced and consumed in the same phase), greedy mode.
"""
import numpy as np
import pytest
import torch

from paper_2601_20357_b200 import workloads as W

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import gpu_harness as H
    from paper_2601_20357_b200 import binding as TB


def wl_small(*, d=256, heads=4, kv_heads=2, ffn=640, vocab=3000, m=3, B=1, gamma=4, layers=2, prefixes=None,
             cap=256, mode=W.MODE_SAMPLE, sigma=0.3, cid=61, policy=W.POLICY_SOFTMAX_INV_ERR, alpha=None):
    cfg = W.DrafterCfg(layers, d, heads, kv_heads, ffn, vocab, "bf16")
    if prefixes is None:
        prefixes = ((("embeds", 37), ("tokens", 9)), (("tokens", 5),), (("tokens", 130),))[:m]
    if alpha is None:
        alpha = tuple([0.5, 0.3, 0.2][:m]) if m == 3 else tuple([1.0 / m] * m)
    return W.Workload(name=f"persist{cid}", config_id=cid, drafter=cfg, n_inputs=m, n_requests=B, gamma=gamma, window_h=4,
                      rounds=6, policy=policy, prefixes=prefixes, kv_capacity=cap, alpha=alpha,
                      sigma_schedule=((0, sigma),), sample_mode=mode)


def run_lockstep(wl, rounds, override=True):
    pair = H.build_pair(wl)
    assert pair.gpu.current_path() == TB.PATH_PERSISTENT
    for rnd in range(rounds):
        H.lockstep_round(pair, rnd, override=override)
    return pair


def test_path_selection():
    pair = H.build_pair(wl_small())
    g = pair.gpu
    assert g.current_path() == TB.PATH_PERSISTENT
    g.select_path(TB.PATH_PER_OP)
    assert g.current_path() == TB.PATH_PER_OP
    g.select_path(TB.PATH_AUTO)
    assert g.current_path() == TB.PATH_PERSISTENT
    g.destroy()
    tiny = H.build_pair(W.TINY)                       # fp32 drafter: per-operation kernels only
    assert tiny.gpu.current_path() == TB.PATH_PER_OP
    with pytest.raises(TB.TabedError) as e:
        tiny.gpu.select_path(TB.PATH_PERSISTENT)
    assert e.value.code == -7
    tiny.gpu.destroy()


def test_lockstep_gqa_head64_three_inputs():
    """R = 3 slots, grouped-query attention 4/2, one row longer than an attention split (merge by ticket)."""
    run_lockstep(wl_small(), 5).gpu.destroy()


def test_lockstep_two_pending_tokens_every_round():
    """m = 1 makes q = p, every block is fully accepted, so every round after the first feeds two
    pending tokens in one weight pass: the second slot reads the first slot's K,V of the same phase."""
    wl = wl_small(m=1, B=2, sigma=0.0, prefixes=((("tokens", 21),),), alpha=(1.0,), cid=62, policy=W.POLICY_STATIC)
    pair = run_lockstep(wl, 4)
    assert int(pair.orc.n_accept.min()) == wl.gamma
    pair.gpu.destroy()


def test_lockstep_mixed_pending_counts_across_requests():
    """Two requests, two inputs each (R = 4, up to 8 slots); sigma small so that some blocks are fully
    accepted and others not: slots of the second half are active for some requests only."""
    wl = wl_small(m=2, B=2, sigma=0.05, prefixes=((("tokens", 140),), (("embeds", 12), ("tokens", 3))), alpha=(0.9, 0.1),
                  cid=63, gamma=3)
    pair = run_lockstep(wl, 6)
    pair.gpu.destroy()


def test_lockstep_six_rows_extra_pass_every_round():
    """R = 6 rows (more than half of the kernel's 8 slots): both pending tokens of a fully accepted block no longer fit
    into one weight pass, the first is fed in a pass of its own (all layers, no LM head) before step 0.  m = 1 with a
    noise-free target makes q = p, so every block is fully accepted and every round after the first takes that pass."""
    wl = wl_small(m=1, B=6, sigma=0.0, prefixes=((("tokens", 21),),), alpha=(1.0,), cid=81, policy=W.POLICY_STATIC)
    pair = run_lockstep(wl, 4)
    assert int(pair.orc.n_accept.min()) == wl.gamma
    pair.gpu.destroy()


@pytest.mark.parametrize("B,m", [(2, 3), (4, 2), (1, 5), (1, 8)])
def test_lockstep_five_to_eight_rows_mixed_pending(B, m):
    """5 - 8 rows on the persistent kernel; sigma small so that some requests' blocks are fully accepted and others'
    not: in the extra pass only the rows with two pending tokens are active, the others wait for step 0."""
    prefixes = ((("tokens", 140),), (("embeds", 12), ("tokens", 3)), (("tokens", 40),), (("tokens", 7),),
                (("embeds", 20),), (("tokens", 64),), (("tokens", 3),), (("tokens", 90),))[:m]
    alpha = tuple([0.9] + [0.1 / (m - 1)] * (m - 1))
    wl = wl_small(m=m, B=B, sigma=0.05, prefixes=prefixes, alpha=alpha, cid=82 + B * 10 + m, gamma=3)
    pair = run_lockstep(wl, 6)
    pair.gpu.destroy()


@pytest.mark.parametrize("heads,kv_heads,d", [(8, 2, 256), (2, 1, 256), (4, 4, 512)])
def test_lockstep_head_sizes(heads, kv_heads, d):
    """head_dim 32 (8 heads, 4 per KV head), 128 (2 heads sharing one KV head), 128 without grouping."""
    wl = wl_small(d=d, heads=heads, kv_heads=kv_heads, ffn=512, cid=64 + heads)
    run_lockstep(wl, 3).gpu.destroy()


def test_lockstep_ragged_vocabulary_and_greedy():
    """V = 3001 (not a multiple of the 16-row LM-head tile nor of the 128-bit vector), greedy decoding."""
    wl = wl_small(vocab=3001, mode=W.MODE_GREEDY, cid=71)
    run_lockstep(wl, 3).gpu.destroy()
    wl = wl_small(vocab=2050, cid=72)
    run_lockstep(wl, 3).gpu.destroy()


def test_free_run_matches_per_operation_path_on_first_round():
    """Both paths from the same state, no logits override: the forward passes agree within the bf16
    bound and, fed the same logits, give the same decisions (checked against the checker above)."""
    wl = wl_small(cid=73)
    a, b = H.build_pair(wl), H.build_pair(wl)
    b.gpu.select_path(TB.PATH_PER_OP)
    ud, _, _ = W.round_uniforms(wl, 0)
    toks = torch.empty((1, wl.gamma), dtype=torch.int32, device=H.DEV)
    a.gpu.draft_round(H.t(ud), toks)
    b.gpu.draft_round(H.t(ud), toks.clone())
    torch.cuda.synchronize()
    la = a.gpu.debug_view(TB.VIEW_LOGITS)[0].cpu().numpy()
    lb = b.gpu.debug_view(TB.VIEW_LOGITS)[0].cpu().numpy()
    assert np.max(np.abs(la - lb)) <= 2 * H.logit_tols(wl)[0]        # two CUDA paths, each within the bound of the checker
    H.check_error_flag(a.gpu)
    # the in-kernel ensemble on the kernel's own logits (row maxima gathered by the LM-head epilogue)
    # equals, bit for bit, the stand-alone ensemble step applied to those logits
    own = a.gpu.debug_view(TB.VIEW_LOGITS).clone()
    qk_r = a.gpu.debug_view(TB.VIEW_QK).clone()
    q_r = a.gpu.debug_view(TB.VIEW_Q).clone()
    y = torch.empty(1, dtype=torch.int32, device=H.DEV)
    q = torch.empty((1, wl.drafter.vocab), device=H.DEV)
    qk = torch.empty((1, wl.n_inputs, wl.drafter.vocab), device=H.DEV)
    for i in range(wl.gamma):
        a.gpu.ensemble_step(own[i].contiguous(), None, H.t(ud[:, i].copy()), y, q, qk)
        torch.cuda.synchronize()
        assert torch.equal(qk[0], qk_r[0, i]) and torch.equal(q[0], q_r[0, i])
        assert int(y[0]) == int(toks[0, i])
    a.gpu.destroy(); b.gpu.destroy()


def test_phase_trace_is_monotonic():
    wl = wl_small(cid=74)
    pair = H.build_pair(wl)
    pair.gpu.debug_trace(True)
    H.lockstep_round(pair, 0, override=True)
    tr = pair.gpu.debug_view(TB.VIEW_TRACE).cpu().numpy().astype(np.int64)
    n_bar = 5 * wl.drafter.n_layers + 4                # one more record per step while logits are overridden
    flat = tr[:, :n_bar, 0].reshape(-1)
    assert np.all(flat > 0) and np.all(np.diff(flat) > 0)
    assert (flat[-1] - flat[0]) < 50_000_000          # one round stays far below 50 ms
    pair.gpu.destroy()
