"""GPU parity tests of the drafting path whose projections run as tcgen05 contractions over all rows
(TABED_PATH_TENSOR_CORE: bf16 drafter, 16 or more shared-weight rows), through the C boundary.

Same bars as tests/test_gpu_parity.py (lock step with the checker: integer results and q, q^(k), p
bit-exact on the checker's logits; the kernel's own logits within the bf16 bound, probabilities
within 1e-5).  The shapes are chosen for what is special here: input dimensions that are not a
multiple of the 128-column pipeline stage, an output dimension that is not a multiple of the
128-row tile (ragged LM-head tile), row counts that are not a multiple of 16, requests with one and
with two pending tokens in the same step (the second half of the slots is projected in a pass of its
own that is skipped when nobody needs it)."""
import numpy as np
import pytest
import torch

from paper_2601_20357_b200 import workloads as W

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import gpu_harness as H
    from paper_2601_20357_b200 import binding as TB


def wl_rows(*, B, m, d=256, heads=4, kv_heads=2, ffn=640, vocab=3000, gamma=3, sigma=0.3, cid=81, alpha=None):
    cfg = W.DrafterCfg(2, d, heads, kv_heads, ffn, vocab, "bf16")
    prefixes = ((("embeds", 11), ("tokens", 7)), (("tokens", 5),), (("tokens", 40),))[:m]
    if alpha is None:
        alpha = tuple([0.5, 0.3, 0.2][:m]) if m == 3 else tuple([1.0 / m] * m)
    return W.Workload(name=f"tensor{cid}", config_id=cid, drafter=cfg, n_inputs=m, n_requests=B, gamma=gamma, window_h=4,
                      rounds=4, policy=W.POLICY_SOFTMAX_INV_ERR if m != 2 else W.POLICY_GRID_MT, prefixes=prefixes,
                      kv_capacity=128, alpha=alpha, sigma_schedule=((0, sigma),))


def test_tensor_path_is_selected_for_many_rows():
    pair = H.build_pair(wl_rows(B=6, m=3))
    assert pair.gpu.current_path() == TB.PATH_TENSOR_CORE
    pair.gpu.select_path(TB.PATH_PER_OP)
    assert pair.gpu.current_path() == TB.PATH_PER_OP
    pair.gpu.destroy()


def test_lockstep_18_rows_ragged_dimensions():
    """R = 18 rows (MMA N = 32), d = 256, F = 640 (5 stages), V = 3000 (last LM-head tile has 56 rows)."""
    wl = wl_rows(B=6, m=3)
    pair = H.build_pair(wl)
    for rnd in range(3):
        H.lockstep_round(pair, rnd, override=True)
    pair.gpu.destroy()


def test_lockstep_mixed_pending_counts_40_rows():
    """20 requests x 2 inputs; small sigma so that some requests accept whole blocks (two pending tokens)
    while others do not: the pass over the second half of the slots runs with most slots inactive."""
    wl = wl_rows(B=20, m=2, sigma=0.05, alpha=(0.9, 0.1), cid=82, gamma=2)
    pair = H.build_pair(wl)
    full = 0
    for rnd in range(4):
        H.lockstep_round(pair, rnd, override=True)
        full += int((pair.orc.n_accept == wl.gamma).sum())
    assert 0 < full < 4 * wl.n_requests
    pair.gpu.destroy()


def test_tensor_path_agrees_with_per_operation_path():
    wl = wl_rows(B=8, m=3, cid=83)
    a, b = H.build_pair(wl), H.build_pair(wl)
    b.gpu.select_path(TB.PATH_PER_OP)
    ud, _, _ = W.round_uniforms(wl, 0)
    toks = torch.empty((wl.n_requests, wl.gamma), dtype=torch.int32, device=H.DEV)
    a.gpu.draft_round(H.t(ud), toks)
    b.gpu.draft_round(H.t(ud), toks.clone())
    torch.cuda.synchronize()
    la = a.gpu.debug_view(TB.VIEW_LOGITS)[0].cpu().numpy()
    lb = b.gpu.debug_view(TB.VIEW_LOGITS)[0].cpu().numpy()
    assert np.max(np.abs(la - lb)) <= 2 * H.logit_tols(wl)[0]        # two CUDA paths, each within the bound of the checker
    H.check_error_flag(a.gpu)
    a.gpu.destroy(); b.gpu.destroy()


# ------------------------------------------------------------------------------------------------
# TMA / tensor-core attention of the per-operation paths (bf16 caches, head size 64)
# ------------------------------------------------------------------------------------------------
def wl_attn(*, heads, kv_heads, d, prefixes, cap, B=1, cid=90, gamma=3, sigma=0.3, layers=2):
    m = len(prefixes)
    # vocabulary 8000: with a few thousand words the largest probabilities are so large that one bf16 ulp in
    # a cache entry (the checker rounds fp64 values, the kernels fp32 ones) moves them by more than 1e-5
    cfg = W.DrafterCfg(layers, d, heads, kv_heads, 512, 8000, "bf16")
    alpha = tuple([1.0 / m] * m)
    return W.Workload(name=f"attn{cid}", config_id=cid, drafter=cfg, n_inputs=m, n_requests=B, gamma=gamma, window_h=4,
                      rounds=4, policy=W.POLICY_SOFTMAX_INV_ERR if m != 2 else W.POLICY_GRID_MT, prefixes=prefixes,
                      kv_capacity=cap, alpha=alpha, sigma_schedule=((0, sigma),))


@pytest.mark.parametrize("heads,kv_heads,d", [(4, 2, 256), (8, 2, 512), (14, 2, 896)])
def test_attention_caches_spread_over_many_ctas(heads, kv_heads, d):
    """Per-operation path, few rows with long caches: fewer chunks of 128 positions than CTAs, so every
    cache longer than one chunk is cut into one-chunk segments on different CTAs (with idle CTAs in
    between) and put together by the last warp to finish (ticket).  Ragged last chunks (700 % 128, 130 %
    128), a cache shorter than one chunk, groups of 2, 4 and 7 query heads per KV head."""
    wl = wl_attn(heads=heads, kv_heads=kv_heads, d=d, cap=1024, cid=90 + heads,
                 prefixes=((("tokens", 700),), (("tokens", 130),), (("embeds", 37), ("tokens", 9))))
    pair = H.build_pair(wl)
    pair.gpu.select_path(TB.PATH_PER_OP)
    for rnd in range(3):
        H.lockstep_round(pair, rnd, override=True)
    pair.gpu.destroy()


def test_attention_many_rows_several_chunks_each():
    """Tensor-core path, 36 rows with 2 to 4 chunks per cache: segments that start and end inside a CTA's
    range next to caches that straddle two CTAs; two pending tokens for some requests (inactive slots)."""
    wl = wl_attn(heads=4, kv_heads=2, d=256, cap=512, B=12, cid=97, sigma=0.05, gamma=2,
                 prefixes=((("tokens", 390),), (("tokens", 260),), (("embeds", 120), ("tokens", 30))))
    pair = H.build_pair(wl)
    assert pair.gpu.current_path() == TB.PATH_TENSOR_CORE
    for rnd in range(3):
        H.lockstep_round(pair, rnd, override=True)
    pair.gpu.destroy()


# ------------------------------------------------------------------------------------------------
# prompts fed in chunks of 256 positions through the tensor-core kernels
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("heads,kv_heads,d", [(4, 2, 256), (8, 2, 256)])
def test_chunked_prefill_matches_position_by_position_prefill(heads, kv_heads, d):
    """The same prompts (700 tokens = 2 full chunks + 188; 130 and 37 embeddings + 9 tokens: short chunks) fed as
    chunks of positions (tcgen05 projections, every position attending up to itself) and one position at a
    time (per-operation kernels): both handles then follow the checker in lock step, and their first
    drafting step agrees within the bf16 bound.  Head sizes 64 (TMA attention) and 32 (split kernels)."""
    wl = wl_attn(heads=heads, kv_heads=kv_heads, d=d, cap=1024, cid=120 + heads,
                 prefixes=((("tokens", 700),), (("tokens", 130),), (("embeds", 37), ("tokens", 9))))
    a = H.build_pair(wl)
    b = H.build_pair(wl, prefill_path=TB.PATH_PER_OP)
    ud, _, _ = W.round_uniforms(wl, 0)
    toks = torch.empty((1, wl.gamma), dtype=torch.int32, device=H.DEV)
    for p in (a, b):
        p.gpu.select_path(TB.PATH_PER_OP)
    a.gpu.draft_round(H.t(ud), toks)
    b.gpu.draft_round(H.t(ud), toks.clone())
    torch.cuda.synchronize()
    la = a.gpu.debug_view(TB.VIEW_LOGITS)[0].cpu().numpy()
    lb = b.gpu.debug_view(TB.VIEW_LOGITS)[0].cpu().numpy()
    assert np.max(np.abs(la - lb)) <= 2 * H.logit_tols(wl)[0]        # two CUDA paths, each within the bound of the checker
    H.check_error_flag(a.gpu); H.check_error_flag(b.gpu)
    a.gpu.destroy(); b.gpu.destroy()
    for path in (None, TB.PATH_PER_OP):
        pair = H.build_pair(wl, prefill_path=path)
        for rnd in range(2):
            H.lockstep_round(pair, rnd, override=True)
        pair.gpu.destroy()


def test_tensor_path_forced_on_few_rows():
    """The tensor-core kernels are set up for every bf16 drafter (they feed the prompts); forcing them for the
    drafting steps of a 3-row workload (6 slots padded to 16 MMA columns, half of them inactive most rounds)
    must follow the checker like the automatic choice does."""
    wl = wl_attn(heads=4, kv_heads=2, d=256, cap=512, cid=131, sigma=0.05, gamma=3,
                 prefixes=((("tokens", 150),), (("tokens", 40),), (("embeds", 20), ("tokens", 3))))
    pair = H.build_pair(wl)
    assert pair.gpu.current_path() == TB.PATH_PERSISTENT
    pair.gpu.select_path(TB.PATH_TENSOR_CORE)
    assert pair.gpu.current_path() == TB.PATH_TENSOR_CORE
    for rnd in range(4):
        H.lockstep_round(pair, rnd, override=True)
    pair.gpu.select_path(TB.PATH_AUTO)
    H.lockstep_round(pair, 4, override=True)         # and back on the persistent kernel, same caches
    pair.gpu.destroy()
