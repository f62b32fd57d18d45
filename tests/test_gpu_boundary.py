"""Boundary behaviour of the library that needs a device: how device-side failures reach the caller, what a
corrupt snapshot does, pointers that are only element-aligned, handles of different shapes living side by side,
and the exact cache-length bookkeeping of the host-buffer round."""
import struct

import numpy as np
import pytest
import torch

import gpu_harness as H
from paper_2601_20357_b200 import binding as TB
from paper_2601_20357_b200 import workloads as W

pytestmark = pytest.mark.gpu


def small_wl(*, d=256, heads=4, kv_heads=2, ffn=640, vocab=3000, B=1, gamma=3, cap=256, cid=70):
    cfg = W.DrafterCfg(2, d, heads, kv_heads, ffn, vocab, "bf16")
    return W.Workload(name=f"boundary_{cid}", config_id=cid, drafter=cfg, n_inputs=3, n_requests=B, gamma=gamma, window_h=4,
                      rounds=4, policy=W.POLICY_SOFTMAX_INV_ERR, kv_capacity=cap, alpha=(0.5, 0.3, 0.2),
                      prefixes=((("embeds", 21), ("tokens", 9)), (("tokens", 5),), (("tokens", 40),)),
                      sigma_schedule=((0, 0.3),))


def host_round(pair, rnd, target=None):
    wl, g = pair.wl, pair.gpu
    B, G, m, V = wl.n_requests, wl.gamma, wl.n_inputs, wl.drafter.vocab
    ud, ua, ur = W.round_uniforms(wl, rnd)
    tl = target if target is not None else W.substream(wl.config_id, "host_target", rnd).standard_normal((B, G + 1, V)).astype(np.float32)
    out = (torch.empty((B, G), dtype=torch.int32), torch.empty(B, dtype=torch.int32), torch.empty(B, dtype=torch.int32),
           torch.empty((B, m)), torch.empty(B, dtype=torch.int32))
    g.round_host(torch.from_numpy(ud), torch.from_numpy(ua), torch.from_numpy(ur), torch.from_numpy(tl), *out)
    return out


def test_device_error_word_reaches_the_caller():
    """A set bit of the device-side error word comes back as the return code of the synchronising calls and is
    cleared by them (the word is preset through its view: nothing is made to fail on the device)."""
    pair = H.build_pair(small_wl())
    g = pair.gpu
    flag = g.debug_view(TB.VIEW_ERROR_FLAG)
    assert g.last_device_error() == 0
    for bits, code in ((8, TB.ERR_TIMEOUT), (16, TB.ERR_TIMEOUT), (4, TB.ERR_KV_OVERFLOW), (1, TB.ERR_NUMERIC), (2, TB.ERR_NUMERIC),
                       (4 | 8, TB.ERR_TIMEOUT)):
        flag.fill_(bits)
        assert g.last_device_error() == code
        assert g.last_device_error() == 0 and int(flag.cpu()[0]) == 0
    snap = g.state_export()
    flag.fill_(16)
    with pytest.raises(TB.TabedError) as e:
        host_round(pair, 0)
    assert e.value.code == TB.ERR_TIMEOUT
    assert g.last_device_error() == 0                     # cleared by the call that reported it
    g.state_import(snap)
    host_round(pair, 0)                                   # and the handle works on
    g.destroy()


def test_a_bounded_wait_that_runs_out_is_reported_and_the_gpu_keeps_answering():
    pair = H.build_pair(small_wl(cid=71))
    g = pair.gpu
    assert g.current_path() == TB.PATH_PERSISTENT
    assert g.debug_barrier_timeout() == TB.ERR_TIMEOUT    # one CTA, an arrival count nobody completes: the wait gives up
    assert g.last_device_error() == 0
    for rnd in range(2):                                  # the persistent kernel's own barriers are intact afterwards
        H.lockstep_round(pair, rnd, override=True)
    g.destroy()


def test_non_finite_logits_are_reported_not_drawn_from():
    V, B, m = 5000, 2, 3
    g = TB.Tabed(n_inputs=m, n_requests=B, gamma=1, window_h=1, policy=TB.POLICY_STATIC, vocab=V)
    lg = torch.full((B, m, V), float("nan"), device=H.DEV)
    u = torch.full((B,), 0.5, device=H.DEV)
    y = torch.full((B,), -1, dtype=torch.int32, device=H.DEV)
    g.ensemble_step(lg, None, u, y)
    assert g.last_device_error() == TB.ERR_NUMERIC and y.cpu().tolist() == [0, 0]
    g.destroy()
    w = torch.full((B, m), 1.0 / m, device=H.DEV)
    q = torch.empty((B, V), device=H.DEV)
    assert TB.static_last_error() == 0
    TB.ensemble_step_static(lg, w, u, y, q)
    assert TB.static_last_error() == TB.ERR_NUMERIC and TB.static_last_error() == 0


def test_corrupt_snapshots_are_rejected_before_anything_is_written():
    wl = small_wl(cid=72)
    pair = H.build_pair(wl)
    g = pair.gpu
    host_round(pair, 0)
    snap = g.state_export()
    B, m, h = wl.n_requests, wl.n_inputs, wl.window_h
    off_pend = 24 + B * m * 4
    off_pushed = off_pend + B * 12 + B * h * TB.MAX_DEV * 8 + B * TB.MAX_DEV * 8
    off_head = off_pushed + B * 8
    off_count, off_j, off_len = off_head + B * 4, off_head + 2 * B * 4, off_head + 3 * B * 4

    def patched(off, value):
        b = bytearray(snap)
        b[off:off + 4] = struct.pack("<i", value)
        return bytes(b)

    bad = [patched(off_pend, 3), patched(off_pend, 0), patched(off_pend + 4, wl.drafter.vocab), patched(off_pend + 4, -1),
           patched(off_head, h), patched(off_head, -1), patched(off_count, h + 1), patched(off_j, 11),
           patched(off_len, wl.kv_capacity + 1), patched(off_len, -1), patched(0, 0x1234)]
    before = [g.debug_view(v).clone() for v in (TB.VIEW_WEIGHTS, TB.VIEW_PENDING, TB.VIEW_KV_LEN, TB.VIEW_WINDOW_SUM)]
    for blob in bad:
        with pytest.raises(TB.TabedError) as e:
            g.state_import(blob)
        assert e.value.code == TB.ERR_INVALID_ARG
    after = [g.debug_view(v) for v in (TB.VIEW_WEIGHTS, TB.VIEW_PENDING, TB.VIEW_KV_LEN, TB.VIEW_WINDOW_SUM)]
    assert all(torch.equal(x, y) for x, y in zip(before, after))
    g.state_import(snap)
    host_round(pair, 1)
    assert g.last_device_error() == 0
    g.destroy()


def test_offset_views_take_the_element_wise_path_with_identical_results():
    """q / qk / logits pointers that are only 4-byte aligned (views with a storage offset)."""
    wl = W.LLAVA_SMALL.replace(n_requests=2)
    V, m, B = wl.drafter.vocab, 3, 2
    g = H.make_gpu(wl)
    lg = H.t(W.logits_like_drafter(wl, 3)[0])
    u = H.t(W.lattice_uniforms(W.substream(2, "off_u"), (B,)))
    y0 = torch.empty(B, dtype=torch.int32, device=H.DEV); q0 = torch.empty((B, V), device=H.DEV); qk0 = torch.empty((B, m, V), device=H.DEV)
    g.ensemble_step(lg, None, u, y0, q0, qk0)
    big_q = torch.zeros(B * V + 8, device=H.DEV); big_qk = torch.zeros(B * m * V + 8, device=H.DEV); big_lg = torch.zeros(B * m * V + 8, device=H.DEV)
    q1 = big_q[1:1 + B * V].view(B, V); qk1 = big_qk[3:3 + B * m * V].view(B, m, V); lg1 = big_lg[1:1 + B * m * V].view(B, m, V)
    lg1.copy_(lg)
    assert q1.data_ptr() % 16 == 4 and qk1.data_ptr() % 16 == 12 and lg1.data_ptr() % 16 == 4
    y1 = torch.empty(B, dtype=torch.int32, device=H.DEV)
    g.ensemble_step(lg1, None, u, y1, q1, qk1)
    torch.cuda.synchronize()
    assert torch.equal(y0, y1) and torch.equal(q0, q1) and torch.equal(qk0, qk1)
    assert big_q[0] == 0 and big_q[1 + B * V] == 0 and big_qk[2] == 0 and big_qk[3 + B * m * V] == 0
    y2 = torch.empty(B, dtype=torch.int32, device=H.DEV)
    w = g.debug_view(TB.VIEW_WEIGHTS).clone()
    q1.zero_(); qk1.zero_()
    TB.ensemble_step_static(lg1, w, u, y2, q1, qk1)
    torch.cuda.synchronize()
    assert torch.equal(y0, y2) and torch.equal(q0, q1) and torch.equal(qk0, qk1)
    g.destroy()


def test_two_handles_of_different_shapes_alternate():
    """Two live handles whose persistent kernels need different amounts of shared memory."""
    pa = H.build_pair(small_wl(d=512, heads=8, kv_heads=2, ffn=1280, cid=73))
    pb = H.build_pair(small_wl(d=128, heads=2, kv_heads=1, ffn=320, vocab=1500, cid=74))
    assert pa.gpu.current_path() == TB.PATH_PERSISTENT and pb.gpu.current_path() == TB.PATH_PERSISTENT
    for rnd in range(2):
        H.lockstep_round(pa, rnd, override=True)
        H.lockstep_round(pb, rnd, override=True)
    pa.gpu.destroy()
    H.lockstep_round(pb, 2, override=True)
    pb.gpu.destroy()


def test_host_round_keeps_exact_cache_lengths():
    """With the host-buffer round the overflow check works on exact lengths: a capacity that the per-round worst
    case (gamma + 1 positions) would exhaust after a few rounds lasts as long as the caches really have room."""
    G = 3
    wl = small_wl(gamma=G, cap=40 + 30, cid=75)          # longest prefix 40; worst case 4 per round -> 6 rounds
    pair = H.build_pair(wl)
    g = pair.gpu
    V = wl.drafter.vocab
    reject = np.full((1, G + 1, V), -30.0, np.float32)    # the target puts all its mass on one token: the first draft is
    reject[:, :, 7] = 30.0                                # (almost surely) rejected and a round keeps one position per row
    rounds = 0
    try:
        while rounds < 40:
            toks, a, z, w, am = host_round(pair, rounds, target=reject)
            rounds += 1
    except TB.TabedError as e:
        assert e.code == TB.ERR_KV_OVERFLOW
    lens = g.debug_view(TB.VIEW_KV_LEN).cpu().numpy()
    assert rounds >= 15                                   # far more rounds than the worst-case bound (6) allows
    assert lens.max() + 2 + G - 1 > wl.kv_capacity        # and it stopped only when the next round could really overflow
    assert g.last_device_error() == 0
    # the asynchronous calls are conservative; tabed_sync_lengths makes the bound exact again
    g.destroy()
    pair = H.build_pair(wl.replace(config_id=76))
    g = pair.gpu
    toks = torch.empty((1, G), dtype=torch.int32, device=H.DEV)
    u = torch.full((1, G), 0.5, device=H.DEV)
    a = torch.empty(1, dtype=torch.int32, device=H.DEV)
    n_async = 0
    for _ in range(40):
        try:
            g.draft_round(u, toks)
        except TB.TabedError as e:
            assert e.code == TB.ERR_KV_OVERFLOW
            g.sync_lengths()
            if int(g.debug_view(TB.VIEW_KV_LEN).max()) + 2 + G - 1 > wl.kv_capacity:
                break
            g.draft_round(u, toks)
        g.verify(H.t(reject), u, u[:, 0].contiguous(), a, a.clone())
        g.update_weights()
        n_async += 1
    assert n_async >= 15 and g.last_device_error() == 0
    g.destroy()


def test_random_policy_needs_its_uniforms():
    wl = W.TINY.replace(policy=W.POLICY_RANDOM)
    g = H.make_gpu(wl)
    B, G, V = wl.n_requests, wl.gamma, wl.drafter.vocab
    u = torch.full((B, G), 0.5, device=H.DEV)
    toks = torch.empty((B, G), dtype=torch.int32, device=H.DEV)
    a = torch.empty(B, dtype=torch.int32, device=H.DEV)
    g.draft_round_logits(torch.zeros((G, B, wl.n_inputs, V), device=H.DEV), u, toks)
    g.verify(torch.zeros((B, G + 1, V), device=H.DEV), u, u[:, 0].contiguous(), a, a.clone())
    with pytest.raises(TB.TabedError) as e:
        g.update_weights()
    assert e.value.code == TB.ERR_BAD_STATE
    g.set_policy_uniforms(torch.full((B, wl.n_inputs), 0.25, device=H.DEV))
    w = torch.empty((B, wl.n_inputs), device=H.DEV)
    g.update_weights(w)
    torch.cuda.synchronize()
    assert torch.allclose(w, torch.full_like(w, 0.5)) and g.last_device_error() == 0
    with pytest.raises(TB.TabedError):
        TB.Tabed(n_inputs=3, n_requests=1, gamma=3, window_h=2, policy=TB.POLICY_GRID_HARD, vocab=100)
    g.destroy()
