"""The allocation-free ensemble step against the handle-based one.

tabed_ensemble_step_static serves callers that cannot allocate device memory where they draft
(a server whose pool already owns the GPU, a fixed memory budget, a path that must avoid
cudaMalloc), so it keeps its scratch in a fixed array inside the library.  It must return exactly
what tabed_ensemble_step returns: token ids and distributions bit for bit (the arithmetic is
order-independent), on two calls in a row, because the shared scratch keeps the previous call's
contents.  This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from paper_2601_20357_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _case(B, m, V, seed, mode):
    from paper_2601_20357_b200 import binding as TB
    dev = torch.device("cuda", 0)
    g = torch.Generator(device="cpu").manual_seed(seed)
    logits = (torch.randn((B, m, V), generator=g) * 1.3).to(dev)
    w = torch.softmax(torch.randn((B, m), generator=g), dim=-1).to(dev).contiguous()
    u = torch.from_numpy(W.lattice_uniforms(np.random.default_rng(seed), (B,))).to(dev)
    return TB, dev, logits, w, u


@pytest.mark.parametrize("B,m,V,mode", [(2, 3, 32000, 0), (1, 2, 1000, 0), (4, 4, 5003, 1)])
def test_static_entry_point_matches_handle_entry_point_twice(B, m, V, mode):
    TB, dev, logits, w, u = _case(B, m, V, 11, mode)
    h = TB.Tabed(n_inputs=m, n_requests=B, gamma=1, window_h=1, policy=TB.POLICY_STATIC, vocab=V, sample_mode=mode)
    for call in range(2):
        if call == 1:                                    # second call: new inputs over the used scratch
            TB, dev, logits, w, u = _case(B, m, V, 12, mode)
        y0 = torch.empty(B, dtype=torch.int32, device=dev); q0 = torch.empty((B, V), device=dev)
        qk0 = torch.empty((B, m, V), device=dev)
        h.ensemble_step(logits, w, u, y0, q0, qk0)
        y1 = torch.full((B,), -1, dtype=torch.int32, device=dev); q1 = torch.zeros((B, V), device=dev)
        qk1 = torch.zeros((B, m, V), device=dev)
        TB.ensemble_step_static(logits, w, u, y1, q1, qk1, sample_mode=mode)
        torch.cuda.synchronize()
        assert torch.equal(y0, y1)
        assert torch.equal(q0, q1) and torch.equal(qk0, qk1)      # tolerance 0: bitwise, as in the other tests
        # ... and against the CPU checker itself, not only against the other entry point
        from oracle import exact32 as X
        lg_h, w_h, u_h = logits.cpu().numpy(), w.cpu().numpy(), u.cpu().numpy()
        for b in range(B):
            qk_o = X.softmax_exact(lg_h[b]); q_o = X.ensemble_exact(qk_o, w_h[b])
            assert np.array_equal(qk1[b].cpu().numpy(), qk_o) and np.array_equal(q1[b].cpu().numpy(), q_o)
            assert int(y1[b]) == (X.argmax_lowest(q_o) if mode == 1 else X.draw(X.masses(q_o), u_h[b]))
    h.destroy()


def test_static_entry_point_rejects_sizes_beyond_its_scratch():
    from paper_2601_20357_b200 import binding as TB
    dev = torch.device("cuda", 0)
    B, m, V = 600, 2, 8                                  # 1200 rows > 1024
    logits = torch.zeros((B, m, V), device=dev); w = torch.full((B, m), 0.5, device=dev)
    u = torch.full((B,), 0.5, device=dev)
    y = torch.empty(B, dtype=torch.int32, device=dev); q = torch.empty((B, V), device=dev)
    with pytest.raises(TB.TabedError) as e:
        TB.ensemble_step_static(logits, w, u, y, q)
    assert e.value.code == -7
