"""Pins for oracle/drafter.py (CPU only): the forward pass against library routines and identities."""
import numpy as np
import pytest
import torch

from oracle.drafter import OracleDrafter, round_bf16
from paper_2601_20357_b200 import workloads as W

SMALL_FP32 = W.DrafterCfg(2, 64, 4, 4, 160, 97, "fp32")
SMALL_BF16 = W.DrafterCfg(2, 64, 4, 2, 160, 97, "bf16")


def small_workload(cfg, cid=91):
    return W.Workload(name="t", config_id=cid, drafter=cfg, n_inputs=2, n_requests=1, gamma=2,
                      window_h=2, rounds=1, policy=W.POLICY_STATIC)


def make(cfg):
    wl = small_workload(cfg)
    return OracleDrafter(cfg, W.make_weights(wl)), W.make_weights(wl)


def torch_forward(cfg, weights, tokens):
    """Independent fp64 restatement with torch library ops (full sequence, no cache)."""
    t = lambda a: torch.tensor(np.asarray(a), dtype=torch.float64)
    bf = (lambda x: x.to(torch.float32).to(torch.bfloat16).to(torch.float64)) if cfg.dtype == "bf16" else (lambda x: x)
    T, H, Hkv, hd = len(tokens), cfg.n_heads, cfg.n_kv_heads, cfg.head_dim
    x = t(weights["embed"])[torch.tensor(tokens, dtype=torch.long)]
    pos = torch.arange(T, dtype=torch.float64)
    inv = cfg.rope_theta ** (-torch.arange(0, hd, 2, dtype=torch.float64) / hd)
    ang = torch.outer(pos, inv)
    cos, sin = torch.cos(ang).repeat(1, 2)[:, None, :], torch.sin(ang).repeat(1, 2)[:, None, :]

    def rot(v):  # rotate-half convention
        half = hd // 2
        return torch.cat([-v[..., half:], v[..., :half]], dim=-1)

    def norm(v, g):
        return torch.nn.functional.rms_norm(v, (cfg.d_model,), t(g), cfg.rms_eps)

    for l in range(cfg.n_layers):
        a = bf(norm(x, weights["norm1"][l]))
        q = torch.nn.functional.linear(a, t(weights["wq"][l])).view(T, H, hd)
        k = torch.nn.functional.linear(a, t(weights["wk"][l])).view(T, Hkv, hd)
        v = torch.nn.functional.linear(a, t(weights["wv"][l])).view(T, Hkv, hd)
        q = bf(q * cos + rot(q) * sin)
        k = bf(k * cos + rot(k) * sin)
        v = bf(v)
        o = torch.nn.functional.scaled_dot_product_attention(
            q.transpose(0, 1)[None], k.transpose(0, 1)[None], v.transpose(0, 1)[None],
            is_causal=True, enable_gqa=(H != Hkv))[0].transpose(0, 1).reshape(T, H * hd)
        x = x + torch.nn.functional.linear(bf(o), t(weights["wo"][l]))
        b = bf(norm(x, weights["norm2"][l]))
        g = torch.nn.functional.linear(b, t(weights["w_gate"][l]))
        u = torch.nn.functional.linear(b, t(weights["w_up"][l]))
        x = x + torch.nn.functional.linear(bf(torch.nn.functional.silu(g) * u), t(weights["w_down"][l]))
    return torch.nn.functional.linear(bf(norm(x, weights["final_norm"])), t(weights["lm_head"])).numpy()


@pytest.mark.parametrize("cfg", [SMALL_FP32, SMALL_BF16], ids=["fp32", "bf16_gqa"])
def test_forward_matches_torch_library_restatement(cfg):
    dr, weights = make(cfg)
    # non-trivial norm gains so that a dropped gain fails
    rng = np.random.default_rng(0)
    for l in range(cfg.n_layers):
        weights["norm1"][l] = W.to_bf16_grid(1 + 0.1 * rng.standard_normal(cfg.d_model).astype(np.float32))
        weights["norm2"][l] = W.to_bf16_grid(1 + 0.1 * rng.standard_normal(cfg.d_model).astype(np.float32))
    weights["final_norm"] = W.to_bf16_grid(1 + 0.1 * rng.standard_normal(cfg.d_model).astype(np.float32))
    # larger weights so that attention is far from uniform
    for nm in W.WEIGHT_NAMES_PER_LAYER:
        weights[nm] = [W.to_bf16_grid(w * 8) for w in weights[nm]]
    dr = OracleDrafter(cfg, weights)
    tokens = rng.integers(0, cfg.vocab, size=23)
    cache = dr.new_cache(64)
    got = dr.forward(cache, dr.embed_tokens(tokens))
    ref = torch_forward(cfg, weights, tokens)
    if cfg.dtype == "fp32":
        np.testing.assert_allclose(got, ref, rtol=0, atol=1e-11)
    else:
        # bf16 rounding points identical; a value within 1e-16 of a rounding boundary may flip
        assert np.mean(np.abs(got - ref)) < 1e-6 and np.max(np.abs(got - ref)) < 1e-3


@pytest.mark.parametrize("cfg", [SMALL_FP32, SMALL_BF16], ids=["fp32", "bf16_gqa"])
def test_chunked_prefill_equals_token_by_token_decode(cfg):
    dr, _ = make(cfg)
    rng = np.random.default_rng(1)
    tokens = rng.integers(0, cfg.vocab, size=17)
    c1 = dr.new_cache(32)
    full = dr.forward(c1, dr.embed_tokens(tokens))
    c2 = dr.new_cache(32)
    dr.forward(c2, dr.embed_tokens(tokens[:9]), want_logits=False)
    step = [dr.forward(c2, dr.embed_tokens(tokens[i:i + 1]))[0] for i in range(9, 17)]
    assert c1.length == c2.length == 17
    if cfg.dtype == "fp32":
        np.testing.assert_allclose(np.stack(step), full[9:], atol=1e-12)
        np.testing.assert_allclose(c1.k[:, :, :17], c2.k[:, :, :17], atol=1e-13)
    else:
        assert np.mean(np.abs(np.stack(step) - full[9:])) < 1e-6


def test_rope_relative_position_identity():
    dr, _ = make(SMALL_FP32)
    rng = np.random.default_rng(2)
    hd = SMALL_FP32.head_dim
    q, k = rng.standard_normal((1, 1, hd)), rng.standard_normal((1, 1, hd))
    def dot(a, b):
        return float(np.sum(dr.rope(q, np.array([a])) * dr.rope(k, np.array([b]))))
    assert dot(5, 3) == pytest.approx(dot(105, 103), abs=1e-10)
    assert dot(5, 3) == pytest.approx(dot(2, 0), abs=1e-10)
    assert dot(0, 0) == pytest.approx(float(np.sum(q * k)), abs=1e-12)
    assert dot(7, 3) != pytest.approx(dot(3, 7), abs=1e-6)
    # norm preserved
    assert np.linalg.norm(dr.rope(q, np.array([11]))) == pytest.approx(np.linalg.norm(q))


def test_single_position_attention_returns_value_and_equal_prefixes_equal_logits():
    cfg = SMALL_FP32
    dr, w = make(cfg)
    tok = np.array([5])
    cache = dr.new_cache(8)
    dr.forward(cache, dr.embed_tokens(tok))
    # with one cached position softmax weight is 1: the layer-0 attention output is V[0]; check via
    # a hand computation of layer 0's contribution
    x = dr.embed_tokens(tok)
    a = dr.rmsnorm(x, dr.layers[0]["norm1"])
    v = a @ dr.layers[0]["wv"].T
    np.testing.assert_allclose(cache.v[0, :, 0, :].reshape(-1), v[0], atol=1e-14)
    # two rows with the same prefix give the same logits
    rng = np.random.default_rng(3)
    tokens = rng.integers(0, cfg.vocab, size=9)
    l1 = dr.forward(dr.new_cache(16), dr.embed_tokens(tokens))
    l2 = dr.forward(dr.new_cache(16), dr.embed_tokens(tokens))
    assert np.array_equal(l1, l2)
    # and a different prefix gives different logits for the same last token
    t2 = tokens.copy(); t2[0] = (t2[0] + 1) % cfg.vocab
    l3 = dr.forward(dr.new_cache(16), dr.embed_tokens(t2))
    assert np.max(np.abs(l3[-1] - l1[-1])) > 1e-9


def test_round_bf16_against_torch():
    rng = np.random.default_rng(4)
    x = np.concatenate([rng.standard_normal(10000) * 3, [0.0, 1.00390625, 1.01171875, -1.00390625, 3.0e-39]])
    ref = torch.tensor(x, dtype=torch.float64).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(round_bf16(x), ref)


def test_workload_bf16_grid_helpers_against_torch():
    rng = np.random.default_rng(5)
    x = (rng.standard_normal(5000) * 0.02).astype(np.float32)
    g = W.to_bf16_grid(x)
    t = torch.tensor(x).to(torch.bfloat16)
    assert np.array_equal(g, t.to(torch.float32).numpy())
    assert np.array_equal(W.f32_to_bf16_bits(g), t.view(torch.int16).numpy().view(np.uint16))


def test_bf16_rounding_flip_noise_sets_the_logit_tolerance():
    """Two evaluations that differ by 1e-7 relative before each bf16 rounding (what fp32 against fp64
    accumulation amounts to) disagree on some roundings; this measures how far the logits move and
    checks it stays inside the bound the GPU parity tests use for a bf16 drafter."""
    cfg = W.DrafterCfg(2, 256, 4, 2, 640, 3000, "bf16")
    wl = W.Workload(name="flip", config_id=41, drafter=cfg, n_inputs=1, n_requests=1, gamma=2, window_h=2,
                    rounds=1, policy=W.POLICY_STATIC)
    weights = W.make_weights(wl)

    class Perturbed(OracleDrafter):
        def rb(self, x):
            return round_bf16(x * (1 + 1e-7 * self.noise.standard_normal(x.shape)))

    a, b = OracleDrafter(cfg, weights), Perturbed(cfg, weights)
    b.noise = np.random.default_rng(0)
    tokens = np.random.default_rng(1).integers(0, cfg.vocab, size=150)
    ca, cb = a.new_cache(160), b.new_cache(160)
    a.forward(ca, a.embed_tokens(tokens[:-1]), want_logits=False)
    b.forward(cb, b.embed_tokens(tokens[:-1]), want_logits=False)
    la = a.forward(ca, a.embed_tokens(tokens[-1:]))
    lb = b.forward(cb, b.embed_tokens(tokens[-1:]))
    err = np.abs(la - lb)
    assert 1e-5 < err.mean() < 1e-2 and err.max() < 6e-2
    # and the probabilities stay inside the 1e-5 bar
    from oracle import definitions as D
    assert np.max(np.abs(D.softmax(la) - D.softmax(lb))) < 1e-5
