"""Pins of the oracle's model arithmetic against an independent dense forward.

The dense forward below is a different formulation from the oracle's: whole
sequence at once, float64 matrices, a full causal score matrix instead of a
cache, complex multiplication for the rotary embedding.  A dropped residual, a
transposed operand, a wrong norm, a wrong RoPE pairing or an off-by-one in the
cache indexing in the oracle fails these tests.
"""
import numpy as np
import pytest

from conftest import tiny_cfg
from paper_2507_23777_b200 import inputs


def dense_forward(cfg, wf32, cond, tokens):
    """Logits [n, V] and final normed hidden [n, d] for a whole token sequence."""
    W = {n: inputs.tensor_view(cfg, wf32, n).astype(np.float64) for n, _, _ in inputs.weight_tensors(cfg)}
    d, H, dh = cfg["d_model"], cfg["n_heads"], cfg["d_head"]
    n = len(tokens)
    eps = cfg["rms_eps"]

    def norm(x, g):
        return x / np.sqrt((x * x).mean(-1, keepdims=True) + eps) * g

    def rot(x):  # x [n, H, dh]; pair (i, i+dh/2) as one complex number
        half = dh // 2
        z = x[..., :half] + 1j * x[..., half:]
        ang = np.arange(n)[:, None, None] * cfg["rope_theta"] ** (-2.0 * np.arange(half) / dh)[None, None, :]
        z = z * np.exp(1j * ang)
        return np.concatenate([z.real, z.imag], -1)

    def softmax(s):
        s = s - s.max(-1, keepdims=True)
        e = np.exp(s)
        return e / e.sum(-1, keepdims=True)

    h = W["E"][np.asarray(tokens)]
    mask = np.triu(np.full((n, n), -np.inf), 1)
    c = cond.astype(np.float64)
    for l in range(cfg["n_layers"]):
        p = f"l{l}."
        u = norm(h, W[p + "g1"])
        q = rot((u @ W[p + "Wq"].T).reshape(n, H, dh))
        k = rot((u @ W[p + "Wk"].T).reshape(n, H, dh))
        v = (u @ W[p + "Wv"].T).reshape(n, H, dh)
        s = np.einsum("ihd,jhd->hij", q, k) / np.sqrt(dh) + mask
        a = np.einsum("hij,jhd->ihd", softmax(s), v).reshape(n, d)
        h = h + a @ W[p + "Wo"].T
        u = norm(h, W[p + "g2"])
        q = (u @ W[p + "Wqc"].T).reshape(n, H, dh)
        kc = (c @ W[p + "Wkc"].T).reshape(-1, H, dh)
        vc = (c @ W[p + "Wvc"].T).reshape(-1, H, dh)
        s = np.einsum("ihd,jhd->hij", q, kc) / np.sqrt(dh)
        a = np.einsum("hij,jhd->ihd", softmax(s), vc).reshape(n, d)
        h = h + a @ W[p + "Woc"].T
        u = norm(h, W[p + "g3"])
        ga, up = u @ W[p + "Wgate"].T, u @ W[p + "Wup"].T
        h = h + (ga / (1 + np.exp(-ga)) * up) @ W[p + "Wdown"].T
    g = norm(h, W["gf"])
    return g @ W["W0"].T, g, W


@pytest.mark.parametrize("dtype", [0, 1])
def test_row_forward_matches_dense_forward(oracle_mod, dtype):
    cfg = tiny_cfg(dtype=dtype)
    w = inputs.make_weights(cfg, random_gains=True)
    wf = inputs.weights_as_f32(cfg, w)
    cond = inputs.make_cond(cfg, 1)[0]
    rng = np.random.default_rng(5)
    toks = rng.integers(0, cfg["vocab"], 23)
    ref_logits, ref_g, W = dense_forward(cfg, wf, cond, toks)
    orc = oracle_mod.Oracle(cfg, w, n_pages=8)
    s = orc.new_seq(cond, 0, max_positions=32)
    for p, t in enumerate(toks):
        z, g = s.forward_row(int(t), p)
        np.testing.assert_allclose(z, ref_logits[p], rtol=2e-5, atol=2e-5)
        np.testing.assert_allclose(g, ref_g[p], rtol=2e-5, atol=2e-5)
    # decoding head: logits = Wout (g + SiLU(W1 g)), checked on the dense g
    for i in (1, 2):
        g = ref_g[7].astype(np.float32)
        t = W[f"h{i}.W1"] @ g.astype(np.float64)
        y = g + t / (1 + np.exp(-t))
        np.testing.assert_allclose(orc.head(i, g), W[f"h{i}.Wout"] @ y, rtol=2e-5, atol=2e-5)


def test_cache_row_is_rotated_key_and_plain_value(oracle_mod):
    """The cache holds the key after RoPE at its absolute position and the value as projected."""
    cfg = tiny_cfg(n_layers=1)
    w = inputs.make_weights(cfg, random_gains=True)
    cond = inputs.make_cond(cfg, 1)[0]
    toks = [3, 9, 9, 1, 40, 17]
    _, _, W = dense_forward(cfg, w, cond, toks)
    h = W["E"][np.asarray(toks)]
    u = h / np.sqrt((h * h).mean(-1, keepdims=True) + cfg["rms_eps"]) * W["l0.g1"]
    k = (u @ W["l0.Wk"].T).reshape(len(toks), cfg["n_heads"], cfg["d_head"])
    v = u @ W["l0.Wv"].T
    half = cfg["d_head"] // 2
    orc = oracle_mod.Oracle(cfg, w, n_pages=4)
    s = orc.new_seq(cond, 0, max_positions=16)
    for p, t in enumerate(toks):
        s.forward_row(t, p)
    for p in range(len(toks)):
        th = p * cfg["rope_theta"] ** (-2.0 * np.arange(half) / cfg["d_head"])
        kr = np.concatenate([k[p, :, :half] * np.cos(th) - k[p, :, half:] * np.sin(th),
                             k[p, :, :half] * np.sin(th) + k[p, :, half:] * np.cos(th)], -1).reshape(-1)
        np.testing.assert_allclose(s.kv(0, 0, p), kr, rtol=1e-5, atol=1e-6)
        np.testing.assert_allclose(s.kv(0, 1, p), v[p], rtol=1e-5, atol=1e-6)


def test_position_zero_rope_is_identity_and_single_key_returns_value(oracle_mod):
    """At position 0 the rotation is the identity and attention over one key returns its value,
    so with Wo = I-like access through the cache: k row == Wk u exactly as projected."""
    cfg = tiny_cfg(n_layers=1)
    w = inputs.make_weights(cfg)
    cond = inputs.make_cond(cfg, 1)[0]
    W = {n: inputs.tensor_view(cfg, w, n).astype(np.float64) for n, _, _ in inputs.weight_tensors(cfg)}
    orc = oracle_mod.Oracle(cfg, w, n_pages=2)
    s = orc.new_seq(cond, 0, max_positions=8)
    s.forward_row(7, 0)
    h = W["E"][7]
    u = h / np.sqrt((h * h).mean() + cfg["rms_eps"])
    np.testing.assert_allclose(s.kv(0, 0, 0), W["l0.Wk"] @ u, rtol=1e-5, atol=1e-7)


def test_bf16_storage_reads_the_rounded_values(oracle_mod):
    """dtype 1 must use exactly the bf16 values: same logits as an fp32 oracle given the widened buffer."""
    cfg = tiny_cfg(dtype=1)
    w16 = inputs.make_weights(cfg)
    cond = inputs.make_cond(cfg, 1)[0]
    cfg32 = dict(cfg, dtype=0)
    w32 = np.ascontiguousarray(inputs.bf16_bits_to_f32(w16))
    a = oracle_mod.Oracle(cfg, w16, n_pages=4).new_seq(cond, 0, 16)
    b = oracle_mod.Oracle(cfg32, w32, n_pages=4).new_seq(cond, 0, 16)
    for p, t in enumerate([1, 2, 3, 4, 5]):
        za, _ = a.forward_row(t, p)
        zb, _ = b.forward_row(t, p)
        assert np.array_equal(za, zb)


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, -0.1], dtype=np.float32)
    r = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(x))
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == np.float32(1.0 + 2.0 ** -6) and r[3] == np.float32(1 + 2.0 ** -7)
    assert abs(r[4] + 0.1) < 0.1 * 2.0 ** -8
