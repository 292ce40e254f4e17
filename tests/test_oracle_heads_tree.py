"""Pins of the oracle's cross-attention decoding head (Eq. 3) and of its probability-tree sampler (Appendix)."""
import itertools

import numpy as np
import pytest

from conftest import tiny_cfg
from paper_2507_23777_b200 import inputs


def _softmax(s):
    s = s - s.max(-1, keepdims=True)
    e = np.exp(s)
    return e / e.sum(-1, keepdims=True)


@pytest.mark.parametrize("dtype", [0, 1])
def test_cross_attention_head_matches_a_dense_statement(oracle_mod, dtype):
    """Head i on a hidden state g: y = g + Wo Attn(Wq g, Wk c, Wv c), logits = Wout y, written here with float64
    matrices and one einsum per product (a transposed operand, a dropped residual, a wrong head split or scale in the
    oracle fails this); and the step routine feeds the heads the final hidden state of every window row."""
    cfg = tiny_cfg(dtype=dtype, head_kind=1, n_draft=3)
    w = inputs.make_weights(cfg, random_gains=True)
    wf = inputs.weights_as_f32(cfg, w)
    W = {n: inputs.tensor_view(cfg, wf, n).astype(np.float64) for n, _, _ in inputs.weight_tensors(cfg)}
    cond = inputs.make_cond(cfg, 1)[0]
    orc = oracle_mod.Oracle(cfg, w)
    s = orc.new_seq(cond, 0)
    H, dh, d = cfg["n_heads"], cfg["d_head"], cfg["d_model"]
    rng = np.random.default_rng(3)
    c = cond.astype(np.float64)
    for i in range(1, 4):
        g = rng.standard_normal(d).astype(np.float32)
        q = (W[f"h{i}.Wq"] @ g).reshape(H, dh)
        k = (c @ W[f"h{i}.Wk"].T).reshape(-1, H, dh)
        v = (c @ W[f"h{i}.Wv"].T).reshape(-1, H, dh)
        p = _softmax(np.einsum("hd,jhd->hj", q, k) / np.sqrt(dh))
        a = np.einsum("hj,jhd->hd", p, v).reshape(d)
        y = g + W[f"h{i}.Wo"] @ a
        np.testing.assert_allclose(s.head(i, g), W[f"h{i}.Wout"] @ y, rtol=3e-5, atol=3e-5)
    # the decoding step evaluates head i on g of every row
    dc = oracle_mod.decode_config(cfg)
    s.begin([0], dc)
    win, n = s.window(), s.len
    _, _, z0, zh = s.step(dc, want_logits=True)
    ref = orc.new_seq(cond, 0)
    for j in range(len(win)):
        _, g = ref.forward_row(int(win[j]), n + j)
        for i in range(1, 4):
            np.testing.assert_array_equal(zh[i - 1][j], ref.head(i, g))
    orc.close()


def _brute_tree(zh, ks, u):
    """Every root-to-leaf path over the top-ks tokens of each head, in depth-first order with children by rank; weight
    = product of full-softmax probabilities; paths with a running product below 1e-5 removed; inverse CDF."""
    D, V = zh.shape
    tok, m = [], []
    for d in range(D):
        p = _softmax(zh[d].astype(np.float64))
        order = np.lexsort((np.arange(V), -zh[d]))[:ks]
        tok.append(order)
        m.append(p[order])
    leaves = []
    for idx in itertools.product(range(ks), repeat=D):
        wgt, ok = 1.0, True
        for d, k in enumerate(idx):
            wgt *= m[d][k]
            if wgt < 1e-5:
                ok = False
                break
        if ok:
            leaves.append(([int(tok[d][k]) for d, k in enumerate(idx)], wgt))
    if not leaves:
        return [int(tok[d][0]) for d in range(D)], leaves
    total = sum(wg for _, wg in leaves)
    cum = 0.0
    for path, wg in leaves:
        cum += wg
        if cum > u * total:
            return path, leaves
    return leaves[-1][0], leaves


def test_tree_sampler_against_brute_force_enumeration(oracle_mod):
    rng = np.random.default_rng(0)
    for D, V, ks, scale in [(1, 9, 3, 2.0), (2, 7, 2, 1.0), (3, 12, 3, 3.0), (4, 10, 4, 1.5), (3, 300, 3, 0.3)]:
        zh = (rng.standard_normal((D, V)) * scale).astype(np.float32)
        for _ in range(60):
            r = int(rng.integers(0, 1 << 24))
            want, leaves = _brute_tree(zh, ks, r / 2.0 ** 24)
            got = oracle_mod.sample_tree(zh, ks, r)
            # a draw within 1e-9 of a CDF edge may legitimately fall either way
            total = sum(wg for _, wg in leaves) or 1.0
            edges = np.cumsum([wg for _, wg in leaves]) / total
            if len(edges) and np.min(np.abs(edges - r / 2.0 ** 24)) < 1e-9:
                continue
            assert got.tolist() == want, (D, V, ks, r)


def test_tree_sampler_invariants(oracle_mod):
    """One head: the tree is the inverse CDF over the top-k_s probabilities.  Peaked heads (nothing pruned): paths
    are drawn like independent draws from every head's renormalised top-k_s.  Pruned branches never appear.  When
    every complete path is pruned the most probable token of every head is returned."""
    rng = np.random.default_rng(1)
    V = 8
    z = np.log(np.array([0.4, 0.25, 0.15, 0.1, 0.04, 0.03, 0.02, 0.01], dtype=np.float64)).astype(np.float32)
    for r, want in [(0, 0), (int(0.49 * 2 ** 24), 0), (int(0.51 * 2 ** 24), 1), (int(0.82 * 2 ** 24), 2), ((1 << 24) - 1, 2)]:
        assert oracle_mod.sample_tree(z[None, :], 3, r)[0] == want       # 0.4 / 0.8 = 0.5, 0.65 / 0.8 = 0.8125
    # two peaked heads, nothing pruned: joint frequencies = product of the renormalised marginals
    z2 = np.stack([z, z[::-1].copy()])
    counts = np.zeros((2, 2))
    n = 20000
    for r in rng.integers(0, 1 << 24, n):
        a, b = oracle_mod.sample_tree(z2, 2, int(r))
        counts[[0, 1].index(a), [7, 6].index(b)] += 1
    p = np.array([0.4, 0.25]) / 0.65
    expect = np.outer(p, p) * n
    assert ((counts - expect) ** 2 / expect).sum() < 16.3          # chi-square, 3 degrees of freedom, p = 0.001
    # pruning: second tokens of probability 1e-3 each: the path (second, second, second) weighs 1e-9 and never appears,
    # the path (first, first, second) weighs about 1e-3 and does
    zp = np.log(np.array([0.998, 0.001, 0.001], dtype=np.float64)).astype(np.float32)
    z3 = np.stack([zp, zp, zp])
    seen = set()
    for r in list(rng.integers(0, 1 << 24, 4000)) + [(1 << 24) - 1]:
        seen.add(tuple(oracle_mod.sample_tree(z3, 2, int(r)).tolist()))
    assert (1, 1, 1) not in seen and (1, 1, 0) not in seen and (0, 0, 0) in seen and (0, 0, 1) in seen
    # every complete path below 1e-5 (eight flat heads over 64 tokens): the most probable token of every head
    zf = (rng.standard_normal((8, 64)) * 0.01).astype(np.float32)
    got = oracle_mod.sample_tree(zf, 4, 12345)
    assert got.tolist() == [int(np.lexsort((np.arange(64), -zf[d]))[0]) for d in range(8)]


def test_tree_mode_decoding_step(oracle_mod):
    """sample_mode 2 in the decoding loop: x_{s*} is drawn from the backbone's row as in mode 1, the drafts are one
    path of the tree over the heads' rows of the first rejection (slot 1's random number)."""
    cfg = tiny_cfg(n_draft=3, verify_mode=1, k_accept=3, sample_mode=2, k_sample=3, temperature=0.7)
    w = inputs.make_weights(cfg)
    cond = inputs.make_cond(cfg, 1)[0]
    orc = oracle_mod.Oracle(cfg, w)
    dc = oracle_mod.decode_config(cfg)
    s = orc.new_seq(cond, 0)
    s.begin([0], dc)
    for _ in range(6):
        step = s.step_idx
        toks, a, z0, zh = s.step(dc, want_logits=True)
        nw = s.window()
        one = oracle_mod.decode_config(dict(cfg, sample_mode=1))
        assert nw[0] == oracle_mod.sample(z0[a], one, oracle_mod.rand24(cfg["seed"], 0, step, 0, 0))
        want = oracle_mod.sample_tree(zh[:, a], 3, oracle_mod.rand24(cfg["seed"], 0, step, 1, 0))
        assert np.array_equal(nw[1:], want)
    orc.close()
