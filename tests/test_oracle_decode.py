"""Pins of the oracle's decoding loop (Algorithm 1), acceptance rules, sampling and RNG."""
import os

import numpy as np
import pytest

from conftest import tiny_cfg
from paper_2507_23777_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _mk(oracle_mod, cfg, n_pages=64, batch=1):
    w = inputs.make_weights(cfg, random_gains=True)
    cond = inputs.make_cond(cfg, batch)
    return oracle_mod.Oracle(cfg, w, n_pages=n_pages), cond


def test_philox_known_answers(oracle_mod):
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) if l[0] != "#"]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        assert oracle_mod.philox4x32_10(v[0:4], v[4:6]) == v[6:10]


def test_philox_agrees_with_curand_host_generator(oracle_mod):
    """cuRAND's Philox4_32_10 host generator, called as a library: with seed s and offset 0 it emits the four words
    of counter (n, 0, t, 0), key (s_lo, s_hi), for t = 0 .. T-1 (one block per generator thread), then n + 1.  The
    oracle's block function must give the same words (round function, key schedule, word order)."""
    import ctypes as C
    try:
        lib = C.CDLL("libcurand.so")
    except OSError:
        try:
            lib = C.CDLL("/usr/local/cuda/lib64/libcurand.so")
        except OSError:
            pytest.skip("libcurand not found")
    PHILOX4_32_10 = 161
    gen = C.c_void_p()
    if lib.curandCreateGeneratorHost(C.byref(gen), PHILOX4_32_10) != 0:
        pytest.skip("no cuRAND host generator")
    seed = 0x0123_4567_89AB_CDEF
    key = [seed & 0xFFFFFFFF, seed >> 32]
    assert lib.curandSetPseudoRandomGeneratorSeed(gen, C.c_ulonglong(seed)) == 0
    assert lib.curandSetGeneratorOffset(gen, C.c_ulonglong(0)) == 0
    n = 4 * 70000
    out = np.zeros(n, dtype=np.uint32)
    assert lib.curandGenerate(gen, out.ctypes.data_as(C.c_void_p), C.c_size_t(n)) == 0
    lib.curandDestroyGenerator(gen)
    blocks = out.reshape(-1, 4)
    for t in (0, 1, 2, 63, 1000):
        assert list(blocks[t]) == oracle_mod.philox4x32_10([0, 0, t, 0], key), t
    nxt = oracle_mod.philox4x32_10([1, 0, 0, 0], key)
    T = next(i for i in range(1, len(blocks)) if list(blocks[i]) == nxt)       # generator threads
    assert list(blocks[T + 5]) == oracle_mod.philox4x32_10([1, 0, 5, 0], key)
    assert list(blocks[T - 1]) == oracle_mod.philox4x32_10([0, 0, T - 1, 0], key)


def test_rand24_addressing(oracle_mod):
    """key = (seed_lo ^ seq_id, seed_hi), counter = (step, slot, purpose, 0), top 24 bits of word 0."""
    seed = 0x1234_5678_9ABC_DEF0
    for seq, step, slot, purpose in [(0, 0, 0, 0), (3, 17, 2, 0), (15, 4000, 4, 1)]:
        o = oracle_mod.philox4x32_10([step, slot, purpose, 0], [(seed & 0xFFFFFFFF) ^ seq, seed >> 32])
        assert oracle_mod.rand24(seed, seq, step, slot, purpose) == o[0] >> 8


# ---------------------------------------------------------------- acceptance

def test_strict_and_topk_acceptance(oracle_mod):
    z = np.array([0.1, 2.0, -1.0, 2.0, 0.5, 1.9], dtype=np.float32)   # order: 1, 3, 5, 4, 0, 2
    order = [1, 3, 5, 4, 0, 2]
    DC = oracle_mod.DecodeConfig
    for ka in range(1, 7):
        dc = DC(1, ka, 0.0, 0, 1, 1.0, 0)
        assert [oracle_mod.accept(z, x, dc) for x in range(6)] == [order.index(x) < ka for x in range(6)]
    strict = DC(0, 99, 0.0, 0, 1, 1.0, 0)          # k_accept ignored: K_a = 1, ties -> lowest index
    assert [oracle_mod.accept(z, x, strict) for x in range(6)] == [x == 1 for x in range(6)]
    assert not oracle_mod.accept(z, -1, strict) and not oracle_mod.accept(z, 6, strict)


def test_threshold_acceptance(oracle_mod):
    rng = np.random.default_rng(0)
    DC = oracle_mod.DecodeConfig
    for _ in range(20):
        z = rng.normal(0, 2, 40).astype(np.float32)
        p = np.exp(z.astype(np.float64) - z.max())
        p /= p.sum()
        for delta in (0.05, 0.2, 0.5):
            dc = DC(2, 1, delta, 0, 1, 1.0, 0)
            for x in range(40):
                if abs(p[x] - delta) > 1e-6:
                    assert oracle_mod.accept(z, x, dc) == (p[x] > delta)
        assert all(oracle_mod.accept(z, x, DC(2, 1, -1.0, 0, 1, 1.0, 0)) for x in range(40))   # delta < 0
        assert not any(oracle_mod.accept(z, x, DC(2, 1, 1.0, 0, 1, 1.0, 0)) for x in range(40))  # delta >= 1
    two = np.array([0.0, 0.0], dtype=np.float32)       # p = 0.5 exactly: strict inequality rejects
    assert not oracle_mod.accept(two, 0, DC(2, 1, 0.5, 0, 1, 1.0, 0))


# ------------------------------------------------------------------ sampling

def test_argmax_sampling_ties_to_lowest_index(oracle_mod):
    dc = oracle_mod.DecodeConfig(0, 1, 0.0, 0, 1, 1.0, 0)
    assert oracle_mod.sample(np.array([1, 3, 3, 2], dtype=np.float32), dc, 12345) == 1


def test_topk_temperature_sampling_distribution(oracle_mod):
    """Frequencies over 2^24-spaced u match softmax(z_topk / T); tokens outside the top k never appear."""
    z = np.array([0.3, 1.2, -0.5, 1.2, 0.9, 0.0, -2.0, 0.7], dtype=np.float32)
    k, T = 5, 0.5
    dc = oracle_mod.DecodeConfig(1, k, 0.0, 1, k, T, 0)
    order = sorted(range(8), key=lambda v: (-z[v], v))[:k]
    w = np.exp((z[order].astype(np.float64) - z[order[0]]) / T)
    p = w / w.sum()
    n = 1 << 14
    us = (np.arange(n, dtype=np.uint64) * ((1 << 24) // n) + 7).astype(np.uint32)   # stratified u
    draws = np.array([oracle_mod.sample(z, dc, int(u)) for u in us])
    assert set(draws.tolist()) <= set(order)
    freq = np.array([(draws == t).mean() for t in order])
    np.testing.assert_allclose(freq, p, atol=2.0 / n * k + 1e-4)
    # inverse CDF over the ordered candidates: first j with cum > u
    cdf = np.cumsum(p)
    for u24 in (0, 1, (1 << 23), (1 << 24) - 1, 5_000_000, 11_111_111):
        u = u24 / 2 ** 24
        if np.min(np.abs(cdf - u)) > 1e-9:
            assert oracle_mod.sample(z, dc, u24) == order[int(np.searchsorted(cdf, u, side="right"))]


def test_cdf_edge_is_strict(oracle_mod):
    """Two equal logits, T = 1: the CDF edge is exactly 0.5; u = 0.5 is not below it, so the second wins."""
    dc = oracle_mod.DecodeConfig(1, 2, 0.0, 1, 2, 1.0, 0)
    z = np.array([-3.0, 1.5, 1.5, 0.0], dtype=np.float32)
    assert oracle_mod.sample(z, dc, (1 << 23) - 1) == 1
    assert oracle_mod.sample(z, dc, 1 << 23) == 2


def test_low_temperature_limit_is_argmax(oracle_mod):
    rng = np.random.default_rng(1)
    for _ in range(10):
        z = rng.normal(0, 1, 64).astype(np.float32)
        dc = oracle_mod.DecodeConfig(1, 5, 0.0, 1, 5, 1e-4, 0)
        assert oracle_mod.sample(z, dc, int(rng.integers(0, 1 << 24))) == int(np.argmax(z))


# -------------------------------------------------------- Algorithm 1 itself

def _plain(orc, cond, dc, n, prompt=(0,)):
    return orc.new_seq(cond, 0).generate_plain(list(prompt), dc, n)


@pytest.mark.parametrize("dtype", [0, 1])
def test_strict_greedy_speculation_equals_plain_greedy(oracle_mod, dtype):
    """With K_a = 1 acceptance and argmax resampling the committed sequence is plain greedy decoding,
    whatever the heads and the initial drafts are (Sec. 3.1, Sec. 4.2)."""
    cfg = tiny_cfg(dtype=dtype)
    orc, cond = _mk(oracle_mod, cfg)
    dc = oracle_mod.decode_config(cfg)
    ref = _plain(orc, cond[0], dc, 48)
    for seed in (0, 1, 2):
        dcs = oracle_mod.decode_config(dict(cfg, seed=seed))   # other initial drafts
        s = orc.new_seq(cond[0], 0)
        s.begin([0], dcs)
        toks, steps, hist = s.generate(dcs, 48)
        assert np.array_equal(toks, ref)
        assert sum(h * (a + 1) for a, h in enumerate(hist)) >= 48 and sum(hist) == steps


def test_scripted_drafts_accept_all_or_none(oracle_mod):
    """Drafts equal to the true continuation are all accepted (a = K every step); drafts that are never
    the argmax are all rejected (a = 0).  Either way the output is the greedy sequence."""
    cfg = tiny_cfg()
    K, V = cfg["n_draft"], cfg["vocab"]
    orc, cond = _mk(oracle_mod, cfg)
    dc = oracle_mod.decode_config(cfg)
    ref = _plain(orc, cond[0], dc, 40)
    full = np.concatenate([[0], ref])
    for good in (True, False):
        s = orc.new_seq(cond[0], 0)
        s.begin([0], dc)
        out = []
        while len(out) < 30:
            n = s.len
            truth = full[n + 1:n + 1 + K]
            s.set_drafts(truth if good else (truth + 1) % V)
            toks, a, _, _ = s.step(dc)
            assert a == (K if good else 0) and len(toks) == a + 1
            out.extend(toks.tolist())
        assert out == ref[:len(out)].tolist()


def test_accept_everything_reduces_to_taking_all_drafts(oracle_mod):
    """delta < 0: the 'straightforward approach' of Sec. 4.2, every step commits K drafts + 1 sample."""
    cfg = tiny_cfg(verify_mode=inputs.VERIFY_THRESHOLD, delta=-1.0)
    orc, cond = _mk(oracle_mod, cfg)
    dc = oracle_mod.decode_config(cfg)
    s = orc.new_seq(cond[0], 0)
    s.begin([0], dc)
    for _ in range(5):
        w = s.window()
        toks, a, _, _ = s.step(dc)
        assert a == cfg["n_draft"] and np.array_equal(toks[:-1], w[1:])
    cfg2 = tiny_cfg(verify_mode=inputs.VERIFY_THRESHOLD, delta=1.0)
    dc2 = oracle_mod.decode_config(cfg2)
    s = orc.new_seq(cond[0], 0)
    s.begin([0], dc2)
    toks, steps, hist = s.generate(dc2, 20)
    assert steps == 20 and hist == [20, 0, 0]     # one backbone token per step: SCR = 1.000 (Table 3 row A)
    assert np.array_equal(toks, _plain(orc, cond[0], dc2, 20))


def test_no_heads_is_plain_decoding(oracle_mod):
    cfg = tiny_cfg(n_draft=0)
    orc, cond = _mk(oracle_mod, cfg)
    for mode in (0, 1):
        c = dict(cfg, sample_mode=mode, k_sample=4, temperature=0.8, verify_mode=mode, k_accept=4, seed=9)
        dc = oracle_mod.decode_config(c)
        s = orc.new_seq(cond[0], 0)
        s.begin([0], dc)
        toks, steps, hist = s.generate(dc, 25)
        assert steps == 25 and hist == [25]
        assert np.array_equal(toks, _plain(orc, cond[0], dc, 25))


def test_sampled_tokens_lie_in_backbone_topk(oracle_mod):
    """Top-k acceptance + top-k sampling: every committed token is within the backbone's top k at its
    position, and the step's output follows from its logits by the stated rules."""
    cfg = tiny_cfg(verify_mode=1, k_accept=3, sample_mode=1, k_sample=3, temperature=0.7, seed=4, sigma=0.6)
    K, V = cfg["n_draft"], cfg["vocab"]
    orc, cond = _mk(oracle_mod, cfg)
    dc = oracle_mod.decode_config(cfg)
    s = orc.new_seq(cond[0], 0)
    s.begin([0], dc)
    seen_accept = 0
    for step in range(40):
        if step % 2 == 0:   # plant a first draft that the backbone ranks second at row 0: it must be accepted
            w = s.window()
            z_peek, _ = s.forward_row(int(w[0]), s.len)
            second = sorted(range(V), key=lambda v: (-z_peek[v], v))[1]
            s.set_drafts([second] + w[2:].tolist())
        w = s.window()
        toks, a, z0, zh = s.step(dc, want_logits=True)
        exp_a = 0
        while exp_a < K and oracle_mod.accept(z0[exp_a], w[exp_a + 1], dc):
            exp_a += 1
        assert a == exp_a and (step % 2 or a >= 1)
        seen_accept += a
        for j, t in enumerate(toks):
            rank = sum(1 for v in range(V) if (z0[j][v] > z0[j][t]) or (z0[j][v] == z0[j][t] and v < t))
            assert rank < 3
        nw = s.window()
        assert nw[0] == toks[-1] == oracle_mod.sample(z0[a], dc, oracle_mod.rand24(4, 0, step, 0, 0))
        for i in range(1, K + 1):
            assert nw[i] == oracle_mod.sample(zh[i - 1][a], dc, oracle_mod.rand24(4, 0, step, i, 0))
    assert seen_accept >= 20


def test_initial_drafts_are_uniform_integers(oracle_mod):
    cfg = tiny_cfg(n_draft=4, seed=77)
    orc, cond = _mk(oracle_mod, cfg)
    dc = oracle_mod.decode_config(cfg)
    s = orc.new_seq(cond[0], 5)
    s.begin([0], dc)
    w = s.window()
    assert w[0] == 0 and s.len == 0 and s.step_idx == 0
    for i in range(1, 5):
        assert w[i] == (oracle_mod.rand24(77, 5, 0, i, 1) * cfg["vocab"]) >> 24
    # uniform on [0, V): mean and range over many sequence ids
    xs = np.array([(oracle_mod.rand24(1, q, 0, 1, 1) * 50) >> 24 for q in range(4000)])
    assert xs.min() == 0 and xs.max() == 49 and abs(xs.mean() - 24.5) < 1.0


def test_rollback_cache_equals_never_speculated_cache(oracle_mod):
    """After a run with mixed accept lengths the logical cache (positions < len) is bit-equal to the
    cache of a run that fed the final sequence one token at a time; page accounting is exact."""
    cfg = tiny_cfg(n_draft=3)
    K, V, P = 3, cfg["vocab"], cfg["page_size"]
    orc, cond = _mk(oracle_mod, cfg, n_pages=40)
    dc = oracle_mod.decode_config(cfg)
    ref = _plain(orc, cond[0], dc, 60)
    full = np.concatenate([[0], ref])
    free0 = orc.free_pages()
    s = orc.new_seq(cond[0], 0)
    s.begin([0], dc)
    rng = np.random.default_rng(3)
    lens = []
    while s.len < 40:
        n = s.len
        good = int(rng.integers(0, K + 1))           # accept exactly `good` drafts this step
        dr = full[n + 1:n + 1 + K].copy()
        dr[good:] = (dr[good:] + 1 + rng.integers(0, V - 1, K - good)) % V
        if good < K:
            dr[good] = (full[n + 1 + good] + 1) % V
        s.set_drafts(dr)
        _, a, _, _ = s.step(dc)
        assert a == good
        lens.append(a)
        assert s.blocks == -(-(s.len + K + 1) // P)
        assert orc.free_pages() == free0 - s.blocks
    assert len(set(lens)) == K + 1
    t = orc.new_seq(cond[0], 0)
    for p in range(s.len):
        t.forward_row(int(full[p]), p)
    for layer in range(cfg["n_layers"]):
        for kv in (0, 1):
            for p in range(s.len):
                assert np.array_equal(s.kv(layer, kv, p), t.kv(layer, kv, p))
    n_s, n_t = s.blocks, t.blocks
    s.close(); t.close()
    assert orc.free_pages() == free0 and n_s >= n_t


def test_interleaved_sequences_equal_separate_runs(oracle_mod):
    """Sequences sharing the page pool and stepped in turn give what each gives alone."""
    cfg = tiny_cfg(verify_mode=1, k_accept=2, sample_mode=1, k_sample=4, temperature=0.9, seed=21)
    orc, cond = _mk(oracle_mod, cfg, n_pages=64, batch=3)
    dc = oracle_mod.decode_config(cfg)
    alone = []
    for b in range(3):
        s = orc.new_seq(cond[b], b)
        s.begin([0], dc)
        alone.append(s.generate(dc, 24)[0])
        s.close()
    seqs = [orc.new_seq(cond[b], b) for b in range(3)]
    outs = [[] for _ in seqs]
    for s in seqs:
        s.begin([0], dc)
    for _ in range(24):
        for b, s in enumerate(seqs):
            outs[b].extend(s.step(dc)[0].tolist())
    for b in range(3):
        assert outs[b][:24] == alone[b].tolist()
    assert not np.array_equal(alone[0], alone[1])


def test_prompt_and_eos(oracle_mod):
    cfg = tiny_cfg()
    orc, cond = _mk(oracle_mod, cfg)
    dc = oracle_mod.decode_config(cfg)
    prompt = [0, 5, 6, 7]
    ref = _plain(orc, cond[0], dc, 30, prompt)
    s = orc.new_seq(cond[0], 0)
    s.begin(prompt, dc)
    assert s.len == 3 and s.window()[0] == 7
    assert np.array_equal(s.generate(dc, 30)[0], ref)
    eos = int(ref[10])
    first = int(np.argmax(ref == eos))
    cfg_e = tiny_cfg(eos_id=eos)
    orc_e = oracle_mod.Oracle(cfg_e, inputs.make_weights(cfg_e, random_gains=True), n_pages=64)
    s = orc_e.new_seq(cond[0], 0)
    s.begin(prompt, dc)
    toks, _, _ = s.generate(dc, 30)
    assert toks.tolist() == ref[:first + 1].tolist()


def test_capacity_is_an_error_not_a_crash(oracle_mod):
    cfg = tiny_cfg()
    orc, cond = _mk(oracle_mod, cfg, n_pages=2)      # 8 positions in all
    dc = oracle_mod.decode_config(cfg)
    s = orc.new_seq(cond[0], 0)
    s.begin([0], dc)
    with pytest.raises(RuntimeError):
        for _ in range(20):
            s.step(dc)
