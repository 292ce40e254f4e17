"""The offline head-fitting script: its backbone forward against the oracle, and the fit itself on a hand-sized
model (CPU; the corpus comes from the oracle's plain loop here, from the library's K = 0 path in real use)."""
import numpy as np
import pytest

from conftest import tiny_cfg
from paper_2507_23777_b200 import fit_heads, inputs

torch = pytest.importorskip("torch")


def test_backbone_hidden_matches_the_oracle_row_by_row(oracle_mod):
    cfg = tiny_cfg()
    w = inputs.make_weights(cfg, random_gains=True)
    cond = inputs.make_cond(cfg, 1)
    orc = oracle_mod.Oracle(cfg, w)
    s = orc.new_seq(cond[0])
    toks = np.random.default_rng(3).integers(0, cfg["vocab"], 14)
    g_ref = np.stack([s.forward_row(int(t), p)[1] for p, t in enumerate(toks)])
    Wf = torch.from_numpy(inputs.weights_as_f32(cfg, w).astype(np.float32, copy=True))
    g = fit_heads.backbone_hidden(cfg, Wf, toks, cond[0], device="cpu").numpy()
    assert np.abs(g - g_ref).max() < 2e-4 * max(1.0, np.abs(g_ref).max())


def test_fit_changes_only_the_heads_and_never_loses_on_held_out_meshes(oracle_mod):
    cfg = tiny_cfg(n_draft=2)
    w = inputs.make_weights(cfg)
    orc = oracle_mod.Oracle(cfg, w)
    seqs, conds = [], []
    for i in range(8):
        c = dict(cfg, seed=100 + i)
        cond = inputs.make_cond(c, 1)[0]
        toks = orc.new_seq(cond, i).generate_plain([0], oracle_mod.decode_config(c), 40)
        seqs.append(np.concatenate([[0], toks]))
        conds.append(cond)
    fitted, rep = fit_heads.fit_from_corpus(cfg, w, seqs, conds, iters=60, lr=2e-3, eval_every=10, batch=128, device="cpu")
    assert rep["held_out_loss_kept"] <= rep["held_out_loss_start"]
    assert rep["curve"][0]["iteration"] == 0 and rep["held_out_meshes"] == 1
    offs = inputs.weight_offsets(cfg)
    first_head = offs["h1.W1"][0]
    assert np.array_equal(fitted[:first_head], w[:first_head])
    assert fitted.shape == w.shape and fitted.dtype == w.dtype
    if rep["kept_iteration"] == 0:      # the starting point: copies of the LM head behind an empty residual block
        W0 = inputs.tensor_view(cfg, w, "W0")
        for i in (1, 2):
            assert np.array_equal(inputs.tensor_view(cfg, fitted, f"h{i}.Wout"), W0)
            assert not inputs.tensor_view(cfg, fitted, f"h{i}.W1").any()
    else:
        assert not np.array_equal(fitted[first_head:], w[first_head:])
