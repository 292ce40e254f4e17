"""Scripted drafts (the benchmark's load generator for Sec. 5.1's speedup formula) on the hand-sized model."""
import numpy as np
import pytest

from conftest import gpu_cfg
from paper_2507_23777_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mean_accept", [0.0, 0.5, 1.25, 3.0])
def test_scripted_drafts_force_the_accept_length(mean_accept):
    """With the backbone's own greedy continuation as the script and strict-greedy verification, step t accepts
    floor((t+1) a) - floor(t a) drafts: SCR = 1 + a up to the first step and the truncated last one, and the tokens
    are exactly the plain greedy ones (Sec. 4.2: a draft is accepted only where the backbone agrees)."""
    import torch
    assert torch.cuda.is_available(), "this test needs a B200"
    from paper_2507_23777_b200 import binding, build
    build.build()
    K, T = 3, 80
    cfg = gpu_cfg(dtype=1, n_draft=K, sigma=0.05, max_seq_len=128)
    cfg0 = dict(cfg, n_draft=0)
    w = inputs.make_weights(cfg, random_gains=True)
    w0 = np.ascontiguousarray(w[:inputs.n_weight_elements(cfg0)])
    cond = inputs.make_cond(cfg, 1)
    dc = binding.decode_config(cfg)
    ctx0 = binding.Context(cfg0, w0)
    ctx0.prefill(cond, [0], dc)
    ref, _, st0 = ctx0.generate(T)
    ctx0.xsm_destroy()
    assert st0.steps == T
    script = np.concatenate([[0], ref[0], np.zeros(K + 2, dtype=np.int32)]).astype(np.int32)[None, :]
    ctx = binding.Context(cfg, w)
    ctx.prefill(cond, [0], dc)
    ctx.xsm_debug_set_script(script, mean_accept)
    toks, lens, st = ctx.generate(T)
    assert lens[0] == T and np.array_equal(toks[0], ref[0])
    # the first step still verifies the random initial drafts; every later step t accepts the scheduled number
    hist = np.array(list(st.accept_hist)[:K + 1])
    sched = [int((t + 1) * round(mean_accept * 1024) // 1024 - t * round(mean_accept * 1024) // 1024) for t in range(1, int(st.steps))]
    want = np.bincount(sched, minlength=K + 1)
    assert np.abs(hist - want).sum() <= 4, (hist, want)       # first step and the truncated last one aside
    assert abs(st.scr - (1.0 + mean_accept)) < 0.25          # 80 tokens: the first step (random drafts) weighs up to 0.2
    # the script is switched off by the next prefill
    ctx.prefill(cond, [0], dc)
    _, _, st2 = ctx.generate(T)
    assert st2.scr < 1.0 + mean_accept or mean_accept == 0.0
    ctx.xsm_destroy()
