"""Head fitting end to end on the GPU: corpus from the library's K = 0 path, fit, decode with the fitted heads."""
import numpy as np
import pytest

from paper_2507_23777_b200 import inputs

pytestmark = pytest.mark.gpu


def test_fitted_heads_are_accepted_far_more_often_than_the_configured_ones():
    import torch
    assert torch.cuda.is_available(), "this test needs a B200"
    from paper_2507_23777_b200 import binding, build, fit_heads
    build.build()
    cfg = inputs.config(2, n_layers=4, max_seq_len=1024 + 64)
    w = inputs.make_weights(cfg)
    fitted, rep = fit_heads.fit(cfg, w, n_meshes=12, n_tokens=256, iters=50, eval_every=25)
    first_head = inputs.weight_offsets(cfg)["h1.W1"][0]
    assert np.array_equal(fitted[:first_head], w[:first_head]) and not np.array_equal(fitted[first_head:], w[first_head:])
    assert rep["held_out_loss_kept"] <= rep["held_out_loss_start"]
    scr = {}
    for name, ww in (("configured", w), ("fitted", fitted)):
        ctx = binding.Context(cfg, ww, max_batch=1)
        ctx.prefill(inputs.make_cond(cfg, 1), [cfg["bos_id"]], binding.decode_config(cfg))
        toks, lens, st = ctx.generate(1024)
        assert int(lens[0]) == 1024 and sum(st.accept_hist) == st.steps
        scr[name] = st.scr
        ctx.xsm_destroy()
    assert scr["configured"] < 1.1           # independent heads: about k / V of the drafts pass
    assert scr["fitted"] > 1.5, scr
