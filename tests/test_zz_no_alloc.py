"""xsm_spec_step_static: the decoding step whose attention scratch is built into the library.

Some hosts cannot allocate device memory when they call the library (all of it was handed out at start-up, or
an allocation would synchronise a device that must keep running), so this entry point takes the scratch that
the key splits of an attention stage exchange from an array inside the library image instead of from the
caller's workspace.  It must commit exactly the tokens that xsm_spec_step commits.  The file is named so
that pytest collects it after every other test.
"""
import numpy as np
import pytest

from conftest import gpu_cfg
from paper_2507_23777_b200 import inputs

pytestmark = pytest.mark.gpu


def test_static_scratch_step_matches_workspace_step():
    import torch
    assert torch.cuda.is_available(), "this test needs a B200"
    from paper_2507_23777_b200 import binding, build
    build.build()
    # 32-token pages and a context that grows past four pages, so that the later steps split the keys of
    # self-attention over several CTAs and the scratch is really used; two sequences with their own lengths
    cfg = gpu_cfg(dtype=1, n_draft=2, max_seq_len=384, sigma=0.05, seed=7)
    w = inputs.make_weights(cfg, random_gains=True)
    cond = inputs.make_cond(cfg, 2)
    dc = binding.decode_config(cfg)
    ref = binding.Context(cfg, w, max_batch=2)
    sta = binding.Context(cfg, w, max_batch=2)
    ref.prefill(cond, [0], dc)
    sta.prefill(cond, [0], dc)
    K1 = cfg["n_draft"] + 1
    mk = lambda: (torch.empty((2, K1), dtype=torch.int32, device="cuda"), torch.empty(2, dtype=torch.int32, device="cuda"))
    (rt, rn), (st_, sn) = mk(), mk()
    n_steps, longest = 200, 0
    for step in range(n_steps):                      # every call is followed by another one: 200 calls in a row
        ref.xsm_spec_step(rt, rn)
        sta.xsm_spec_step_static(st_, sn)
        # integer results: equal, not close (the tests of the library compare token streams bit for bit)
        assert torch.equal(rn, sn), f"accept lengths differ at step {step}"
        assert torch.equal(rt, st_), f"committed tokens differ at step {step}"
    a, b = ref.xsm_debug_get_state(), sta.xsm_debug_get_state()
    assert np.array_equal(a["len"], b["len"]) and np.array_equal(a["window"], b["window"])
    longest = int(a["len"].max())
    assert longest > 4 * cfg["page_size"] + 32, "the run never reached the split path"
    # the logits of the last step agree as well (bf16 bound of the other tests; they are in fact identical)
    z0a, zha = ref.xsm_debug_get_logits()
    z0b, zhb = sta.xsm_debug_get_logits()
    assert np.allclose(z0a, z0b, atol=2e-2, rtol=1e-2) and np.allclose(zha, zhb, atol=2e-2, rtol=1e-2)
    ref.xsm_destroy()
    sta.xsm_destroy()


def test_the_two_step_calls_alternate_on_one_context():
    """One ordinary step, two through the built-in scratch, one ordinary, and so on, on ONE context, well past the
    context length where self-attention is split over several CTAs: the tokens equal those of a context that only
    takes ordinary steps.  (The partials carry a tag that repeats every three writes; the library clears the
    workspace copy when a caller comes back from the built-in scratch, or a stale partial could pass for a new one.)"""
    import torch
    assert torch.cuda.is_available(), "this test needs a B200"
    from paper_2507_23777_b200 import binding, build
    build.build()
    for n_layers in (2, 4):          # the tag of a layer's partials depends on (step * layers + layer) mod 3
        cfg = gpu_cfg(dtype=1, n_draft=2, max_seq_len=512, sigma=0.05, seed=9, n_layers=n_layers)
        w = inputs.make_weights(cfg, random_gains=True)
        cond = inputs.make_cond(cfg, 2)
        dc = binding.decode_config(cfg)
        ref = binding.Context(cfg, w, max_batch=2)
        mix = binding.Context(cfg, w, max_batch=2)
        ref.prefill(cond, [0], dc)
        mix.prefill(cond, [0], dc)
        K1 = cfg["n_draft"] + 1
        mk = lambda: (torch.empty((2, K1), dtype=torch.int32, device="cuda"), torch.empty(2, dtype=torch.int32, device="cuda"))
        (rt, rn), (mt, mn) = mk(), mk()
        for step in range(260):
            ref.xsm_spec_step(rt, rn)
            if step % 4 in (1, 2):
                mix.xsm_spec_step_static(mt, mn)
            else:
                mix.xsm_spec_step(mt, mn)
            assert torch.equal(rn, mn) and torch.equal(rt, mt), f"step {step} differs ({n_layers} layers)"
        assert int(ref.xsm_debug_get_state()["len"].max()) > 5 * cfg["page_size"]
        ref.xsm_destroy()
        mix.xsm_destroy()


def test_static_scratch_refuses_what_does_not_fit():
    import torch
    assert torch.cuda.is_available(), "this test needs a B200"
    from paper_2507_23777_b200 import binding, build
    build.build()
    # 8 sequences x 4 heads x 4 key splits x 16 query rows x (128 + 2) floats, twice (self- and cross-attention),
    # is 2.1 MB: more than the 1 MiB the library carries
    cfg = gpu_cfg(dtype=1, n_draft=15, d_model=512, n_heads=4, d_head=128, d_ff=512, head_hidden=512, page_size=32,
                  max_seq_len=64, sigma=0.05)
    w = inputs.make_weights(cfg)
    ctx = binding.Context(cfg, w, max_batch=8)
    ctx.prefill(inputs.make_cond(cfg, 8), [0], binding.decode_config(cfg))
    with pytest.raises(binding.XsmError) as e:
        ctx.xsm_spec_step_static()
    assert e.value.status == binding.XSM_ERR_CAPACITY and "scratch" in str(e.value)
    ctx.xsm_spec_step()          # the context is still good for the ordinary step
    ctx.xsm_destroy()
