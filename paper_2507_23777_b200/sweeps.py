"""Measured sweeps around the benchmark's headline number (all through the C ABI; the oracle is not involved).

* scripted_drafts: Sec. 5.1's speedup = SCR x latency(K = 0) / latency(K), traced on this hardware by forcing the
  accept length of every step (xsm_debug_set_script): the backbone's own greedy continuation is the script, a fixed
  schedule leaves the first a_t drafts of step t intact, so SCR = 1 + mean(a_t) whatever the heads are.  A projection:
  it says what a given acceptance would be worth, not what acceptance trained heads reach.
* threshold: the paper's acceptance rule p0(x) > delta (Sec. 4.2; Sec. 5.4 sweeps delta) with heads fitted to the
  synthetic backbone: SCR, step latency and tokens/s per delta.
* heads: the number of decoding heads D (Sec. 5.4: speedup peaks at D = 4 on the paper's hardware), heads fitted per D.
"""
from __future__ import annotations

import numpy as np

from . import binding, inputs, metrics

UNIT = "tokens/s"


def _timed(cfg, weights, cond, T, script=None, mean_accept=0.0, warm=128):
    ctx = binding.Context(cfg, weights, max_batch=1)
    gdc = binding.decode_config(cfg)
    out = None
    for n in (min(T, warm), T):                       # a short warm-up pass, then the timed one
        ctx.prefill(cond[:1], [cfg["bos_id"]], gdc)
        if script is not None:
            ctx.xsm_debug_set_script(script, mean_accept)
        toks, lens, st = ctx.generate(n)
        out = (toks[0], int(lens[0]), st)
    ctx.xsm_destroy()
    toks, n, st = out
    assert n == T
    return toks, {"value": T / st.wall_ms * 1e3, "unit": UNIT, "scr": st.scr, "steps": int(st.steps),
                  "step_latency_us": st.wall_ms * 1e3 / st.steps,
                  "accept_hist": [int(x) for x in list(st.accept_hist)[:cfg["n_draft"] + 1]]}


def scripted_drafts(cfg, weights, cond, T=2048, targets=(1.0, 1.18, 1.33, 1.91, 2.02, 3.0, 5.0)):
    """tokens/s against SCR under forced accept lengths; strict-greedy verification and argmax resampling, so that the
    backbone reproduces the script (its own greedy continuation from the library's K = 0 path)."""
    K = cfg["n_draft"]
    g = dict(cfg, verify_mode=inputs.VERIFY_STRICT_GREEDY, k_accept=1, sample_mode=inputs.SAMPLE_ARGMAX, k_sample=1)
    g0 = dict(g, n_draft=0)
    w0 = np.ascontiguousarray(weights[:inputs.n_weight_elements(g0)])
    ref, k0 = _timed(g0, w0, cond, T)
    script = np.concatenate([[cfg["bos_id"]], ref, np.zeros(K + 2, dtype=np.int32)]).astype(np.int32)[None, :]
    rows = []
    for scr in targets:
        a = min(max(scr - 1.0, 0.0), float(K))
        toks, r = _timed(g, weights, cond, T, script=script, mean_accept=a)
        r.update({"scr_target": 1.0 + a, "reproduces_k0_tokens": bool(np.array_equal(toks, ref)),
                  "speedup_vs_k0": r["value"] / k0["value"],
                  "formula": metrics.speedup(r["scr"], k0["step_latency_us"], r["step_latency_us"])})
        rows.append(r)
    return {"note": "projection (Sec. 5.1): accept lengths forced by a script, strict-greedy verification; not a measurement of "
                    "what trained heads accept", "tokens": T, "k0": k0, "rows": rows}


def threshold(cfg, fitted, cond, k0_value, T=2048, deltas=(0.1, 0.3, 0.5, 0.7, 0.9)):
    """p0(x) > delta acceptance (temperature-1 softmax of the backbone logits), candidates resampled as configured."""
    rows = []
    for d in deltas:
        c = dict(cfg, verify_mode=inputs.VERIFY_THRESHOLD, delta=float(d))
        _, r = _timed(c, fitted, cond, T)
        r.update({"delta": float(d), "speedup_vs_k0": r["value"] / k0_value})
        rows.append(r)
    return {"tokens": T, "rows": rows, "note": "fitted heads; K = 0 reference is the configured sampling rule's"}


def heads(cfg, weights_of, cond, seqs, conds, k0_value, T=2048, counts=(1, 2, 3, 4, 6, 8), iters=150):
    """SCR, step latency and speedup against the number of decoding heads; weights_of(K) gives the configured model
    with K heads (same backbone), whose heads are then fitted on the same corpus."""
    from . import fit_heads
    rows = []
    for K in counts:
        c = dict(cfg, n_draft=K)
        fitted, _ = fit_heads.fit_from_corpus(c, weights_of(K), seqs, conds, iters=iters, eval_every=25)
        _, r = _timed(c, fitted, cond, T)
        r.update({"n_draft": K, "speedup_vs_k0": r["value"] / k0_value})
        rows.append(r)
    return {"tokens": T, "rows": rows}
