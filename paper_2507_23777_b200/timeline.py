"""Per-stage timeline of one decoding step (xsm_debug_trace_step), as a table.

    python -m paper_2507_23777_b200.timeline --config 2 --warm 64

Runs `warm` decoding steps of the chosen configuration (batch 1 unless --batch), then one traced step, and prints
for every kind of stage: how long the step spends in it (last CTA of the previous stage done -> last CTA of this
stage done), how long a CTA waits for its inputs after finishing the previous stage, and how long it takes from
"inputs are in shared memory" to "outputs are published".  Every mark is a read of the GPU's global timer plus a
store (a few hundred nanoseconds), so a traced step is slower than an untraced one; compare shares, not totals.
"""
from __future__ import annotations

import argparse

import numpy as np

from . import binding, build, inputs

LAYER_STAGES = ["RMSNorm + QKV", "self-attention", "out-projection + residual", "RMSNorm + cross q", "cross-attention",
                "cross out-projection + residual", "RMSNorm + gate/up + SiLU*mul", "down projection + residual"]


def stage_names(cfg):
    tail = ["LM head + head blocks"] + (["head output projections"] if cfg["n_draft"] else []) + ["verify / resample", "commit"]
    return LAYER_STAGES, tail


def table(cfg, t: np.ndarray) -> str:
    t = t.astype(np.int64)
    rows, G = t.shape
    L = cfg["n_layers"]
    layer, tail = stage_names(cfg)
    end_prev = t[0].copy()
    acc: dict[str, list] = {}
    for p in range((rows - 1) // 2):
        a, e = t[1 + 2 * p], t[2 + 2 * p]
        name = layer[p % 8] if p < 8 * L else tail[p - 8 * L]
        has = a > 0
        wait = (a[has] - end_prev[has]) if has.any() else np.zeros(1)
        comp = (e[has] - a[has]) if has.any() else np.zeros(1)
        acc.setdefault(name, []).append((e.max() - end_prev.max(), wait.mean(), comp.mean(), int(has.sum())))
        end_prev = e
    total = t[-1].max() - t[0].min()
    out = [f"traced step: {total / 1e3:.1f} us, {G} CTAs", f"{'stage':34s} {'n':>3s} {'us each':>8s} {'share':>7s} {'wait in':>8s} {'compute':>8s} {'CTAs':>5s}"]
    for k, v in acc.items():
        v = np.array(v, dtype=float)
        out.append(f"{k:34s} {len(v):3d} {v[:, 0].mean() / 1e3:8.2f} {100 * v[:, 0].sum() / total:6.1f}% {v[:, 1].mean() / 1e3:8.2f} {v[:, 2].mean() / 1e3:8.2f} {v[:, 3].mean():5.0f}")
    return "\n".join(out)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--warm", type=int, default=64)
    ap.add_argument("--batch", type=int, default=1)
    args = ap.parse_args()
    build.build()
    cfg = inputs.config(args.config)
    w = inputs.make_weights(cfg)
    ctx = binding.Context(cfg, w, max_batch=args.batch)
    ctx.prefill(inputs.make_cond(cfg, args.batch), [cfg["bos_id"]], binding.decode_config(cfg))
    for _ in range(args.warm):
        ctx.xsm_spec_step()
    print(f"config {args.config} ({cfg['name']}), batch {args.batch}, context {int(ctx.xsm_debug_get_state()['len'][0])}")
    print(table(cfg, ctx.xsm_debug_trace_step()))
    ctx.xsm_destroy()


if __name__ == "__main__":
    main()
