"""Benchmark of the speculative decoding hot path on synthetic mesh-model-shaped inputs.

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--config I] [--k0]

One "step" is one whole generation of the workload's token count (prefill + every decoding step of
Algorithm 1) for one batch of synthetic meshes.  The metric is generated mesh tokens per second per
mesh.  `value` is measured with the condition latents already on the device; `e2e` goes through
xsm_generate_host with pinned host buffers (host-to-device copy of the condition and prompt, device-
to-host copy of the tokens, both inside the timed region).  `--impl reference` times the CPU oracle
instead (rank 0 only).  With N > 1 every rank runs an independent replica (meshes are independent;
there is no exchange step), and `value` is the aggregate over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2507_23777_b200 import inputs, metrics  # noqa: E402

METRIC = "generated mesh tokens/s per mesh"
UNIT = "tokens/s"


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows, self.proc, self.index = [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "200"], stdout=subprocess.PIPE, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm = [float(r[0]) for r in self.rows if len(r) >= 6 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 6 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) >= 6 and r[2 + i] == "Active" for r in self.rows)]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def workload(args):
    cfg = inputs.config(args.config)
    if args.k0:
        cfg["n_draft"] = 0
    if args.tokens:
        cfg["gen_tokens"] = args.tokens
    if args.head_kind:
        cfg["head_kind"] = 1
    return cfg


def oracle_sample(cfg, weights, cond, seconds_budget=20.0, min_steps=4):
    """Times the oracle, as it stands, on the first decoding steps of the workload."""
    import oracle
    oracle.build()
    orc = oracle.Oracle(cfg, weights, n_pages=2 * ((256 + cfg["n_draft"] + 1) // cfg["page_size"] + 2))
    dc = oracle.decode_config(cfg)
    s = orc.new_seq(cond[0], 0)
    s.begin([cfg["bos_id"]], dc)
    t0 = time.perf_counter()
    toks = steps = 0
    while (time.perf_counter() - t0 < seconds_budget or steps < min_steps) and steps < 256:
        t, _, _, _ = s.step(dc)
        toks += len(t)
        steps += 1
    dt = time.perf_counter() - t0
    return toks / dt, steps, dt, os.cpu_count()


def spot_check(cfg, weights, cond, n_steps=12):
    """The library against the oracle on one decoding step of the benchmark's own model: after n_steps steps the oracle
    is brought to the same state (the committed tokens run through its forward) and both evaluate the next window."""
    import oracle
    from paper_2507_23777_b200 import binding
    oracle.build()
    ctx = binding.Context(cfg, weights, max_batch=1)
    ctx.prefill(cond[:1], [cfg["bos_id"]], binding.decode_config(cfg))
    toks = [cfg["bos_id"]]
    for _ in range(n_steps):
        nt, nn = ctx.step()
        toks.extend(int(t) for t in nt[0][:nn[0]])
    st = ctx.xsm_debug_get_state()
    n, win = int(st["len"][0]), st["window"][0].copy()
    assert n == len(toks) - 1 and win[0] == toks[-1]
    ctx.step()
    z0g, zhg = ctx.xsm_debug_get_logits()
    ctx.xsm_destroy()
    P = cfg["page_size"]
    orc = oracle.Oracle(cfg, weights, n_pages=(n + 2 * cfg["n_draft"] + 2) // P + 2)
    dc = oracle.decode_config(cfg)
    s = orc.new_seq(cond[0], 0)
    s.begin(toks, dc)
    s.set_window(win)
    _, _, z0, zh = s.step(dc, want_logits=True)
    err = float(np.abs(z0g[0] - z0).max())
    bound = 2e-2 + 1e-2 * np.abs(z0)
    ok = bool((np.abs(z0g[0] - z0) <= bound).all())
    if cfg["n_draft"]:
        err = max(err, float(np.abs(zhg[:, 0] - zh).max()))
        ok = ok and bool((np.abs(zhg[:, 0] - zh) <= 2e-2 + 1e-2 * np.abs(zh)).all())
    orc.close()
    return {"context": n, "max_logit_err": err, "bound": "2e-2 + 1e-2 |ref|", "ok": ok}


def run_reference(args):
    cfg = workload(args)
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = inputs.make_weights(cfg)
    cond = inputs.make_cond(cfg, 1)
    vals, sample = [], ""
    per = args.reference_seconds or max(4.0, min(30.0, 120.0 / max(1, args.steps + args.warmup)))
    for i in range(args.warmup + args.steps):
        v, steps, dt, cores = oracle_sample(cfg, w, cond, seconds_budget=per)
        if i >= args.warmup:
            vals.append((v, dt))
        sample = f"first {steps} decoding steps of one mesh (context < {steps * (cfg['n_draft'] + 1)} tokens)"
    value = float(np.mean([v for v, _ in vals]))
    ms = float(np.mean([dt for _, dt in vals])) * 1e3
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64 accumulate over fp32 state", "data": "synthetic",
        "config": {"workload": f"config {args.config} ({cfg['name']}): oracle on a bounded prefix", "batch": 1,
                   "n_draft": cfg["n_draft"]},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def fitted_heads_arm(args, cfg, w, cond, T):
    """The same mesh decoded twice more: by the library's K = 0 path, and by the K-head path with heads fitted to
    the backbone (fit_heads: first training stage of Sec. 4.3 on sequences the backbone generated for other
    meshes).  The configured heads are drawn independently of the backbone, so they show the cost of a step but
    accept nothing; the paper's speedup is SCR / latency ratio with trained heads."""
    from paper_2507_23777_b200 import binding, fit_heads
    gdc = binding.decode_config(cfg)

    def timed(c, ww):
        ctx = binding.Context(c, ww, max_batch=1)
        ctx.prefill(cond[:1], [c["bos_id"]], gdc)
        ctx.generate(min(T, 256))                           # warm-up
        ctx.prefill(cond[:1], [c["bos_id"]], gdc)
        _, lens, st = ctx.generate(T)
        assert int(lens[0]) == T
        ctx.xsm_destroy()
        return {"value": T / st.wall_ms * 1e3, "unit": UNIT, "scr": st.scr, "step_latency_us": st.wall_ms * 1e3 / st.steps,
                "accept_hist": [int(x) for x in list(st.accept_hist)[:c["n_draft"] + 1]]}

    cfg0 = dict(cfg, n_draft=0)
    k0 = timed(cfg0, np.ascontiguousarray(w[:inputs.n_weight_elements(cfg0)]))
    seqs, conds = fit_heads.corpus(cfg, w, args.fit_meshes, 512)
    fitted, report = fit_heads.fit_from_corpus(cfg, w, seqs, conds)
    report.update({"tokens_per_mesh": 512, "corpus_seed0": 5000})
    report.pop("curve")
    fh = timed(cfg, fitted)
    fh["speedup_vs_k0"] = fh["value"] / k0["value"]
    fh["fit"] = report
    fh["note"] = ("heads = copies of the LM head fine-tuned on the frozen backbone's own sequences of other meshes "
                  "(stage-1 loss, w(d) = 0.8^d, best held-out checkpoint); backbone and K = 0 path unchanged; the "
                  "synthetic backbone's token dynamics are far more repetitive than a trained mesh model's")
    out = {"k0": k0, "fitted_heads": fh}
    from paper_2507_23777_b200 import sweeps
    Ts = min(T, 2048)
    # the paper's own acceptance rule, delta swept (Sec. 5.4), with the fitted heads
    out["threshold_sweep"] = sweeps.threshold(cfg, fitted, cond, k0["value"], T=Ts)
    if args.head_sweep:
        out["head_sweep"] = sweeps.heads(cfg, lambda K: inputs.make_weights(dict(cfg, n_draft=K, seed=args.config)), cond, seqs, conds,
                                         k0["value"], T=Ts)
    return out


def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2507_23777_b200 import binding, build, replicas

    world, rank, local = replicas.env_ranks()
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    build.build()
    cfg = workload(args)
    cfg["seed"] = replicas.replica_seed(cfg["seed"], rank, world)           # every replica has its own meshes
    B, T, K = cfg["batch"], cfg["gen_tokens"], cfg["n_draft"]
    w = inputs.make_weights(dict(cfg, seed=args.config))
    cond = inputs.make_cond(cfg, B)
    ctx = binding.Context(cfg, w, max_batch=B)
    gdc = binding.decode_config(cfg)
    d_cond = ctx.cond_to_device(cond)
    prompt = np.full((B, 1), cfg["bos_id"], dtype=np.int32)
    d_prompt = torch.from_numpy(prompt).cuda()
    d_tokens = torch.empty((B, T), dtype=torch.int32, device="cuda")
    d_lengths = torch.empty(B, dtype=torch.int32, device="cuda")
    h_cond = torch.from_numpy(ctx.cond_to_host(cond).view(np.int16 if cfg["dtype"] == 1 else np.float32)).pin_memory()
    h_prompt = torch.from_numpy(prompt).pin_memory()
    h_tokens = torch.empty((B, T), dtype=torch.int32).pin_memory()
    h_lengths = torch.empty(B, dtype=torch.int32).pin_memory()

    def one_pass():
        ctx.xsm_prefill(d_cond, d_prompt, 1, gdc)
        return ctx.xsm_generate(T, d_tokens, d_lengths)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        one_pass()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    barrier()
    l0 = ctx.xsm_kernel_launches()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    stats, kernel_ms = [], 0.0
    for _ in range(args.steps):
        st = one_pass()
        stats.append((st.steps, st.tokens, list(st.accept_hist)))
        kernel_ms += st.wall_ms
    ev1.record()
    barrier()
    launches = ctx.xsm_kernel_launches() - l0
    ms = ev0.elapsed_time(ev1)
    # end to end through host buffers
    ctx.xsm_generate_host(h_cond.numpy(), h_prompt.numpy(), gdc, T, h_tokens.numpy(), h_lengths.numpy())
    barrier()
    e0 = time.perf_counter()
    ev0.record()
    n_e2e = max(1, min(args.steps, 2))
    for _ in range(n_e2e):
        ctx.xsm_generate_host(h_cond.numpy(), h_prompt.numpy(), gdc, T, h_tokens.numpy(), h_lengths.numpy())
    ev1.record()
    barrier()
    ms_e2e = max(ev0.elapsed_time(ev1), (time.perf_counter() - e0) * 1e3)
    clocks = sampler.stop() if rank == 0 else None
    assert int(h_lengths.numpy().min()) == T
    tokens_total = sum(s[1] for s in stats)
    steps_total = sum(s[0] for s in stats)
    job = replicas.reduce_totals(tokens_total, B, ms, ms_e2e, device="cuda")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    ms, ms_e2e = job.ms, job.ms_e2e
    scr = tokens_total / steps_total
    value = job.tokens_per_s_per_mesh()
    e2e = world * n_e2e * T / (ms_e2e / 1e3)
    peaks, which = measured_peaks()
    # roofline of the persistent step kernel: algorithmic bytes of all its steps / time inside xsm_generate
    alg = metrics.algorithmic_bytes(cfg, B)
    mean_n = (T / 2.0)
    bytes_per_step = alg["fixed"] + alg["per_position"] * mean_n
    steps_per_pass = steps_total / args.steps / 1.0
    n_step_launches = sum(-(-int(s[0] // B) // 64) for s in stats) or 1
    achieved = bytes_per_step * (steps_total / B) / (kernel_ms / 1e3) / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 weights, fp16 cache, f32 arithmetic" if cfg["dtype"] == 1 else "f32", "data": "synthetic",
        "config": {"workload": f"config {args.config} ({cfg['name']}): batch {B}, K={K} {'cross-attention ' if cfg.get('head_kind') else ''}heads, {T} tokens per mesh, "
                               f"verify_mode {cfg['verify_mode']}, k={cfg['k_accept']}, T={cfg['temperature']}",
                   "weights": "iid N(0, sigma) as configured (heads untrained)", "l2": "inputs larger than L2 "
                   f"({alg['fixed'] / 1e6:.0f} MB of weights streamed per decoding step)", "parallelism": "replicas"},
        "scr": scr, "decode_steps_per_pass": steps_per_pass, "step_latency_us": kernel_ms * 1e3 / (steps_total / B),
        "accept_hist": [int(sum(s[2][a] for s in stats)) for a in range(K + 1)],
        "e2e": {"value": e2e, "unit": UNIT, "h2d_bytes_per_step": int(h_cond.numel() * h_cond.element_size() + h_prompt.numel() * 4),
                "d2h_bytes_per_step": int(h_tokens.numel() * 4 + h_lengths.numel() * 4)},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": achieved / peaks["hbm_gbs"],
                     "traffic": metrics.measured_traffic(args.config if not args.k0 else -1, bytes_per_step * steps_total / B / n_step_launches,
                                                                 cfg.get("head_kind", 0)),
                     "peak_source": f"{which} copy bandwidth (MEASURED_PEAKS.json)" if which == "measured" else "fallback",
                     "kernel": "xsm::step_kernel (persistent, 148 CTAs; one launch = up to 64 decoding steps)",
                     "bytes_per_launch": bytes_per_step * steps_total / B / n_step_launches,
                     "avg_launch_ms": kernel_ms / n_step_launches},
        "clocks": clocks,
    }
    if world == 1 and K >= 1 and not args.k0 and not args.no_fitted_heads:
        line.update(fitted_heads_arm(args, cfg, w, cond, T))
    if world == 1 and K >= 1 and not args.k0 and not args.no_scripted and B == 1:
        from paper_2507_23777_b200 import sweeps
        line["scripted_drafts"] = sweeps.scripted_drafts(cfg, w, cond, T=min(T, 2048))
    if not args.no_cpu_baseline and world == 1:
        import oracle
        line["oracle_spot_check"] = spot_check(cfg, w, cond)
        assert line["oracle_spot_check"]["ok"], line["oracle_spot_check"]
        v, steps, dt, cores = oracle_sample(cfg, w, cond, seconds_budget=15.0)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"first {steps} decoding steps of one mesh ({dt:.1f} s)"}
        oracle.set_threads(1)
        v1, steps1, dt1, _ = oracle_sample(cfg, w, cond, seconds_budget=8.0, min_steps=2)
        oracle.set_threads(cores)
        line["cpu_baseline"]["one_thread"] = {"value": v1, "unit": UNIT, "cores": 1,
                                              "sample": f"first {steps1} decoding steps of one mesh ({dt1:.1f} s)"}
    print(json.dumps(line))
    ctx.xsm_destroy()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="xsm", choices=["xsm", "reference"])
    ap.add_argument("--config", type=int, default=2, help="workload: index into the five configurations")
    ap.add_argument("--k0", action="store_true", help="non-speculative path of the same library (n_draft = 0)")
    ap.add_argument("--tokens", type=int, default=0, help="override tokens per mesh")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-fitted-heads", action="store_true", help="skip the K = 0 and fitted-heads runs of the same mesh")
    ap.add_argument("--fit-meshes", type=int, default=64, help="meshes of 512 tokens the heads are fitted on")
    ap.add_argument("--no-scripted", action="store_true", help="skip the scripted-draft sweep (tokens/s against forced SCR)")
    ap.add_argument("--head-kind", type=int, default=0, choices=[0, 1],
                    help="1: cross-attention decoding heads (Eq. 3) in place of the configured MLP heads")
    ap.add_argument("--head-sweep", action="store_true", help="also sweep the number of decoding heads (heads fitted per count)")
    ap.add_argument("--reference-seconds", type=float, default=0.0,
                    help="--impl reference: CPU seconds per step (default: 120 s spread over the steps, 4 to 30 s each)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
