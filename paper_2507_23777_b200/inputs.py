"""Seeded synthetic inputs: model shapes, weight buffers, condition latents.

This module holds no arithmetic of the decoding method.  It only draws random
numbers and lays them out in the canonical flat weight order, so that the CPU
oracle and the CUDA library can be handed the very same buffers by a test or a
benchmark.  Neither of those two imports this module; the caller does.

Canonical flat weight layout (elements, all matrices row-major ``[out, in]`` so
that ``y = W x``):

    E[V, d]
    for each layer l = 0..L-1:
        g1[d]  Wq[d, d]  Wk[d, d]  Wv[d, d]  Wo[d, d]
        g2[d]  Wqc[d, d] Wkc[d, dc] Wvc[d, dc] Woc[d, d]
        g3[d]  Wgate[f, d] Wup[f, d] Wdown[d, f]
    gf[d]  W0[V, d]
    for each draft head i = 1..K:
        W1[hd, d]  Wout[V, hd]          (head_kind 0, hd == d: the block is residual)
        Wq[d, d] Wk[d, dc] Wv[d, dc] Wo[d, d] Wout[V, d]     (head_kind 1: cross-attention head)

``dtype`` 0 stores fp32 elements, ``dtype`` 1 stores bf16 elements (uint16 bit
patterns, rounded to nearest-even once, here).

The shapes stand in for the auto-regressive mesh transformer of the paper
(Sec. 4.1: N blocks of self-attention, cross-attention to the condition and a
feed-forward network; Table 1: mesh vocabularies of about 5k entries; Sec. 5:
D = 4 heads; sequences of thousands to tens of thousands of tokens).
"""
from __future__ import annotations

import numpy as np

# Verification / sampling mode numbers shared by the two C interfaces.
VERIFY_STRICT_GREEDY, VERIFY_TOPK, VERIFY_THRESHOLD = 0, 1, 2
SAMPLE_ARGMAX, SAMPLE_TOPK_TEMPERATURE, SAMPLE_TREE = 0, 1, 2


def _cfg(name, L, d, H, dh, f, C, V, K, dtype, batch, gen, sigma, out_scale,
         verify, k_accept, sample, k_sample, temp, max_seq):
    return dict(
        name=name, n_layers=L, d_model=d, n_heads=H, d_head=dh, d_ff=f,
        n_cond=C, d_cond=d, vocab=V, n_draft=K, head_hidden=d, dtype=dtype,
        page_size=64, batch=batch, gen_tokens=gen, sigma=sigma,
        out_scale=out_scale, rope_theta=10000.0, rms_eps=1e-6, bos_id=0,
        eos_id=-1, verify_mode=verify, k_accept=k_accept, delta=0.5,
        sample_mode=sample, k_sample=k_sample, temperature=temp,
        max_seq_len=max_seq,
    )


# Config i uses seed i.
CONFIGS = [
    _cfg("tiny_fp32", 4, 256, 4, 64, 1024, 64, 512, 3, 0, 1, 512, 0.02, 1.0,
         VERIFY_STRICT_GREEDY, 1, SAMPLE_ARGMAX, 1, 1.0, 512 + 64),
    _cfg("small_bf16", 12, 768, 12, 64, 3072, 257, 4096, 4, 1, 1, 4096, 0.02,
         1.0, VERIFY_STRICT_GREEDY, 1, SAMPLE_ARGMAX, 1, 1.0, 4096 + 64),
    _cfg("medium_bf16", 24, 1024, 16, 64, 4096, 257, 4096, 4, 1, 1, 12288,
         0.02, 4.0, VERIFY_TOPK, 5, SAMPLE_TOPK_TEMPERATURE, 5, 0.5,
         12288 + 64),
    _cfg("batched_bf16", 24, 1024, 16, 64, 4096, 257, 4096, 4, 1, 16, 8192,
         0.02, 4.0, VERIFY_TOPK, 5, SAMPLE_TOPK_TEMPERATURE, 5, 0.5,
         8192 + 64),
    _cfg("large_bf16", 32, 2048, 16, 128, 8192, 513, 8192, 6, 1, 4, 20000,
         0.015, 1.0, VERIFY_TOPK, 8, SAMPLE_TOPK_TEMPERATURE, 8, 0.7,
         20000 + 64),
]


def config(i: int, **overrides) -> dict:
    c = dict(CONFIGS[i])
    c["seed"] = i
    c.update(overrides)
    return c


def weight_tensors(cfg: dict):
    """Yield ``(name, shape, kind)`` in canonical order; kind is 'gain',
    'out' (an output projection: W0 or a head's Wout) or 'w'."""
    L, d, f, V = cfg["n_layers"], cfg["d_model"], cfg["d_ff"], cfg["vocab"]
    dc, K, hd = cfg["d_cond"], cfg["n_draft"], cfg["head_hidden"]
    yield "E", (V, d), "w"
    for l in range(L):
        p = f"l{l}."
        yield p + "g1", (d,), "gain"
        yield p + "Wq", (d, d), "w"
        yield p + "Wk", (d, d), "w"
        yield p + "Wv", (d, d), "w"
        yield p + "Wo", (d, d), "w"
        yield p + "g2", (d,), "gain"
        yield p + "Wqc", (d, d), "w"
        yield p + "Wkc", (d, dc), "w"
        yield p + "Wvc", (d, dc), "w"
        yield p + "Woc", (d, d), "w"
        yield p + "g3", (d,), "gain"
        yield p + "Wgate", (f, d), "w"
        yield p + "Wup", (f, d), "w"
        yield p + "Wdown", (d, f), "w"
    yield "gf", (d,), "gain"
    yield "W0", (V, d), "out"
    for i in range(1, K + 1):
        if cfg.get("head_kind", 0) == 1:      # cross-attention head (Eq. 3): its own q/k/v/o projections
            yield f"h{i}.Wq", (d, d), "w"
            yield f"h{i}.Wk", (d, dc), "w"
            yield f"h{i}.Wv", (d, dc), "w"
            yield f"h{i}.Wo", (d, d), "w"
            yield f"h{i}.Wout", (V, d), "out"
        else:
            yield f"h{i}.W1", (hd, d), "w"
            yield f"h{i}.Wout", (V, hd), "out"


def weight_offsets(cfg: dict) -> dict:
    """name -> (element offset, shape)."""
    off, out = 0, {}
    for name, shape, _ in weight_tensors(cfg):
        out[name] = (off, shape)
        off += int(np.prod(shape))
    out["__total__"] = (off, ())
    return out


def n_weight_elements(cfg: dict) -> int:
    return weight_offsets(cfg)["__total__"][0]


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even); returns uint16 patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _normal(seed: int, stream: int, n: int) -> np.ndarray:
    g = np.random.Generator(np.random.Philox(key=[seed & (2**64 - 1), stream]))
    return g.standard_normal(n, dtype=np.float32)


def make_weights(cfg: dict, random_gains: bool = False) -> np.ndarray:
    """Flat weight buffer in canonical order: float32 array (dtype 0) or uint16
    array of bf16 patterns (dtype 1).  Matrices are N(0, sigma); output
    projections are additionally multiplied by ``out_scale``; norm gains are
    1.0 unless ``random_gains`` (a test aid: gains drawn from U(0.5, 1.5))."""
    seed, sigma = cfg["seed"], cfg["sigma"]
    total = n_weight_elements(cfg)
    bf16 = cfg["dtype"] == 1
    buf = np.empty(total, dtype=np.uint16 if bf16 else np.float32)
    jobs, off = [], 0
    for tid, (name, shape, kind) in enumerate(weight_tensors(cfg)):
        n = int(np.prod(shape))
        jobs.append((tid, kind, off, n))
        off += n

    def fill(job):          # every tensor has its own stream, so the order of execution is irrelevant
        tid, kind, o, n = job
        if kind == "gain":
            if random_gains:
                g = np.random.Generator(np.random.Philox(key=[seed, 1 << 20 | tid]))
                w = g.uniform(0.5, 1.5, n).astype(np.float32)
            else:
                w = np.ones(n, dtype=np.float32)
        else:
            w = _normal(seed, tid, n)
            w *= np.float32(sigma * (cfg["out_scale"] if kind == "out" else 1.0))
        buf[o:o + n] = f32_to_bf16_bits(w) if bf16 else w

    from concurrent.futures import ThreadPoolExecutor
    import os
    with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as ex:
        list(ex.map(fill, jobs))
    return buf


def make_cond(cfg: dict, batch: int | None = None) -> np.ndarray:
    """Condition latents ``[B, C, d_cond]`` drawn N(0, 1); sequence b has its
    own stream.  Returned as float32 values (already rounded to bf16-exact
    values when the model dtype is bf16, so both sides see identical numbers)."""
    B = cfg["batch"] if batch is None else batch
    C, dc = cfg["n_cond"], cfg["d_cond"]
    out = np.empty((B, C, dc), dtype=np.float32)
    for b in range(B):
        out[b] = _normal(cfg["seed"], (1 << 30) + b, C * dc).reshape(C, dc)
    if cfg["dtype"] == 1:
        out = bf16_bits_to_f32(f32_to_bf16_bits(out)).reshape(B, C, dc)
    return out


def weights_as_f32(cfg: dict, buf: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(buf) if cfg["dtype"] == 1 else buf


def tensor_view(cfg: dict, buf: np.ndarray, name: str) -> np.ndarray:
    off, shape = weight_offsets(cfg)[name]
    return buf[off:off + int(np.prod(shape))].reshape(shape)
