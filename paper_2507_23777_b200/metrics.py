"""Host-side bookkeeping: algorithmic HBM bytes of a decoding step and the paper's speedup formula."""
from __future__ import annotations


def algorithmic_bytes(cfg: dict, batch: int) -> dict:
    """Bytes one decoding step must move when every hot weight and every cached key/value is read
    once: `fixed` (hot weights + cross-attention cache of `batch` sequences) and `per_position` (self-
    attention cache per committed position, all sequences).  Not counted: embedding rows, the cross
    Wk/Wv (prefill only), activations."""
    e = 2 if cfg["dtype"] == 1 else 4
    L, d, f, V, C, K = (cfg[k] for k in ("n_layers", "d_model", "d_ff", "vocab", "n_cond", "n_draft"))
    backbone = L * (6 * d * d + 3 * d * f) * e
    lm = d * V * e
    heads = K * (d * d + d * V) * e
    cross = batch * L * 2 * C * d * e
    if cfg.get("head_kind", 0) == 1:      # cross-attention heads: Wq, Wo, Wout and each head's keys and values of the condition
        heads = K * (2 * d * d + d * V) * e
        cross += batch * K * 2 * C * d * e
    return {"fixed": backbone + lm + heads + cross, "per_position": batch * L * 2 * d * e,
            "backbone": backbone, "lm": lm, "heads": heads, "cross_kv": cross}


def speedup(scr: float, latency_base: float, latency_spec: float) -> float:
    """Speedup from the step compression ratio and the two step latencies (Sec. 5.1)."""
    return scr * latency_base / latency_spec


# DRAM traffic of the step kernel measured with ncu (dram__bytes_read.sum + dram__bytes_write.sum of one launch of 64
# decoding steps at contexts 0..63, see profiles/), as a ratio to the algorithmic bytes of the same launch.  Traffic
# grows in proportion to the units processed (weights once per step plus the cache), so a launch of the benchmark is
# its algorithmic bytes times this ratio.  None: no capture of the current kernel for that configuration.
_TRAFFIC_RATIO = {1: (19.537792e9 + 47.306752e6) / 19304546304.0,
                  2: (63.641296e9 + 80.708864e6) / 63021514752.0}


def measured_traffic(config_index: int, algorithmic_bytes_per_launch: float, head_kind: int = 0):
    """None where no capture exists: other configurations, the K = 0 path, cross-attention heads."""
    r = _TRAFFIC_RATIO.get(config_index) if head_kind == 0 else None
    return None if r is None else r * algorithmic_bytes_per_launch
