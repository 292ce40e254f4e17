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
    return {"fixed": backbone + lm + heads + cross, "per_position": batch * L * 2 * d * e,
            "backbone": backbone, "lm": lm, "heads": heads, "cross_kv": cross}


def speedup(scr: float, latency_base: float, latency_spec: float) -> float:
    """Speedup from the step compression ratio and the two step latencies (Sec. 5.1)."""
    return scr * latency_base / latency_spec


# DRAM traffic of one decoding step measured with ncu (dram__bytes_read.sum + dram__bytes_write.sum of the
# step kernel, scaled to one step); None until a capture exists for that configuration.  See profiles/.
_TRAFFIC_PER_LAUNCH = {}


def measured_traffic(config_index: int):
    return _TRAFFIC_PER_LAUNCH.get(config_index)
