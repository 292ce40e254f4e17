"""Lock-step comparison of the CUDA library with the CPU oracle (helpers for the GPU tests).

The oracle is teacher-forced on the GPU's token stream: before every step it is given the GPU's window
and length, so both sides evaluate the same tokens at the same positions; their logits and their
accept / resample decisions are compared step by step.  A decision may differ only where it hangs on
a margin smaller than ``margin`` (a near-tie of logits, a probability at the threshold, a uniform draw
at a CDF edge); such steps are counted and reported.
"""
from __future__ import annotations

import numpy as np

import oracle
from paper_2507_23777_b200 import binding, inputs


def logits_close(gpu, ref, atol, rtol):
    """|gpu - ref| <= atol + rtol |ref|.  Rounding errors of the hidden state show up in every logit in
    proportion to the scale of the row, so the absolute part is never taken below 2e-5 of the largest
    |ref| (only models with logits far above 10 are affected)."""
    scale = float(np.abs(ref).max()) if ref.size else 0.0
    return np.abs(gpu - ref) <= max(atol, 2e-5 * scale) + rtol * np.abs(ref)


def _rank_margin(z, x, k):
    """Distance of logit z[x] from the boundary between rank k-1 and rank k."""
    order = np.lexsort((np.arange(z.size), -z))
    srt = z[order]
    if k >= z.size:
        return np.inf
    rank = int(np.where(order == x)[0][0])
    return abs(z[x] - srt[k]) if rank < k else abs(z[x] - srt[k - 1])


def accept_margin(z, x, dc):
    if dc.verify_mode == 2:
        p = np.exp(z.astype(np.float64) - z.max())
        p /= p.sum()
        return abs(p[x] - dc.delta)
    return _rank_margin(z, x, 1 if dc.verify_mode == 0 else dc.k_accept)


def sample_excused(z, dc, r24, margin):
    """Could a perturbation of the logits by `margin` change the sampled token?"""
    order = np.lexsort((np.arange(z.size), -z))
    if dc.sample_mode == 0:
        return z[order[0]] - z[order[1]] < margin
    k = min(dc.k_sample, z.size)
    top = z[order[:k + 1]].astype(np.float64)
    if np.min(-np.diff(top)) < margin:       # membership or order of the candidates is in doubt
        return True
    w = np.exp((top[:k] - top[0]) / dc.temperature)
    cdf = np.cumsum(w) / w.sum()
    return np.min(np.abs(cdf - r24 / 2.0 ** 24)) < margin


def tree_excused(zh, ks, r24, margin):
    """Probability-tree sampling (sample_mode 2): could a perturbation of the heads' logits zh [K, V] by `margin` change
    the drawn path?  Yes if the candidates of a head nearly tie, if a path's weight lies at the pruning bound, or if
    the uniform draw lies within `margin` of an edge of the cumulative path weights."""
    import itertools
    K, V = zh.shape
    ks = min(ks, V)
    m = []
    for d in range(K):
        order = np.lexsort((np.arange(V), -zh[d]))
        top = zh[d][order[:ks + 1]].astype(np.float64)
        if np.min(-np.diff(top)) < margin:
            return True
        p = np.exp(zh[d].astype(np.float64) - zh[d].max())
        m.append((p / p.sum())[order[:ks]])
    w = []
    for idx in itertools.product(range(ks), repeat=K):
        wg = 1.0
        for d, k in enumerate(idx):
            wg *= m[d][k]
        if abs(wg - 1e-5) < 1e-5 * 10 * margin:
            return True
        w.append(wg if wg >= 1e-5 else 0.0)
    w = np.asarray(w)
    if w.sum() <= 0:
        return False
    edges = np.cumsum(w) / w.sum()
    return bool(np.min(np.abs(edges - r24 / 2.0 ** 24)) < margin)


def assert_logits(gpu, ref, atol, rtol, what):
    """Every logit within atol + rtol |ref| (no exceptions)."""
    ok = logits_close(gpu, ref, atol, rtol)
    assert ok.all(), f"{what} off by {float(np.abs(gpu - ref).max())} ({int((~ok).sum())} of {ok.size} beyond the bound)"


class LockStep:
    def __init__(self, cfg, batch=1, random_gains=False, weights=None, phase_launch=False, workspace_bytes=None):
        self.cfg = dict(cfg)
        self.B, self.K, self.V = batch, cfg["n_draft"], cfg["vocab"]
        self.w = weights if weights is not None else inputs.make_weights(cfg, random_gains=random_gains)
        self.cond = inputs.make_cond(cfg, batch)
        P = cfg["page_size"]
        self.orc = oracle.Oracle(cfg, self.w, n_pages=batch * ((cfg["max_seq_len"] + self.K + 1 + P - 1) // P))
        self.odc = oracle.decode_config(cfg)
        self.gdc = binding.decode_config(cfg)
        self.ctx = binding.Context(cfg, self.w, max_batch=batch, workspace_bytes=workspace_bytes)
        if phase_launch:
            self.ctx.xsm_debug_set_phase_launch(True)
        self.seqs = [self.orc.new_seq(self.cond[b], b) for b in range(batch)]
        self.excused = 0
        self.steps = 0
        self.max_logit_err = 0.0

    def begin(self, prompt=(0,)):
        self.ctx.prefill(self.cond, list(prompt), self.gdc)
        for s in self.seqs:
            s.begin(list(prompt), self.odc)
        st = self.ctx.xsm_debug_get_state()
        for b, s in enumerate(self.seqs):
            assert st["len"][b] == s.len, (st["len"], s.len)
            assert np.array_equal(st["window"][b], s.window()), (st["window"][b], s.window())
        return st

    def step(self, atol, rtol, margin=1e-2, drafts=None, check_logits=True):
        """One step on both sides.  Returns (tokens per sequence, accept lengths) of the GPU."""
        if drafts is not None:
            self.ctx.xsm_debug_set_drafts(drafts)
            for b, s in enumerate(self.seqs):
                s.set_drafts(np.asarray(drafts).reshape(self.B, self.K)[b])
        before = self.ctx.xsm_debug_get_state()
        nt, nn = self.ctx.step()
        after = self.ctx.xsm_debug_get_state()
        z0g, zhg = self.ctx.xsm_debug_get_logits()
        out_toks, out_a = [], []
        for b, s in enumerate(self.seqs):
            if before["finished"][b]:
                assert nn[b] == 0
                out_toks.append([]); out_a.append(-1)
                continue
            assert s.len == before["len"][b] and np.array_equal(s.window(), before["window"][b])
            step_idx = s.step_idx
            win = s.window()
            otoks, oa, z0, zh = s.step(self.odc, want_logits=True)
            if check_logits:
                assert_logits(z0g[b], z0, atol, rtol, f"backbone logits (seq {b}, step {self.steps})")
                if self.K:
                    assert_logits(zhg[:, b], zh, atol, rtol, f"head logits (seq {b}, step {self.steps})")
                    self.max_logit_err = max(self.max_logit_err, float(np.abs(zhg[:, b] - zh).max()))
                self.max_logit_err = max(self.max_logit_err, float(np.abs(z0g[b] - z0).max()))
            ga = int(nn[b]) - 1
            gw = after["window"][b]
            excused = False
            if ga != oa:      # the first differing accept decision must hang on a small margin
                j = min(ga, oa)
                assert accept_margin(z0[j], int(win[j + 1]), self.odc) < margin, \
                    f"accept length {ga} vs oracle {oa} without a small margin (seq {b}, step {self.steps})"
                excused = True
            else:
                onw = s.window()
                tree = self.odc.sample_mode == 2
                for slot in range(self.K + 1):
                    if gw[slot] != onw[slot]:
                        if tree and slot >= 1:      # the drafts are one path of the tree, drawn with slot 1's number
                            r = oracle.rand24(self.cfg["seed"], b, step_idx, 1, 0)
                            assert tree_excused(zh[:, oa], self.odc.k_sample, r, margin), \
                                f"tree path: gpu {gw[1:]} vs oracle {onw[1:]} (seq {b}, step {self.steps})"
                            excused = True
                            break
                        z = z0[oa] if slot == 0 else zh[slot - 1][oa]
                        r = oracle.rand24(self.cfg["seed"], b, step_idx, slot, 0)
                        one = oracle.decode_config(dict(self.cfg, sample_mode=1)) if tree else self.odc
                        assert sample_excused(z, one, r, margin), \
                            f"slot {slot}: gpu {gw[slot]} vs oracle {onw[slot]} (seq {b}, step {self.steps})"
                        excused = True
                assert np.array_equal(nt[b][:ga], win[1:1 + ga])
                assert nt[b][ga] == gw[0] and (nt[b][ga + 1:] == -1).all()
            self.excused += int(excused)
            # teacher forcing: the oracle continues from the GPU's state
            s.set_window(gw)
            s.set_len(int(after["len"][b]))
            assert after["len"][b] == before["len"][b] + ga + 1
            out_toks.append(nt[b][:ga + 1].tolist())
            out_a.append(ga)
        self.steps += 1
        return out_toks, out_a

    def compare_cache(self, atol, rtol, layers=None):
        st = self.ctx.xsm_debug_get_state()
        for b, s in enumerate(self.seqs):
            n = int(st["len"][b])
            for layer in (layers if layers is not None else range(self.cfg["n_layers"])):
                k, v = self.ctx.xsm_debug_get_kv(layer, b, 0, n)
                ok = np.stack([s.kv(layer, 0, p) for p in range(n)])
                ov = np.stack([s.kv(layer, 1, p) for p in range(n)])
                assert logits_close(k, ok, atol, rtol).all(), f"keys differ, layer {layer} seq {b}"
                assert logits_close(v, ov, atol, rtol).all(), f"values differ, layer {layer} seq {b}"

    def close(self):
        self.ctx.xsm_destroy()
