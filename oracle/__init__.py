"""ctypes front end of the CPU oracle (``xsm_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
benchmark's CPU-baseline leg; the CUDA product never imports it.  The wrapper
only marshals arguments; all arithmetic is in the C file.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import weakref

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "xsm_oracle.c")


def _cpu_tag() -> str:
    """The library is built with -march=native, so its name carries a hash of
    this host's CPU flags: a copy built on another machine is never loaded."""
    import hashlib
    flags = ""
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    flags = line
                    break
    except OSError:
        pass
    return hashlib.md5(flags.encode()).hexdigest()[:8]


_LIB = os.path.join(_HERE, f"libxsm_oracle_{_cpu_tag()}.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over output rows only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-ftree-vectorize", "-march=native", "-fopenmp", "-fPIC",
                               "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class ModelConfig(C.Structure):
    _fields_ = [(n, C.c_int) for n in (
        "n_layers", "d_model", "n_heads", "d_head", "d_ff", "vocab", "n_cond", "d_cond",
        "n_draft", "head_hidden", "wdtype", "page_size", "n_pages")] + [
        ("rope_theta", C.c_float), ("rms_eps", C.c_float), ("bos_id", C.c_int), ("eos_id", C.c_int),
        ("head_kind", C.c_int)]


class DecodeConfig(C.Structure):
    _fields_ = [("verify_mode", C.c_int), ("k_accept", C.c_int), ("delta", C.c_float),
                ("sample_mode", C.c_int), ("k_sample", C.c_int), ("temperature", C.c_float),
                ("seed", C.c_uint64)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        vp, ip, fp = C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_float)
        L.orc_weight_elements.restype = C.c_size_t
        L.orc_weight_elements.argtypes = [C.POINTER(ModelConfig)]
        L.orc_create.argtypes = [C.POINTER(ModelConfig), vp, C.POINTER(vp)]
        L.orc_destroy.argtypes = [vp]
        L.orc_free_pages.argtypes = [vp]
        L.orc_philox4x32_10.argtypes = [C.POINTER(C.c_uint32), C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)]
        L.orc_rand24.restype = C.c_uint32
        L.orc_rand24.argtypes = [C.c_uint64, C.c_int, C.c_uint32, C.c_uint32, C.c_uint32]
        L.orc_accept.argtypes = [fp, C.c_int, C.c_int, C.POINTER(DecodeConfig)]
        L.orc_sample.argtypes = [fp, C.c_int, C.POINTER(DecodeConfig), C.c_uint32]
        L.orc_seq_create.argtypes = [vp, fp, C.c_int, C.c_int, C.POINTER(vp)]
        L.orc_seq_destroy.argtypes = [vp]
        for n in ("orc_seq_len", "orc_seq_blocks", "orc_seq_finished"):
            getattr(L, n).argtypes = [vp]
        L.orc_seq_step_idx.restype = C.c_uint32
        L.orc_seq_step_idx.argtypes = [vp]
        L.orc_seq_get_window.argtypes = [vp, ip]
        L.orc_seq_set_window.argtypes = [vp, ip]
        L.orc_seq_set_drafts.argtypes = [vp, ip]
        L.orc_seq_set_len.argtypes = [vp, C.c_int]
        L.orc_seq_set_step_idx.argtypes = [vp, C.c_uint32]
        L.orc_seq_get_kv.argtypes = [vp, C.c_int, C.c_int, C.c_int, fp]
        L.orc_forward_row.argtypes = [vp, C.c_int, C.c_int, fp, fp]
        L.orc_head.argtypes = [vp, C.c_int, fp, fp]
        L.orc_head.restype = None
        L.orc_seq_head.argtypes = [vp, C.c_int, fp, fp]
        L.orc_seq_head.restype = None
        L.orc_sample_tree.argtypes = [fp, C.c_int, C.c_int, C.c_int, C.c_uint32, ip]
        L.orc_sample_tree.restype = None
        L.orc_seq_begin.argtypes = [vp, ip, C.c_int, C.POINTER(DecodeConfig)]
        L.orc_step.argtypes = [vp, C.POINTER(DecodeConfig), ip, C.POINTER(C.c_int), fp, fp, fp]
        L.orc_generate.argtypes = [vp, C.POINTER(DecodeConfig), C.c_int, C.c_int, ip,
                                   C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
        L.orc_generate_plain.argtypes = [vp, ip, C.c_int, C.POINTER(DecodeConfig), C.c_int, ip]
        _lib = L
    return _lib


def set_threads(n: int) -> None:
    """Number of OpenMP threads the oracle's row loops use from now on (results do not depend on it)."""
    lib()
    C.CDLL("libgomp.so.1").omp_set_num_threads(int(n))


def _fp(a):
    return a.ctypes.data_as(C.POINTER(C.c_float)) if a is not None else None


def _ip(a):
    return a.ctypes.data_as(C.POINTER(C.c_int32))


def decode_config(cfg: dict) -> DecodeConfig:
    return DecodeConfig(cfg["verify_mode"], cfg["k_accept"], cfg["delta"], cfg["sample_mode"],
                        cfg["k_sample"], cfg["temperature"], cfg["seed"])


def philox4x32_10(ctr, key):
    c = (C.c_uint32 * 4)(*ctr)
    k = (C.c_uint32 * 2)(*key)
    o = (C.c_uint32 * 4)()
    lib().orc_philox4x32_10(c, k, o)
    return [int(x) for x in o]


def rand24(seed, seq_id, step, slot, purpose):
    return int(lib().orc_rand24(seed, seq_id, step, slot, purpose))


def accept(z: np.ndarray, x: int, dc: DecodeConfig) -> bool:
    z = np.ascontiguousarray(z, dtype=np.float32)
    return bool(lib().orc_accept(_fp(z), z.size, int(x), C.byref(dc)))


def sample_tree(zh: np.ndarray, k_s: int, r24: int) -> np.ndarray:
    """One path of the top-k_s probability tree over the heads' logits zh [D, V] (Appendix)."""
    zh = np.ascontiguousarray(zh, dtype=np.float32)
    out = np.empty(zh.shape[0], dtype=np.int32)
    lib().orc_sample_tree(_fp(zh), zh.shape[0], zh.shape[1], int(k_s), int(r24), _ip(out))
    return out


def sample(z: np.ndarray, dc: DecodeConfig, r24: int) -> int:
    z = np.ascontiguousarray(z, dtype=np.float32)
    return int(lib().orc_sample(_fp(z), z.size, C.byref(dc), r24))


class Oracle:
    """Model + shared page pool."""

    def __init__(self, cfg: dict, weights: np.ndarray, n_pages: int | None = None):
        self.cfg = dict(cfg)
        P = cfg["page_size"]
        if n_pages is None:
            n_pages = cfg.get("batch", 1) * ((cfg["max_seq_len"] + cfg["n_draft"] + 1 + P - 1) // P)
        self.mc = ModelConfig(cfg["n_layers"], cfg["d_model"], cfg["n_heads"], cfg["d_head"], cfg["d_ff"],
                              cfg["vocab"], cfg["n_cond"], cfg["d_cond"], cfg["n_draft"], cfg["head_hidden"],
                              cfg["dtype"], P, n_pages, cfg["rope_theta"], cfg["rms_eps"], cfg["bos_id"],
                              cfg["eos_id"], cfg.get("head_kind", 0))
        want = np.uint16 if cfg["dtype"] == 1 else np.float32
        assert weights.dtype == want and weights.flags.c_contiguous
        assert weights.size == lib().orc_weight_elements(C.byref(self.mc))
        self._w = weights
        self._h = C.c_void_p()
        self._seqs = weakref.WeakSet()
        rc = lib().orc_create(C.byref(self.mc), weights.ctypes.data_as(C.c_void_p), C.byref(self._h))
        if rc:
            raise RuntimeError(f"orc_create failed: {rc}")

    def free_pages(self) -> int:
        return lib().orc_free_pages(self._h)

    def new_seq(self, cond: np.ndarray, seq_id: int = 0, max_positions: int | None = None) -> "Seq":
        s = Seq(self, cond, seq_id, max_positions)
        self._seqs.add(s)
        return s

    def head(self, i: int, g: np.ndarray) -> np.ndarray:
        g = np.ascontiguousarray(g, dtype=np.float32)
        out = np.empty(self.cfg["vocab"], dtype=np.float32)
        lib().orc_head(self._h, i, _fp(g), _fp(out))
        return out

    def close(self):
        # sequences hand their pages back to the context: they go first, whatever order the collector picks
        for s in list(getattr(self, "_seqs", ())):
            s.close()
        if self._h:
            lib().orc_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Seq:
    def __init__(self, orc: Oracle, cond: np.ndarray, seq_id: int, max_positions: int | None):
        self.orc = orc
        cfg = orc.cfg
        self.K, self.V, self.d = cfg["n_draft"], cfg["vocab"], cfg["d_model"]
        self.max_positions = max_positions or (cfg["max_seq_len"] + self.K + 1)
        cond = np.ascontiguousarray(cond, dtype=np.float32)
        assert cond.shape == (cfg["n_cond"], cfg["d_cond"])
        self._h = C.c_void_p()
        lib().orc_seq_create(orc._h, _fp(cond), seq_id, self.max_positions, C.byref(self._h))

    # --- state
    @property
    def len(self):
        return lib().orc_seq_len(self._h)

    @property
    def blocks(self):
        return lib().orc_seq_blocks(self._h)

    @property
    def step_idx(self):
        return int(lib().orc_seq_step_idx(self._h))

    def window(self) -> np.ndarray:
        w = np.empty(self.K + 1, dtype=np.int32)
        lib().orc_seq_get_window(self._h, _ip(w))
        return w

    def set_window(self, w):
        w = np.ascontiguousarray(w, dtype=np.int32)
        assert w.size == self.K + 1
        lib().orc_seq_set_window(self._h, _ip(w))

    def set_drafts(self, dr):
        dr = np.ascontiguousarray(dr, dtype=np.int32)
        assert dr.size == self.K
        if self.K:
            lib().orc_seq_set_drafts(self._h, _ip(dr))

    def set_len(self, n):
        lib().orc_seq_set_len(self._h, int(n))

    def set_step_idx(self, n):
        lib().orc_seq_set_step_idx(self._h, int(n))

    def kv(self, layer: int, kv: int, pos: int) -> np.ndarray:
        out = np.empty(self.d, dtype=np.float32)
        if lib().orc_seq_get_kv(self._h, layer, kv, pos, _fp(out)):
            raise IndexError(pos)
        return out

    # --- compute
    def head(self, i: int, g: np.ndarray) -> np.ndarray:
        """Logits of decoding head i (1-based) on final hidden state g, whichever kind the model has."""
        g = np.ascontiguousarray(g, dtype=np.float32)
        out = np.empty(self.V, dtype=np.float32)
        lib().orc_seq_head(self._h, i, _fp(g), _fp(out))
        return out

    def forward_row(self, token: int, pos: int):
        z = np.empty(self.V, dtype=np.float32)
        g = np.empty(self.d, dtype=np.float32)
        rc = lib().orc_forward_row(self._h, int(token), int(pos), _fp(z), _fp(g))
        if rc:
            raise RuntimeError(f"orc_forward_row failed: {rc}")
        return z, g

    def begin(self, prompt, dc: DecodeConfig):
        p = np.ascontiguousarray(prompt, dtype=np.int32)
        rc = lib().orc_seq_begin(self._h, _ip(p), p.size, C.byref(dc))
        if rc:
            raise RuntimeError(f"orc_seq_begin failed: {rc}")

    def step(self, dc: DecodeConfig, want_logits: bool = False):
        """One iteration of Algorithm 1's loop.  Returns (committed tokens, a,
        logits0[K+1,V], head_logits[K,K+1,V]) (the arrays are None unless asked)."""
        M = self.K + 1
        nt = np.empty(M, dtype=np.int32)
        n = C.c_int()
        z0 = np.empty((M, self.V), dtype=np.float32) if want_logits else None
        zh = np.empty((self.K, M, self.V), dtype=np.float32) if want_logits else None
        rc = lib().orc_step(self._h, C.byref(dc), _ip(nt), C.byref(n), _fp(z0), _fp(zh), None)
        if rc:
            raise RuntimeError(f"orc_step failed: {rc}")
        return nt[:n.value].copy(), n.value - 1, z0, zh

    def generate(self, dc: DecodeConfig, max_new: int):
        toks = np.empty(max_new, dtype=np.int32)
        steps = C.c_uint64()
        hist = (C.c_uint64 * (self.K + 1))()
        n = lib().orc_generate(self._h, C.byref(dc), max_new, self.max_positions, _ip(toks),
                               C.byref(steps), hist)
        if n < 0:
            raise RuntimeError(f"orc_generate failed: {n}")
        return toks[:n].copy(), int(steps.value), [int(x) for x in hist]

    def generate_plain(self, prompt, dc: DecodeConfig, max_new: int):
        p = np.ascontiguousarray(prompt, dtype=np.int32)
        toks = np.empty(max_new, dtype=np.int32)
        n = lib().orc_generate_plain(self._h, _ip(p), p.size, C.byref(dc), max_new, _ip(toks))
        if n < 0:
            raise RuntimeError(f"orc_generate_plain failed: {n}")
        return toks[:n].copy()

    def close(self):
        if self._h:
            lib().orc_seq_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
