"""ctypes binding of libxsm.so: the same entry points as include/xsm.h.

Argument marshalling only.  PyTorch is used for device memory and the CUDA
stream; every step of the decoding path runs in the library's kernels.  There
is no fallback: if the library is missing or a call fails, an exception is
raised.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libxsm.so")

XSM_OK, XSM_ERR_INVALID_ARG, XSM_ERR_STATE, XSM_ERR_CAPACITY, XSM_ERR_CUDA, XSM_ERR_TIMEOUT = range(6)
XSM_MAX_DRAFT = 16

EXPORTS = [
    "xsm_weights_bytes", "xsm_workspace_bytes", "xsm_create", "xsm_prefill", "xsm_spec_step", "xsm_generate",
    "xsm_generate_host", "xsm_destroy", "xsm_last_error", "xsm_kernel_launches", "xsm_debug_get_logits",
    "xsm_debug_get_kv", "xsm_debug_set_drafts", "xsm_debug_get_state", "xsm_debug_set_phase_launch",
    "xsm_debug_trace_step", "xsm_spec_step_static", "xsm_debug_set_wait_limits", "xsm_debug_launch_stage",
    "xsm_debug_set_script",
]


class XsmError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"xsm status {status}: {msg}")
        self.status = status


class ModelConfig(C.Structure):
    _fields_ = [(n, C.c_int) for n in (
        "n_layers", "d_model", "n_heads", "d_head", "d_ff", "vocab", "n_cond", "d_cond", "n_draft", "head_hidden",
        "head_kind", "dtype", "page_size", "max_batch", "max_seq_len")] + [
        ("rope_theta", C.c_float), ("rms_eps", C.c_float), ("bos_id", C.c_int), ("eos_id", C.c_int)]


class DecodeConfig(C.Structure):
    _fields_ = [("verify_mode", C.c_int), ("k_accept", C.c_int), ("delta", C.c_float), ("sample_mode", C.c_int),
                ("k_sample", C.c_int), ("temperature", C.c_float), ("seed", C.c_uint64)]


class Stats(C.Structure):
    _fields_ = [("steps", C.c_uint64), ("tokens", C.c_uint64), ("accept_hist", C.c_uint64 * (XSM_MAX_DRAFT + 1)),
                ("wall_ms", C.c_double), ("scr", C.c_double)]


_lib = None


def load(path: str | None = None):
    """Loads the library; raises if it has not been built."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise FileNotFoundError(f"{p} not found: build it with `python -m paper_2507_23777_b200.build`")
    L = C.CDLL(p)
    vp, ip, fp = C.c_void_p, C.c_void_p, C.c_void_p
    L.xsm_weights_bytes.restype = C.c_size_t
    L.xsm_weights_bytes.argtypes = [C.POINTER(ModelConfig)]
    L.xsm_workspace_bytes.restype = C.c_size_t
    L.xsm_workspace_bytes.argtypes = [C.POINTER(ModelConfig)]
    L.xsm_create.argtypes = [C.POINTER(ModelConfig), vp, vp, C.c_size_t, vp, C.POINTER(vp)]
    L.xsm_prefill.argtypes = [vp, C.c_int, vp, ip, C.c_int, C.POINTER(DecodeConfig)]
    L.xsm_spec_step.argtypes = [vp, ip, ip]
    L.xsm_spec_step_static.argtypes = [vp, ip, ip]
    L.xsm_generate.argtypes = [vp, C.c_int, ip, ip, C.POINTER(Stats)]
    L.xsm_generate_host.argtypes = [vp, C.c_int, vp, ip, C.c_int, C.POINTER(DecodeConfig), C.c_int, ip, ip,
                                    C.POINTER(Stats)]
    L.xsm_destroy.argtypes = [vp]
    L.xsm_last_error.restype = C.c_char_p
    L.xsm_last_error.argtypes = [vp]
    L.xsm_kernel_launches.restype = C.c_uint64
    L.xsm_kernel_launches.argtypes = [vp]
    L.xsm_debug_get_logits.argtypes = [vp, fp, fp]
    L.xsm_debug_get_kv.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.c_int, fp, fp]
    L.xsm_debug_set_drafts.argtypes = [vp, ip]
    L.xsm_debug_get_state.argtypes = [vp, ip, ip, ip, ip, ip]
    L.xsm_debug_set_phase_launch.argtypes = [vp, C.c_int]
    L.xsm_debug_set_script.argtypes = [vp, ip, C.c_int, C.c_float]
    L.xsm_debug_set_wait_limits.argtypes = [vp, C.c_uint32, C.c_uint32]
    L.xsm_debug_launch_stage.argtypes = [vp, C.c_int]
    L.xsm_debug_trace_step.argtypes = [vp, vp, C.c_size_t, C.POINTER(C.c_int), C.POINTER(C.c_int)]
    if path is None:
        _lib = L
    return L


def model_config(cfg: dict, max_batch: int | None = None) -> ModelConfig:
    return ModelConfig(cfg["n_layers"], cfg["d_model"], cfg["n_heads"], cfg["d_head"], cfg["d_ff"], cfg["vocab"],
                       cfg["n_cond"], cfg["d_cond"], cfg["n_draft"], cfg["head_hidden"], cfg.get("head_kind", 0),
                       cfg["dtype"], cfg["page_size"], max_batch or cfg.get("batch", 1), cfg["max_seq_len"],
                       cfg["rope_theta"], cfg["rms_eps"], cfg["bos_id"], cfg["eos_id"])


def decode_config(cfg: dict) -> DecodeConfig:
    return DecodeConfig(cfg["verify_mode"], cfg["k_accept"], cfg["delta"], cfg["sample_mode"], cfg["k_sample"],
                        cfg["temperature"], cfg["seed"])


def xsm_weights_bytes(mc: ModelConfig) -> int:
    return load().xsm_weights_bytes(C.byref(mc))


def xsm_workspace_bytes(mc: ModelConfig) -> int:
    return load().xsm_workspace_bytes(C.byref(mc))


def _np_ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


class Context:
    """One xsm_ctx bound to torch-allocated weights and workspace on the current CUDA device."""

    def __init__(self, cfg: dict, weights: np.ndarray, max_batch: int | None = None, workspace_bytes: int | None = None,
                 stream=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("xsm needs a CUDA device; there is no CPU path")
        self.lib = load()
        self.cfg = dict(cfg)
        self.mc = model_config(cfg, max_batch)
        self.K, self.V, self.d = cfg["n_draft"], cfg["vocab"], cfg["d_model"]
        nbytes = xsm_weights_bytes(self.mc)
        if nbytes == 0:
            raise XsmError(XSM_ERR_INVALID_ARG, "invalid model configuration")
        if weights.nbytes != nbytes:
            raise XsmError(XSM_ERR_INVALID_ARG, f"weight buffer has {weights.nbytes} bytes, expected {nbytes}")
        self.torch = torch
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        self.d_weights = torch.from_numpy(weights.view(np.uint8)).cuda()
        ws = workspace_bytes if workspace_bytes is not None else xsm_workspace_bytes(self.mc)
        self.d_ws = torch.empty(ws, dtype=torch.uint8, device="cuda")
        self._h = C.c_void_p()
        st = self.lib.xsm_create(C.byref(self.mc), self.d_weights.data_ptr(), self.d_ws.data_ptr(), ws,
                                 self.stream.cuda_stream, C.byref(self._h))
        if st != XSM_OK:
            raise XsmError(st, self.lib.xsm_last_error(None).decode())
        self.batch = 0

    # ---- helpers
    def _check(self, st):
        if st != XSM_OK:
            raise XsmError(st, self.lib.xsm_last_error(self._h).decode())

    def cond_to_device(self, cond: np.ndarray):
        """float32 condition latents [B, C, dc] -> device tensor of the model dtype."""
        t = self.torch.from_numpy(np.ascontiguousarray(cond, dtype=np.float32)).cuda()
        return t.to(self.torch.bfloat16).contiguous() if self.cfg["dtype"] == 1 else t

    def cond_to_host(self, cond: np.ndarray) -> np.ndarray:
        """float32 condition latents -> host array of the model dtype (bf16 bit patterns as uint16)."""
        c = np.ascontiguousarray(cond, dtype=np.float32)
        if self.cfg["dtype"] == 1:
            u = c.view(np.uint32)
            return ((u + (((u >> 16) & 1) + 0x7FFF)) >> 16).astype(np.uint16)
        return c

    # ---- the C ABI, one method per entry point
    def xsm_prefill(self, d_cond, d_prompt, prompt_len: int, dc: DecodeConfig):
        batch = d_prompt.shape[0]
        self._keep = (d_cond, d_prompt)
        self._check(self.lib.xsm_prefill(self._h, batch, d_cond.data_ptr(), d_prompt.data_ptr(), prompt_len, C.byref(dc)))
        self.batch = batch

    def xsm_spec_step(self, d_new_tokens=None, d_n_new=None):
        self._check(self.lib.xsm_spec_step(self._h, d_new_tokens.data_ptr() if d_new_tokens is not None else None,
                                           d_n_new.data_ptr() if d_n_new is not None else None))

    def xsm_spec_step_static(self, d_new_tokens=None, d_n_new=None):
        self._check(self.lib.xsm_spec_step_static(self._h, d_new_tokens.data_ptr() if d_new_tokens is not None else None,
                                                  d_n_new.data_ptr() if d_n_new is not None else None))

    def xsm_generate(self, max_new: int, d_tokens=None, d_lengths=None) -> Stats:
        st = Stats()
        self._check(self.lib.xsm_generate(self._h, max_new, d_tokens.data_ptr() if d_tokens is not None else None,
                                          d_lengths.data_ptr() if d_lengths is not None else None, C.byref(st)))
        return st

    def xsm_generate_host(self, h_cond: np.ndarray, h_prompt: np.ndarray, dc: DecodeConfig, max_new: int,
                          h_tokens: np.ndarray, h_lengths: np.ndarray) -> Stats:
        st = Stats()
        batch, prompt_len = h_prompt.shape
        self._check(self.lib.xsm_generate_host(self._h, batch, _np_ptr(h_cond), _np_ptr(h_prompt), prompt_len,
                                               C.byref(dc), max_new, _np_ptr(h_tokens), _np_ptr(h_lengths), C.byref(st)))
        self.batch = batch
        return st

    def xsm_kernel_launches(self) -> int:
        return int(self.lib.xsm_kernel_launches(self._h))

    def xsm_debug_get_logits(self):
        B, M = self.batch, self.K + 1
        z0 = np.empty((B, M, self.V), dtype=np.float32)
        zh = np.empty((self.K, B, M, self.V), dtype=np.float32)
        self._check(self.lib.xsm_debug_get_logits(self._h, _np_ptr(z0), _np_ptr(zh) if self.K else None))
        return z0, zh

    def xsm_debug_get_kv(self, layer: int, seq: int, pos0: int, n: int):
        k = np.empty((n, self.d), dtype=np.float32)
        v = np.empty((n, self.d), dtype=np.float32)
        self._check(self.lib.xsm_debug_get_kv(self._h, layer, seq, pos0, n, _np_ptr(k), _np_ptr(v)))
        return k, v

    def xsm_debug_set_drafts(self, drafts):
        a = np.ascontiguousarray(drafts, dtype=np.int32).reshape(self.batch, self.K)
        self._check(self.lib.xsm_debug_set_drafts(self._h, _np_ptr(a)))

    def xsm_debug_get_state(self):
        B = self.batch
        ln = np.empty(B, dtype=np.int32)
        win = np.empty((B, self.K + 1), dtype=np.int32)
        fin = np.empty(B, dtype=np.int32)
        pages = np.empty(B, dtype=np.int32)
        free = np.empty(1, dtype=np.int32)
        self._check(self.lib.xsm_debug_get_state(self._h, _np_ptr(ln), _np_ptr(win), _np_ptr(fin), _np_ptr(pages),
                                                 _np_ptr(free)))
        return dict(len=ln, window=win, finished=fin, pages=pages, free_pages=int(free[0]))

    def xsm_debug_trace_step(self) -> np.ndarray:
        """Timeline of one decoding step: uint64 [1 + 2 * stages, CTAs] nanoseconds (see include/xsm.h)."""
        cap = (1 + 2 * (8 * self.cfg["n_layers"] + 6)) * 256
        buf = np.zeros(cap, dtype=np.uint64)
        rows, ctas = C.c_int(), C.c_int()
        self._check(self.lib.xsm_debug_trace_step(self._h, _np_ptr(buf), cap, C.byref(rows), C.byref(ctas)))
        return buf[:rows.value * ctas.value].reshape(rows.value, ctas.value)

    def xsm_debug_set_phase_launch(self, on: bool):
        self._check(self.lib.xsm_debug_set_phase_launch(self._h, int(on)))

    def xsm_debug_set_script(self, tokens, mean_accept: float):
        """tokens: [batch, n] token of every absolute position (None: off)."""
        if tokens is None:
            self._check(self.lib.xsm_debug_set_script(self._h, None, 0, 0.0))
            return
        a = np.ascontiguousarray(tokens, dtype=np.int32).reshape(self.batch, -1)
        self._check(self.lib.xsm_debug_set_script(self._h, _np_ptr(a), a.shape[1], float(mean_accept)))

    def xsm_debug_set_wait_limits(self, polls: int = 0, barrier_tries: int = 0):
        self._check(self.lib.xsm_debug_set_wait_limits(self._h, polls, barrier_tries))

    def xsm_debug_launch_stage(self, stage: int):
        self._check(self.lib.xsm_debug_launch_stage(self._h, stage))

    def xsm_destroy(self):
        if self._h:
            self.lib.xsm_destroy(self._h)
            self._h = C.c_void_p()

    # ---- conveniences built from the calls above
    def prefill(self, cond: np.ndarray, prompt, dc: DecodeConfig):
        torch = self.torch
        p = np.ascontiguousarray(prompt, dtype=np.int32)
        if p.ndim == 1:
            p = np.tile(p, (cond.shape[0], 1))
        self.xsm_prefill(self.cond_to_device(cond), torch.from_numpy(p).cuda(), p.shape[1], dc)

    def step(self):
        torch = self.torch
        nt = torch.empty((self.batch, self.K + 1), dtype=torch.int32, device="cuda")
        nn = torch.empty(self.batch, dtype=torch.int32, device="cuda")
        self.xsm_spec_step(nt, nn)
        return nt.cpu().numpy(), nn.cpu().numpy()

    def generate(self, max_new: int):
        torch = self.torch
        toks = torch.empty((self.batch, max_new), dtype=torch.int32, device="cuda")
        lens = torch.empty(self.batch, dtype=torch.int32, device="cuda")
        st = self.xsm_generate(max_new, toks, lens)
        return toks.cpu().numpy(), lens.cpu().numpy(), st

    def __del__(self):
        try:
            self.xsm_destroy()
        except Exception:
            pass
