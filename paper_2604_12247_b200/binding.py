"""Thin ctypes binding of the C-ABI CUDA library (``include/specbound.h``).

Argument marshalling only: every step of the decode path runs in the library's kernels.
PyTorch supplies device memory and the stream.  If the shared library is missing the
import of this module's ``lib()`` fails loudly -- there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path
from typing import Optional, Sequence

import numpy as np
import torch

from . import inputs

_LIB_PATH = Path(__file__).resolve().parent / "libspecbound_b200.so"
MAX_W = 8
MAX_LAYERS = 64
OPT_GEMM = 1


class Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab")] + [
        ("rope_base", C.c_float), ("rms_eps", C.c_float), ("dtype", C.c_int32), ("max_seq", C.c_int32),
        ("kv_page", C.c_int32)]


class LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down")]


class Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p),
                ("layers", C.POINTER(LayerWeights)), ("exit_head", C.POINTER(C.c_void_p)),
                ("exit_norm", C.POINTER(C.c_void_p))]


class Stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("rounds", "rows", "accepted_drafts", "emitted", "probes", "layer_steps",
                                         "layer_row_steps")] + [
        ("exit_hist", C.c_int64 * (MAX_LAYERS + 1)), ("width_hist", C.c_int64 * (MAX_W + 1)),
        ("us_prefill", C.c_double), ("us_decode", C.c_double), ("us_decode_dev", C.c_double), ("us_draft", C.c_double),
        ("us_verify", C.c_double), ("us_unified", C.c_double), ("unified_layer_steps", C.c_int64),
        ("unified_kv_positions", C.c_int64), ("us_probe_kernels", C.c_double), ("kernel_launches", C.c_int64),
        ("h2d_bytes", C.c_int64), ("d2h_bytes", C.c_int64), ("probes_timed", C.c_int64), ("rounds_timed", C.c_int64)]


class Round(C.Structure):
    _fields_ = [("w", C.c_int32), ("D", C.c_int32), ("emitted", C.c_int32), ("accepted_drafts", C.c_int32),
                ("exit_layer", C.c_int32 * MAX_W), ("draft", C.c_int32 * MAX_W), ("g", C.c_int32 * MAX_W),
                ("conf", C.c_float * MAX_W)]


class State(C.Structure):
    _fields_ = [("n", C.c_int32), ("pending", C.c_int32), ("rows", C.c_int32), ("depth", C.c_int32 * MAX_W)]


class SBError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib().sb_strerror(status).decode()} ({status})")


EXPORTS = ("sb_workspace_bytes", "sb_create", "sb_destroy", "sb_load_weights", "sb_reset", "sb_get_state",
           "sb_selftest_wait_timeout",
           "sb_read_hidden", "sb_prefill", "sb_draft_push", "sb_draft_advance", "sb_exit_confidence", "sb_verify",
           "sb_generate", "sb_generate_ar", "sb_set_sampling", "sb_sample_uniform", "sb_k_sample", "sb_k_sample_scratch_bytes", "sb_k_scratch_bytes", "sb_k_exit_confidence", "sb_k_exit_confidence_static",
           "sb_k_layer", "sb_k_layer_chain", "sb_k_rope_table", "sb_k_rope_table_bytes",
           "sb_tau_schedule", "sb_model_speedup", "sb_plan_gemm", "sb_set_option", "sb_set_default_option", "sb_strerror")

_lib = None


def lib():
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2604_12247_b200.build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(str(_LIB_PATH))
        vp, i32, f32 = C.c_void_p, C.c_int32, C.c_float
        L.sb_workspace_bytes.restype = C.c_size_t
        L.sb_workspace_bytes.argtypes = [C.POINTER(Config)]
        L.sb_k_scratch_bytes.restype = C.c_size_t
        L.sb_k_scratch_bytes.argtypes = [C.POINTER(Config)]
        L.sb_create.argtypes = [C.POINTER(Config), vp, C.c_size_t, vp, C.POINTER(vp)]
        L.sb_destroy.argtypes = [vp]
        L.sb_destroy.restype = None
        L.sb_load_weights.argtypes = [vp, C.POINTER(Weights)]
        L.sb_reset.argtypes = [vp]
        L.sb_get_state.argtypes = [vp, C.POINTER(State)]
        L.sb_selftest_wait_timeout.argtypes = [vp, i32]
        L.sb_read_hidden.argtypes = [vp, i32, vp]
        L.sb_prefill.argtypes = [vp, vp, i32, C.POINTER(i32)]
        L.sb_draft_push.argtypes = [vp, i32]
        L.sb_draft_advance.argtypes = [vp, i32]
        L.sb_exit_confidence.argtypes = [vp, i32, f32, f32, C.POINTER(f32), C.POINTER(i32), C.POINTER(i32)]
        L.sb_verify.argtypes = [vp, vp, i32, vp, C.POINTER(i32)]
        L.sb_generate.argtypes = [vp, vp, i32, i32, i32, i32, vp, f32, vp, C.POINTER(i32), C.POINTER(Stats), vp, i32,
                                  C.POINTER(i32)]
        L.sb_generate_ar.argtypes = [vp, vp, i32, i32, vp, C.POINTER(i32), C.POINTER(Stats)]
        L.sb_set_sampling.argtypes = [vp, f32, f32, C.c_uint64]
        L.sb_sample_uniform.argtypes = [C.c_uint64, C.c_int64]
        L.sb_sample_uniform.restype = C.c_double
        L.sb_k_sample.argtypes = [vp, i32, i32, f32, f32, C.c_uint64, C.c_int64, vp, vp, C.c_size_t, vp]
        L.sb_k_sample_scratch_bytes.argtypes = [i32, i32]
        L.sb_k_sample_scratch_bytes.restype = C.c_size_t
        L.sb_k_exit_confidence.argtypes = [C.POINTER(Config), vp, i32, vp, vp, f32, vp, vp, vp, vp, C.c_size_t, vp]
        L.sb_k_exit_confidence_static.argtypes = [C.POINTER(Config), vp, i32, vp, vp, f32, vp, vp, vp]
        L.sb_k_layer.argtypes = [C.POINTER(Config), C.POINTER(LayerWeights), vp, i32, vp, vp, vp, i32, vp, C.c_size_t, vp]
        L.sb_k_rope_table_bytes.restype = C.c_size_t
        L.sb_k_rope_table_bytes.argtypes = [C.POINTER(Config)]
        L.sb_k_rope_table.argtypes = [C.POINTER(Config), vp, C.c_size_t, vp]
        L.sb_k_layer_chain.argtypes = [C.POINTER(Config), C.POINTER(LayerWeights), i32, vp, i32, C.POINTER(vp), C.POINTER(vp), vp,
                                       i32, vp, vp, C.c_size_t, vp]
        L.sb_tau_schedule.argtypes = [f32, i32, vp]
        L.sb_model_speedup.restype = C.c_double
        L.sb_model_speedup.argtypes = [i32, C.c_double, i32, i32]
        L.sb_plan_gemm.argtypes = [i32, vp, i32, i32, i32, vp, vp, vp]
        L.sb_set_option.argtypes = [vp, i32, i32]
        L.sb_set_default_option.argtypes = [i32, i32]
        L.sb_strerror.restype = C.c_char_p
        L.sb_strerror.argtypes = [C.c_int]
        _lib = L
    return _lib


def _check(status: int, where: str):
    if status != 0:
        raise SBError(status, where)


def make_config(shape: inputs.Shape, max_seq: int, kv_page: int = 64) -> Config:
    return Config(shape.n_layers, shape.d_model, shape.n_heads, shape.n_kv_heads, shape.head_dim, shape.d_ffn,
                  shape.vocab, shape.rope_base, shape.rms_eps, {"f32": 0, "bf16": 1}[shape.dtype], max_seq, kv_page)


def layer_weights(lw: dict) -> LayerWeights:
    return LayerWeights(*[lw[n].data_ptr() for n, _ in LayerWeights._fields_])


def _np_ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _stream_handle(stream: Optional[torch.cuda.Stream]):
    return C.c_void_p(stream.cuda_stream if stream is not None else torch.cuda.current_stream().cuda_stream)


def tau_schedule(alpha: float, L: int) -> np.ndarray:
    out = np.zeros(L, dtype=np.float32)
    _check(lib().sb_tau_schedule(alpha, L, _np_ptr(out)), "sb_tau_schedule")
    return out


def model_speedup(L: int, a: float, w: int, d_max: int) -> float:
    return lib().sb_model_speedup(L, a, w, d_max)


def plan_gemm(mode: int, n_rows: Sequence[int], k: int, units: int):
    """sb_plan_gemm: (rows per CTA, k splits, work items) of a weight-streaming GEMM on `units` CTAs or clusters."""
    nr = np.ascontiguousarray(n_rows, dtype=np.int32)
    r, s_, n = C.c_int32(), C.c_int32(), C.c_int32()
    _check(lib().sb_plan_gemm(mode, _np_ptr(nr), len(nr), k, units, C.byref(r), C.byref(s_), C.byref(n)), "sb_plan_gemm")
    return r.value, s_.value, n.value


def sample_uniform(seed: int, pos: int) -> float:
    """sb_sample_uniform: the uniform number that decides the token at sequence position pos."""
    return float(lib().sb_sample_uniform(int(seed), int(pos)))


def set_default_gemm(value: int):
    _check(lib().sb_set_default_option(OPT_GEMM, value), "sb_set_default_option")


class Context:
    """One sequence on one GPU.  ``weights``: dict of CUDA tensors from ``inputs.make_weights``."""

    def __init__(self, shape: inputs.Shape, weights: dict, max_seq: int, kv_page: int = 64,
                 stream: Optional[torch.cuda.Stream] = None, gemm: Optional[int] = None):
        self.shape = shape
        self.cfg = make_config(shape, max_seq, kv_page)
        nbytes = lib().sb_workspace_bytes(C.byref(self.cfg))
        if nbytes == 0:
            raise SBError(-1, "sb_workspace_bytes")
        self.workspace = torch.empty(nbytes + 1024, dtype=torch.uint8, device="cuda")
        base = (self.workspace.data_ptr() + 1023) & ~1023
        self._weights = weights
        self.stream = stream
        h = C.c_void_p()
        _check(lib().sb_create(C.byref(self.cfg), C.c_void_p(base), nbytes, _stream_handle(stream), C.byref(h)), "sb_create")
        self.h = h
        self._layers = (LayerWeights * shape.n_layers)(*[layer_weights(lw) for lw in weights["layers"]])
        def table(key):   # optional per-layer exit heads / norm gains: list of tensors or None entries
            items = weights.get(key)
            if not items:
                return None
            assert len(items) == shape.n_layers
            return (C.c_void_p * shape.n_layers)(*[t.data_ptr() if t is not None else None for t in items])
        self._exit_head, self._exit_norm = table("exit_head"), table("exit_norm")
        self._w = Weights(weights["embed"].data_ptr(), weights["final_norm"].data_ptr(), weights["lm_head"].data_ptr(),
                          self._layers, self._exit_head, self._exit_norm)
        _check(lib().sb_load_weights(self.h, C.byref(self._w)), "sb_load_weights")
        if gemm is not None:
            _check(lib().sb_set_option(self.h, OPT_GEMM, gemm), "sb_set_option")

    def close(self):
        if getattr(self, "h", None):
            lib().sb_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self):
        _check(lib().sb_reset(self.h), "sb_reset")

    def selftest_wait_timeout(self, budget_ms: int = 20) -> int:
        """Returns the status of a kernel whose bounded wait is made to run out (expected: -5)."""
        return lib().sb_selftest_wait_timeout(self.h, budget_ms)

    def state(self) -> State:
        s = State()
        _check(lib().sb_get_state(self.h, C.byref(s)), "sb_get_state")
        return s

    def read_hidden(self, row: int) -> np.ndarray:
        out = np.zeros(self.shape.d_model, dtype=np.float32)
        _check(lib().sb_read_hidden(self.h, row, _np_ptr(out)), "sb_read_hidden")
        return out

    def prefill(self, prompt: Sequence[int]) -> int:
        pr = np.ascontiguousarray(prompt, dtype=np.int32)
        t = C.c_int32()
        _check(lib().sb_prefill(self.h, _np_ptr(pr), len(pr), C.byref(t)), "sb_prefill")
        return t.value

    def draft_push(self, token: int):
        _check(lib().sb_draft_push(self.h, token), "sb_draft_push")

    def draft_advance(self, to_layer: int):
        _check(lib().sb_draft_advance(self.h, to_layer), "sb_draft_advance")

    def exit_confidence(self, layer: int, tau_l: float, threshold: float):
        conf, tok, flag = C.c_float(), C.c_int32(), C.c_int32()
        _check(lib().sb_exit_confidence(self.h, layer, tau_l, threshold, C.byref(conf), C.byref(tok), C.byref(flag)),
               "sb_exit_confidence")
        return conf.value, tok.value, bool(flag.value)

    def verify(self, drafts: Sequence[int]):
        d = np.ascontiguousarray(drafts, dtype=np.int32)
        out = np.zeros(MAX_W, dtype=np.int32)
        n = C.c_int32()
        _check(lib().sb_verify(self.h, _np_ptr(d), len(d), _np_ptr(out), C.byref(n)), "sb_verify")
        return out[:n.value].copy()

    def generate(self, prompt: Sequence[int], n_gen: int, d_max: int, w_max: int, tau: Sequence[float], threshold: float,
                 trace: bool = False):
        pr = np.ascontiguousarray(prompt, dtype=np.int32)
        tau = np.ascontiguousarray(tau, dtype=np.float32)
        out = np.zeros(n_gen, dtype=np.int32)
        n, nr = C.c_int32(), C.c_int32()
        st = Stats()
        rounds = (Round * n_gen)() if trace else None
        _check(lib().sb_generate(self.h, _np_ptr(pr), len(pr), n_gen, d_max, w_max, _np_ptr(tau), threshold, _np_ptr(out),
                                 C.byref(n), C.byref(st), C.cast(rounds, C.c_void_p) if trace else None,
                                 n_gen if trace else 0, C.byref(nr)), "sb_generate")
        res = {"tokens": out[:n.value], "stats": st}
        if trace:
            res["rounds"] = [rounds[i] for i in range(nr.value)]
        return res

    def set_sampling(self, temperature: float, seed: int = 0, top_p: float = 1.0):
        """sb_set_sampling: temperature 0 restores greedy decoding; top_p < 1 = nucleus sampling."""
        _check(lib().sb_set_sampling(self.h, float(temperature), float(top_p), int(seed)), "sb_set_sampling")

    def generate_ar(self, prompt: Sequence[int], n_gen: int):
        pr = np.ascontiguousarray(prompt, dtype=np.int32)
        out = np.zeros(n_gen, dtype=np.int32)
        n = C.c_int32()
        st = Stats()
        _check(lib().sb_generate_ar(self.h, _np_ptr(pr), len(pr), n_gen, _np_ptr(out), C.byref(n), C.byref(st)),
               "sb_generate_ar")
        return {"tokens": out[:n.value], "stats": st}


class KernelScratch:
    """Scratch for the stateless kernel entry points."""

    def __init__(self, cfg: Config):
        self.nbytes = lib().sb_k_scratch_bytes(C.byref(cfg))
        if self.nbytes == 0:
            raise SBError(-1, "sb_k_scratch_bytes")
        self.buf = torch.empty(self.nbytes + 1024, dtype=torch.uint8, device="cuda")
        self.ptr = (self.buf.data_ptr() + 1023) & ~1023


def k_exit_confidence(cfg: Config, h: torch.Tensor, final_norm: torch.Tensor, lm_head: torch.Tensor, tau_l: float,
                      scratch: KernelScratch, want_logits: bool = False, stream=None):
    """h: CUDA fp32 [m, d].  Returns (conf [m] fp32, token [m] int32[, logits [m, V] fp32]) as CUDA tensors."""
    m = h.shape[0]
    assert h.is_cuda and h.dtype == torch.float32 and h.is_contiguous()
    conf = torch.empty(m, dtype=torch.float32, device="cuda")
    tok = torch.empty(m, dtype=torch.int32, device="cuda")
    logits = torch.empty((m, cfg.vocab), dtype=torch.float32, device="cuda") if want_logits else None
    _check(lib().sb_k_exit_confidence(C.byref(cfg), h.data_ptr(), m, final_norm.data_ptr(), lm_head.data_ptr(), tau_l,
                                      conf.data_ptr(), tok.data_ptr(), logits.data_ptr() if want_logits else None,
                                      C.c_void_p(scratch.ptr), scratch.nbytes, _stream_handle(stream)),
           "sb_k_exit_confidence")
    return (conf, tok, logits) if want_logits else (conf, tok)


def k_sample(logits: torch.Tensor, temperature: float, seed: int, pos0: int, top_p: float = 1.0, stream=None) -> torch.Tensor:
    """sb_k_sample on a [m, vocab] fp32 device tensor -> int32 tokens [m] (device)."""
    assert logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous() and logits.dim() == 2
    tok = torch.empty(logits.shape[0], dtype=torch.int32, device=logits.device)
    nbytes = lib().sb_k_sample_scratch_bytes(logits.shape[0], logits.shape[1])
    scratch = torch.empty(nbytes // 8, dtype=torch.float64, device=logits.device)
    _check(lib().sb_k_sample(logits.data_ptr(), logits.shape[0], logits.shape[1], float(temperature), float(top_p), int(seed), int(pos0),
                             tok.data_ptr(), scratch.data_ptr(), nbytes, _stream_handle(stream)), "sb_k_sample")
    return tok


def k_exit_confidence_static(cfg: Config, h: torch.Tensor, final_norm: torch.Tensor, lm_head: torch.Tensor, tau_l: float,
                             stream=None):
    """Exit confidence for callers that may not allocate device memory and have no scratch to lend:
    the library's own fixed device array serves as scratch (d_model <= 8192).  Calls on one device
    share that array, so do not let two of them overlap on the GPU.  The output tensors made here
    are the binding's convenience; the C entry point itself allocates nothing.
    Returns (conf [m] fp32, token [m] int32) as CUDA tensors."""
    m = h.shape[0]
    assert h.is_cuda and h.dtype == torch.float32 and h.is_contiguous()
    conf = torch.empty(m, dtype=torch.float32, device="cuda")
    tok = torch.empty(m, dtype=torch.int32, device="cuda")
    _check(lib().sb_k_exit_confidence_static(C.byref(cfg), h.data_ptr(), m, final_norm.data_ptr(), lm_head.data_ptr(),
                                             tau_l, conf.data_ptr(), tok.data_ptr(), _stream_handle(stream)),
           "sb_k_exit_confidence_static")
    return conf, tok


def k_layer(cfg: Config, lw: dict, h: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor,
            page_table: torch.Tensor, first_pos: int, scratch: KernelScratch, stream=None):
    """One decoder layer in place on h (CUDA fp32 [m, d]); appends to the paged caches."""
    assert h.is_cuda and h.dtype == torch.float32 and h.is_contiguous()
    L = lw if isinstance(lw, LayerWeights) else layer_weights(lw)
    _check(lib().sb_k_layer(C.byref(cfg), C.byref(L), h.data_ptr(), h.shape[0], k_cache.data_ptr(), v_cache.data_ptr(),
                            page_table.data_ptr(), first_pos, C.c_void_p(scratch.ptr), scratch.nbytes,
                            _stream_handle(stream)), "sb_k_layer")


def k_rope_table(cfg: Config, stream=None) -> torch.Tensor:
    """sb_k_rope_table: the cos/sin table of the rotation angles for this config, as a device tensor."""
    nbytes = lib().sb_k_rope_table_bytes(C.byref(cfg))
    tab = torch.empty(nbytes // 4, dtype=torch.float32, device="cuda")
    _check(lib().sb_k_rope_table(C.byref(cfg), tab.data_ptr(), nbytes, _stream_handle(stream)), "sb_k_rope_table")
    return tab


class LayerChain:
    """Marshalled arguments of sb_k_layer_chain: n layers' weights and caches (kept alive here)."""

    def __init__(self, lws: Sequence[dict], k_caches: Sequence[torch.Tensor], v_caches: Sequence[torch.Tensor]):
        n = len(lws)
        assert n == len(k_caches) == len(v_caches)
        self.n = n
        self._keep = (lws, k_caches, v_caches)
        self.lw = (LayerWeights * n)(*[l if isinstance(l, LayerWeights) else layer_weights(l) for l in lws])
        self.kc = (C.c_void_p * n)(*[t.data_ptr() for t in k_caches])
        self.vc = (C.c_void_p * n)(*[t.data_ptr() for t in v_caches])


def k_layer_chain(cfg: Config, chain: LayerChain, h: torch.Tensor, page_table: torch.Tensor, first_pos: int,
                  scratch: KernelScratch, rope_table: Optional[torch.Tensor] = None, stream=None):
    """n consecutive decoder layers in place on h (CUDA fp32 [m, d]), one launch sequence."""
    assert h.is_cuda and h.dtype == torch.float32 and h.is_contiguous()
    _check(lib().sb_k_layer_chain(C.byref(cfg), chain.lw, chain.n, h.data_ptr(), h.shape[0], chain.kc, chain.vc,
                                  page_table.data_ptr(), first_pos, rope_table.data_ptr() if rope_table is not None else None,
                                  C.c_void_p(scratch.ptr), scratch.nbytes, _stream_handle(stream)), "sb_k_layer_chain")
