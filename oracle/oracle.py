"""ctypes front end of the C oracle (``specbound_oracle.c``).

TEST INFRASTRUCTURE: imported only by ``tests/``, the smoke check and the
benchmark's CPU-baseline leg.  It never imports the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "specbound_oracle.c"
_LIB = _HERE / "libspecbound_oracle.so"
MAX_W = 8


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (plain -O2, OpenMP over output rows)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c99", "-o", str(tmp),
                               str(_SRC), "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab")] + [
        ("rope_base", C.c_double), ("rms_eps", C.c_double), ("wdtype", C.c_int32), ("max_seq", C.c_int32),
        ("kv_round_bf16", C.c_int32)]


class _Layer(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down")]


class _Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p), ("layers", C.POINTER(_Layer))]


class Round(C.Structure):
    _fields_ = [("w", C.c_int32), ("D", C.c_int32), ("emitted", C.c_int32), ("accepted_drafts", C.c_int32),
                ("layer_steps", C.c_int32), ("probes", C.c_int32),
                ("exit_layer", C.c_int32 * MAX_W), ("draft", C.c_int32 * MAX_W), ("g", C.c_int32 * MAX_W),
                ("layers_done", C.c_int32 * MAX_W), ("depth_after", (C.c_int32 * MAX_W) * MAX_W),
                ("conf", C.c_double * MAX_W)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(str(build()))
        L.orc_create.restype = C.c_void_p
        L.orc_create.argtypes = [C.POINTER(_Config), C.POINTER(_Weights)]
        L.orc_destroy.argtypes = [C.c_void_p]
        L.orc_tau_schedule.argtypes = [C.c_double, C.c_int, C.c_void_p]
        for f in ("orc_round_cost", "orc_expected_accepted", "orc_speedup"):
            getattr(L, f).restype = C.c_double
        L.orc_round_cost.argtypes = [C.c_int, C.c_int, C.c_int]
        L.orc_expected_accepted.argtypes = [C.c_double, C.c_int]
        L.orc_speedup.argtypes = [C.c_int, C.c_double, C.c_int, C.c_int]
        L.orc_exit_confidence.argtypes = [C.c_void_p, C.c_void_p, C.c_double, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_confidence.argtypes = [C.c_void_p, C.c_int, C.c_double, C.c_void_p, C.c_void_p]
        L.orc_set_exit_head.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_exit_confidence_at.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_double, C.c_void_p, C.c_void_p]
        L.orc_mix64.restype = C.c_uint64
        L.orc_mix64.argtypes = [C.c_uint64, C.c_int64]
        L.orc_uniform.restype = C.c_double
        L.orc_uniform.argtypes = [C.c_uint64, C.c_int64]
        L.orc_sample_token.argtypes = [C.c_void_p, C.c_int, C.c_double, C.c_double, C.c_double, C.c_void_p]
        L.orc_nucleus_threshold.restype = C.c_double
        L.orc_nucleus_threshold.argtypes = [C.c_void_p, C.c_int, C.c_double, C.c_double]
        L.orc_set_sampling.argtypes = [C.c_void_p, C.c_double, C.c_double, C.c_uint64]
        L.orc_set_kv.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_get_kv.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_layer_forward.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_int]
        L.orc_embed.argtypes = [C.c_void_p, C.c_int, C.c_void_p]
        L.orc_final_logits.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_prefill.argtypes = [C.c_void_p, C.c_void_p, C.c_int]
        L.orc_ar_generate.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_bruteforce_generate.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p]
        L.orc_teacher_forced.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int] + [C.c_void_p] * 4
        L.orc_specbound_generate.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p,
                                             C.c_double, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int]
        _lib = L
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def tau_schedule(alpha: float, L: int) -> np.ndarray:
    out = np.zeros(L, dtype=np.float64)
    lib().orc_tau_schedule(alpha, L, _ptr(out))
    return out


def round_cost(L, w, d_max):
    return lib().orc_round_cost(L, w, d_max)


def expected_accepted(a, w):
    return lib().orc_expected_accepted(a, w)


def speedup(L, a, w, d_max):
    return lib().orc_speedup(L, a, w, d_max)


def mix64(seed: int, pos: int) -> int:
    """Counter-based 64-bit hash behind the sampling uniforms (splitmix64 output function)."""
    return int(lib().orc_mix64(seed, pos))


def uniform(seed: int, pos: int) -> float:
    """u(seed, pos) in (0, 1): the uniform number that decides the token at sequence position pos."""
    return float(lib().orc_uniform(seed, pos))


def sample_token(z: np.ndarray, temperature: float, u: float, top_p: float = 1.0):
    """Inverse-CDF sample, in vocabulary order, of softmax(z / temperature) restricted to its top-p nucleus
    -> (token, slack)."""
    z = np.ascontiguousarray(z, dtype=np.float64)
    slack = C.c_double()
    t = lib().orc_sample_token(_ptr(z), z.size, float(temperature), float(top_p), float(u), C.byref(slack))
    return int(t), float(slack.value)


def nucleus_threshold(z: np.ndarray, temperature: float, top_p: float) -> float:
    """Smallest logit inside the top-p nucleus of softmax(z / temperature) (-inf for top_p >= 1)."""
    z = np.ascontiguousarray(z, dtype=np.float64)
    return float(lib().orc_nucleus_threshold(_ptr(z), z.size, float(temperature), float(top_p)))


def confidence(z: np.ndarray, T: float):
    z = np.ascontiguousarray(z, dtype=np.float64)
    conf = C.c_double()
    tok = C.c_int32()
    lib().orc_confidence(_ptr(z), z.shape[0], T, C.byref(conf), C.byref(tok))
    return conf.value, tok.value


class Oracle:
    """A decoder with its own KV cache.  ``weights`` is the dict of CPU tensors the input
    generator returns (fp32 or bf16 storage); the tensors are borrowed and kept alive."""

    def __init__(self, shape, weights: dict, max_seq: int, kv_round_bf16: Optional[bool] = None):
        self.shape = shape
        self._keep = weights
        wd = {"f32": 0, "bf16": 1}[shape.dtype]
        if kv_round_bf16 is None:
            kv_round_bf16 = shape.dtype == "bf16"
        self.cfg = _Config(shape.n_layers, shape.d_model, shape.n_heads, shape.n_kv_heads, shape.head_dim, shape.d_ffn,
                           shape.vocab, shape.rope_base, shape.rms_eps, wd, max_seq, int(kv_round_bf16))
        want = torch.float32 if wd == 0 else torch.bfloat16

        def p(t: torch.Tensor):
            assert t.device.type == "cpu" and t.dtype == want and t.is_contiguous()
            return t.data_ptr()

        self._layers = (_Layer * shape.n_layers)()
        for i, lw in enumerate(weights["layers"]):
            for name, _ in _Layer._fields_:
                setattr(self._layers[i], name, p(lw[name]))
        self._w = _Weights(p(weights["embed"]), p(weights["final_norm"]), p(weights["lm_head"]), self._layers)
        self.h = lib().orc_create(C.byref(self.cfg), C.byref(self._w))
        if not self.h:
            raise MemoryError("oracle KV cache allocation failed")
        self._want = want
        self._exit_keep = {}
        heads, norms = weights.get("exit_head"), weights.get("exit_norm")   # optional per-layer exit heads / norm gains
        for l in range(1, shape.n_layers + 1):
            eh = heads[l - 1] if heads else None
            en = norms[l - 1] if norms else None
            if eh is not None or en is not None:
                self.set_exit_head(l, eh, en)

    def close(self):
        if self.h:
            lib().orc_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_sampling(self, temperature: float, seed: int = 0, top_p: float = 1.0):
        """Sampling decoding (Section 4.3): temperature 0 restores greedy decoding; top_p < 1 = nucleus sampling."""
        lib().orc_set_sampling(self.h, float(temperature), float(top_p), int(seed))

    def set_exit_head(self, layer: int, head: Optional[torch.Tensor], norm: Optional[torch.Tensor] = None):
        """Head [vocab, d_model] (and norm gain [d_model]) of the exit test after `layer`; None = the shared ones."""
        for t in (head, norm):
            assert t is None or (t.device.type == "cpu" and t.dtype == self._want and t.is_contiguous())
        self._exit_keep[layer] = (head, norm)
        lib().orc_set_exit_head(self.h, layer, head.data_ptr() if head is not None else None,
                                norm.data_ptr() if norm is not None else None)

    # ---- single operations ------------------------------------------------
    def exit_confidence_at(self, layer: int, h, T: float):
        h = np.ascontiguousarray(h, dtype=np.float64)
        conf, tok = C.c_double(), C.c_int32()
        lib().orc_exit_confidence_at(self.h, layer, _ptr(h), T, C.byref(conf), C.byref(tok))
        return conf.value, tok.value

    def exit_confidence(self, h, T: float, want_logits: bool = False):
        h = np.ascontiguousarray(h, dtype=np.float64)
        conf, tok = C.c_double(), C.c_int32()
        z = np.zeros(self.shape.vocab, dtype=np.float64) if want_logits else None
        lib().orc_exit_confidence(self.h, _ptr(h), T, C.byref(conf), C.byref(tok), _ptr(z) if want_logits else None)
        return (conf.value, tok.value, z) if want_logits else (conf.value, tok.value)

    def final_logits(self, h):
        h = np.ascontiguousarray(h, dtype=np.float64)
        z = np.zeros(self.shape.vocab, dtype=np.float64)
        lib().orc_final_logits(self.h, _ptr(h), _ptr(z))
        return z

    def embed(self, tok: int):
        h = np.zeros(self.shape.d_model, dtype=np.float64)
        lib().orc_embed(self.h, tok, _ptr(h))
        return h

    def set_kv(self, layer: int, pos: int, k, v):
        k = np.ascontiguousarray(k, dtype=np.float64)
        v = np.ascontiguousarray(v, dtype=np.float64)
        lib().orc_set_kv(self.h, layer, pos, _ptr(k), _ptr(v))

    def get_kv(self, layer: int, pos: int):
        kvd = self.shape.n_kv_heads * self.shape.head_dim
        k, v = np.zeros(kvd), np.zeros(kvd)
        lib().orc_get_kv(self.h, layer, pos, _ptr(k), _ptr(v))
        return k, v

    def layer_forward(self, layer: int, h, first_pos: int):
        h = np.array(h, dtype=np.float64, order="C", copy=True)
        assert h.ndim == 2
        lib().orc_layer_forward(self.h, layer, _ptr(h), h.shape[0], first_pos)
        return h

    # ---- generation ---------------------------------------------------------
    def ar_generate(self, prompt: Sequence[int], n_gen: int, want_margins: bool = False):
        pr = np.ascontiguousarray(prompt, dtype=np.int32)
        out = np.zeros(n_gen, dtype=np.int32)
        mg = np.zeros(n_gen, dtype=np.float64)
        r = lib().orc_ar_generate(self.h, _ptr(pr), len(pr), n_gen, _ptr(out), _ptr(mg))
        if r < 0:
            raise ValueError("ar_generate: bad arguments / capacity")
        return (out, mg) if want_margins else out

    def bruteforce_generate(self, prompt: Sequence[int], n_gen: int):
        pr = np.ascontiguousarray(prompt, dtype=np.int32)
        out = np.zeros(n_gen, dtype=np.int32)
        lib().orc_bruteforce_generate(self.h, _ptr(pr), len(pr), n_gen, _ptr(out))
        return out

    def teacher_forced(self, tokens: Sequence[int], start: int):
        """``tokens`` = prompt + generated; ``start`` = index of the first generated token."""
        tk = np.ascontiguousarray(tokens, dtype=np.int32)
        n = len(tk) - start
        top1 = np.zeros(n, dtype=np.int32)
        top2 = np.zeros(n, dtype=np.int32)
        margin = np.zeros(n)
        deficit = np.zeros(n)
        r = lib().orc_teacher_forced(self.h, _ptr(tk), len(tk), start, _ptr(top1), _ptr(top2), _ptr(margin), _ptr(deficit))
        if r < 0:
            raise ValueError("teacher_forced: bad arguments / capacity")
        return top1, top2, margin, deficit

    def specbound_generate(self, prompt: Sequence[int], n_gen: int, d_max: int, w_max: int, tau: Sequence[float],
                           threshold: float, script: Optional[Sequence[int]] = None, max_rounds: Optional[int] = None):
        pr = np.ascontiguousarray(prompt, dtype=np.int32)
        out = np.zeros(max(n_gen, 1), dtype=np.int32)
        tau = np.ascontiguousarray(tau, dtype=np.float64)
        assert len(tau) >= d_max
        max_rounds = max_rounds or max(n_gen, 1)
        rounds = (Round * max_rounds)()
        sc = np.ascontiguousarray(script, dtype=np.int32) if script is not None else None
        r = lib().orc_specbound_generate(self.h, _ptr(pr), len(pr), n_gen, d_max, w_max, _ptr(tau), threshold,
                                         _ptr(sc) if sc is not None else None, len(sc) if sc is not None else 0,
                                         _ptr(out), C.cast(rounds, C.c_void_p), max_rounds)
        if r < 0:
            raise ValueError("specbound_generate: bad arguments / capacity")
        return out[:n_gen], [rounds[i] for i in range(min(r, max_rounds))]
