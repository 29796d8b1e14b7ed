"""Seeded synthetic inputs: model shapes, random-init weights, random prompts.

This module holds NO arithmetic of the decoding method.  It only names the
workload shapes and draws random tensors, so that the CUDA library and the CPU
oracle (which share no code) can be handed the very same bytes.

Recipe (stands in for the Spec-Bench prompts and the Vicuna / CodeLlama weights
the paper's experiments section uses, none of which exist offline):

* every linear weight and the embedding ~ N(0, 0.02), drawn in fp32 from ONE
  ``torch.Generator`` seeded ``seed`` in the fixed order
  ``embed; per layer wq, wk, wv, wo, w_gate, w_up, w_down; lm_head``;
* the LM head is multiplied by ``head_scale`` before the cast to the storage
  dtype (so shallow-layer softmax is peaked enough for exits to happen);
* RMSNorm gains are 1.0 (a N(0, 0.02) gain would zero the activations);
* optional ``damp_rho``: W_o and W_down of layer l (1-based) are multiplied by
  ``max(rho**(l-1), 0.01)`` -- a "damped deep layers" variant in which a shallow
  layer's prediction often equals the final one, the synthetic stand-in for
  the trained exit heads of the paper;
* prompts: ``randint(0, vocab)`` from a second generator seeded ``seed + 1``.
"""
from __future__ import annotations

from dataclasses import dataclass, field, asdict
from typing import Dict, List, Optional

import torch


@dataclass(frozen=True)
class Shape:
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rope_base: float = 10000.0
    rms_eps: float = 1e-5
    dtype: str = "bf16"          # storage dtype of weights and KV cache: "f32" | "bf16"
    head_scale: float = 4.0


@dataclass(frozen=True)
class Run:
    """One workload: a shape plus the decoding hyper-parameters of a config."""
    shape: Shape
    n_prompt: int
    n_gen: int
    d_max: int
    w_max: int
    tau: tuple                   # per-layer temperature T_l for l = 1..d_max
    threshold: float
    seed: int = 0
    damp_rho: Optional[float] = None


def tau_linear(d_max: int, first: float, last: float) -> tuple:
    """Temperatures falling linearly from ``first`` at layer 1 to ``last`` at layer d_max."""
    if d_max == 1:
        return (last,)
    return tuple(first + (last - first) * (l - 1) / (d_max - 1) for l in range(1, d_max + 1))


TINY = Shape("tiny", 4, 256, 4, 4, 64, 688, 1024, 10000.0, 1e-5, "f32", 8.0)
LLAMA2_7B = Shape("llama2-7b-shape", 32, 4096, 32, 32, 128, 11008, 32000, 10000.0, 1e-5, "bf16", 4.0)
LLAMA3_8B = Shape("llama3-8b-shape", 32, 4096, 32, 8, 128, 14336, 128256, 500000.0, 1e-5, "bf16", 4.0)
LLAMA_13B = Shape("13b-shape", 40, 5120, 40, 40, 128, 13824, 32000, 10000.0, 1e-5, "bf16", 4.0)


def scaled(shape: Shape, **kw) -> Shape:
    """A copy of ``shape`` with some fields replaced (e.g. fewer layers for a parity case)."""
    d = asdict(shape)
    d.update(kw)
    return Shape(**d)


# The named workloads (shape + decoding hyper-parameters); labelled additions are marked.
RUNS: Dict[str, Run] = {
    # tiny decoder, fp32: tau_l = 1 + 0.5 (d_max - l)
    "tiny": Run(TINY, 16, 32, 2, 4, (1.5, 1.0), 0.3, seed=0),
    # addition: damped deep layers + sharper head so that exits happen at both layers, drafts get
    # accepted in runs of 0..4 and both round-termination causes occur within 32 tokens
    "tiny-damped": Run(scaled(TINY, name="tiny-damped", head_scale=16.0), 16, 32, 2, 4, (1.5, 1.0), 0.3, seed=0,
                       damp_rho=0.2),
    "7b": Run(LLAMA2_7B, 512, 512, 6, 4, tau_linear(6, 2.0, 1.0), 0.6, seed=0),
    # addition, the synthetic stand-in for trained exit heads: W_o and W_down of layer l scaled by
    # max(0.3^(l-1), 0.01) and a sharper head (x8), so that a confident shallow prediction usually is the
    # full model's token; the paper's own hyper-parameters: d_max 10, w_max 8, Eq. 1 with alpha 0.2,
    # confidence threshold 0.55
    "7b-damped": Run(scaled(LLAMA2_7B, name="llama2-7b-shape-damped", head_scale=8.0), 512, 512, 10, 8,
                     tuple(1.0 + 0.2 * (1.0 - l / 32.0) for l in range(1, 11)), 0.55, seed=0, damp_rho=0.3),
    "l3-8b": Run(LLAMA3_8B, 1024, 2048, 8, 6, tau_linear(8, 2.0, 1.0), 0.5, seed=0),
    "13b": Run(LLAMA_13B, 2048, 1024, 8, 4, tau_linear(8, 2.0, 1.0), 0.6, seed=0),
}


def torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


LAYER_MATS = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")


def layer_mat_shapes(s: Shape) -> Dict[str, tuple]:
    q = s.n_heads * s.head_dim
    kv = s.n_kv_heads * s.head_dim
    return {
        "wq": (q, s.d_model), "wk": (kv, s.d_model), "wv": (kv, s.d_model), "wo": (s.d_model, q),
        "w_gate": (s.d_ffn, s.d_model), "w_up": (s.d_ffn, s.d_model), "w_down": (s.d_model, s.d_ffn),
    }


def make_weights(s: Shape, seed: int = 0, device: str = "cpu", damp_rho: Optional[float] = None,
                 std: float = 0.02) -> dict:
    """Random-init weights of shape ``s`` as a dict of tensors in the storage dtype.

    Returns ``{"embed", "final_norm", "lm_head", "layers": [ {attn_norm, wq, ...}, ... ]}``.
    Every matrix is row-major ``[out_features, in_features]``.  Draws happen on ``device``
    (a CPU generator gives the same bytes on every machine; a CUDA generator is only
    reproducible on the same GPU model, which is all the large shapes need).
    """
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    dt = torch_dtype(s.dtype)

    def draw(shape, scale=1.0):
        t = torch.empty(shape, dtype=torch.float32, device=device)
        t.normal_(0.0, std, generator=g)
        if scale != 1.0:
            t.mul_(scale)
        return t.to(dt).contiguous()

    out = {"embed": draw((s.vocab, s.d_model)), "layers": []}
    shapes = layer_mat_shapes(s)
    for l in range(1, s.n_layers + 1):
        damp = 1.0 if damp_rho is None else max(damp_rho ** (l - 1), 0.01)
        lw = {}
        for name in LAYER_MATS:
            lw[name] = draw(shapes[name], damp if name in ("wo", "w_down") else 1.0)
        lw["attn_norm"] = torch.ones(s.d_model, dtype=dt, device=device)
        lw["mlp_norm"] = torch.ones(s.d_model, dtype=dt, device=device)
        out["layers"].append(lw)
    out["lm_head"] = draw((s.vocab, s.d_model), s.head_scale)
    out["final_norm"] = torch.ones(s.d_model, dtype=dt, device=device)
    return out


def make_prompt(s: Shape, n: int, seed: int = 0) -> torch.Tensor:
    """``n`` uniform-random token ids (int32, CPU) from a generator seeded ``seed + 1``."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed + 1)
    return torch.randint(0, s.vocab, (n,), generator=g, dtype=torch.int64).to(torch.int32)


def make_hidden(m: int, d: int, seed: int, scale: float = 1.0) -> torch.Tensor:
    """``m`` random hidden-state rows ~ N(0, scale^2), fp32, CPU."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return torch.randn((m, d), generator=g, dtype=torch.float32) * scale


def make_kv(n_pos: int, kv_dim: int, seed: int, dtype: str) -> tuple:
    """Random K and V contents ``[n_pos, kv_dim]`` ~ N(0,1) in the storage dtype (CPU)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    k = torch.randn((n_pos, kv_dim), generator=g, dtype=torch.float32).to(torch_dtype(dtype))
    v = torch.randn((n_pos, kv_dim), generator=g, dtype=torch.float32).to(torch_dtype(dtype))
    return k, v


def add_exit_heads(w: dict, s: Shape, seed: int = 0, noise: float = 0.5) -> dict:
    """Synthetic per-layer exit heads (stand-ins for the lightweight heads Section 3.2 trains): for every layer a
    head = shared LM head + ``noise`` x an independent draw of the same scale, and a norm gain close to 1.  Adds
    ``exit_head`` / ``exit_norm`` (lists of n_layers tensors) to ``w`` in place and returns it."""
    dev = w["lm_head"].device
    g = torch.Generator(device=dev)
    g.manual_seed(seed + 1000)
    dt = torch_dtype(s.dtype)
    heads, norms = [], []
    base = w["lm_head"].float()
    for _ in range(s.n_layers):
        n = torch.empty_like(base).normal_(0.0, 0.02 * s.head_scale, generator=g)
        heads.append((base + noise * n).to(dt).contiguous())
        gn = torch.empty(s.d_model, dtype=torch.float32, device=dev).normal_(0.0, 0.1, generator=g)
        norms.append((1.0 + gn).to(dt).contiguous())
    w["exit_head"], w["exit_norm"] = heads, norms
    return w


def weights_to(w: dict, device: str) -> dict:
    def move(v):
        if isinstance(v, torch.Tensor):
            return v.to(device)
        if isinstance(v, list):
            return [move(x) for x in v]
        return v
    out = {k: move(v) for k, v in w.items() if k != "layers"}
    out["layers"] = [{k: v.to(device) for k, v in lw.items()} for lw in w["layers"]]
    return out


def weight_bytes(s: Shape) -> Dict[str, int]:
    """Storage bytes of one layer's matrices, of the LM head and of the whole model."""
    es = 4 if s.dtype == "f32" else 2
    per_layer = sum(a * b for a, b in layer_mat_shapes(s).values()) * es
    head = s.vocab * s.d_model * es
    return {"layer": per_layer, "head": head, "model": per_layer * s.n_layers + head}
