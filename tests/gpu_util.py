"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch

from oracle import oracle
from paper_2604_12247_b200 import binding, inputs

# Tolerances of the parity tests: logits within 1e-4 (fp32 models) / 2e-2 (bf16 models) absolute,
# exit confidences within 1e-3.  Hidden states are compared relative to their own scale.
LOGIT_TOL = {"f32": 1e-4, "bf16": 2e-2}
CONF_TOL = 1e-3
HIDDEN_TOL = {"f32": 2e-5, "bf16": 4e-3}


def gpu_ctx(shape, weights_cpu, max_seq, kv_page=16, gemm=None):
    wg = inputs.weights_to(weights_cpu, "cuda")
    return binding.Context(shape, wg, max_seq, kv_page=kv_page, gemm=gemm), wg


def near_tie_count(shape, weights_cpu, prompt, gpu_tokens, tol):
    """Teacher-forced oracle check of a GPU token sequence.  Returns (n_not_top1, worst_deficit):
    every GPU token must be the oracle's top-1 or lie within `tol` of it."""
    toks = np.concatenate([np.asarray(prompt, dtype=np.int32), np.asarray(gpu_tokens, dtype=np.int32)])
    o = oracle.Oracle(shape, weights_cpu, len(toks) + 1)
    top1, _, margin, deficit = o.teacher_forced(toks, len(prompt))
    return int((top1 != gpu_tokens).sum()), float(deficit.min())


def gemm_modes(shape):
    """GEMM back ends a model of this dtype can use: 0 = CUDA-core kernels, 1 = TMA + tcgen05
    (bf16 only; test_gpu_generate.test_tcgen05_backend_is_built fails if it is missing)."""
    if shape.dtype == "f32":
        return [0]
    ok = binding.lib().sb_set_default_option(binding.OPT_GEMM, 1) == 0
    binding.lib().sb_set_default_option(binding.OPT_GEMM, -1)
    return [0, 1] if ok else [0]
