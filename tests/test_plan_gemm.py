"""Host logic of the weight-streaming GEMMs' work decomposition (no GPU): every shape of the workloads is covered by its
work items, the tile sizes are ones the kernels can run, and no CTA or cluster gets much more than its share."""
import math

import pytest

from paper_2604_12247_b200 import binding, inputs

SHAPES = [inputs.LLAMA2_7B, inputs.LLAMA3_8B, inputs.LLAMA_13B,
          inputs.scaled(inputs.LLAMA3_8B, name="small", n_layers=4, d_model=512, n_heads=8, n_kv_heads=2, head_dim=64,
                        d_ffn=1416, vocab=2048)]


def _gemms(s):
    qd, kvd = s.n_heads * s.head_dim, s.n_kv_heads * s.head_dim
    return {"qkv": ([qd, kvd, kvd], s.d_model), "o": ([s.d_model], qd), "down": ([s.d_model], s.d_ffn)}


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: s.name)
@pytest.mark.parametrize("mode,units", [(0, 296), (0, 148), (2, 74), (2, 72)])
def test_split_gemm_plans_cover_their_matrices(shape, mode, units):
    per = 2 if mode == 2 else 1                       # CTAs that share a work item
    for name, (n_rows, k) in _gemms(shape).items():
        R, S, items = binding.plan_gemm(mode, n_rows, k, units)
        assert R % 8 == 0 and (8 if mode == 2 else 64) <= R <= 128, (name, R)
        assert (per * R) % 16 == 0 or mode == 0       # the pair kernel's MMA width 2R is a multiple of 16
        kb = math.ceil(k / 64)
        assert 1 <= S <= min(8, kb), (name, S)
        slabs = sum(math.ceil(n / (per * R)) for n in n_rows)
        assert items == slabs * S                     # every row of every matrix lies in exactly one slab, every k block in one split
        # the busiest unit's work (slab rows x k blocks) against a perfectly even share of the matrices
        busiest = math.ceil(items / units) * per * R * math.ceil(kb / S)
        ideal = sum(n_rows) * kb / units
        if shape.name != "small":                     # (a matrix of a few hundred rows cannot fill 296 CTAs)
            assert busiest <= 1.6 * ideal, (name, R, S, items, busiest / ideal)


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: s.name)
@pytest.mark.parametrize("mode,units", [(1, 296), (3, 74)])
def test_gate_up_plans(shape, mode, units):
    h, S, items = binding.plan_gemm(mode, [shape.d_ffn], shape.d_model, units)
    assert S == 1                                     # the SwiGLU epilogue needs whole sums: never split along k
    assert h % 8 == 0 and (32 <= h <= 64 if mode == 1 else 8 <= h <= 128)
    assert items == math.ceil(shape.d_ffn / h)        # every FFN column in exactly one item


def test_plan_query_rejects_bad_arguments():
    with pytest.raises(binding.SBError):
        binding.plan_gemm(4, [4096], 4096, 148)
    with pytest.raises(binding.SBError):
        binding.plan_gemm(0, [4096, 0], 4096, 148)
    with pytest.raises(binding.SBError):
        binding.plan_gemm(2, [4096], 0, 74)
    with pytest.raises(binding.SBError):
        binding.plan_gemm(2, [4096], 4096, 0)
