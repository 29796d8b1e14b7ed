"""The allocation-free exit-confidence entry point (collected last on purpose: if it fails, a run
that stops at the first failure has already been through every other test).

`sb_k_exit_confidence_static` serves callers that cannot call cudaMalloc and have no scratch buffer
to lend: its scratch is a fixed array inside the library.  It must give what the ordinary entry
point gives, also on a second call that finds the array dirty from the first."""
import numpy as np
import pytest
import torch

from paper_2604_12247_b200 import binding, inputs
from gpu_util import CONF_TOL

pytestmark = pytest.mark.gpu

BF16 = inputs.scaled(inputs.LLAMA2_7B, name="noalloc-bf16", n_layers=1, d_model=512, n_heads=8, n_kv_heads=8,
                     head_dim=64, d_ffn=64, vocab=5000)


def _head(shape, seed):
    g = torch.Generator().manual_seed(seed)
    dt = inputs.torch_dtype(shape.dtype)
    lm = (torch.randn((shape.vocab, shape.d_model), generator=g) * 0.02 * shape.head_scale).to(dt).cuda()
    gain = (1.0 + 0.2 * torch.randn(shape.d_model, generator=g)).to(dt).cuda()
    return lm, gain


@pytest.mark.parametrize("shape", [inputs.TINY, BF16], ids=["f32", "bf16"])
def test_static_scratch_entry_point_matches_the_ordinary_one(shape):
    cfg = binding.make_config(shape, 64, 16)
    lm, gain = _head(shape, 41)
    scratch = binding.KernelScratch(cfg)
    # two calls in a row; the second uses other rows, another row count and another temperature, and
    # finds the shared array as the first call left it
    for call, (m, tau) in enumerate(((8, 1.7), (3, 1.0))):
        h = inputs.make_hidden(m, shape.d_model, 300 + call, scale=1.5).cuda()
        want_conf, want_tok = binding.k_exit_confidence(cfg, h, gain, lm, tau, scratch)
        got_conf, got_tok = binding.k_exit_confidence_static(cfg, h, gain, lm, tau)
        torch.cuda.synchronize()
        assert np.allclose(got_conf.cpu().numpy(), want_conf.cpu().numpy(), atol=CONF_TOL, rtol=0), call
        assert np.array_equal(got_tok.cpu().numpy(), want_tok.cpu().numpy()), call
        assert np.all(got_conf.cpu().numpy() > 0) and np.all(got_conf.cpu().numpy() <= 1 + 1e-6)


def test_static_scratch_entry_point_refuses_what_does_not_fit():
    big = inputs.scaled(BF16, name="too-wide", d_model=16384, n_heads=128, head_dim=128, n_kv_heads=128)
    cfg = binding.make_config(big, 64, 16)
    x = torch.zeros((1, 8), device="cuda")
    with pytest.raises(binding.SBError) as e:      # refused before any pointer is touched
        binding.lib()  # make sure the library is loaded
        binding._check(binding.lib().sb_k_exit_confidence_static(cfg, x.data_ptr(), 1, x.data_ptr(), x.data_ptr(), 1.0,
                                                                  x.data_ptr(), x.data_ptr(), None), "static")
    assert e.value.status == -3                    # capacity: d_model beyond the 8192 the fixed array holds
    ok_cfg = binding.make_config(BF16, 64, 16)
    with pytest.raises(binding.SBError) as e:
        binding._check(binding.lib().sb_k_exit_confidence_static(ok_cfg, x.data_ptr(), 9, x.data_ptr(), x.data_ptr(), 1.0,
                                                                  x.data_ptr(), x.data_ptr(), None), "static")
    assert e.value.status == -1                    # more than 8 rows
