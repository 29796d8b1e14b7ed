"""The allocation-free exit-confidence entry point (collected last on purpose: if it fails, a run
that stops at the first failure has already been through every other test).

`sb_k_exit_confidence_static` serves callers that cannot call cudaMalloc and have no scratch buffer
to lend: its scratch is a fixed array inside the library.  It must give what the ordinary entry
point gives, also on a second call that finds the array dirty from the first."""
import numpy as np
import pytest
import torch

from oracle import oracle
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
        # and against the CPU oracle's exit test on the same rows (Eq. 2), directly
        w = inputs.make_weights(inputs.scaled(shape, vocab=8), 0)
        w["lm_head"], w["final_norm"] = lm.cpu(), gain.cpu()
        o = oracle.Oracle(shape, w, 4)
        for i in range(m):
            p, t = o.exit_confidence(h[i].cpu().numpy(), tau)
            assert abs(float(got_conf[i]) - p) < CONF_TOL and int(got_tok[i]) == t, (call, i)
        o.close()


def test_static_scratch_call_allocates_no_device_memory():
    """What the entry point is for: with the outputs preallocated, a call leaves the device's free memory where it
    was (no cudaMalloc behind the caller's back), also at the widest model the fixed array takes (d_model 8192)."""
    wide = inputs.scaled(BF16, name="noalloc-wide", d_model=8192, n_heads=64, n_kv_heads=64, head_dim=128, vocab=512)
    for shape in (BF16, wide):
        cfg = binding.make_config(shape, 64, 16)
        lm, gain = _head(shape, 43)
        h = inputs.make_hidden(8, shape.d_model, 77).cuda()
        conf = torch.empty(8, dtype=torch.float32, device="cuda")
        tok = torch.empty(8, dtype=torch.int32, device="cuda")
        call = lambda: binding._check(binding.lib().sb_k_exit_confidence_static(
            cfg, h.data_ptr(), 8, gain.data_ptr(), lm.data_ptr(), 1.3, conf.data_ptr(), tok.data_ptr(), None), "static")
        call()                                   # the first call on a device looks up the array's address
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        for _ in range(3):
            call()
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert free1 == free0, (shape.name, free0, free1)
        assert np.all(conf.cpu().numpy() > 0) and np.all((tok.cpu().numpy() >= 0) & (tok.cpu().numpy() < shape.vocab))


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
