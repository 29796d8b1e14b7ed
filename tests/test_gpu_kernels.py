"""Kernel-level parity of the CUDA path against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2604_12247_b200 import binding, inputs
from gpu_util import LOGIT_TOL, CONF_TOL, HIDDEN_TOL

pytestmark = pytest.mark.gpu

HEAD_BF16 = inputs.scaled(inputs.LLAMA2_7B, name="head-bf16", n_layers=1, d_model=512, n_heads=8, n_kv_heads=8,
                          head_dim=64, d_ffn=64, vocab=5000)
HEAD_7B = inputs.scaled(inputs.LLAMA2_7B, name="head-7b", n_layers=1, d_ffn=64)


def head_weights(shape, seed):
    g = torch.Generator().manual_seed(seed)
    dt = inputs.torch_dtype(shape.dtype)
    lm = (torch.randn((shape.vocab, shape.d_model), generator=g) * 0.02 * shape.head_scale).to(dt)
    gain = (1.0 + 0.2 * torch.randn(shape.d_model, generator=g)).to(dt)
    return lm, gain


def oracle_head(shape, lm, gain):
    """An oracle instance that only serves exit_confidence (one dummy layer)."""
    w = inputs.make_weights(inputs.scaled(shape, vocab=8), 0)
    w["lm_head"], w["final_norm"] = lm, gain
    return oracle.Oracle(shape, w, 4)


def run_exit(shape, lm, gain, h, tau, gemm):
    cfg = binding.make_config(shape, 64, 16)
    binding.set_default_gemm(gemm)
    try:
        sc = binding.KernelScratch(cfg)
        conf, tok, logits = binding.k_exit_confidence(cfg, h.cuda(), gain.cuda(), lm.cuda(), tau, sc, want_logits=True)
        torch.cuda.synchronize()
    finally:
        binding.set_default_gemm(-1)
    return conf.cpu().numpy(), tok.cpu().numpy(), logits.cpu().numpy()


from gpu_util import gemm_modes


@pytest.mark.parametrize("shape,ms", [(inputs.TINY, (1, 3, 8)), (HEAD_BF16, (1, 5, 8)), (HEAD_7B, (2,))],
                         ids=["tiny-f32", "bf16-ragged-vocab", "7b-head"])
def test_exit_confidence_matches_oracle(shape, ms):
    lm, gain = head_weights(shape, 11)
    o = oracle_head(shape, lm, gain)
    for gemm in gemm_modes(shape):
        for m in ms:
            h = inputs.make_hidden(m, shape.d_model, 100 + m, scale=1.7)
            for tau in (2.0, 1.5, 1.0):
                conf, tok, logits = run_exit(shape, lm, gain, h, tau, gemm)
                for i in range(m):
                    p, t, z = o.exit_confidence(h[i].numpy(), tau, want_logits=True)
                    err = np.abs(logits[i] - z).max()
                    assert err < LOGIT_TOL[shape.dtype], (gemm, m, tau, err)
                    assert abs(conf[i] - p) < CONF_TOL, (gemm, m, tau, conf[i], p)
                    srt = np.sort(z)
                    if srt[-1] - srt[-2] > 2 * LOGIT_TOL[shape.dtype]:
                        assert tok[i] == t
                    else:                      # near tie: either of the two is a correct argmax
                        assert z[tok[i]] >= srt[-1] - 2 * LOGIT_TOL[shape.dtype]


@pytest.mark.parametrize("shape", [inputs.TINY, HEAD_BF16], ids=["f32", "bf16"])
def test_exit_confidence_special_cases(shape):
    lm, gain = head_weights(shape, 12)
    h = inputs.make_hidden(2, shape.d_model, 5)
    for gemm in gemm_modes(shape):
        # all-zero head: every logit equal -> conf = 1/V, argmax = lowest index
        conf, tok, _ = run_exit(shape, torch.zeros_like(lm), gain, h, 1.3, gemm)
        assert np.allclose(conf, 1.0 / shape.vocab, rtol=1e-5) and (tok == 0).all()
        # two identical dominant rows: the tie goes to the lower index, conf ~ 1/2
        lm2 = lm.clone()
        x = (h[0] * gain.float())
        lm2[7] = (x / x.norm() * 3).to(lm.dtype)
        lm2[shape.vocab - 5] = lm2[7]
        conf, tok, _ = run_exit(shape, lm2, gain, h[:1], 1.0, gemm)
        o = oracle_head(shape, lm2, gain)
        p, t = o.exit_confidence(h[0].numpy(), 1.0)
        assert t == 7 and tok[0] == 7 and abs(conf[0] - p) < CONF_TOL and conf[0] <= 0.5 + 1e-6


def test_exit_confidence_deterministic():
    shape = HEAD_BF16
    lm, gain = head_weights(shape, 13)
    h = inputs.make_hidden(8, shape.d_model, 6)
    for gemm in gemm_modes(shape):
        a = run_exit(shape, lm, gain, h, 1.4, gemm)
        b = run_exit(shape, lm, gain, h, 1.4, gemm)
        assert all(np.array_equal(x, y) for x, y in zip(a, b))
        # a row's result does not depend on its companions
        c = run_exit(shape, lm, gain, h[3:4], 1.4, gemm)
        assert c[0][0] == a[0][3] and c[1][0] == a[1][3]


def test_exit_confidence_rejects_bad_arguments():
    shape = HEAD_BF16
    lm, gain = head_weights(shape, 14)
    cfg = binding.make_config(shape, 64, 16)
    sc = binding.KernelScratch(cfg)
    h = inputs.make_hidden(2, shape.d_model, 1).cuda()
    with pytest.raises(binding.SBError) as e:
        binding.k_exit_confidence(cfg, h, gain.cuda(), lm.cuda(), 0.0, sc)          # tau must be > 0
    assert e.value.status == -1
    sc.nbytes = 1024
    with pytest.raises(binding.SBError) as e:
        binding.k_exit_confidence(cfg, h, gain.cuda(), lm.cuda(), 1.0, sc)          # scratch too small
    assert e.value.status == -3


# ---------------------------------------------------------------------------------------------
LAYER_BF16 = inputs.scaled(inputs.LLAMA3_8B, name="layer-bf16", n_layers=1, d_model=512, n_heads=8, n_kv_heads=2,
                           head_dim=64, d_ffn=1408, vocab=64)
LAYER_F32 = inputs.scaled(inputs.TINY, name="layer-f32", n_layers=1, vocab=64)
LAYER_HD128 = inputs.scaled(inputs.LLAMA2_7B, name="layer-hd128", n_layers=1, d_model=512, n_heads=4, n_kv_heads=4,
                            head_dim=128, d_ffn=1024, vocab=64)


def run_layer(shape, w, h, k_hist, v_hist, first_pos, max_seq, page, gemm):
    """GPU layer on rows h at first_pos.. over a cache pre-filled with k_hist/v_hist[0:first_pos].
    Physical pages are deliberately permuted.  Returns (h_out, K rows, V rows of the new positions)."""
    cfg = binding.make_config(shape, max_seq, page)
    kvd = shape.n_kv_heads * shape.head_dim
    n_pages = (max_seq + page - 1) // page
    perm = torch.randperm(n_pages, generator=torch.Generator().manual_seed(3)).to(torch.int32)
    dt = inputs.torch_dtype(shape.dtype)
    kc = torch.zeros((n_pages, page, kvd), dtype=dt)
    vc = torch.zeros((n_pages, page, kvd), dtype=dt)
    for p in range(first_pos):
        kc[perm[p // page], p % page] = k_hist[p]
        vc[perm[p // page], p % page] = v_hist[p]
    kc, vc, pt = kc.cuda(), vc.cuda(), perm.cuda()
    hg = h.clone().cuda()
    binding.set_default_gemm(gemm)
    try:
        sc = binding.KernelScratch(cfg)
        lw = {k: v.cuda() for k, v in w["layers"][0].items()}
        binding.k_layer(cfg, lw, hg, kc, vc, pt, first_pos, sc)
        torch.cuda.synchronize()
    finally:
        binding.set_default_gemm(-1)
    m = h.shape[0]
    kn = torch.stack([kc[perm[p // page], p % page] for p in range(first_pos, first_pos + m)]).float().cpu().numpy()
    vn = torch.stack([vc[perm[p // page], p % page] for p in range(first_pos, first_pos + m)]).float().cpu().numpy()
    return hg.cpu().numpy(), kn, vn


def oracle_layer(shape, w, h, k_hist, v_hist, first_pos, max_seq):
    o = oracle.Oracle(shape, w, max_seq)
    for p in range(first_pos):
        o.set_kv(1, p, k_hist[p].double().numpy(), v_hist[p].double().numpy())
    out = o.layer_forward(1, h.double().numpy(), first_pos)
    kv = [o.get_kv(1, p) for p in range(first_pos, first_pos + h.shape[0])]
    return out, np.stack([k for k, _ in kv]), np.stack([v for _, v in kv])


@pytest.mark.parametrize("shape", [LAYER_F32, LAYER_BF16, LAYER_HD128], ids=lambda s: s.name)
def test_layer_matches_oracle(shape):
    w = inputs.make_weights(shape, 21, std=0.05)
    g = torch.Generator().manual_seed(1)
    for lw in w["layers"]:
        for k in ("attn_norm", "mlp_norm"):
            lw[k] = (1.0 + 0.2 * torch.randn(shape.d_model, generator=g)).to(lw[k].dtype)
    page, max_seq = 16, 160
    kvd = shape.n_kv_heads * shape.head_dim
    k_hist, v_hist = inputs.make_kv(max_seq, kvd, 31, shape.dtype)
    worst = 0.0
    cases = [(1, 0), (8, 0), (3, 1), (1, 15), (4, 14), (8, 16), (2, 17), (5, 100), (8, max_seq - 8)]
    for gemm in gemm_modes(shape):
        for m, first_pos in cases:
            h = inputs.make_hidden(m, shape.d_model, 7 * m + first_pos)
            got_h, got_k, got_v = run_layer(shape, w, h, k_hist, v_hist, first_pos, max_seq, page, gemm)
            ref_h, ref_k, ref_v = oracle_layer(shape, w, h, k_hist, v_hist, first_pos, max_seq)
            scale = np.abs(ref_h).max()
            err = np.abs(got_h - ref_h).max() / scale
            worst = max(worst, err)
            assert err < HIDDEN_TOL[shape.dtype], (gemm, m, first_pos, err)
            # appended cache rows: equal up to one rounding step of the storage type
            ulp = 2.0 ** -7 if shape.dtype == "bf16" else 2.0 ** -20
            for got, ref in ((got_k, ref_k), (got_v, ref_v)):
                assert np.all(np.abs(got - ref) <= ulp * np.abs(ref) + 1e-5), (gemm, m, first_pos)
    print(f"\n[{shape.name}] worst relative hidden error {worst:.3e}")


@pytest.mark.parametrize("shape", [LAYER_F32, LAYER_BF16], ids=lambda s: s.name)
def test_layer_rows_do_not_depend_on_companions(shape):
    """Row i of an m-row pass is bit-identical to the same row run alone once the earlier rows'
    K,V are in the cache -- what makes speculative and autoregressive decoding agree exactly."""
    w = inputs.make_weights(shape, 22, std=0.05)
    page, max_seq = 16, 96
    kvd = shape.n_kv_heads * shape.head_dim
    k_hist, v_hist = inputs.make_kv(max_seq, kvd, 32, shape.dtype)
    k_hist, v_hist = k_hist.clone(), v_hist.clone()
    for gemm in gemm_modes(shape):
        m, first_pos = 6, 37
        h = inputs.make_hidden(m, shape.d_model, 9)
        all_h, all_k, all_v = run_layer(shape, w, h, k_hist, v_hist, first_pos, max_seq, page, gemm)
        kh, vh = k_hist.clone(), v_hist.clone()
        dt = inputs.torch_dtype(shape.dtype)
        for i in range(m):
            one_h, one_k, one_v = run_layer(shape, w, h[i:i + 1], kh, vh, first_pos + i, max_seq, page, gemm)
            assert np.array_equal(one_h[0], all_h[i]), (gemm, i)
            assert np.array_equal(one_k[0], all_k[i]) and np.array_equal(one_v[0], all_v[i])
            kh[first_pos + i] = torch.from_numpy(one_k[0]).to(dt)
            vh[first_pos + i] = torch.from_numpy(one_v[0]).to(dt)


@pytest.mark.parametrize("shape", [LAYER_BF16, LAYER_HD128], ids=lambda s: s.name)
def test_layer_under_fusion_and_prefetch_options(shape):
    """The L2 prefetch of later weights (SB_OPT_L2_PREFETCH) and the one-launch attention (SB_OPT_FUSE
    bit 1: RoPE, cache append, attention and chunk merge in one kernel) do the same arithmetic in the same
    order as the separate kernels: bit-identical results.  SwiGLU in the gate/up GEMM's epilogue
    (SB_OPT_FUSE bit 0) runs that GEMM without a k split, so it may sum in another order than the separate
    kernels: equal to fp32 rounding, not bit for bit."""
    w = inputs.make_weights(shape, 24, std=0.05)
    page, max_seq = 16, 2200
    kvd = shape.n_kv_heads * shape.head_dim
    k_hist, v_hist = inputs.make_kv(max_seq, kvd, 33, shape.dtype)
    lib = binding.lib()
    outs = {}
    # (rows, first position): one chunk, a round that straddles a chunk boundary, 8 chunks, a round whose last rows
    # need a 9th chunk, 9 and 17 chunks (separate kernels either way)
    cases = ((1, 0), (5, 40), (8, 124), (8, 130), (3, 1000), (4, 1022), (2, 1090), (3, 2100))
    try:
        for fuse, prefetch in ((3, 4), (3, 0), (3, 1), (1, 4), (0, 0)):
            assert lib.sb_set_default_option(7, fuse) == 0 and lib.sb_set_default_option(5, prefetch) == 0
            outs[fuse, prefetch] = [run_layer(shape, w, inputs.make_hidden(m, shape.d_model, 3 + m), k_hist, v_hist, pos,
                                              max_seq, page, 1) for m, pos in cases]
    finally:
        lib.sb_set_default_option(7, 3)
        lib.sb_set_default_option(5, 4)
    for key in ((3, 0), (3, 1), (1, 4)):
        for a, b in zip(outs[3, 4], outs[key]):
            assert all(np.array_equal(x, y) for x, y in zip(a, b)), key
    for a, b in zip(outs[3, 4], outs[0, 0]):
        assert np.array_equal(a[1], b[1]) and np.array_equal(a[2], b[2])          # cache rows come before the MLP
        assert np.abs(a[0] - b[0]).max() <= 1e-5 * np.abs(b[0]).max()


@pytest.mark.parametrize("first_pos,m", [(40, 5), (1100, 3)])
def test_layer_chain_equals_single_layer_calls(first_pos, m):
    """sb_k_layer_chain (n layers in one launch sequence, optionally with the rotation-angle table of sb_k_rope_table) gives
    bit for bit what n successive sb_k_layer calls give: hidden rows and the K/V rows appended to every layer's cache."""
    shape = inputs.scaled(LAYER_HD128, name="chain-hd128", n_layers=3)
    w = inputs.make_weights(shape, 25, std=0.05)
    page, max_seq = 16, 1200
    kvd = shape.n_kv_heads * shape.head_dim
    cfg = binding.make_config(shape, max_seq, page)
    n_pages = (max_seq + page - 1) // page
    pt = torch.arange(n_pages, dtype=torch.int32, device="cuda")
    hist = [inputs.make_kv(max_seq, kvd, 40 + l, shape.dtype) for l in range(shape.n_layers)]
    assert n_pages * page == max_seq

    def caches():   # fresh per-layer caches holding the history
        return ([k.reshape(n_pages, page, kvd).clone().cuda() for k, _ in hist],
                [v.reshape(n_pages, page, kvd).clone().cuda() for _, v in hist])

    lws = [{k: v.cuda() for k, v in lw.items()} for lw in w["layers"]]
    h0 = inputs.make_hidden(m, shape.d_model, 91).cuda()
    binding.set_default_gemm(1)
    try:
        sc = binding.KernelScratch(cfg)
        kc1, vc1 = caches()
        h1 = h0.clone()
        for l in range(shape.n_layers):
            binding.k_layer(cfg, lws[l], h1, kc1[l], vc1[l], pt, first_pos, sc)
        torch.cuda.synchronize()
        tab = binding.k_rope_table(cfg)
        for table in (None, tab):
            kc2, vc2 = caches()
            h2 = h0.clone()
            binding.k_layer_chain(cfg, binding.LayerChain(lws, kc2, vc2), h2, pt, first_pos, sc, table)
            torch.cuda.synchronize()
            assert torch.equal(h1, h2)
            for l in range(shape.n_layers):
                assert torch.equal(kc1[l], kc2[l]) and torch.equal(vc1[l], vc2[l])
    finally:
        binding.set_default_gemm(-1)
    with pytest.raises(binding.SBError) as e:
        binding.k_layer_chain(cfg, binding.LayerChain(lws, kc2, vc2), h2, pt, max_seq - 1, sc, None)   # rows past max_seq
    assert e.value.status == -3


def test_layer_rejects_bad_arguments():
    shape = LAYER_BF16
    w = inputs.make_weights(shape, 23)
    cfg = binding.make_config(shape, 64, 16)
    sc = binding.KernelScratch(cfg)
    lw = {k: v.cuda() for k, v in w["layers"][0].items()}
    kvd = shape.n_kv_heads * shape.head_dim
    kc = torch.zeros((4, 16, kvd), dtype=torch.bfloat16, device="cuda")
    pt = torch.arange(4, dtype=torch.int32, device="cuda")
    h = torch.zeros((4, shape.d_model), device="cuda")
    with pytest.raises(binding.SBError) as e:
        binding.k_layer(cfg, lw, h, kc, kc.clone(), pt, 61, sc)       # 61 + 4 > max_seq
    assert e.value.status == -3
    with pytest.raises(binding.SBError) as e:
        binding.k_layer(cfg, lw, h, kc, kc.clone(), pt, -1, sc)
    assert e.value.status == -1
