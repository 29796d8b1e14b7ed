"""Pins of the oracle's decoder: each block against torch CPU library routines (rms_norm, linear,
scaled_dot_product_attention, silu; RoPE written as a complex rotation), the KV-cached forward
against a no-cache brute force, and the bf16 storage handling against torch's own casts."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import oracle
from paper_2604_12247_b200 import inputs

GQA = inputs.scaled(inputs.TINY, name="tiny-gqa", n_layers=2, d_model=128, n_heads=8, n_kv_heads=2, head_dim=16,
                    d_ffn=200, vocab=300, rope_base=500000.0)


def torch_rope(x, pos, base):
    """x: [n, heads, hd]; rotate-half pairing as a complex multiplication."""
    n, h, hd = x.shape
    half = hd // 2
    inv = base ** (-torch.arange(half, dtype=torch.float64) * 2.0 / hd)
    ang = pos.to(torch.float64)[:, None] * inv[None, :]
    rot = torch.polar(torch.ones_like(ang), ang)[:, None, :]
    z = torch.complex(x[..., :half], x[..., half:]) * rot
    return torch.cat([z.real, z.imag], dim=-1)


def torch_forward(shape, w, tokens):
    """Whole-sequence forward with library routines in fp64; returns per-layer hidden states
    ([L+1] list of [n, d]) and final logits [n, V]."""
    W = lambda t: t.to(torch.float64)
    n = len(tokens)
    x = W(w["embed"])[torch.as_tensor(tokens, dtype=torch.long)]
    pos = torch.arange(n)
    H, Hkv, hd = shape.n_heads, shape.n_kv_heads, shape.head_dim
    hs = [x.clone()]
    for lw in w["layers"]:
        a = F.rms_norm(x, (shape.d_model,), W(lw["attn_norm"]), shape.rms_eps)
        q = torch_rope(F.linear(a, W(lw["wq"])).view(n, H, hd), pos, shape.rope_base)
        k = torch_rope(F.linear(a, W(lw["wk"])).view(n, Hkv, hd), pos, shape.rope_base)
        v = F.linear(a, W(lw["wv"])).view(n, Hkv, hd)
        k = k.repeat_interleave(H // Hkv, dim=1)
        v = v.repeat_interleave(H // Hkv, dim=1)
        o = F.scaled_dot_product_attention(q.transpose(0, 1)[None], k.transpose(0, 1)[None], v.transpose(0, 1)[None],
                                           is_causal=True)[0].transpose(0, 1).reshape(n, H * hd)
        x = x + F.linear(o, W(lw["wo"]))
        m = F.rms_norm(x, (shape.d_model,), W(lw["mlp_norm"]), shape.rms_eps)
        x = x + F.linear(F.silu(F.linear(m, W(lw["w_gate"]))) * F.linear(m, W(lw["w_up"])), W(lw["w_down"]))
        hs.append(x.clone())
    z = F.linear(F.rms_norm(x, (shape.d_model,), W(w["final_norm"]), shape.rms_eps), W(w["lm_head"]))
    return hs, z


def perturbed_gains(w, seed=5):
    """Non-trivial norm gains so that a dropped or misplaced gain would show."""
    g = torch.Generator().manual_seed(seed)
    for lw in w["layers"]:
        for k in ("attn_norm", "mlp_norm"):
            lw[k] = (1.0 + 0.3 * torch.randn(lw[k].shape, generator=g)).to(lw[k].dtype)
    w["final_norm"] = (1.0 + 0.3 * torch.randn(w["final_norm"].shape, generator=g)).to(w["final_norm"].dtype)
    return w


@pytest.mark.parametrize("shape", [inputs.TINY, GQA, inputs.scaled(GQA, name="gqa-bf16", dtype="bf16")], ids=lambda s: s.name)
def test_layers_and_head_match_torch_library(shape):
    w = perturbed_gains(inputs.make_weights(shape, 3))
    toks = inputs.make_prompt(shape, 11, 3).tolist()
    hs, z = torch_forward(shape, w, toks)
    o = oracle.Oracle(shape, w, 32, kv_round_bf16=False)
    h = np.stack([o.embed(t) for t in toks])
    assert np.array_equal(h, hs[0].numpy())
    # layer by layer, rows fed in uneven batches so that later rows read earlier rows' cache
    for l in range(1, shape.n_layers + 1):
        h = np.concatenate([o.layer_forward(l, h[:4], 0), o.layer_forward(l, h[4:5], 4), o.layer_forward(l, h[5:], 5)])
        np.testing.assert_allclose(h, hs[l].numpy(), rtol=1e-10, atol=1e-12)
    for i in (0, 5, 10):
        np.testing.assert_allclose(o.final_logits(h[i]), z[i].numpy(), rtol=1e-10, atol=1e-11)
        p, t, zz = o.exit_confidence(h[i], 1.3, want_logits=True)
        ref = torch.softmax(z[i] / 1.3, dim=0)
        assert t == int(ref.argmax()) and p == pytest.approx(float(ref.max()), rel=1e-10)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_per_layer_exit_head_matches_torch_library(dtype):
    """Exit test with a layer's own head and norm gain (Section 3.2): equals torch's rms_norm -> linear ->
    softmax(z / T).max() with THAT layer's tensors, and falls back to the shared head where none is set."""
    shape = inputs.scaled(GQA, name="gqa-heads", dtype=dtype)
    w = inputs.add_exit_heads(perturbed_gains(inputs.make_weights(shape, 5)), shape, seed=2)
    w["exit_head"][1] = None      # layer 2 keeps the shared head but has its own norm gain
    o = oracle.Oracle(shape, w, 8)
    h = torch.randn(shape.d_model, dtype=torch.float64, generator=torch.Generator().manual_seed(4))
    for l in range(1, shape.n_layers + 1):
        head = w["exit_head"][l - 1] if w["exit_head"][l - 1] is not None else w["lm_head"]
        gain = w["exit_norm"][l - 1]
        x = torch.nn.functional.rms_norm(h, (shape.d_model,), gain.double(), shape.rms_eps)
        ref = torch.softmax(torch.nn.functional.linear(x, head.double()) / 1.7, dim=0)
        p, t = o.exit_confidence_at(l, h.numpy(), 1.7)
        assert t == int(ref.argmax()) and p == pytest.approx(float(ref.max()), rel=1e-10)
    o.set_exit_head(1, None, None)
    p_shared, t_shared = o.exit_confidence(h.numpy(), 1.7)
    assert o.exit_confidence_at(1, h.numpy(), 1.7) == (p_shared, t_shared)


def test_rope_properties():
    """Position 0 is the identity; q.k after rotation depends only on the position difference."""
    shape = inputs.scaled(GQA, n_layers=1)
    w = inputs.make_weights(shape, 1)
    o = oracle.Oracle(shape, w, 64, kv_round_bf16=False)
    hs, _ = torch_forward(shape, w, [5])
    np.testing.assert_allclose(o.layer_forward(1, o.embed(5)[None], 0), hs[1].numpy(), rtol=1e-10, atol=1e-13)
    # same single token at position 0 and at position 37 with an empty past: only itself to attend
    # to, so softmax = 1 and the output must not depend on the position at all.
    o2 = oracle.Oracle(shape, w, 64, kv_round_bf16=False)
    h0 = o2.layer_forward(1, o2.embed(5)[None], 0)
    k0, v0 = o2.get_kv(1, 0)
    # relative-position invariance on the cached keys: rotate the same key to two positions
    x = torch.from_numpy(k0).view(1, shape.n_kv_heads, shape.head_dim)
    a = torch_rope(x, torch.tensor([3]), shape.rope_base)
    b = torch_rope(x, torch.tensor([10]), shape.rope_base)
    c = torch_rope(x, torch.tensor([13]), shape.rope_base)
    d = torch_rope(x, torch.tensor([20]), shape.rope_base)
    assert float((a * b).sum()) == pytest.approx(float((c * d).sum()), rel=1e-9)
    assert np.isfinite(h0).all()


@pytest.mark.parametrize("shape", [inputs.TINY, GQA], ids=lambda s: s.name)
def test_cached_ar_equals_no_cache_bruteforce(shape):
    w = inputs.make_weights(shape, 0)
    pr = inputs.make_prompt(shape, 6, 0).numpy()
    o = oracle.Oracle(shape, w, 64)
    ar = o.ar_generate(pr, 10)
    bf = oracle.Oracle(shape, w, 64).bruteforce_generate(pr, 10)
    assert np.array_equal(ar, bf)
    # and the library forward predicts the same greedy continuation
    _, z = torch_forward(shape, w, list(pr) + list(ar[:-1]))
    assert np.array_equal(z[len(pr) - 1:].argmax(dim=1).numpy(), ar)


def test_teacher_forced_reports_margins(tiny_weights):
    shape = inputs.TINY
    pr = inputs.make_prompt(shape, 8, 0).numpy()
    o = oracle.Oracle(shape, tiny_weights, 64)
    ar, mg = o.ar_generate(pr, 6, want_margins=True)
    toks = np.concatenate([pr, ar])
    t1, t2, margin, deficit = oracle.Oracle(shape, tiny_weights, 64).teacher_forced(toks, len(pr))
    assert np.array_equal(t1, ar) and np.allclose(margin, mg) and np.all(deficit == 0) and np.all(margin > 0)
    _, z = torch_forward(shape, tiny_weights, toks.tolist())
    top2 = z[len(pr) - 1:-1].topk(2, dim=1)
    assert np.array_equal(top2.indices[:, 1].numpy(), t2)
    np.testing.assert_allclose(margin, (top2.values[:, 0] - top2.values[:, 1]).numpy(), rtol=1e-8)
    # a wrong token shows up as a negative deficit
    bad = toks.copy()
    bad[len(pr) + 2] = (bad[len(pr) + 2] + 1) % shape.vocab
    _, _, _, d2 = oracle.Oracle(shape, tiny_weights, 64).teacher_forced(bad, len(pr))
    assert d2[2] < 0


def test_bf16_cache_rounding_matches_torch_cast():
    shape = inputs.scaled(GQA, name="gqa-bf16", dtype="bf16", n_layers=1)
    w = inputs.make_weights(shape, 2)
    exact = oracle.Oracle(shape, w, 16, kv_round_bf16=False)
    rounded = oracle.Oracle(shape, w, 16, kv_round_bf16=True)
    h = np.stack([exact.embed(t) for t in (1, 2, 3)])
    exact.layer_forward(1, h, 0)
    rounded.layer_forward(1, h, 0)
    for p in range(3):
        ke, ve = exact.get_kv(1, p)
        kr, vr = rounded.get_kv(1, p)
        for e, r in ((ke, kr), (ve, vr)):
            want = torch.from_numpy(e).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
            assert np.array_equal(r, want)
