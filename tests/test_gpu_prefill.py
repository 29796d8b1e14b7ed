"""Wide prefill passes (up to 128 prompt rows per launch of the weight-streaming GEMMs) against the 8-row passes and the
oracle.  What prefill leaves behind is the K/V cache of every layer and the first generated token; both are checked
through what is computed from them: the first token, the hidden state of that token after every layer (it attends
over all cached prompt positions of each layer), and the tokens decoded afterwards."""
import numpy as np
import pytest

from oracle import oracle
from paper_2604_12247_b200 import binding, inputs
from gpu_util import gpu_ctx, near_tie_count, HIDDEN_TOL, LOGIT_TOL

pytestmark = pytest.mark.gpu

SMALL_BF16 = inputs.scaled(inputs.LLAMA3_8B, name="small-bf16", n_layers=4, d_model=512, n_heads=8, n_kv_heads=2,
                           head_dim=64, d_ffn=1408, vocab=2048, head_scale=16.0)
# the same with an FFN width that is not a multiple of the GEMMs' 64-wide k block (the down projection's last k block
# is filled up with zeros by the tensor-map's out-of-range rule) nor of the widest tile
ODD_FFN_BF16 = inputs.scaled(SMALL_BF16, name="small-bf16-odd-ffn", d_ffn=1416)
OPT_WIDE_PREFILL = 9


def _hidden_after_prefill(ctx, prompt, n_layers):
    """First token, and its hidden state after every layer (one row pushed and advanced through the whole stack)."""
    first = ctx.prefill(prompt)
    ctx.draft_push(first)
    hid = []
    for l in range(1, n_layers + 1):
        ctx.draft_advance(l)
        hid.append(ctx.read_hidden(0).astype(np.float64))
    return first, hid


# 16: the smallest wide pass; 64, 70, 100: one ragged wide pass (70 and 100 end in a partial block of 8 rows); 128: a
# whole pass; 130: a whole pass + 2 rows through an 8-row pass; 300: two whole passes and a ragged one.  Page size 16
# wide_mode 1: wide GEMMs on CTA pairs + the tiled tensor-core attention kernel (the default); 2: the decode attention
# kernels; 3: as 1 with the wide GEMMs on single CTAs
@pytest.mark.parametrize("wide_mode", [1, 2, 3])
@pytest.mark.parametrize("n_prompt", [16, 64, 70, 100, 128, 130, 300])
def test_wide_prefill_matches_narrow_passes_and_oracle(n_prompt, wide_mode):
    _wide_against_narrow_and_oracle(SMALL_BF16, n_prompt, wide_mode)


@pytest.mark.parametrize("n_prompt", [70, 130])
def test_wide_prefill_with_a_ragged_last_k_block(n_prompt):
    _wide_against_narrow_and_oracle(ODD_FFN_BF16, n_prompt, 1)


def _wide_against_narrow_and_oracle(shape, n_prompt, wide_mode):
    w = inputs.make_weights(shape, 5, damp_rho=0.3)
    pr = inputs.make_prompt(shape, n_prompt, 17).numpy()
    max_seq = n_prompt + 24
    L = shape.n_layers
    assert binding.lib().sb_set_default_option(OPT_WIDE_PREFILL, 0) == 0
    try:
        ctx_n, _ = gpu_ctx(shape, w, max_seq, gemm=1)
        first_n, hid_n = _hidden_after_prefill(ctx_n, pr, L)
        launches_n = ctx_n.generate_ar(pr, 12)["stats"].kernel_launches
        ar_n = ctx_n.generate_ar(pr, 12)["tokens"]
        ctx_n.close()
    finally:
        assert binding.lib().sb_set_default_option(OPT_WIDE_PREFILL, wide_mode) == 0
    try:
        ctx, _ = gpu_ctx(shape, w, max_seq, gemm=1)
        first, hid = _hidden_after_prefill(ctx, pr, L)
        res = ctx.generate_ar(pr, 12)
        sp = ctx.generate(pr, 12, 2, 4, inputs.tau_linear(2, 1.5, 1.0), 0.3)
    finally:
        assert binding.lib().sb_set_default_option(OPT_WIDE_PREFILL, 1) == 0
    ar = res["tokens"]
    assert res["stats"].kernel_launches < launches_n          # the wide passes really ran
    # against the 8-row passes: the same arithmetic up to the split-K summation order
    assert first == first_n
    for l in range(L):
        assert np.abs(hid[l] - hid_n[l]).max() / np.abs(hid_n[l]).max() < 1e-4, l
    # against the oracle: the first token's hidden state after every layer (attention over the whole cached prompt)
    o = oracle.Oracle(shape, w, max_seq)
    o.ar_generate(pr, 1)                                     # fills the oracle's cache with the prompt
    h = o.embed(first)[None, :]
    for l in range(1, L + 1):
        h = o.layer_forward(l, h, n_prompt)
        err = np.abs(hid[l - 1] - h[0]).max() / np.abs(h[0]).max()
        assert err < HIDDEN_TOL["bf16"], (l, err)
    # decoding from the wide-prefilled cache: every token is the oracle's top-1 or within the logit tolerance of it
    n_off, worst = near_tie_count(shape, w, pr, ar, LOGIT_TOL["bf16"])
    assert worst > -2 * LOGIT_TOL["bf16"]
    if n_off == 0:
        assert np.array_equal(ar, ar_n)
    # speculative decoding from the same cache equals autoregressive decoding, bit for bit
    assert np.array_equal(sp["tokens"], ar)
    ctx.close()


def test_wide_prefill_at_the_bench_shape_matches_narrow_first_token_and_tokens():
    """7B shape, 200-token prompt (a whole wide pass + a ragged one of 72 rows): same first token and decoded tokens as the
    8-row passes (which the 7B-shape run tests compare with the oracle), in well under their time.  The wide passes
    themselves are compared with the oracle on the small model above and, at the 7B attention geometry with a 512-token
    prompt, by test_bench_lengths_on_7b_attention_geometry_match_oracle."""
    run = inputs.RUNS["7b-damped"]
    wg = inputs.make_weights(run.shape, run.seed, device="cuda", damp_rho=run.damp_rho)
    pr = inputs.make_prompt(run.shape, 200, run.seed).numpy()
    n_gen = 8
    assert binding.lib().sb_set_default_option(OPT_WIDE_PREFILL, 0) == 0
    try:
        ctx_n = binding.Context(run.shape, wg, 256, kv_page=64)
        out_n = ctx_n.generate_ar(pr, n_gen)
        ctx_n.close()
    finally:
        assert binding.lib().sb_set_default_option(OPT_WIDE_PREFILL, 1) == 0
    ctx = binding.Context(run.shape, wg, 256, kv_page=64)
    out = ctx.generate_ar(pr, n_gen)
    print(f"\n[7b, 200-token prompt] prefill {out_n['stats'].us_prefill / 1e3:.1f} ms in 8-row passes, "
          f"{out['stats'].us_prefill / 1e3:.1f} ms in wide passes")
    assert out["stats"].us_prefill < 0.6 * out_n["stats"].us_prefill
    assert np.array_equal(out["tokens"], out_n["tokens"])
    ctx.close()
