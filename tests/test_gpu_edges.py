"""Edge cases of the CUDA decode path against the oracle: shortest and ragged inputs, exact capacity,
KV-page boundaries inside a round, widest rounds, full acceptance through the primitives."""
import numpy as np
import pytest

from oracle import oracle
from paper_2604_12247_b200 import binding, inputs
from gpu_util import gemm_modes, gpu_ctx

pytestmark = pytest.mark.gpu

SMALL_BF16 = inputs.scaled(inputs.LLAMA3_8B, name="small-bf16", n_layers=4, d_model=512, n_heads=8, n_kv_heads=2,
                           head_dim=64, d_ffn=1408, vocab=2048, head_scale=16.0)


def _models(tiny_damped_weights):
    yield inputs.RUNS["tiny-damped"].shape, tiny_damped_weights
    yield SMALL_BF16, inputs.make_weights(SMALL_BF16, 5, damp_rho=0.3)


def test_shortest_and_ragged_inputs(tiny_damped_weights):
    for shape, w in _models(tiny_damped_weights):
        for gemm in gemm_modes(shape):
            # (prompt length, generated tokens): one-token prompt, one generated token (prefill only),
            # prompt lengths around the 8-row prefill chunk
            for n_prompt, n_gen in ((1, 1), (1, 9), (7, 5), (8, 5), (9, 5), (17, 3)):
                pr = inputs.make_prompt(shape, n_prompt, 3).numpy()
                max_seq = n_prompt + n_gen + 8          # exactly the capacity a w_max = 8 run needs
                ctx, _ = gpu_ctx(shape, w, max_seq, kv_page=16, gemm=gemm)
                ar = ctx.generate_ar(pr, n_gen)["tokens"]
                sp = ctx.generate(pr, n_gen, 2, 8, (1.5, 1.0), 0.2, trace=True)
                assert np.array_equal(sp["tokens"], ar), (shape.name, gemm, n_prompt, n_gen)
                assert len(sp["tokens"]) == n_gen
                assert sum(r.emitted for r in sp["rounds"]) == n_gen - 1
                if shape.dtype == "f32":
                    ref = oracle.Oracle(shape, w, max_seq).ar_generate(pr, n_gen)
                    assert np.array_equal(ar, ref)
                with pytest.raises(binding.SBError) as e:   # one token more does not fit
                    ctx.generate(pr, n_gen + 1, 2, 8, (1.5, 1.0), 0.2)
                assert e.value.status == -3
                ctx.close()


def test_rounds_that_cross_kv_page_boundaries(tiny_damped_weights):
    """16-position pages; prompts placed so that rounds of up to 8 rows straddle a page boundary."""
    run = inputs.RUNS["tiny-damped"]
    for n_prompt in (13, 14, 15, 16, 29, 31):
        pr = inputs.make_prompt(run.shape, n_prompt, 11).numpy()
        ref = oracle.Oracle(run.shape, tiny_damped_weights, 96).ar_generate(pr, 20)
        ctx, _ = gpu_ctx(run.shape, tiny_damped_weights, 96, kv_page=16)
        res = ctx.generate(pr, 20, 2, 8, (1.5, 1.0), 0.0, trace=True)   # threshold 0: every round is 8 rows wide
        assert np.array_equal(res["tokens"], ref), n_prompt
        assert all(r.w == 8 for r in res["rounds"][:-1])
        ctx.close()


def test_full_width_acceptance_through_the_primitives(tiny_damped_weights):
    """Drafts equal to what the full model will say are all accepted: the round emits w tokens, the
    last draft becomes the pending token and no bonus token is produced."""
    run = inputs.RUNS["tiny-damped"]
    shape = run.shape
    pr = inputs.make_prompt(shape, 10, 2).numpy()
    ref = oracle.Oracle(shape, tiny_damped_weights, 64).ar_generate(pr, 12)
    ctx, _ = gpu_ctx(shape, tiny_damped_weights, 64)
    first = ctx.prefill(pr)
    assert first == ref[0]
    w = 8
    # feed the true continuation as inputs, stopping each row after one shallow layer
    for i in range(w):
        ctx.draft_push(int(ref[i]))
        ctx.draft_advance(1)
    st = ctx.state()
    assert st.rows == w and list(st.depth[:w]) == [1] * w
    out = ctx.verify([int(t) for t in ref[1:w + 1]])          # row i drafted ref[i+1]
    assert list(out) == [int(t) for t in ref[1:w + 1]]
    st = ctx.state()
    assert st.rows == 0 and st.n == len(pr) + w and st.pending == ref[w]
    # and a wrong draft in the middle cuts the round there, replaced by the model's token
    ctx.reset()
    ctx.prefill(pr)
    for i in range(4):
        ctx.draft_push(int(ref[i]))
        ctx.draft_advance(2)
    wrong = [int(ref[1]), int((ref[2] + 1) % shape.vocab), int(ref[3]), int(ref[4])]
    out = ctx.verify(wrong)
    assert list(out) == [int(ref[1]), int(ref[2])]
    assert ctx.state().n == len(pr) + 2 and ctx.state().pending == ref[2]
    ctx.close()


def test_context_reuse_across_sequences(tiny_damped_weights):
    """One context, several sequences: stale KV of a longer earlier sequence must never leak."""
    run = inputs.RUNS["tiny-damped"]
    ctx, _ = gpu_ctx(run.shape, tiny_damped_weights, 96)
    for seed, n_prompt, n_gen in ((1, 40, 30), (2, 5, 12), (3, 21, 17)):
        pr = inputs.make_prompt(run.shape, n_prompt, seed).numpy()
        ref = oracle.Oracle(run.shape, tiny_damped_weights, 96).ar_generate(pr, n_gen)
        assert np.array_equal(ctx.generate(pr, n_gen, 2, 4, (1.5, 1.0), 0.3)["tokens"], ref)
        assert np.array_equal(ctx.generate_ar(pr, n_gen)["tokens"], ref)
    ctx.close()


def test_bounded_device_wait_runs_out_and_context_survives(tiny_damped_weights):
    """Failure detection without a GPU fault: a wait on a barrier that nothing completes gives up
    after its budget, the kernel returns, the call reports SB_ERR_DEVICE_TIMEOUT, later calls keep
    reporting it until sb_reset, and the context then works as before."""
    run = inputs.RUNS["tiny-damped"]
    pr = inputs.make_prompt(run.shape, 6, 4).numpy()
    ctx, _ = gpu_ctx(run.shape, tiny_damped_weights, 48)
    ref = ctx.generate_ar(pr, 6)["tokens"]
    assert ctx.selftest_wait_timeout(20) == -5
    ctx.draft_push(1)                                # launches only; the next call that reads a result sees the status
    ctx.draft_advance(1)
    with pytest.raises(binding.SBError) as e:        # the status word is sticky until the sequence is reset
        ctx.exit_confidence(1, 1.0, 0.5)
    assert e.value.status == -5
    ctx.reset()
    assert np.array_equal(ctx.generate_ar(pr, 6)["tokens"], ref)
    ctx.close()
