"""Parity of sampling decoding (Section 4.3, "decoding strategies") on the GPU against the oracle.

What is unique is compared exactly: the uniform numbers, and -- on the GPU itself -- speculative
sampling against autoregressive sampling (bit-identical token sequences).  Against the fp64 oracle a
sampled token may differ only where the uniform number falls within the floating-point error of a
CDF interval edge; those cases are counted and their distance to the edge is checked."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2604_12247_b200 import binding, inputs
from gpu_util import gpu_ctx

pytestmark = pytest.mark.gpu


def f32(x):
    """The temperature as the C ABI receives it (a float), so that both sides divide by the same number."""
    return float(np.float32(x))


SMALL_BF16 = inputs.scaled(inputs.LLAMA3_8B, name="small-bf16", n_layers=4, d_model=512, n_heads=8, n_kv_heads=2,
                           head_dim=64, d_ffn=1408, vocab=2048, head_scale=16.0)


def _compare_with_oracle_samples(logits_cpu: np.ndarray, temperature, seed, pos0, gpu_tokens, edge_tol, top_p=1.0):
    """Row by row: equal tokens, or the oracle's uniform number lies within edge_tol of the edge between the two."""
    n_edge = 0
    for j, z in enumerate(logits_cpu):
        u = oracle.uniform(seed, pos0 + j)
        t, slack = oracle.sample_token(z.astype(np.float64), temperature, u, top_p)
        if t != gpu_tokens[j]:
            assert abs(int(gpu_tokens[j]) - t) >= 1 and slack < edge_tol, (j, t, int(gpu_tokens[j]), slack)
            # the GPU's token must be the neighbour across that edge (skipping tokens without mass)
            p = torch.softmax(torch.from_numpy(z.astype(np.float64)) / temperature, 0).numpy()
            lo, hi = sorted((t, int(gpu_tokens[j])))
            assert p[lo + 1:hi].sum() < edge_tol
            n_edge += 1
    return n_edge


@pytest.mark.parametrize("vocab", [1, 5, 127, 128, 129, 1000, 32000, 128256, 262144])
@pytest.mark.parametrize("temperature", [0.3, 1.0])
def test_sampling_kernel_matches_oracle(vocab, temperature):
    """Vocabulary sizes below one cell, at cell edges, ragged, at the two model sizes and at the maximum."""
    g = torch.Generator().manual_seed(vocab)
    m = 8
    z = torch.randn(m, vocab, generator=g) * 2.5
    z[1] *= 4.0                       # a peaked row
    z[2] = 0.0                        # a flat row: every interval has the same width
    if vocab > 4:
        z[3, : vocab // 2] = -200.0   # half the vocabulary without mass
    seed, pos0, temperature = 77, 1000, f32(temperature)
    tok = binding.k_sample(z.cuda(), temperature, seed, pos0).cpu().numpy()
    assert ((tok >= 0) & (tok < vocab)).all()
    # equal logits, fp64 on both sides: only the summation order differs
    n_edge = _compare_with_oracle_samples(z.numpy(), temperature, seed, pos0, tok, edge_tol=1e-10)
    assert n_edge == 0
    # same inputs, same tokens: the kernel is a pure function of (logits, u)
    assert np.array_equal(binding.k_sample(z.cuda(), temperature, seed, pos0).cpu().numpy(), tok)
    # rows are independent of their neighbours and of m
    one = binding.k_sample(z[5:6].contiguous().cuda(), temperature, seed, pos0 + 5).cpu().numpy()
    assert one[0] == tok[5]


@pytest.mark.parametrize("vocab", [1, 7, 128, 1000, 32000, 128256, 262144])
@pytest.mark.parametrize("temperature,top_p", [(1.0, 0.9), (0.3, 0.9), (1.0, 0.5), (2.0, 0.999), (1.0, 1e-6)])
def test_nucleus_sampling_kernel_matches_oracle(vocab, temperature, top_p):
    """top-p: the radix select must land on the oracle's logit threshold -- random rows, a peaked row, a flat row
    (every token tied: the whole vocabulary is the nucleus), rows with few distinct values (ties at the threshold
    enter together), signed zeros, half the vocabulary without mass."""
    g = torch.Generator().manual_seed(1000 + vocab)
    m = 8
    z = torch.randn(m, vocab, generator=g) * 2.5
    z[1] *= 4.0
    z[2] = 0.0
    if vocab > 4:
        z[3, : vocab // 2] = -200.0
        z[4] = torch.randint(-3, 4, (vocab,), generator=g).float()            # 7 distinct values, massive ties
        z[5] = torch.where(torch.rand(vocab, generator=g) < 0.5, 0.0, -0.0)   # +0 and -0 are one value
        z[6] = torch.round(z[6] * 4) / 4                                      # ties on a grid, negative and positive
    seed, pos0 = 31, 77
    temperature, top_p = f32(temperature), f32(top_p)
    tok = binding.k_sample(z.cuda(), temperature, seed, pos0, top_p=top_p).cpu().numpy()
    assert ((tok >= 0) & (tok < vocab)).all()
    for j in range(m):   # every token lies inside the oracle's nucleus
        zs = oracle.nucleus_threshold(z[j].double().numpy(), temperature, top_p)
        assert float(z[j, tok[j]]) >= zs, (j, tok[j], zs)
    assert _compare_with_oracle_samples(z.numpy(), temperature, seed, pos0, tok, edge_tol=1e-9, top_p=top_p) == 0
    assert np.array_equal(binding.k_sample(z.cuda(), temperature, seed, pos0, top_p=top_p).cpu().numpy(), tok)
    if top_p < 1e-3:     # the nucleus is the set of maxima
        assert all(float(z[j, tok[j]]) == float(z[j].max()) for j in range(m))


def test_sampling_kernel_frequencies_follow_softmax():
    g = torch.Generator().manual_seed(1)
    V, T, N = 200, 0.9, 4000
    z = (torch.randn(V, generator=g) * 2).repeat(8, 1).contiguous().cuda()
    counts = np.zeros(V)
    for k in range(N // 8):
        for t in binding.k_sample(z, T, 5, 8 * k).cpu().numpy():
            counts[t] += 1
    p = torch.softmax(z[0].double().cpu() / T, 0).numpy()
    big = p * N >= 5
    chi2 = (((counts - p * N) ** 2) / (p * N))[big].sum()
    dof = int(big.sum())
    assert chi2 < dof + 5 * np.sqrt(2 * dof), (chi2, dof)


def test_sampling_argument_errors(tiny_weights):
    run = inputs.RUNS["tiny"]
    ctx, _ = gpu_ctx(run.shape, tiny_weights, 64)
    for bad in (-1.0, float("nan")):
        with pytest.raises(binding.SBError):
            ctx.set_sampling(bad, 0)
    for bad_p in (0.0, -0.5, 1.5, float("nan")):
        with pytest.raises(binding.SBError):
            ctx.set_sampling(1.0, 0, top_p=bad_p)
        with pytest.raises(binding.SBError):
            binding.k_sample(torch.zeros(2, 10, device="cuda"), 1.0, 0, 0, top_p=bad_p)
    z = torch.zeros(2, 10, device="cuda")
    with pytest.raises(binding.SBError):
        binding.k_sample(z, 0.0, 0, 0)
    with pytest.raises(binding.SBError):
        binding.k_sample(torch.zeros(9, 10, device="cuda"), 1.0, 0, 0)
    ctx.close()


@pytest.mark.parametrize("which", ["tiny", "tiny-damped"])
def test_tiny_sampled_generation_matches_oracle_and_ar(which, tiny_weights, tiny_damped_weights):
    run = inputs.RUNS[which]
    w = tiny_weights if which == "tiny" else tiny_damped_weights
    pr = inputs.make_prompt(run.shape, run.n_prompt, run.seed).numpy()
    n_gen, max_seq = 24, 64
    ctx, _ = gpu_ctx(run.shape, w, max_seq)
    greedy = ctx.generate_ar(pr, n_gen)["tokens"]
    accepted = {}
    for T, seed, top_p in ((f32(0.3), 1, 1.0), (1.0, 2, 1.0), (1.0, 3, 1.0), (1.0, 3, f32(0.9)), (f32(1.5), 4, 0.5)):
        o = oracle.Oracle(run.shape, w, max_seq)
        o.set_sampling(T, seed, top_p)
        ref, slack = o.ar_generate(pr, n_gen, want_margins=True)
        ctx.set_sampling(T, seed, top_p)
        ar = ctx.generate_ar(pr, n_gen)["tokens"]
        # fp32 model: logits agree to ~1e-6, so a token can differ only within that of a CDF edge
        diff = np.nonzero(ar != ref)[0]
        if len(diff):
            assert slack[diff[0]] < 1e-5, (T, seed, diff[0], slack[diff[0]])
        else:
            assert np.array_equal(ar, ref)
        accepted[(T, seed)] = accepted.get((T, seed), 0)
        for d_max, w_max, thr in ((1, 8, 0.0), (2, 4, 0.25), (3, 3, 0.2), (3, 8, 2.0)):
            tau = inputs.tau_linear(d_max, 1.5, 1.0)
            res = ctx.generate(pr, n_gen, d_max, w_max, tau, thr, trace=True)
            assert np.array_equal(res["tokens"], ar), (T, seed, d_max, w_max, thr)     # lossless, sample by sample
            accepted[(T, seed)] += res["stats"].accepted_drafts
            if not len(diff):
                o2 = oracle.Oracle(run.shape, w, max_seq)
                o2.set_sampling(T, seed, top_p)
                _, rounds = o2.specbound_generate(pr, n_gen, d_max, w_max, tau, thr)
                assert [(r.w, r.emitted, r.accepted_drafts) for r in res["rounds"]] == \
                       [(r.w, r.emitted, r.accepted_drafts) for r in rounds]
    assert not np.array_equal(ar, greedy)
    ctx.set_sampling(1.0, 3, 1e-6)
    assert np.array_equal(ctx.generate_ar(pr, n_gen)["tokens"], greedy)                # top_p -> 0: the top-1 alone
    ctx.set_sampling(0.0, 0)
    assert np.array_equal(ctx.generate_ar(pr, n_gen)["tokens"], greedy)                # switching back restores greedy
    ctx.set_sampling(1e-4, 9)
    assert np.array_equal(ctx.generate_ar(pr, n_gen)["tokens"], greedy)                # T -> 0 limit
    ctx.close()
    if which == "tiny-damped":
        assert accepted[(f32(0.3), 1)] > 0


def test_bf16_sampled_speculative_equals_ar_and_oracle_edges():
    """bf16 GQA model with damped deep layers, both GEMM back ends: speculative sampling is bit-identical to
    autoregressive sampling; teacher-forced against the oracle, every sampled token is the oracle's sample or
    sits across a CDF edge that the bf16 logit tolerance can move past u."""
    from gpu_util import gemm_modes, LOGIT_TOL
    shape = SMALL_BF16
    w = inputs.make_weights(shape, 5, damp_rho=0.3)
    pr = inputs.make_prompt(shape, 20, 5).numpy()
    n_gen, max_seq, T, seed = 40, 96, f32(0.7), 4
    for gemm in gemm_modes(shape):
        ctx, _ = gpu_ctx(shape, w, max_seq, gemm=gemm)
        ctx.set_sampling(T, seed)
        ar = ctx.generate_ar(pr, n_gen)["tokens"]
        acc = 0
        for d_max, w_max, thr in ((2, 4, 0.3), (3, 8, 0.2), (1, 6, 0.0)):
            res = ctx.generate(pr, n_gen, d_max, w_max, inputs.tau_linear(d_max, 1.5, 1.0), thr)
            assert np.array_equal(res["tokens"], ar), (gemm, d_max, w_max)
            acc += res["stats"].accepted_drafts
        assert acc > 0
        # teacher-forced oracle logits along the GPU's own sequence
        seq = np.concatenate([pr, ar]).astype(np.int32)
        o = oracle.Oracle(shape, w, max_seq)
        h = np.stack([o.embed(int(t)) for t in seq[:-1]])
        for l in range(1, shape.n_layers + 1):
            h = o.layer_forward(l, h, 0)
        z = np.stack([o.final_logits(h[len(pr) - 1 + i]) for i in range(n_gen)])
        # a logit error of eps moves a CDF edge by at most ~eps / T (relative mass), summed over both sides
        n_edge = _compare_with_oracle_samples(z, T, seed, len(pr), ar, edge_tol=4 * LOGIT_TOL["bf16"] / T)
        print(f"\n[gemm={gemm}] sampled tokens across a CDF edge from the oracle's: {n_edge} of {n_gen}")
        assert n_edge <= n_gen // 4
        ctx.close()


def test_7b_damped_sampled_run_equals_ar():
    """Bench shape (V = 32000, tcgen05 head with the logits written for the sampler): speculative sampling
    equals autoregressive sampling, and drafts are still accepted at T = 0.3."""
    run = inputs.RUNS["7b-damped"]
    wg = inputs.make_weights(run.shape, run.seed, device="cuda", damp_rho=run.damp_rho)
    pr = inputs.make_prompt(run.shape, 24, run.seed).numpy()
    n_gen = 32
    ctx = binding.Context(run.shape, wg, 96, kv_page=64)
    greedy = ctx.generate_ar(pr, n_gen)["tokens"]
    for T, top_p in ((0.3, 1.0), (1.0, 1.0), (1.0, 0.9)):
        ctx.set_sampling(T, 123, top_p)
        ar = ctx.generate_ar(pr, n_gen)["tokens"]
        sp = ctx.generate(pr, n_gen, run.d_max, run.w_max, run.tau, run.threshold)
        assert np.array_equal(sp["tokens"], ar), (T, top_p)
        print(f"\n[7b-damped T={T} top_p={top_p}] accepted drafts {sp['stats'].accepted_drafts}, rounds {sp['stats'].rounds}, "
              f"differs from greedy at {int((ar != greedy).sum())} of {n_gen}")
        if T == 0.3:
            assert sp["stats"].accepted_drafts > 0
    ctx.close()
