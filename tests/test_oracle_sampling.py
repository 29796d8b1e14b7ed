"""Pins of the oracle's sampling decoding (Section 4.3, "decoding strategies"; Table 2).

The paper names temperature sampling but prints no acceptance rule, so what is pinned here is
the reading the oracle states: the token at position p is the inverse-CDF sample of
softmax(z / T_s) at a counter-based uniform u(seed, p); a draft is accepted iff it equals it.

* the generator against the published splitmix64 output stream,
* the inverse-CDF sampler against a library softmax by stratified counting (a wrong
  temperature, a dropped max-shift, a reversed scan or an off-by-one interval edge fails),
* the T_s -> 0 limit (greedy) and the T_s -> infinity limit (uniform),
* sampling really is autoregressive sampling from the model: each generated token equals the
  sampler applied to logits recomputed by the no-cache brute-force path,
* speculative == autoregressive, token for token, over a (d_max, w_max, threshold, T_s) grid,
* the empirical frequency of the first generated token over many seeds against its softmax,
* top-p: the nucleus against a library sort + cumulative sum, ties entering together, the
  renormalised counts inside the nucleus, the top_p -> 1 and top_p -> 0 limits, and
  speculative == autoregressive under nucleus sampling.
"""
import itertools

import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2604_12247_b200 import inputs

# first outputs of splitmix64 seeded with 0 (Steele, Lea & Flood 2014; the reference
# implementation's well-known test vector)
SPLITMIX64_SEED0 = [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F, 0xF88BB8A8724C81EC]


def test_generator_reproduces_published_splitmix64_stream():
    assert [oracle.mix64(0, p) for p in range(4)] == SPLITMIX64_SEED0


def test_uniforms_are_open_interval_well_spread_and_keyed_by_seed_and_position():
    u = np.array([[oracle.uniform(s, p) for p in range(2000)] for s in (0, 1, 12345)])
    assert (u > 0).all() and (u < 1).all()
    assert abs(u.mean() - 0.5) < 0.01 and abs(u.var() - 1 / 12) < 0.005
    assert len(np.unique(u)) == u.size
    # the top 53 bits of the hash, centred in their cell
    assert oracle.uniform(0, 0) == ((SPLITMIX64_SEED0[0] >> 11) + 0.5) / 2.0 ** 53
    # lag-1 correlation along positions and across seeds is noise
    assert abs(np.corrcoef(u[0, :-1], u[0, 1:])[0, 1]) < 0.06
    assert abs(np.corrcoef(u[0], u[1])[0, 1]) < 0.06


@pytest.mark.parametrize("temperature", [0.3, 1.0, 2.5])
def test_inverse_cdf_counts_match_library_softmax(temperature):
    g = torch.Generator().manual_seed(7)
    z = (torch.randn(37, generator=g, dtype=torch.float64) * 3).numpy()
    p = torch.softmax(torch.from_numpy(z) / temperature, 0).numpy()
    N = 20000
    counts = np.zeros(z.size, dtype=np.int64)
    prev = -1
    for k in range(N):
        t, slack = oracle.sample_token(z, temperature, (k + 0.5) / N)
        assert t >= prev and slack >= 0        # monotone in u: the CDF is scanned in vocabulary order
        prev = t
        counts[t] += 1
    # a stratified grid of N points puts p_v * N +- 1 of them into token v's CDF interval
    assert np.abs(counts - p * N).max() <= 1.0 + 1e-6
    # interval edges: just below / above the first boundary
    assert oracle.sample_token(z, temperature, p[0] * (1 - 1e-9))[0] == 0
    assert oracle.sample_token(z, temperature, p[0] * (1 + 1e-9))[0] == 1
    assert oracle.sample_token(z, temperature, 1 - 1e-15)[0] == z.size - 1


def test_sampler_limits_greedy_and_uniform():
    g = torch.Generator().manual_seed(3)
    z = torch.randn(50, generator=g, dtype=torch.float64).numpy()
    for u in (0.001, 0.31, 0.77, 0.999):          # none on a cell edge k / 50
        assert oracle.sample_token(z, 1e-4, u)[0] == int(np.argmax(z))         # T -> 0: all mass on the top-1
        assert oracle.sample_token(z, 1e9, u)[0] == int(np.floor(u * z.size))  # T -> inf: uniform over tokens
    # zero-mass tokens are never returned, whatever u
    z2 = np.array([-1e4, 0.0, -1e4, 0.0, -1e4])
    assert {oracle.sample_token(z2, 1.0, u)[0] for u in np.linspace(1e-6, 1 - 1e-6, 101)} == {1, 3}


def test_large_shifted_logits_do_not_overflow():
    z = np.array([1000.0, 1001.0, 999.0])
    p = torch.softmax(torch.tensor(z, dtype=torch.float64), 0).numpy()
    assert oracle.sample_token(z, 1.0, p[0] * 0.99)[0] == 0
    assert oracle.sample_token(z, 1.0, p[0] * 1.01)[0] == 1
    assert oracle.sample_token(z, 1.0, (p[0] + p[1]) * 1.001)[0] == 2


@pytest.fixture(scope="module")
def tiny(tiny_weights):
    run = inputs.RUNS["tiny"]
    return run, tiny_weights, inputs.make_prompt(run.shape, run.n_prompt, run.seed).numpy()


def test_sampled_ar_is_sampling_from_the_model(tiny):
    """Each token of the sampled sequence is the sampler applied, at that position's uniform, to
    logits recomputed by a different organisation of the mathematics (teacher-forced pass)."""
    run, w, pr = tiny
    T, seed, n_gen = 0.8, 11, 12
    o = oracle.Oracle(run.shape, w, 64)
    o.set_sampling(T, seed)
    out, slack = o.ar_generate(pr, n_gen, want_margins=True)
    greedy = oracle.Oracle(run.shape, w, 64).ar_generate(pr, n_gen)
    assert not np.array_equal(out, greedy)                 # at T = 0.8 on random weights sampling leaves the greedy path
    assert (slack >= 0).all() and (slack <= 0.5).all()
    # brute force (no cache) under the same sampling setting reproduces it
    b = oracle.Oracle(run.shape, w, 64)
    b.set_sampling(T, seed)
    assert np.array_equal(b.bruteforce_generate(pr, n_gen), out)
    # final logits of every position from the layer-forward / final-logits path
    seq = np.concatenate([pr, out])
    f = oracle.Oracle(run.shape, w, 64)
    h = np.stack([f.embed(int(t)) for t in seq[:-1]])
    for l in range(1, run.shape.n_layers + 1):
        h = f.layer_forward(l, h, 0)
    for i in range(n_gen):
        pos = len(pr) + i                                   # position of the i-th generated token
        z = f.final_logits(h[pos - 1])
        t, _ = oracle.sample_token(z, T, oracle.uniform(seed, pos))
        assert t == out[i], i


def test_tiny_temperature_reproduces_greedy_sequence(tiny):
    run, w, pr = tiny
    greedy = oracle.Oracle(run.shape, w, 64).ar_generate(pr, 16)
    o = oracle.Oracle(run.shape, w, 64)
    o.set_sampling(1e-5, 99)
    assert np.array_equal(o.ar_generate(pr, 16), greedy)
    o.set_sampling(0.0, 99)                                 # 0 switches sampling off
    assert np.array_equal(o.ar_generate(pr, 16), greedy)


GRID = list(itertools.product((1, 2, 3), (1, 3, 8), (0.0, 0.25, 2.0), (0.3, 1.0)))


@pytest.mark.parametrize("which", ["tiny", "tiny-damped"])
def test_speculative_sampling_equals_autoregressive_sampling(which, tiny_weights, tiny_damped_weights):
    run = inputs.RUNS[which]
    w = tiny_weights if which == "tiny" else tiny_damped_weights
    pr = inputs.make_prompt(run.shape, run.n_prompt, run.seed).numpy()
    n_gen = 20
    ars = {}
    accepted = {0.3: 0, 1.0: 0}
    for d_max, w_max, thr, T in GRID:
        seed = 5
        if T not in ars:
            a = oracle.Oracle(run.shape, w, 64)
            a.set_sampling(T, seed)
            ars[T] = a.ar_generate(pr, n_gen)
        o = oracle.Oracle(run.shape, w, 64)
        o.set_sampling(T, seed)
        tau = tuple(1.0 + 0.5 * (d_max - l) for l in range(1, d_max + 1))
        out, rounds = o.specbound_generate(pr, n_gen, d_max, w_max, tau, thr)
        assert np.array_equal(out, ars[T]), (d_max, w_max, thr, T)
        for r in rounds:
            acc = 0
            while acc < r.w and r.draft[acc] >= 0 and r.g[acc] == r.draft[acc]:
                acc += 1
            assert r.accepted_drafts == acc
            accepted[T] += acc
    assert not np.array_equal(ars[0.3], ars[1.0])
    if which == "tiny-damped":
        # greedy drafts survive verification more often at the lower temperature (Table 2's trend)
        assert accepted[0.3] > accepted[1.0] > 0


def test_first_token_frequency_over_seeds_follows_softmax(tiny):
    run, w, pr = tiny
    T = 1.0
    o = oracle.Oracle(run.shape, w, 64)
    h = np.stack([o.embed(int(t)) for t in pr])
    for l in range(1, run.shape.n_layers + 1):
        h = o.layer_forward(l, h, 0)
    z = o.final_logits(h[-1])
    p = torch.softmax(torch.from_numpy(z) / T, 0).numpy()
    N = 1500
    counts = np.zeros(z.size)
    s = oracle.Oracle(run.shape, w, 64)
    for seed in range(N):
        s.set_sampling(T, seed)
        counts[s.ar_generate(pr, 1)[0]] += 1
    # Pearson statistic over the cells with an expected count of at least 5
    big = p * N >= 5
    chi2 = (((counts - p * N) ** 2) / (p * N))[big].sum() + (counts[~big].sum() - (p[~big] * N).sum()) ** 2 / max(
        (p[~big] * N).sum(), 1e-9)
    dof = int(big.sum())
    assert chi2 < dof + 5 * np.sqrt(2 * dof), (chi2, dof)


@pytest.mark.parametrize("temperature,top_p", [(1.0, 0.9), (0.5, 0.5), (2.0, 0.99), (1.0, 0.05)])
def test_nucleus_matches_library_sort_and_cumsum(temperature, top_p):
    g = torch.Generator().manual_seed(13)
    z = (torch.randn(61, generator=g, dtype=torch.float64) * 2).numpy()
    p = torch.softmax(torch.from_numpy(z) / temperature, 0)
    ps, order = torch.sort(p, descending=True)
    k = int(torch.nonzero(torch.cumsum(ps, 0) >= top_p)[0]) + 1        # tokens in the nucleus (no ties in random data)
    members = set(order[:k].tolist())
    zstar = oracle.nucleus_threshold(z, temperature, top_p)
    assert {v for v in range(z.size) if z[v] >= zstar} == members
    assert float(p[list(members)].sum()) >= top_p > float(p[list(members)].sum()) - float(ps[k - 1])   # minimal
    # stratified counts follow the renormalised probabilities inside the nucleus, nothing falls outside
    q = np.where(z >= zstar, p.numpy(), 0.0)
    q /= q.sum()
    N = 8000
    counts = np.zeros(z.size)
    for i in range(N):
        counts[oracle.sample_token(z, temperature, (i + 0.5) / N, top_p)[0]] += 1
    assert np.abs(counts - q * N).max() <= 1.0 + 1e-6
    assert counts[[v for v in range(z.size) if v not in members]].sum() == 0


def test_nucleus_ties_and_limits():
    z = np.array([1.0, 0.0, 1.0, -3.0, 1.0, 0.0])
    # the three tied maxima hold 3e / (3e + 2 + e^-3) = 0.80 of the mass and enter together
    assert oracle.nucleus_threshold(z, 1.0, 0.05) == 1.0
    assert oracle.nucleus_threshold(z, 1.0, 0.79) == 1.0
    assert oracle.nucleus_threshold(z, 1.0, 0.81) == 0.0            # then both zeros together
    assert oracle.nucleus_threshold(z, 1.0, 0.9999) == -3.0
    assert oracle.nucleus_threshold(z, 1.0, 1.0) == -np.inf
    assert {oracle.sample_token(z, 1.0, u, 0.5)[0] for u in np.linspace(0.001, 0.999, 50)} == {0, 2, 4}
    # thirds of the unit interval map to the three maxima in vocabulary order
    assert [oracle.sample_token(z, 1.0, u, 0.5)[0] for u in (0.2, 0.5, 0.9)] == [0, 2, 4]
    g = torch.Generator().manual_seed(2)
    r = torch.randn(40, generator=g, dtype=torch.float64).numpy()
    for u in (0.01, 0.4, 0.8, 0.99):
        assert oracle.sample_token(r, 0.8, u, 1.0) == oracle.sample_token(r, 0.8, u)       # top_p = 1: no restriction
        assert oracle.sample_token(r, 0.8, u, 1e-9)[0] == int(np.argmax(r))               # top_p -> 0: the top-1 alone


def test_speculative_equals_autoregressive_under_nucleus_sampling(tiny_damped_weights):
    run = inputs.RUNS["tiny-damped"]
    w = tiny_damped_weights
    pr = inputs.make_prompt(run.shape, run.n_prompt, run.seed).numpy()
    n_gen = 20
    a = oracle.Oracle(run.shape, w, 64)
    a.set_sampling(1.0, 5, top_p=0.9)
    ar = a.ar_generate(pr, n_gen)
    plain = oracle.Oracle(run.shape, w, 64)
    plain.set_sampling(1.0, 5)
    assert not np.array_equal(ar, plain.ar_generate(pr, n_gen))       # the nucleus changes the sampled sequence
    for d_max, w_max, thr in ((1, 8, 0.0), (2, 4, 0.25), (3, 3, 2.0)):
        o = oracle.Oracle(run.shape, w, 64)
        o.set_sampling(1.0, 5, top_p=0.9)
        out, _ = o.specbound_generate(pr, n_gen, d_max, w_max, inputs.tau_linear(d_max, 1.5, 1.0), thr)
        assert np.array_equal(out, ar), (d_max, w_max, thr)
