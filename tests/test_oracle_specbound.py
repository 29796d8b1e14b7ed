"""Pins of the oracle's round loop (Section 3.3): the exact-equivalence claim, the two bounds,
the paper's two worked scenarios (scripted exits), the work accounting behind Eq. 3 and the
worst case of the robustness appendix."""
import itertools

import numpy as np
import pytest

from oracle import oracle
from paper_2604_12247_b200 import inputs
from test_oracle_closed_forms import read_golden


def _run(shape, w, prompt, n_gen, d_max, w_max, tau, thr, script=None):
    o = oracle.Oracle(shape, w, len(prompt) + n_gen + w_max + 1)
    return o.specbound_generate(prompt, n_gen, d_max, w_max, tau, thr, script=script)


def check_round_invariants(rounds, L, d_max, w_max):
    for r in rounds:
        assert 1 <= r.w <= w_max                                     # width bound
        assert 1 <= r.emitted <= r.w
        assert r.D <= d_max
        for i in range(r.w):
            assert 0 <= r.exit_layer[i] <= d_max                     # depth bound
            assert (r.draft[i] >= 0) == (r.exit_layer[i] >= 1)
            assert r.layers_done[i] == L                             # every row went through all L layers once
        # only the last row may lack a draft (a failed exit ends the round)
        assert all(r.exit_layer[i] >= 1 for i in range(r.w - 1))
        if r.exit_layer[r.w - 1] >= 1:
            assert r.w == w_max                                      # otherwise drafting would have continued
        else:
            assert r.D == d_max
        assert r.layer_steps <= r.w * d_max + (L - r.D)              # Eq. 3 is this bound with D = d_max
        assert r.probes <= r.w * d_max
        acc = 0
        while acc < r.w and r.draft[acc] >= 0 and r.g[acc] == r.draft[acc]:
            acc += 1
        assert r.accepted_drafts == acc


GRID = [(d, wm, thr) for d, wm, thr in itertools.product((1, 2, 3), (1, 2, 4, 8), (0.0, 0.2, 0.3, 2.0))]


@pytest.mark.parametrize("which", ["tiny", "tiny-damped"])
def test_speculative_equals_autoregressive_over_grid(which, tiny_weights, tiny_damped_weights):
    run = inputs.RUNS[which]
    w = tiny_weights if which == "tiny" else tiny_damped_weights
    pr = inputs.make_prompt(run.shape, run.n_prompt, run.seed).numpy()
    n_gen = 24
    ar = oracle.Oracle(run.shape, w, 64).ar_generate(pr, n_gen)
    seen_w, seen_acc, seen_fail, seen_full = set(), set(), 0, 0
    for d_max, w_max, thr in GRID:
        for tau in ((1.0,) * d_max, tuple(1.0 + 0.5 * (d_max - l) for l in range(1, d_max + 1))):
            out, rounds = _run(run.shape, w, pr, n_gen, d_max, w_max, tau, thr)
            assert np.array_equal(out, ar), (d_max, w_max, thr, tau)
            assert sum(r.emitted for r in rounds) == n_gen - 1      # the first token comes from prefill
            check_round_invariants(rounds, run.shape.n_layers, d_max, w_max)
            for r in rounds:
                seen_w.add(r.w); seen_acc.add(r.accepted_drafts)
                seen_fail += r.exit_layer[r.w - 1] == 0
                seen_full += r.exit_layer[r.w - 1] >= 1
            if thr == 0.0:      # always exit at layer 1: every round is a full-width shallow chain
                assert all(r.w == w_max and all(e == 1 for e in r.exit_layer[:r.w]) for r in rounds)
            if thr > 1.0:       # never exit: every round is one AR step that went d_max deep first
                assert all(r.w == 1 and r.D == d_max and r.emitted == 1 and r.draft[0] == -1 for r in rounds)
    assert seen_fail > 0 and seen_full > 0
    if which == "tiny-damped":  # the damped variant must really exercise accepted runs
        assert {0, 1, 2, 3}.issubset(seen_acc) and {1, 2, 4, 8}.issubset(seen_w)


def test_tiny_workloads_run_as_defined(tiny_weights, tiny_damped_weights):
    """Workload 'tiny' as defined, and its damped variant: tokens equal AR, trace is sane."""
    for which, w in (("tiny", tiny_weights), ("tiny-damped", tiny_damped_weights)):
        run = inputs.RUNS[which]
        pr = inputs.make_prompt(run.shape, run.n_prompt, run.seed).numpy()
        ar = oracle.Oracle(run.shape, w, 64).ar_generate(pr, run.n_gen)
        out, rounds = _run(run.shape, w, pr, run.n_gen, run.d_max, run.w_max, run.tau, run.threshold)
        assert np.array_equal(out, ar)
        check_round_invariants(rounds, run.shape.n_layers, run.d_max, run.w_max)
    accs = [r.accepted_drafts for r in rounds]
    assert max(accs) >= 3 and min(accs) == 0
    assert any(r.exit_layer[r.w - 1] == 0 for r in rounds) and any(r.exit_layer[r.w - 1] > 0 for r in rounds)


def test_worst_case_all_rejected_emits_one(tiny_weights):
    """Robustness appendix: full width drafted, everything rejected -> one token per round."""
    run = inputs.RUNS["tiny"]
    pr = inputs.make_prompt(run.shape, run.n_prompt, run.seed).numpy()
    out, rounds = _run(run.shape, tiny_weights, pr, 12, 2, 4, (1.5, 1.0), 0.0)
    rej = [r for r in rounds if r.accepted_drafts == 0]
    assert rej and all(r.emitted == 1 and r.w == 4 for r in rej)


EIGHT = inputs.scaled(inputs.TINY, name="tiny-8l", n_layers=8, d_model=128, n_heads=4, n_kv_heads=4, head_dim=32,
                      d_ffn=256, vocab=200)


def _scenario(name):
    g = read_golden(name)
    exits = [int(x) for x in g["exit_layers"].split()]
    w = inputs.make_weights(EIGHT, 7)
    pr = inputs.make_prompt(EIGHT, 5, 7).numpy()
    ar = oracle.Oracle(EIGHT, w, 64).ar_generate(pr, 8)
    out, rounds = _run(EIGHT, w, pr, 8, int(g["d_max"]), int(g["w_max"]), (1.0,) * 6, 0.5, script=exits)
    assert np.array_equal(out, ar)
    return g, exits, rounds[0]


def test_scenario_difficult_token():
    g, exits, r = _scenario("scenario_difficult_token.txt")
    assert list(r.exit_layer[:r.w]) == exits
    assert r.w == int(g["rows_verified"]) and r.D == int(g["aligned_depth"])
    assert [list(r.depth_after[s][:s + 1]) for s in range(r.w)] == [[2], [4, 4], [6, 6, 6]]
    # draft phase: 2 + 4 + 6 layer passes (earlier rows ride along), then layers 7..8
    assert r.layer_steps == 12 + (EIGHT.n_layers - (int(g["first_verify_layer"]) - 1))
    assert r.probes == 12 and r.draft[2] == -1
    assert all(r.layers_done[i] == EIGHT.n_layers for i in range(r.w))


def test_scenario_long_shallow_chain():
    g, exits, r = _scenario("scenario_long_chain.txt")
    assert list(r.exit_layer[:r.w]) == exits
    assert r.w == int(g["rows_verified"]) and r.D == int(g["aligned_depth"])
    assert [list(r.depth_after[s][:s + 1]) for s in range(r.w)] == [[2], [4, 4], [6, 6, 6], [6, 6, 6, 2]]
    # drafting: 2 + 4 + 6 + 2 passes; alignment: layers 3..6 for the last row alone; then layers 7..8
    assert r.layer_steps == 14 + 4 + 2
    assert r.probes == 14
    assert all(r.layers_done[i] == EIGHT.n_layers for i in range(r.w))


MASKS = [(0, 1, 1), (1, 0, 1), (1, 1, 0), (0, 0, 1), (0, 1, 0), (1, 0, 0), (0, 0, 0)]


def test_probe_layer_mask(tiny_damped_weights):
    """Probe-layer mask (tau_l <= 0: layer l is walked but not tested).  Pins:
    * the output is still plain greedy decoding, for every mask (the exactness claim of Section 3.3 does not depend
      on where exits are looked for);
    * a masked layer never appears as an exit layer, and a row is charged one probe per UNMASKED layer it walked;
    * a masked run is the unmasked algorithm with a test that cannot pass at that layer: temperature 1e30 there makes
      the confidence 1/V < threshold, and that run must agree round for round (width, depth, exit layers, drafts,
      accepted, emitted) -- only the probe count differs, by exactly the probes spent on hopeless layers;
    * masking every layer turns each round into one autoregressive step that went d_max deep (w = 1, no draft)."""
    run = inputs.RUNS["tiny-damped"]
    shape, w = run.shape, tiny_damped_weights
    pr = inputs.make_prompt(shape, run.n_prompt, run.seed).numpy()
    n_gen, d_max, w_max, thr = 24, 3, 4, 0.3
    base = (1.6, 1.3, 1.0)
    ar = oracle.Oracle(shape, w, 64).ar_generate(pr, n_gen)
    seen_exit_layers = set()
    for mask in MASKS:
        tau_masked = tuple(t if on else 0.0 for t, on in zip(base, mask))
        tau_hopeless = tuple(t if on else 1e30 for t, on in zip(base, mask))
        out, rounds = _run(shape, w, pr, n_gen, d_max, w_max, tau_masked, thr)
        out_h, rounds_h = _run(shape, w, pr, n_gen, d_max, w_max, tau_hopeless, thr)
        assert np.array_equal(out, ar) and np.array_equal(out_h, ar), mask
        check_round_invariants(rounds, shape.n_layers, d_max, w_max)
        assert len(rounds) == len(rounds_h)
        for r, q in zip(rounds, rounds_h):
            assert (r.w, r.D, r.emitted, r.accepted_drafts, r.layer_steps) == (q.w, q.D, q.emitted, q.accepted_drafts, q.layer_steps)
            assert list(r.exit_layer[:r.w]) == list(q.exit_layer[:q.w]) and list(r.draft[:r.w]) == list(q.draft[:q.w])
            walked = [e if e else d_max for e in r.exit_layer[:r.w]]          # layers each row's own draft step walked
            assert r.probes == sum(sum(mask[:n]) for n in walked)
            assert q.probes == sum(walked)
            for e in r.exit_layer[:r.w]:
                assert e == 0 or mask[e - 1] == 1
                seen_exit_layers.add(e)
        if not any(mask):
            assert all(r.w == 1 and r.D == d_max and r.draft[0] == -1 and r.probes == 0 for r in rounds)
    assert {1, 2, 3}.issubset(seen_exit_layers)      # the masks really moved exits between layers
    # negative temperatures mask as well, and the unmasked schedule is untouched by the feature
    out_a, rounds_a = _run(shape, w, pr, n_gen, d_max, w_max, (-1.0, 1.3, 1.0), thr)
    out_b, rounds_b = _run(shape, w, pr, n_gen, d_max, w_max, (0.0, 1.3, 1.0), thr)
    assert np.array_equal(out_a, out_b) and [r.probes for r in rounds_a] == [r.probes for r in rounds_b]


def test_bad_arguments_are_refused(tiny_weights):
    run = inputs.RUNS["tiny"]
    pr = inputs.make_prompt(run.shape, 4, 0).numpy()
    o = oracle.Oracle(run.shape, tiny_weights, 16)
    with pytest.raises(ValueError):
        o.specbound_generate(pr, 32, 2, 4, (1.5, 1.0), 0.3)          # capacity
    with pytest.raises(ValueError):
        o.specbound_generate(pr, 4, 9, 4, (1.0,) * 9, 0.3)           # d_max > L
    with pytest.raises(ValueError):
        o.specbound_generate(pr, 4, 2, 9, (1.5, 1.0), 0.3)           # w_max > 8
