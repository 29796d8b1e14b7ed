"""Step- and run-level parity of the CUDA decode path against the CPU oracle (C ABI)."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2604_12247_b200 import binding, inputs
from gpu_util import CONF_TOL, HIDDEN_TOL, LOGIT_TOL, gemm_modes, gpu_ctx, near_tie_count
from test_oracle_closed_forms import read_golden

pytestmark = pytest.mark.gpu


def test_tcgen05_backend_is_built():
    assert gemm_modes(inputs.LLAMA2_7B) == [0, 1]


def compare_traces(gpu_rounds, orc_rounds):
    assert len(gpu_rounds) == len(orc_rounds)
    for g, o in zip(gpu_rounds, orc_rounds):
        assert (g.w, g.D, g.emitted) == (o.w, o.D, o.emitted)
        assert g.accepted_drafts == min(o.accepted_drafts, o.w)
        assert list(g.exit_layer[:g.w]) == list(o.exit_layer[:o.w])
        assert list(g.draft[:g.w]) == list(o.draft[:o.w])
        assert list(g.g[:g.w]) == list(o.g[:o.w])
        for i in range(g.w):
            assert abs(g.conf[i] - o.conf[i]) < CONF_TOL


@pytest.mark.parametrize("which", ["tiny", "tiny-damped"])
def test_tiny_run_matches_oracle_tokens_and_trace(which, tiny_weights, tiny_damped_weights):
    run = inputs.RUNS[which]
    w = tiny_weights if which == "tiny" else tiny_damped_weights
    pr = inputs.make_prompt(run.shape, run.n_prompt, run.seed).numpy()
    max_seq = run.n_prompt + run.n_gen + run.w_max + 1
    orc_ar, margins = oracle.Oracle(run.shape, w, max_seq).ar_generate(pr, run.n_gen, want_margins=True)
    assert margins.min() > 10 * LOGIT_TOL["f32"]          # no near tie in this workload: tokens must be equal
    orc_sp, orc_rounds = oracle.Oracle(run.shape, w, max_seq).specbound_generate(
        pr, run.n_gen, run.d_max, run.w_max, run.tau, run.threshold)
    ctx, _ = gpu_ctx(run.shape, w, max_seq)
    ar = ctx.generate_ar(pr, run.n_gen)
    sp = ctx.generate(pr, run.n_gen, run.d_max, run.w_max, run.tau, run.threshold, trace=True)
    assert np.array_equal(ar["tokens"], orc_ar)
    assert np.array_equal(sp["tokens"], orc_ar) and np.array_equal(orc_sp, orc_ar)
    compare_traces(sp["rounds"], orc_rounds)
    st = sp["stats"]
    assert st.emitted == run.n_gen and st.rounds == len(orc_rounds)
    assert st.probes == sum(r.probes for r in orc_rounds)
    assert st.layer_steps == sum(r.layer_steps for r in orc_rounds)
    assert st.kernel_launches > 0
    # the phase timings and the unified-pass counters cover the event-bracketed rounds: the first and every fourth after it
    timed = [r for i, r in enumerate(orc_rounds) if i % 4 == 0]
    assert st.rounds_timed == len(timed)
    assert st.unified_layer_steps == sum(run.shape.n_layers - r.D for r in timed)   # layers D+1 .. L of each
    assert st.us_unified > 0 and st.us_draft > 0 and st.us_verify >= st.us_unified
    assert 1 <= st.probes_timed <= st.probes
    # determinism: a second run is identical down to the confidence bits
    sp2 = ctx.generate(pr, run.n_gen, run.d_max, run.w_max, run.tau, run.threshold, trace=True)
    assert np.array_equal(sp2["tokens"], sp["tokens"])
    assert all(list(a.conf) == list(b.conf) for a, b in zip(sp["rounds"], sp2["rounds"]))
    ctx.close()


def test_per_layer_exit_heads_match_oracle_trace():
    """Section 3.2's per-layer exit heads (pointer tables exit_head / exit_norm): the exit test after layer l
    uses that layer's head and norm gain, the verify pass the shared head.  Tokens stay those of plain
    autoregressive decoding; exit layers, drafts and confidences follow the oracle run with the same heads,
    and differ from the run with the shared head (the tables are really used)."""
    run = inputs.RUNS["tiny-damped"]
    w = inputs.add_exit_heads(inputs.make_weights(run.shape, run.seed, damp_rho=run.damp_rho), run.shape, seed=3)
    pr = inputs.make_prompt(run.shape, run.n_prompt, run.seed).numpy()
    max_seq = run.n_prompt + run.n_gen + run.w_max + 1
    orc_ar = oracle.Oracle(run.shape, w, max_seq).ar_generate(pr, run.n_gen)
    orc_sp, orc_rounds = oracle.Oracle(run.shape, w, max_seq).specbound_generate(
        pr, run.n_gen, run.d_max, run.w_max, run.tau, run.threshold)
    assert np.array_equal(orc_sp, orc_ar)
    ctx, _ = gpu_ctx(run.shape, w, max_seq)
    sp = ctx.generate(pr, run.n_gen, run.d_max, run.w_max, run.tau, run.threshold, trace=True)
    assert np.array_equal(sp["tokens"], orc_ar)
    compare_traces(sp["rounds"], orc_rounds)
    # the probe primitive with a per-layer head, against the oracle on the same hidden state
    ctx.reset()
    first = ctx.prefill(pr)
    ctx.draft_push(first)
    for l in (1, 2):
        ctx.draft_advance(l)
        conf, tok, _ = ctx.exit_confidence(l, run.tau[l - 1], run.threshold)
        o = oracle.Oracle(run.shape, w, max_seq)
        p_ref, t_ref = o.exit_confidence_at(l, ctx.read_hidden(0).astype(np.float64), run.tau[l - 1])
        assert tok == t_ref and abs(conf - p_ref) < CONF_TOL
        p_shared, _ = o.exit_confidence(ctx.read_hidden(0).astype(np.float64), run.tau[l - 1])
        assert abs(p_shared - p_ref) > 10 * CONF_TOL
    ctx.close()
    shared = {k: v for k, v in w.items() if k not in ("exit_head", "exit_norm")}
    _, shared_rounds = oracle.Oracle(run.shape, shared, max_seq).specbound_generate(
        pr, run.n_gen, run.d_max, run.w_max, run.tau, run.threshold)
    assert [list(r.conf[:r.w]) for r in shared_rounds] != [list(r.conf[:r.w]) for r in orc_rounds]


def test_tiny_hyper_parameter_grid_equals_ar(tiny_damped_weights):
    run = inputs.RUNS["tiny-damped"]
    pr = inputs.make_prompt(run.shape, run.n_prompt, run.seed).numpy()
    ctx, _ = gpu_ctx(run.shape, tiny_damped_weights, 96)
    n_gen = 24
    ar = ctx.generate_ar(pr, n_gen)["tokens"]
    assert np.array_equal(ar, oracle.Oracle(run.shape, tiny_damped_weights, 96).ar_generate(pr, n_gen))
    for d_max in (1, 2, 3):
        for w_max in (1, 2, 4, 8):
            for thr in (0.0, 0.2, 0.3, 2.0):
                tau = [1.0 + 0.5 * (d_max - l) for l in range(1, d_max + 1)]
                res = ctx.generate(pr, n_gen, d_max, w_max, tau, thr, trace=True)
                assert np.array_equal(res["tokens"], ar), (d_max, w_max, thr)
                for r in res["rounds"]:
                    assert 1 <= r.w <= w_max and 1 <= r.emitted <= r.w and r.D <= d_max
                    assert all(0 <= e <= d_max for e in r.exit_layer[:r.w])
                if thr == 0.0:
                    assert all(r.w == w_max for r in res["rounds"][:-1])
                if thr > 1.0:
                    assert all(r.w == 1 and r.emitted == 1 for r in res["rounds"])
    ctx.close()


def test_probe_layer_mask_matches_oracle_trace(tiny_damped_weights):
    """Probe-layer mask (temperature <= 0: the layer is walked but not tested): tokens stay those of autoregressive
    decoding for every mask, and rounds, exit layers, drafts, confidences and the probe count follow the oracle run
    with the same mask."""
    run = inputs.RUNS["tiny-damped"]
    pr = inputs.make_prompt(run.shape, run.n_prompt, run.seed).numpy()
    n_gen, d_max, w_max, thr = 24, 3, 4, 0.3
    base = (1.6, 1.3, 1.0)
    ctx, _ = gpu_ctx(run.shape, tiny_damped_weights, 64)
    ar = ctx.generate_ar(pr, n_gen)["tokens"]
    assert np.array_equal(ar, oracle.Oracle(run.shape, tiny_damped_weights, 64).ar_generate(pr, n_gen))
    for mask in ((1, 1, 1), (0, 1, 1), (1, 0, 1), (1, 1, 0), (0, 0, 1), (0, 1, 0), (1, 0, 0), (0, 0, 0)):
        tau = tuple(t if on else 0.0 for t, on in zip(base, mask))
        _, orc_rounds = oracle.Oracle(run.shape, tiny_damped_weights, 64).specbound_generate(pr, n_gen, d_max, w_max, tau, thr)
        sp = ctx.generate(pr, n_gen, d_max, w_max, tau, thr, trace=True)
        assert np.array_equal(sp["tokens"], ar), mask
        compare_traces(sp["rounds"], orc_rounds)
        assert sp["stats"].probes == sum(r.probes for r in orc_rounds)
        assert sp["stats"].layer_steps == sum(r.layer_steps for r in orc_rounds)
        assert all(mask[e - 1] for r in sp["rounds"] for e in r.exit_layer[:r.w] if e)
    ctx.close()


GEOM_7B_RUN = inputs.scaled(inputs.LLAMA2_7B, name="7b-attention-geometry-7l", n_layers=7, d_model=512, d_ffn=1024, vocab=2048,
                            head_scale=16.0)


def test_bench_lengths_on_7b_attention_geometry_match_oracle():
    """The bench workload's lengths and bounds (512-token prompt, 512 generated tokens, d_max 6, w_max 4, its tau
    schedule and threshold) on a 7-layer model with the 7B attention geometry (32 heads of 128 channels; d_model and
    FFN cut so that the oracle can follow every position): the context grows from 512 to 1028 positions, through
    cluster merges of 5 to 8 chunk CTAs and over the hand-over to the separate attention kernels at the 9th chunk, and
    the prompt goes through the wide prefill passes.  Speculative == autoregressive bit for bit on the GPU; every one of
    the 512 tokens is the oracle's top-1 or within the logit tolerance of it (teacher-forced), near ties counted."""
    run = inputs.RUNS["7b"]
    shape = GEOM_7B_RUN
    w = inputs.make_weights(shape, 5, damp_rho=0.3)
    pr = inputs.make_prompt(shape, run.n_prompt, 9).numpy()
    n_gen = run.n_gen
    max_seq = run.n_prompt + n_gen + run.w_max + 8
    ctx, _ = gpu_ctx(shape, w, max_seq, kv_page=64, gemm=1)
    ar = ctx.generate_ar(pr, n_gen)["tokens"]
    sp = ctx.generate(pr, n_gen, run.d_max, run.w_max, run.tau, run.threshold, trace=True)
    assert np.array_equal(sp["tokens"], ar)
    rounds = sp["rounds"]
    assert all(1 <= r.w <= run.w_max and r.D <= run.d_max and 1 <= r.emitted <= r.w for r in rounds)
    st = sp["stats"]
    assert st.accepted_drafts > 0 and max(r.w for r in rounds) == run.w_max
    ctx.close()
    toks = np.concatenate([pr, ar]).astype(np.int32)
    top1, top2, margin, deficit = oracle.Oracle(shape, w, max_seq).teacher_forced(toks, len(pr))
    n_off = int((top1 != ar).sum())
    near = int((margin < 2 * LOGIT_TOL["bf16"]).sum())
    print(f"\n[7B attention geometry, 512 + 512 tokens] {len(rounds)} rounds, {st.accepted_drafts} drafts accepted; GPU tokens "
          f"that are not the oracle's top-1: {n_off} of {n_gen}; positions with a top-2 margin below tolerance: {near}; "
          f"worst deficit {deficit.min():.2e}")
    assert deficit.min() > -LOGIT_TOL["bf16"]
    assert all(margin[i] < 2 * LOGIT_TOL["bf16"] for i in range(n_gen) if top1[i] != ar[i])


EIGHT = inputs.scaled(inputs.TINY, name="tiny-8l", n_layers=8, d_model=128, n_heads=4, n_kv_heads=4, head_dim=32,
                      d_ffn=256, vocab=200)


@pytest.mark.parametrize("name", ["scenario_difficult_token.txt", "scenario_long_chain.txt"])
def test_worked_scenarios_step_parity(name):
    """The paper's two worked rounds, driven through the draft primitives with scripted exits; the
    hidden-state cache and depths are compared with an oracle replay after every draft step."""
    g = read_golden(name)
    exits = [int(x) for x in g["exit_layers"].split()]
    d_max = int(g["d_max"])
    w = inputs.make_weights(EIGHT, 7)
    pr = inputs.make_prompt(EIGHT, 5, 7).numpy()
    orc = oracle.Oracle(EIGHT, w, 64)
    ref_tokens, ref_rounds = oracle.Oracle(EIGHT, w, 64).specbound_generate(pr, 8, d_max, int(g["w_max"]), (1.0,) * 6, 0.5,
                                                                          script=exits)
    ctx, _ = gpu_ctx(EIGHT, w, 64)
    first = ctx.prefill(pr)
    assert first == ref_tokens[0]
    pending = orc.ar_generate(pr, 1)[0]            # fills the replay oracle's cache for the prompt
    assert pending == first
    n = len(pr)
    hid, depth, drafts, cur = [], [], [], first
    for step, e in enumerate(exits):
        ctx.draft_push(cur)
        hid.append(orc.embed(cur)); depth.append(0)
        tok = None
        for l in range(1, d_max + 1):
            ctx.draft_advance(l)
            r0 = len(depth)
            while r0 > 0 and depth[r0 - 1] == l - 1:
                r0 -= 1
            out = orc.layer_forward(l, np.stack(hid[r0:]), n + r0)
            for i in range(r0, len(depth)):
                hid[i], depth[i] = out[i - r0], l
            conf, tok, _ = ctx.exit_confidence(l, 1.0, 0.5)
            p, t = orc.exit_confidence(hid[-1], 1.0)
            assert abs(conf - p) < CONF_TOL and tok == t
            if l == e:
                break
        st = ctx.state()
        assert list(st.depth[:st.rows]) == depth == list(ref_rounds[0].depth_after[step][:step + 1])
        for i in range(st.rows):
            err = np.abs(ctx.read_hidden(i) - hid[i]).max() / np.abs(hid[i]).max()
            assert err < HIDDEN_TOL["f32"]
        drafts.append(tok if e else -1)
        cur = tok
    out = ctx.verify(drafts)
    r = ref_rounds[0]
    assert len(drafts) == r.w == int(g["rows_verified"])
    assert list(out) == list(r.g[:r.emitted])
    st = ctx.state()
    assert st.rows == 0 and st.n == n + r.emitted and st.pending == r.g[r.emitted - 1]
    ctx.close()


SMALL_BF16 = inputs.scaled(inputs.LLAMA3_8B, name="small-bf16", n_layers=4, d_model=512, n_heads=8, n_kv_heads=2,
                           head_dim=64, d_ffn=1408, vocab=2048, head_scale=16.0)


def test_bf16_model_speculative_equals_ar_and_oracle():
    """A small bf16 GQA model with damped deep layers (so that drafts get accepted): on the GPU,
    speculative and autoregressive decoding are bit-identical for every GEMM back end; against the
    oracle the tokens agree except at near ties, which are counted."""
    shape = SMALL_BF16
    w = inputs.make_weights(shape, 5, damp_rho=0.3)
    pr = inputs.make_prompt(shape, 20, 5).numpy()
    n_gen, max_seq = 40, 96
    orc_ar, margins = oracle.Oracle(shape, w, max_seq).ar_generate(pr, n_gen, want_margins=True)
    for gemm in gemm_modes(shape):
        ctx, _ = gpu_ctx(shape, w, max_seq, gemm=gemm)
        ar = ctx.generate_ar(pr, n_gen)["tokens"]
        seen_acc = 0
        for d_max, w_max, thr in ((2, 4, 0.3), (3, 8, 0.2), (1, 6, 0.0)):
            tau = inputs.tau_linear(d_max, 1.5, 1.0)
            res = ctx.generate(pr, n_gen, d_max, w_max, tau, thr, trace=True)
            assert np.array_equal(res["tokens"], ar), (gemm, d_max, w_max)
            seen_acc += res["stats"].accepted_drafts
        assert seen_acc > 0
        n_off, worst = near_tie_count(shape, w, pr, ar, LOGIT_TOL["bf16"])
        print(f"\n[gemm={gemm}] positions where the GPU token is not the oracle top-1: {n_off}, worst deficit {worst:.2e}")
        assert worst > -2 * LOGIT_TOL["bf16"]
        if margins.min() > 2 * LOGIT_TOL["bf16"]:
            assert np.array_equal(ar, orc_ar)
        ctx.close()


def test_state_and_argument_errors(tiny_weights):
    run = inputs.RUNS["tiny"]
    ctx, _ = gpu_ctx(run.shape, tiny_weights, 40)
    pr = inputs.make_prompt(run.shape, 8, 0).numpy()
    E = binding.SBError
    with pytest.raises(E) as e:
        ctx.draft_push(3)                                   # nothing prefilled yet
    assert e.value.status == -2
    with pytest.raises(E) as e:
        ctx.generate(pr, 32, 2, 4, (1.5, 1.0), 0.3)          # 8 + 32 + 4 > 40
    assert e.value.status == -3
    with pytest.raises(E) as e:
        ctx.generate(pr, 8, 4, 4, (1.0,) * 4, 0.3)           # d_max must stay below the layer count
    assert e.value.status == -1
    with pytest.raises(E) as e:
        ctx.generate(pr, 8, 2, 9, (1.5, 1.0), 0.3)           # w_max > 8
    assert e.value.status == -1
    with pytest.raises(E) as e:
        ctx.generate(pr, 8, 2, 4, (1.5, float("nan")), 0.3)  # a temperature must be a number (<= 0 masks the layer)
    assert e.value.status == -1
    bad = pr.copy(); bad[3] = run.shape.vocab
    with pytest.raises(E) as e:
        ctx.generate_ar(bad, 4)                              # token id outside the vocabulary
    assert e.value.status == -1
    ctx.reset()
    t = ctx.prefill(pr)
    ctx.draft_push(t)
    ctx.draft_advance(1)
    with pytest.raises(E) as e:
        ctx.exit_confidence(2, 1.0, 0.5)                     # newest row is at depth 1, not 2
    assert e.value.status == -2
    with pytest.raises(E) as e:
        ctx.exit_confidence(1, 0.0, 0.5)                     # a masked layer (temperature <= 0) cannot be probed
    assert e.value.status == -1
    with pytest.raises(E) as e:
        ctx.verify([-1, -1])                                 # one row in flight, two given
    assert e.value.status == -2
    assert len(ctx.verify([-1])) == 1                        # the context is still usable
    ctx.close()


def test_7b_shape_run_matches_oracle_on_sampled_positions():
    """The bench workload's shape (32 layers, d = 4096, 32 heads, FFN 11008, vocab 32000, bf16) in the
    launch configuration bench.py times, on a short sequence the oracle can follow.
    * speculative and autoregressive decoding are bit-identical on the GPU;
    * every GPU token is the oracle's top-1 or within the logit tolerance of it (teacher-forced, so
      that one near tie cannot cascade);
    * exit confidences: the exit kernel agrees with the oracle's exit test on the SAME hidden state
      within 1e-3 (measured ~1e-6).  Against the free-running oracle the hidden state itself drifts
      by ~3e-4 per layer, because ~0.3 % of the K/V entries the GPU caches land on the neighbouring
      bf16 value (fp32 vs fp64 value straddling a rounding boundary); that drift is bounded and
      printed, not hidden."""
    run = inputs.RUNS["7b"]
    shape = run.shape
    wg = inputs.make_weights(shape, run.seed, device="cuda")
    # the workload's norm gains are all 1.0, which would hide a dropped or misplaced gain at d = 4096: perturb them here
    g = torch.Generator(device="cuda").manual_seed(77)
    perturbed = lambda t: (1.0 + 0.1 * torch.randn(t.shape, generator=g, device="cuda")).to(t.dtype)
    for lw in wg["layers"]:
        lw["attn_norm"], lw["mlp_norm"] = perturbed(lw["attn_norm"]), perturbed(lw["mlp_norm"])
    wg["final_norm"] = perturbed(wg["final_norm"])
    pr = inputs.make_prompt(shape, 24, run.seed).numpy()
    n_gen, max_seq = 12, 64
    ctx = binding.Context(shape, wg, max_seq, kv_page=64)
    ar = ctx.generate_ar(pr, n_gen)["tokens"]
    sp = ctx.generate(pr, n_gen, run.d_max, run.w_max, run.tau, run.threshold, trace=True)
    assert np.array_equal(sp["tokens"], ar)
    for r in sp["rounds"]:
        assert 1 <= r.w <= run.w_max and r.D <= run.d_max and 1 <= r.emitted <= r.w
    wc = inputs.weights_to(wg, "cpu")
    toks = np.concatenate([pr, ar]).astype(np.int32)
    top1, top2, margin, deficit = oracle.Oracle(shape, wc, max_seq).teacher_forced(toks, len(pr))
    n_off = int((top1 != ar).sum())
    print(f"\n[7b shape] GPU tokens that are not the oracle's top-1: {n_off} of {n_gen}; worst deficit {deficit.min():.2e}; "
          f"smallest top-2 margin {margin.min():.3f}")
    assert deficit.min() > -LOGIT_TOL["bf16"]
    assert all(margin[i] < 2 * LOGIT_TOL["bf16"] for i in range(n_gen) if top1[i] != ar[i])
    # one draft row walked through the shallow layers with the draft primitives
    ctx.reset()
    first = ctx.prefill(pr)
    o = oracle.Oracle(shape, wc, max_seq)
    assert o.ar_generate(pr, 1)[0] == first
    ctx.draft_push(first)
    h = o.embed(first)[None]
    worst_kernel, worst_drift, worst_hidden = 0.0, 0.0, 0.0
    for l in range(1, run.d_max + 1):
        ctx.draft_advance(l)
        h = o.layer_forward(l, h, len(pr))
        gh = ctx.read_hidden(0)
        conf, tok, _ = ctx.exit_confidence(l, run.tau[l - 1], run.threshold)
        p_same, t_same = o.exit_confidence(gh.astype(np.float64), run.tau[l - 1])   # oracle on the GPU's hidden state
        p_free, t_free = o.exit_confidence(h[0], run.tau[l - 1])                    # free-running oracle
        worst_kernel = max(worst_kernel, abs(conf - p_same))
        worst_drift = max(worst_drift, abs(conf - p_free))
        worst_hidden = max(worst_hidden, np.abs(gh - h[0]).max() / np.abs(h[0]).max())
        assert tok == t_same
    print(f"[7b shape] exit confidence vs oracle on the same hidden state: {worst_kernel:.1e}; vs free-running oracle: "
          f"{worst_drift:.1e} (hidden drift {worst_hidden:.1e} after {run.d_max} layers)")
    assert worst_kernel < CONF_TOL
    assert worst_drift < 1e-2 and worst_hidden < HIDDEN_TOL["bf16"]
    ctx.close()


def test_7b_damped_run_accepts_drafts_and_equals_ar():
    """The labelled addition `7b-damped` (damped deep layers: the stand-in for trained exit heads) is what
    exercises long rounds and accepted drafts at the bench shape: speculative decoding must still be
    bit-identical to autoregressive decoding, emit more than one token per round on average, and every token
    must be the oracle's top-1 or within the logit tolerance of it (teacher-forced)."""
    run = inputs.RUNS["7b-damped"]
    shape = run.shape
    wg = inputs.make_weights(shape, run.seed, device="cuda", damp_rho=run.damp_rho)
    pr = inputs.make_prompt(shape, 24, run.seed).numpy()
    n_gen, max_seq = 40, 96
    ctx = binding.Context(shape, wg, max_seq, kv_page=64)
    ar = ctx.generate_ar(pr, n_gen)["tokens"]
    sp = ctx.generate(pr, n_gen, run.d_max, run.w_max, run.tau, run.threshold, trace=True)
    assert np.array_equal(sp["tokens"], ar)
    rounds = sp["rounds"]
    emitted = sum(r.emitted for r in rounds)
    assert emitted == n_gen - 1
    assert all(1 <= r.w <= run.w_max and r.D <= run.d_max and 1 <= r.emitted <= r.w for r in rounds)
    print(f"\n[7b-damped] {len(rounds)} rounds, mean width {np.mean([r.w for r in rounds]):.2f}, "
          f"emitted per round {emitted / len(rounds):.2f}, widest {max(r.w for r in rounds)}")
    assert emitted / len(rounds) > 1.5 and max(r.emitted for r in rounds) >= 3
    wc = inputs.weights_to(wg, "cpu")
    n_chk = 12   # oracle cost: one teacher-forced pass over prompt + n_chk tokens
    toks = np.concatenate([pr, ar[:n_chk]]).astype(np.int32)
    top1, top2, margin, deficit = oracle.Oracle(shape, wc, max_seq).teacher_forced(toks, len(pr))
    assert deficit.min() > -LOGIT_TOL["bf16"]
    assert all(margin[i] < 2 * LOGIT_TOL["bf16"] for i in range(n_chk) if top1[i] != ar[i])
    ctx.close()


@pytest.mark.parametrize("which", ["l3-8b", "13b"])
def test_large_config_tokens_match_oracle(which):
    """Workloads `l3-8b` (Llama-3-8B shape: GQA 32/8 heads, vocabulary 128256) and `13b` (13B shape: 40 layers,
    d = 5120) in the launch configuration bench.py uses, on a sequence short enough for the oracle:
    speculative == autoregressive bit for bit on the GPU, and every token is the oracle's top-1 or within the
    logit tolerance of it (teacher-forced)."""
    run = inputs.RUNS[which]
    shape = run.shape
    wg = inputs.make_weights(shape, run.seed, device="cuda")
    pr = inputs.make_prompt(shape, 12, run.seed).numpy()
    n_gen, max_seq = 8, 48
    ctx = binding.Context(shape, wg, max_seq, kv_page=64)
    ar = ctx.generate_ar(pr, n_gen)["tokens"]
    sp = ctx.generate(pr, n_gen, run.d_max, run.w_max, run.tau, run.threshold, trace=True)
    assert np.array_equal(sp["tokens"], ar)
    for r in sp["rounds"]:
        assert 1 <= r.w <= run.w_max and r.D <= run.d_max and 1 <= r.emitted <= r.w
    ctx.close()
    wc = inputs.weights_to(wg, "cpu")
    del wg
    torch.cuda.empty_cache()
    toks = np.concatenate([pr, ar]).astype(np.int32)
    top1, top2, margin, deficit = oracle.Oracle(shape, wc, max_seq).teacher_forced(toks, len(pr))
    n_off = int((top1 != ar).sum())
    print(f"\n[{which}] GPU tokens that are not the oracle's top-1: {n_off} of {n_gen}; worst deficit {deficit.min():.2e}; "
          f"smallest top-2 margin {margin.min():.3f}")
    assert deficit.min() > -LOGIT_TOL["bf16"]
    assert all(margin[i] < 2 * LOGIT_TOL["bf16"] for i in range(n_gen) if top1[i] != ar[i])


def test_bench_sweep_mode_on_tiny(capsys):
    """bench.py --sweep (depth bound x width bound and threshold sweep): every point decodes the same tokens as
    autoregressive decoding and reports its statistics."""
    import argparse
    import json
    import bench
    bench.sweep_arm(argparse.Namespace(), inputs.RUNS["tiny-damped"])
    line = json.loads(capsys.readouterr().out.strip().splitlines()[-1])
    pts = line["points"]
    assert line["mode"] == "sweep" and len(pts) >= 9
    assert all(p["tokens_equal_ar"] for p in pts)
    assert {p["d_max"] for p in pts} == {1, 2} and {p["w_max"] for p in pts} == {2, 4, 8}
    assert all(1.0 <= p["emitted_per_round"] <= p["w_max"] and 0.0 <= p["draft_acceptance"] <= 1.0 for p in pts)
    assert max(p["emitted_per_round"] for p in pts) > 1.5
    # annealing-strength sweep, component ablation, probe-layer masks and the fitted cost model (Section 4.4's axes)
    assert [p["alpha"] for p in line["alpha_sweep"]] == [0.0, 0.1, 0.2, 0.4, 0.8, 1.6]
    assert len(line["ablation"]) == 4 and line["ablation"][2]["d_max"] == inputs.RUNS["tiny-damped"].shape.n_layers - 1
    assert len(line["probe_mask"]) >= 2 and line["probe_mask"][-1]["probes"] < line["probe_mask"][0]["probes"]
    for group in ("alpha_sweep", "ablation", "probe_mask"):
        assert all(p["tokens_equal_ar"] for p in line[group]), group
    fit = line["cost_model_fit"]
    assert fit["points"] == len(pts) + 6 + 4 + len(line["probe_mask"]) and fit["t_layer_us"] > 0
    strat = line["decoding_strategies"]
    assert [x["strategy"] for x in strat] == ["greedy", "temperature 0.3", "temperature 1.0", "top-p 0.9"]
    assert all(x["tokens_equal_ar"] and x["tokens_per_s"] > 0 and x["ar_tokens_per_s"] > 0 for x in strat)


def test_host_side_options_do_not_change_results(tiny_damped_weights):
    """Work issued ahead while the host waits for an exit decision (SB_OPT_QKV_AHEAD) and programmatic dependent
    launch (SB_OPT_PDL) are scheduling choices: tokens, rounds, exit layers and confidences are bit-identical."""
    run = inputs.RUNS["tiny-damped"]
    pr = inputs.make_prompt(run.shape, run.n_prompt, run.seed).numpy()
    max_seq = run.n_prompt + run.n_gen + run.w_max + 1
    lib = binding.lib()
    results = []
    try:
        for ahead, pdl in ((1, 1), (0, 1), (1, 0), (0, 0)):
            assert lib.sb_set_default_option(8, ahead) == 0 and lib.sb_set_default_option(4, pdl) == 0
            for shape, w in ((run.shape, tiny_damped_weights),):
                ctx, _ = gpu_ctx(shape, w, max_seq)
                sp = ctx.generate(pr, run.n_gen, run.d_max, run.w_max, run.tau, run.threshold, trace=True)
                results.append((sp["tokens"].copy(), [(r.w, r.D, r.emitted, list(r.exit_layer), list(r.conf)) for r in sp["rounds"]]))
                ctx.close()
    finally:
        lib.sb_set_default_option(8, 1)
        lib.sb_set_default_option(4, 1)
    for tokens, rounds in results[1:]:
        assert np.array_equal(tokens, results[0][0]) and rounds == results[0][1]
