"""Pins of the oracle's closed-form parts: Eq. 1 (temperature schedule), Eq. 2 (confidence),
Eq. 3-5 (analytic speed-up model).  Each expected value below comes from the mathematics or
from a library routine, never from the oracle itself or the CUDA path."""
import math
from pathlib import Path

import numpy as np
import pytest
import torch

from oracle import oracle

GOLDEN = Path(__file__).parent / "golden"


def read_golden(name):
    out = {}
    for line in (GOLDEN / name).read_text().splitlines():
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            out[k.strip()] = v.strip()
    return out


# ---- Eq. 1 -----------------------------------------------------------------------------------
@pytest.mark.parametrize("alpha,L", [(0.2, 32), (0.5, 4), (1.0, 40)])
def test_eq1_schedule_endpoints_and_slope(alpha, L):
    T = oracle.tau_schedule(alpha, L)
    assert T.shape == (L,)
    assert T[-1] == pytest.approx(1.0, abs=1e-15)                 # T_L = 1
    assert T[0] == pytest.approx(1 + alpha * (1 - 1 / L), abs=1e-15)  # Eq. 1 at l = 1
    assert np.allclose(T[:-1] - T[1:], alpha / L, atol=1e-15)     # linear, hotter when shallower
    assert np.all(T[:-1] > T[1:])


def test_eq1_paper_setting():
    s = read_golden("paper_settings.txt")
    T = oracle.tau_schedule(float(s["alpha"]), 32)
    # with alpha = 0.2 and L = 32: T_l = 1.2 - 0.00625 l
    assert np.allclose(T, 1.2 - 0.00625 * np.arange(1, 33), atol=1e-14)


# ---- Eq. 2 -----------------------------------------------------------------------------------
def test_eq2_uniform_logits_give_one_over_V():
    for V in (2, 7, 1024):
        p, t = oracle.confidence(np.full(V, 3.25), 1.7)
        assert p == pytest.approx(1.0 / V, rel=1e-14)
        assert t == 0                                              # ties: lowest index


def test_eq2_dominant_logit_gives_one():
    z = np.zeros(100)
    z[37] = 800.0
    p, t = oracle.confidence(z, 1.0)
    assert t == 37 and p == pytest.approx(1.0, abs=1e-15)


def test_eq2_matches_library_softmax_and_is_monotone_in_T():
    rng = np.random.default_rng(0)
    z = rng.normal(0, 5, size=1000)
    last = 1.1
    for T in (0.5, 1.0, 1.2, 1.5, 2.0, 10.0, 1e6):
        p, t = oracle.confidence(z, T)
        ref = torch.softmax(torch.from_numpy(z) / T, dim=0)
        assert t == int(torch.argmax(torch.from_numpy(z)))
        assert p == pytest.approx(float(ref.max()), rel=1e-12)
        assert p <= last + 1e-15                                   # non-increasing in T
        last = p
    assert last == pytest.approx(1e-3, rel=1e-4)                   # T -> inf: 1/V


def test_eq2_two_logit_closed_form():
    # softmax max over {a, b} at temperature T is the logistic of |a-b|/T
    for a, b, T in [(1.0, 0.0, 1.0), (2.5, -1.0, 2.0), (0.3, 0.4, 1.5)]:
        p, t = oracle.confidence(np.array([a, b]), T)
        assert p == pytest.approx(1.0 / (1.0 + math.exp(-abs(a - b) / T)), rel=1e-14)
        assert t == (0 if a >= b else 1)


def test_eq2_tie_break_lowest_index():
    z = np.array([0.0, 4.0, 1.0, 4.0, 4.0])
    p, t = oracle.confidence(z, 1.0)
    assert t == 1


# ---- Eq. 3-5 ---------------------------------------------------------------------------------
def test_eq3_round_cost():
    assert oracle.round_cost(32, 8, 10) == pytest.approx((8 * 10 + 32 - 10) / 32)
    assert oracle.round_cost(32, 1, 32) == pytest.approx(1.0)      # one row, all layers = one AR step


@pytest.mark.parametrize("a", [0.0, 0.1, 0.5, 0.9, 0.99])
@pytest.mark.parametrize("w", [1, 2, 4, 8])
def test_eq4_sum_equals_closed_form(a, w):
    closed = a * (1 - a ** w) / (1 - a)
    assert oracle.expected_accepted(a, w) == pytest.approx(closed, rel=1e-12, abs=1e-15)


def test_eq4_monte_carlo():
    # geometric acceptance: each draft survives with probability a, stop at the first failure
    rng = np.random.default_rng(1)
    a, w = 0.7, 6
    ok = rng.random((200000, w)) < a
    n_acc = np.where(ok.all(axis=1), w, np.argmin(ok, axis=1))
    assert oracle.expected_accepted(a, w) == pytest.approx(n_acc.mean(), rel=5e-3)


def test_eq5_is_eq4_over_eq3_and_paper_setting():
    s = read_golden("paper_settings.txt")
    w, d_max = int(s["w_max"]), int(s["d_max"])
    for L, a in [(32, 0.9), (40, 0.6), (32, 0.3)]:
        sd = oracle.speedup(L, a, w, d_max)
        assert sd == pytest.approx(oracle.expected_accepted(a, w) / oracle.round_cost(L, w, d_max), rel=1e-12)
    # hand value: 32*0.9*(1-0.9^8) / (0.1*(80+22)) = 1.6081...
    assert oracle.speedup(32, 0.9, 8, 10) == pytest.approx(32 * 0.9 * (1 - 0.9 ** 8) / (0.1 * 102), rel=1e-13)
    assert oracle.speedup(32, 0.9, 8, 10) == pytest.approx(1.608, abs=5e-4)
