"""Pins of the step-wise KL oracle against things other than itself: closed forms, a library routine,
brute force in plain Python, and the invariances the definition implies (Sec. "KL-ST Stage")."""
import math

import numpy as np
import pytest

import oracle
from paper_2602_02711_b200 import inputs


def test_identical_logits_give_zero_and_kl_is_nonnegative():
    high, low = inputs.logit_pair(6, 257, seed=1)
    ks, kt = oracle.stepwise_kl(high, high, [0, 6])
    assert np.all(kt == 0.0) and ks[0] == 0.0
    _, kt = oracle.stepwise_kl(high, low, [0, 6])
    assert np.all(kt > 0.0)


def test_two_outcome_closed_form():
    # V = 2, logits (a, 0) and (b, 0): Bernoulli distributions with p = sigmoid(a), q = sigmoid(b)
    for a, b in [(0.3, -1.2), (4.0, 3.5), (-7.0, 2.0), (0.0, 0.0)]:
        p, q = 1 / (1 + math.exp(-a)), 1 / (1 + math.exp(-b))
        want = p * math.log(p / q) + (1 - p) * math.log((1 - p) / (1 - q))
        _, kt = oracle.stepwise_kl(np.array([[a, 0.0]]), np.array([[b, 0.0]]), [0, 1])
        assert kt[0] == pytest.approx(want, rel=1e-12, abs=1e-15)


def test_uniform_against_one_raised_entry_closed_form():
    # p uniform over V entries, q has one logit raised by c: KL = log(V - 1 + e^c) - log V - c / V
    V, c = 1000, 3.0
    b = np.zeros((1, V))
    b[0, 17] = c
    want = math.log(V - 1 + math.exp(c)) - math.log(V) - c / V
    _, kt = oracle.stepwise_kl(np.zeros((1, V)), b, [0, 1])
    assert kt[0] == pytest.approx(want, rel=1e-12)
    # and the other direction is a different number (KL is not symmetric: a swapped operand shows)
    _, kr = oracle.stepwise_kl(b, np.zeros((1, V)), [0, 1])
    q0 = math.exp(c) / (V - 1 + math.exp(c))
    want_r = q0 * c - math.log(V - 1 + math.exp(c)) + math.log(V)
    assert kr[0] == pytest.approx(want_r, rel=1e-12)
    assert abs(kr[0] - kt[0]) > 1e-3


def test_matches_scipy_softmax_and_rel_entr():
    sp = pytest.importorskip("scipy.special")
    high, low = inputs.logit_pair(5, 300, seed=2)
    _, kt = oracle.stepwise_kl(high, low, [0, 5])
    for i in range(5):
        want = float(np.sum(sp.rel_entr(sp.softmax(high[i]), sp.softmax(low[i]))))
        assert kt[i] == pytest.approx(want, rel=1e-10)


def test_brute_force_in_plain_python():
    high, low = inputs.logit_pair(3, 11, seed=3)
    _, kt = oracle.stepwise_kl(high, low, [0, 3])
    for i in range(3):
        za = math.fsum(math.exp(x) for x in high[i])
        zb = math.fsum(math.exp(x) for x in low[i])
        want = math.fsum((math.exp(x) / za) * ((x - math.log(za)) - (y - math.log(zb))) for x, y in zip(high[i], low[i]))
        assert kt[i] == pytest.approx(want, rel=1e-11)


def test_shift_invariance_and_zero_probability_entries():
    high, low = inputs.logit_pair(4, 64, seed=4)
    _, kt = oracle.stepwise_kl(high, low, [0, 4])
    _, k2 = oracle.stepwise_kl(high + 5.0, low - 11.0, [0, 4])     # softmax ignores a constant per row
    assert np.allclose(kt, k2, rtol=1e-11, atol=1e-14)
    # an entry the high-precision model gives probability 0 contributes nothing, whatever the other model says
    h2, l2 = high.copy(), low.copy()
    h2 = np.concatenate([h2, np.full((4, 1), -np.inf)], axis=1)
    for extra in (0.0, -np.inf):
        lx = np.concatenate([l2, np.full((4, 1), extra)], axis=1)
        _, k3 = oracle.stepwise_kl(h2, lx, [0, 4])
        assert np.all(np.isfinite(k3))
    lx = np.concatenate([l2, np.full((4, 1), -np.inf)], axis=1)
    _, k3 = oracle.stepwise_kl(h2, lx, [0, 4])
    assert np.allclose(k3, kt, rtol=1e-11, atol=1e-14)


def test_step_means_and_empty_steps():
    high, low = inputs.logit_pair(10, 50, seed=5)
    offs = [0, 3, 3, 4, 10]
    ks, kt = oracle.stepwise_kl(high, low, offs)
    assert ks[0] == pytest.approx((kt[0] + kt[1] + kt[2]) / 3, rel=1e-14)
    assert ks[1] == 0.0                       # a step without action tokens
    assert ks[2] == kt[3]
    assert ks[3] == pytest.approx(math.fsum(kt[4:10]) / 6, rel=1e-14)


def test_bf16_inputs_are_read_as_their_exact_values():
    high, low = inputs.logit_pair(2, 40, seed=6)
    hb, lb = inputs.f64_to_bf16_bits(high), inputs.f64_to_bf16_bits(low)
    _, k1 = oracle.stepwise_kl(hb, lb, [0, 2])
    _, k2 = oracle.stepwise_kl(inputs.bf16_bits_to_f64(hb), inputs.bf16_bits_to_f64(lb), [0, 2])
    assert np.array_equal(k1, k2)


def test_synthetic_logits_have_a_dense_low_mode_and_a_rare_high_mode():
    # the recipe mirrors what the paper reports about the KL distribution: most steps low, a few far higher
    high, low = inputs.logit_pair(200, 512, seed=7, critical_frac=0.1)
    _, kt = oracle.stepwise_kl(high, low, [0, 200])
    lo, hi = np.sum(kt < 0.05), np.sum(kt > 0.3)
    assert lo > 150 and 5 <= hi <= 40
