"""Pins for the oracle's soft-gated forward (Eq. 6: bias log u_s beyond the window; Eq. 7: the
annealed gate).  Every check computes its expectation by a route of its own: multiplicative key
weights in numpy (the softmax of a score plus log u is the softmax of the score with the key's
exponential multiplied by u), explicit index sets for the limits, closed forms for a zero query."""
import math
import os

import numpy as np
import pytest

import oracle
from paper_2605_14037_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")
D = 128


def f64(bits):
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


def case(seed, T, G, spread=3.0):
    rng = np.random.default_rng(seed)
    K, V = synth.normal_bf16(rng, (T, D)), synth.normal_bf16(rng, (T, D))
    q = synth.normal_bf16(rng, (T, G, D))
    logit = (rng.standard_normal(T) * spread).astype(np.float32)
    return K, V, q, logit


def weighted_attend(q, K, V, weights, scale):
    """sum_s weights_s e^{score_s} v_s / sum_s weights_s e^{score_s} for the G heads of q (numpy)."""
    s = (f64(K) @ f64(q).T).T * scale                        # [G, T]
    e = np.exp(s - s.max(axis=1, keepdims=True)) * weights[None, :]
    return (e / e.sum(axis=1, keepdims=True)) @ f64(V)


def key_weights(t, w, logit, alpha, tau_l):
    """Weight of key s for query t: 0 in the future, 1 in the window, the (annealed) gate before it."""
    T = len(logit)
    u = 1.0 / (1.0 + np.exp(-logit.astype(np.float64)))
    z = (logit >= np.float32(tau_l)).astype(np.float64)
    gate = (1.0 - alpha) * u + alpha * z
    s = np.arange(T)
    return np.where(s > t, 0.0, np.where(t - s < w, 1.0, gate))


def test_gate_bias_extremes_as_the_paper_states_them():
    rows = [l.split() for l in open(os.path.join(GOLD, "soft_gate_extremes.txt")) if l[0] != "#"]
    stated = {float(u): float(b) for u, b in rows}
    assert stated == {0.0: -math.inf, 1.0: 0.0}
    # utility 1 <=> logit -> +inf, utility 0 <=> logit -> -inf
    assert oracle.gate_log_bias(np.inf) == stated[1.0] and abs(oracle.gate_log_bias(40.0)) < 1e-15
    assert oracle.gate_log_bias(-np.inf) == stated[0.0]
    # in between: the logarithm of the sigmoid, formed explicitly here
    for l in (-30.0, -5.0, -0.5, 0.0, 0.5, 5.0, 30.0):
        assert abs(oracle.gate_log_bias(l) - math.log(1.0 / (1.0 + math.exp(-l)))) < 1e-12
    assert abs(oracle.gate_log_bias(0.0) + math.log(2.0)) < 1e-15
    assert abs(oracle.gate_log_bias(-800.0) + 800.0) < 1e-9         # log sigma(l) -> l, no underflow to -inf
    # gates initialised fully open: bias 5 gives u = 0.993 (printed), a mask bias of log 0.993
    assert abs(oracle.gate_log_bias(5.0) - math.log(0.993)) < 5e-4


def test_annealed_gate_interpolates_between_soft_and_binary():
    tl = float(oracle.tau_logit(0.7))
    for l in (-3.0, 0.2, 0.84, 0.85, 2.5):
        l = float(np.float32(l))                 # logits are float32 numbers
        u, z = 1.0 / (1.0 + math.exp(-l)), (1.0 if np.float32(l) >= np.float32(tl) else 0.0)
        for alpha in (0.25, 0.5, 0.9):
            assert abs(oracle.gate_log_bias(l, alpha, tl) - math.log((1 - alpha) * u + alpha * z)) < 1e-12
        want = 0.0 if z else -math.inf
        assert oracle.gate_log_bias(l, 1.0, tl) == want
    # the threshold is inclusive (Eq. 2) and taken on the float32 logit
    assert oracle.gate_log_bias(np.float32(tl), 1.0, tl) == 0.0
    assert oracle.gate_log_bias(np.nextafter(np.float32(tl), np.float32(-9)), 1.0, tl) == -math.inf


@pytest.mark.parametrize("w,G,alpha", [(1, 1, 0.0), (4, 4, 0.0), (16, 2, 0.3), (128, 8, 0.0), (7, 3, 1.0)])
def test_soft_forward_equals_multiplicative_key_weights(w, G, alpha):
    T = 150
    K, V, q, logit = case(10 + w, T, G)
    scale = 1.0 / math.sqrt(D)
    tl = float(oracle.tau_logit(0.6))
    got, lse = oracle.soft_attend_all(K, V, logit, w, q, scale, alpha, tl, want_lse=True)
    for t in range(T):
        wts = key_weights(t, w, logit, alpha, tl)
        assert np.abs(got[t] - weighted_attend(q[t], K, V, wts, scale)).max() < 1e-11
        s = (f64(K) @ f64(q[t]).T).T * scale
        assert np.abs(lse[t] - np.log((np.exp(s) * wts[None, :]).sum(axis=1))).max() < 1e-10
        row = oracle.soft_attend_row(K, V, logit, t, w, q[t], scale, alpha, tl)
        assert np.array_equal(row, got[t])                    # the all-rows driver adds nothing


def np_softmax_attend(q, K, V, idx, scale):
    Kd, Vd, qd = f64(K)[idx], f64(V)[idx], f64(q)
    s = (Kd @ qd.T).T * scale
    p = np.exp(s - s.max(axis=1, keepdims=True))
    return (p / p.sum(axis=1, keepdims=True)) @ Vd


def test_all_gates_open_is_full_causal_attention_and_all_closed_is_the_window():
    T, G, w = 120, 4, 16
    K, V, q, _ = case(3, T, G)
    scale = 1.0 / math.sqrt(D)
    open_, shut = np.full(T, 40.0, np.float32), np.full(T, -np.inf, np.float32)
    nearly_shut = np.full(T, -800.0, np.float32)
    for t in (0, 5, 15, 16, 17, 63, T - 1):
        full = np_softmax_attend(q[t], K, V, list(range(t + 1)), scale)
        win = np_softmax_attend(q[t], K, V, list(range(max(0, t - w + 1), t + 1)), scale)
        assert np.abs(oracle.soft_attend_row(K, V, open_, t, w, q[t], scale) - full).max() < 1e-12
        assert np.abs(oracle.soft_attend_row(K, V, shut, t, w, q[t], scale) - win).max() < 1e-12
        assert np.abs(oracle.soft_attend_row(K, V, nearly_shut, t, w, q[t], scale) - win).max() < 1e-12
        # a window that covers the sequence: the gates do not matter
        assert np.abs(oracle.soft_attend_row(K, V, shut, t, T, q[t], scale) - full).max() < 1e-12


def test_fully_annealed_gate_is_the_hard_gated_forward():
    T, G, w = 140, 2, 8
    K, V, q, logit = case(4, T, G, spread=1.5)
    scale = 1.0 / math.sqrt(D)
    for tau in (0.3, 0.5, 0.8):
        tl = float(oracle.tau_logit(tau))
        for t in (0, 7, 8, 9, 70, T - 1):
            vis = [s for s in range(T) if s <= t and (t - s < w or np.float32(logit[s]) >= np.float32(tl))]
            want = np_softmax_attend(q[t], K, V, vis, scale)
            assert np.abs(oracle.soft_attend_row(K, V, logit, t, w, q[t], scale, 1.0, tl) - want).max() < 1e-12


def test_zero_query_closed_form():
    """q = 0: every score is 0, the weights are 1 inside the window and u_s before it, so the
    output is a weighted mean of the values and the log-sum-exp is the log of the total weight."""
    T, G, w = 90, 3, 10
    K, V, q, logit = case(5, T, G)
    q0 = np.zeros_like(q[0])
    for t in (0, 9, 10, 50, T - 1):
        u = 1.0 / (1.0 + np.exp(-logit.astype(np.float64)))
        n_out = max(0, t - w + 1)
        wts = np.concatenate([u[:n_out], np.ones(t + 1 - n_out)])
        want = (wts[:, None] * f64(V)[:t + 1]).sum(axis=0) / wts.sum()
        got, lse = oracle.soft_attend_row(K, V, logit, t, w, q0, 0.3, want_lse=True)
        assert np.abs(got - want[None, :]).max() < 1e-12
        assert np.abs(lse - math.log(wts.sum())).max() < 1e-12


def test_heads_of_a_group_are_independent_and_use_their_own_query():
    T, G, w = 60, 4, 6
    K, V, q, logit = case(6, T, G)
    scale = 1.0 / math.sqrt(D)
    t = 40
    group = oracle.soft_attend_row(K, V, logit, t, w, q[t], scale)
    for g in range(G):
        alone = oracle.soft_attend_row(K, V, logit, t, w, q[t, g:g + 1], scale)
        assert np.array_equal(alone[0], group[g])
    assert np.abs(group[0] - group[1]).max() > 1e-3
