"""Pins of the oracle's sink-token variant (the "Fixed Attention Sinks" row of the paper's
ablation table; the evaluation protocol keeps four sink tokens for every method): the first
n_sink positions stay visible whatever their gate says.  Checked against brute-force visible
sets, the limits that reduce to known attention patterns, and mask form == streaming form."""
import math

import numpy as np
import pytest

import oracle
from paper_2605_14037_b200 import synth

D = 128


def f64(bits):
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


def visible_set(t, w, logit, tau_l, n_sink):
    return [s for s in range(len(logit))
            if s <= t and ((t - s) < w or np.float32(logit[s]) >= np.float32(tau_l) or s < n_sink)]


def run_stream(K, V, q, logit, w, tau_l, scale, n_sink):
    u = oracle.Unit(w, D, n_sink=n_sink)
    outs = []
    for t in range(K.shape[0]):
        u.append(K[t], V[t], logit[t], tau_l)
        outs.append(u.attend(q[t], scale))
    return np.stack(outs), u


def case(seed, T, G, rate, tl):
    rng = np.random.default_rng(seed)
    K = synth.normal_bf16(rng, (T, D))
    V = synth.normal_bf16(rng, (T, D))
    q = synth.normal_bf16(rng, (T, G, D))
    logit = synth.logits_with_keep_rate(rng, (T,), rate, tl if math.isfinite(tl) else 0.0)
    return K, V, q, logit


@pytest.mark.parametrize("form", ["mask", "stream"])
@pytest.mark.parametrize("w,n_sink,tau", [(1, 4, 0.5), (4, 1, 0.9), (16, 4, np.inf), (128, 4, 0.5),
                                          (8, 20, 0.5)])
def test_visible_set_with_sinks_enumerated(form, w, n_sink, tau):
    """q = 0 gives uniform weights; one-hot values then spell out the visible set."""
    T = 170
    rng = np.random.default_rng(7)
    tl = float(oracle.tau_logit(tau)) if math.isfinite(tau) else tau
    logit = synth.logits_with_keep_rate(rng, (T,), 0.3, tl if math.isfinite(tl) else 0.0)
    K = synth.normal_bf16(rng, (T, D))
    Vf = np.zeros((T, D), np.float32)
    Vf[np.arange(T), np.arange(T) % D] = 1.0 + (np.arange(T) // D)
    V = synth.to_bf16_bits(Vf)
    q = np.zeros((T, 1, D), np.uint16)
    if form == "mask":
        got = oracle.mask_attend_all(K, V, logit, w, tl, q, 1.0, n_sink=n_sink)
    else:
        got, _ = run_stream(K, V, q, logit, w, tl, 1.0, n_sink)
    for t in range(T):
        vis = visible_set(t, w, logit, tl, n_sink)
        want = np.zeros(D)
        for s in vis:
            want[s % D] += (1.0 + s // D) / len(vis)
        np.testing.assert_allclose(got[t, 0], want, rtol=0, atol=1e-14)


@pytest.mark.parametrize("w,G,n_sink,tau", [(1, 1, 4, 0.5), (4, 4, 2, 0.2), (128, 8, 4, 0.5),
                                            (16, 2, 4, np.inf), (16, 2, 4, -np.inf)])
def test_mask_equals_stream_with_sinks(w, G, n_sink, tau):
    T = 260
    tl = float(oracle.tau_logit(tau)) if math.isfinite(tau) else tau
    K, V, q, logit = case(300 + w + G, T, G, 0.35, tl)
    scale = 1.0 / math.sqrt(D)
    a = oracle.mask_attend_all(K, V, logit, w, tl, q, scale, n_sink=n_sink)
    b, u = run_stream(K, V, q, logit, w, tl, scale, n_sink)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-12)
    want_pos = [s for s in range(T)
                if s <= T - 1 - w and (np.float32(logit[s]) >= np.float32(tl) or s < n_sink)]
    pos, kk, vv = u.kept()
    assert pos.tolist() == want_pos
    assert np.array_equal(kk, K[want_pos]) and np.array_equal(vv, V[want_pos])


def test_limits_with_sinks():
    """tau = +inf: sinks + sliding window (the attention-sink pattern); n_sink >= T: full causal
    attention whatever tau; n_sink = 0: the method as defined."""
    T, G, w = 150, 2, 8
    scale = 1.0 / math.sqrt(D)
    K, V, q, logit = case(11, T, G, 0.4, 0.0)
    Kd, Vd = f64(K), f64(V)

    def dense(t, idx):
        s = (Kd[idx] @ f64(q[t]).T).T * scale
        p = np.exp(s - s.max(axis=1, keepdims=True))
        return (p / p.sum(axis=1, keepdims=True)) @ Vd[idx]

    got = oracle.mask_attend_all(K, V, logit, w, np.inf, q, scale, n_sink=4)
    for t in range(T):
        idx = sorted(set(range(min(4, t + 1))) | set(range(max(0, t - w + 1), t + 1)))
        np.testing.assert_allclose(got[t], dense(t, idx), rtol=0, atol=1e-12)
    got = oracle.mask_attend_all(K, V, logit, w, np.inf, q, scale, n_sink=T)
    for t in range(T):
        np.testing.assert_allclose(got[t], dense(t, list(range(t + 1))), rtol=0, atol=1e-12)
    a = oracle.mask_attend_all(K, V, logit, w, 0.0, q, scale, n_sink=0)
    b = oracle.mask_attend_all(K, V, logit, w, 0.0, q, scale)
    assert np.array_equal(a, b)


def test_sinks_change_only_rows_that_lost_a_gated_off_sink():
    """A row differs from the sink-free result iff one of the first n_sink positions is outside
    its window and gated off."""
    T, w, n_sink = 120, 8, 4
    K, V, q, logit = case(12, T, 1, 0.0, 0.0)       # keep rate 0: every gate closed
    scale = 1.0 / math.sqrt(D)
    a = oracle.mask_attend_all(K, V, logit, w, 0.0, q, scale)
    b = oracle.mask_attend_all(K, V, logit, w, 0.0, q, scale, n_sink=n_sink)
    for t in range(T):
        lost = any(t - s >= w for s in range(min(n_sink, t + 1)))
        assert (not np.array_equal(a[t], b[t])) == lost
