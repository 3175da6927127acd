"""Pins for the CPU oracle: closed forms, limiting cases, brute force.

Each test checks the oracle against something fixed by the paper or by the
mathematics and computed here by an independent route (index sets enumerated by
Python loops from the definitions, numpy library routines, printed constants),
never by the oracle's own code.
"""
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


def visible_set(t, w, logit, tau_l):
    """Eq. 2-4 by brute force: s visible for query t."""
    return [s for s in range(len(logit))
            if s <= t and ((t - s) < w or np.float32(logit[s]) >= np.float32(tau_l))]


def np_softmax_attend(q, K, V, idx, scale):
    """Dense softmax attention over an explicit index set (numpy, float64)."""
    Kd, Vd, qd = f64(K)[idx], f64(V)[idx], f64(q)
    s = (Kd @ qd.T).T * scale               # [G, n]
    s = s - s.max(axis=1, keepdims=True)
    p = np.exp(s)
    p /= p.sum(axis=1, keepdims=True)
    return p @ Vd


def rand_case(seed, T, G, rate=0.3, tau=0.5):
    rng = np.random.default_rng(seed)
    K = synth.normal_bf16(rng, (T, D))
    V = synth.normal_bf16(rng, (T, D))
    q = synth.normal_bf16(rng, (T, G, D))
    tl = float(oracle.tau_logit(tau))
    logit = synth.logits_with_keep_rate(rng, (T,), rate, tl if math.isfinite(tl) else 0.0)
    return K, V, q, logit


def run_stream(K, V, q, logit, w, tau_l, scale):
    """Streaming form over a whole sequence: outputs at every t and the final unit."""
    u = oracle.Unit(w, D)
    outs = []
    for t in range(K.shape[0]):
        u.append(K[t], V[t], logit[t], tau_l)
        outs.append(u.attend(q[t], scale))
    return np.stack(outs), u


# ----------------------------------------------------------------- constants

def test_sigmoid_printed_value():
    rows = [l.split() for l in open(os.path.join(GOLD, "sigmoid_init.txt")) if l[0] != "#"]
    for z, printed in rows:
        assert abs(oracle.sigmoid(float(z)) - float(printed)) < 5e-4
    assert oracle.sigmoid(0.0) == 0.5
    assert abs(oracle.sigmoid(-3.0) + oracle.sigmoid(3.0) - 1.0) < 1e-15


def test_tau_logit_limits_and_monotone_equivalence():
    assert oracle.tau_logit(0.5) == 0.0
    assert oracle.tau_logit(0.0) == -np.inf and oracle.tau_logit(-1.0) == -np.inf
    assert oracle.tau_logit(1.0) == np.inf and oracle.tau_logit(2.0) == np.inf
    assert abs(float(oracle.tau_logit(0.9)) - math.log(9.0)) < 1e-6
    rng = np.random.default_rng(0)
    for tau in (0.01, 0.2, 0.5, 0.7, 0.99):
        tl = float(oracle.tau_logit(tau))
        z = rng.standard_normal(2000) * 4
        z = z[np.abs(z - tl) > 1e-4]
        u = np.array([oracle.sigmoid(x) for x in z])
        assert np.array_equal(u >= tau, z.astype(np.float32) >= np.float32(tl))


def test_bf16_widening_exact():
    bits = np.array([0x0000, 0x3F80, 0xBF80, 0x4049, 0x0001, 0x7F7F, 0x8000, 0x3DCC], np.uint16)
    want = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    assert np.array_equal(oracle.bf16_to_double(bits), want)
    assert oracle.bf16_to_double(np.array([0x3F80], np.uint16))[0] == 1.0
    assert oracle.bf16_to_double(np.array([0x4049], np.uint16))[0] == 3.140625


# --------------------------------------------------------------- Eq. 1 scores

def test_score_linear_matches_matmul_and_onehot():
    rng = np.random.default_rng(1)
    x = synth.normal_bf16(rng, (37, 512))
    W = synth.linear_predictor(rng, 3, 512)
    b = rng.standard_normal(3).astype(np.float32)
    got = oracle.score_linear(x, W, b)
    want = f64(x) @ f64(W).T + b.astype(np.float64)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)
    # one-hot rows pick single inputs: logit = x[:, i] + b
    W1 = np.zeros((2, 512), np.float32)
    W1[0, 7] = 1.0
    W1[1, 300] = -2.0
    got = oracle.score_linear(x, synth.to_bf16_bits(W1), b[:2])
    np.testing.assert_array_equal(got[:, 0], f64(x)[:, 7] + float(b[0]))
    np.testing.assert_array_equal(got[:, 1], -2.0 * f64(x)[:, 300] + float(b[1]))


def test_score_mlp_matches_numpy_and_silu_values():
    rng = np.random.default_rng(2)
    x = synth.normal_bf16(rng, (11, 96))
    W1, b1, W2, b2 = synth.mlp_predictor(rng, 4, 96, 40)
    got = oracle.score_mlp(x, W1, b1, W2, b2)
    z = f64(x) @ f64(W1).T + b1.astype(np.float64)
    a = z / (1.0 + np.exp(-z))
    want = a @ f64(W2).T + b2.astype(np.float64)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)
    # d_in = hidden = heads = 1, W1 = W2 = 1, no bias: logit = SiLU(x); SiLU(1) = 1/(1+1/e)
    one = synth.to_bf16_bits(np.ones((1, 1), np.float32))
    zero = np.zeros(1, np.float32)
    got = oracle.score_mlp(one, one, zero, one, zero)
    assert abs(got[0, 0] - 1.0 / (1.0 + math.exp(-1.0))) < 1e-15
    neg = synth.to_bf16_bits(np.full((1, 1), -2.0, np.float32))
    got = oracle.score_mlp(neg, one, zero, one, zero)
    assert abs(got[0, 0] - (-2.0 / (1.0 + math.exp(2.0)))) < 1e-15


# ------------------------------------------------- limiting cases (both forms)

@pytest.mark.parametrize("form", ["mask", "stream"])
@pytest.mark.parametrize("tau,w,expect", [
    (-np.inf, 8, "full"),      # all gates open: full causal attention
    (np.inf, 8, "window"),     # no gate open: sliding-window attention
    (0.5, 1000, "full"),       # window covers the sequence: full for any tau
    (np.inf, 1, "self"),       # w = 1, nothing kept: each query sees only itself
])
def test_limits(form, tau, w, expect):
    T, G = 70, 2
    K, V, q, logit = rand_case(3, T, G)
    tl = float(oracle.tau_logit(tau)) if math.isfinite(tau) else tau
    scale = 1.0 / math.sqrt(D)
    if form == "mask":
        got = oracle.mask_attend_all(K, V, logit, w, tl, q, scale)
    else:
        got, _ = run_stream(K, V, q, logit, w, tl, scale)
    for t in range(T):
        if expect == "full":
            idx = list(range(t + 1))
        elif expect == "window":
            idx = list(range(max(0, t - w + 1), t + 1))
        else:
            idx = [t]
        want = np_softmax_attend(q[t], K, V, idx, scale)
        np.testing.assert_allclose(got[t], want, rtol=0, atol=1e-12)
        if expect == "self":
            np.testing.assert_allclose(got[t], np.broadcast_to(f64(V)[t], (G, D)), atol=1e-15)


# ----------------------------- visible set enumerated with one-hot values, q = 0

@pytest.mark.parametrize("form", ["mask", "stream"])
@pytest.mark.parametrize("w,tau", [(1, 0.5), (4, 0.2), (16, 0.9), (128, 0.5)])
def test_visible_set_enumeration(form, w, tau):
    T, G = 150, 1
    rng = np.random.default_rng(4)
    tl = float(oracle.tau_logit(tau))
    logit = synth.logits_with_keep_rate(rng, (T,), 0.35, tl)
    K = synth.normal_bf16(rng, (T, D))
    # values: token s carries a one at column s mod D and a two-digit "page" marker
    Vf = np.zeros((T, D), np.float32)
    Vf[np.arange(T), np.arange(T) % D] = 1.0 + (np.arange(T) // D)
    V = synth.to_bf16_bits(Vf)
    q = np.zeros((T, G, D), np.uint16)          # zero query: uniform weights
    if form == "mask":
        got = oracle.mask_attend_all(K, V, logit, w, tl, q, 1.0)
    else:
        got, _ = run_stream(K, V, q, logit, w, tl, 1.0)
    for t in range(T):
        vis = visible_set(t, w, logit, tl)
        want = np.zeros(D)
        for s in vis:
            want[s % D] += (1.0 + s // D) / len(vis)
        np.testing.assert_allclose(got[t, 0], want, rtol=0, atol=1e-14)


# ------------------------------------------------------ mask form == streaming

@pytest.mark.parametrize("w", [1, 2, 4, 128])
@pytest.mark.parametrize("G", [1, 4, 8])
@pytest.mark.parametrize("tau", [-np.inf, 0.2, 0.5, 0.9, np.inf])
def test_mask_equals_stream(w, G, tau):
    T = 200 if w < 128 else 300
    K, V, q, logit = rand_case(100 + w + G, T, G, rate=0.4, tau=tau if math.isfinite(tau) else 0.5)
    tl = float(oracle.tau_logit(tau)) if math.isfinite(tau) else tau
    scale = 1.0 / math.sqrt(D)
    a = oracle.mask_attend_all(K, V, logit, w, tl, q, scale)
    b, u = run_stream(K, V, q, logit, w, tl, scale)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-12)
    # kept-set identity: the pairs outside the last query's window that pass the threshold
    want_pos = [s for s in range(T) if s <= T - 1 - w and np.float32(logit[s]) >= np.float32(tl)]
    pos, kk, vv = u.kept()
    assert pos.tolist() == want_pos and len(u) == len(want_pos)
    assert np.array_equal(kk, K[want_pos]) and np.array_equal(vv, V[want_pos])
    wpos, wk, wv, wl = u.window()
    first = max(0, T - w)
    assert wpos.tolist() == list(range(first, T))
    assert np.array_equal(wk, K[first:]) and np.array_equal(wv, V[first:])
    assert np.array_equal(wl, logit[first:])


def test_mask_row_matches_explicit_set_with_random_queries():
    T, G, w = 400, 4, 16
    K, V, q, logit = rand_case(7, T, G, rate=0.25)
    tl = 0.0
    for t in (0, 1, 15, 16, 17, 200, 399):
        got, lse = oracle.mask_attend_row(K, V, logit, t, w, tl, q[t], 0.3, want_lse=True)
        vis = visible_set(t, w, logit, tl)
        want = np_softmax_attend(q[t], K, V, vis, 0.3)
        np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)
        s = (f64(K)[vis] @ f64(q[t]).T).T * 0.3
        want_lse = np.log(np.exp(s - s.max(axis=1, keepdims=True)).sum(axis=1)) + s.max(axis=1)
        np.testing.assert_allclose(lse, want_lse, rtol=0, atol=1e-12)


# --------------------------------------------------------- closed-form cases

@pytest.mark.parametrize("form", ["mask", "stream"])
def test_dominant_key_and_identical_keys(form):
    T, w, G = 40, 4, 2
    rng = np.random.default_rng(8)
    V = synth.normal_bf16(rng, (T, D))
    logit = np.full(T, 1.0, np.float32)       # everything kept
    # (a) identical keys: uniform weights whatever the query -> running mean of v
    K = np.tile(synth.normal_bf16(rng, (1, D)), (T, 1))
    q = synth.normal_bf16(rng, (T, G, D))
    got = (oracle.mask_attend_all(K, V, logit, w, 0.0, q, 1.0) if form == "mask"
           else run_stream(K, V, q, logit, w, 0.0, 1.0)[0])
    for t in range(T):
        np.testing.assert_allclose(got[t, 0], f64(V)[:t + 1].mean(axis=0), atol=1e-12)
    # (b) one key with an enormous score: output is its value, no overflow
    Kf = np.zeros((T, D), np.float32)
    Kf[5, 0] = 200.0
    qf = np.zeros((T, G, D), np.float32)
    qf[:, :, 0] = 100.0
    K, q = synth.to_bf16_bits(Kf), synth.to_bf16_bits(qf)
    got = (oracle.mask_attend_all(K, V, logit, w, 0.0, q, 1.0) if form == "mask"
           else run_stream(K, V, q, logit, w, 0.0, 1.0)[0])
    assert np.isfinite(got).all()
    for t in range(5, T):
        np.testing.assert_allclose(got[t, 1], f64(V)[5], atol=1e-12)


def test_scale_zero_gives_uniform_and_gqa_heads_independent():
    T, w = 30, 4
    K, V, q, logit = rand_case(9, T, 4)
    got = oracle.mask_attend_all(K, V, logit, w, 0.0, q, 0.0)
    for t in range(T):
        vis = visible_set(t, w, logit, 0.0)
        np.testing.assert_allclose(got[t, 2], f64(V)[vis].mean(axis=0), atol=1e-13)
    # each query head of the group is computed from its own query only
    full = oracle.mask_attend_all(K, V, logit, w, 0.0, q, 0.1)
    for g in range(4):
        single = oracle.mask_attend_all(K, V, logit, w, 0.0, np.ascontiguousarray(q[:, g:g + 1]), 0.1)
        np.testing.assert_array_equal(full[:, g], single[:, 0])


def test_log_sum_exp_merge_of_any_partition():
    """Partial softmax results over a partition of the keys, merged by their
    log-sum-exp weights, equal the unsplit result (what a split-K kernel relies on)."""
    n, G = 90, 4
    rng = np.random.default_rng(10)
    K, V = synth.normal_bf16(rng, (n, D)), synth.normal_bf16(rng, (n, D))
    q = synth.normal_bf16(rng, (G, D))
    scale = 0.2

    def ring_only(idx):
        u = oracle.Unit(1000, D)
        for s in idx:
            u.append(K[s], V[s], 0.0, 0.0)
        return u.attend(q, scale, want_lse=True)

    whole, lse_w = ring_only(range(n))
    parts = [range(0, 7), range(7, 64), range(64, 65), range(65, 90)]
    outs, lses = zip(*[ring_only(p) for p in parts])
    lses = np.stack(lses)                                 # [parts, G]
    m = lses.max(axis=0)
    wgt = np.exp(lses - m)
    merged = sum(wgt[i][:, None] * outs[i] for i in range(len(parts))) / wgt.sum(axis=0)[:, None]
    np.testing.assert_allclose(merged, whole, rtol=0, atol=1e-12)
    np.testing.assert_allclose(m + np.log(wgt.sum(axis=0)), lse_w, rtol=0, atol=1e-12)
    np.testing.assert_allclose(whole, np_softmax_attend(q, K, V, list(range(n)), scale), atol=1e-12)


# ------------------------------------------------------- state equivalences

@pytest.mark.parametrize("chunk", [1, 16, 127, 128, 129, 500])
def test_chunked_prefill_equals_token_by_token(chunk):
    T, w, G = 500, 128, 2
    K, V, q, logit = rand_case(11, T, G, rate=0.3)
    scale = 1.0 / math.sqrt(D)
    ref, u_ref = run_stream(K, V, q, logit, w, 0.0, scale)
    u = oracle.Unit(w, D)
    outs = []
    for a in range(0, T, chunk):
        outs.append(u.prefill(K[a:a + chunk], V[a:a + chunk], logit[a:a + chunk], 0.0,
                              q[a:a + chunk], scale))
    np.testing.assert_array_equal(np.concatenate(outs), ref)
    for x, y in zip(u.kept(), u_ref.kept()):
        assert np.array_equal(x, y)
    for x, y in zip(u.window(), u_ref.window()):
        assert np.array_equal(x, y)


def test_threshold_applied_at_window_exit_with_current_tau():
    """A pair is judged when it leaves the ring, with the threshold in force then."""
    w, T = 4, 20
    rng = np.random.default_rng(12)
    K, V = synth.normal_bf16(rng, (T, D)), synth.normal_bf16(rng, (T, D))
    logit = np.linspace(-1.0, 1.0, T).astype(np.float32)
    u = oracle.Unit(w, D)
    for t in range(T):
        tl = -0.5 if t < 12 else 0.5      # position t-w is judged at step t
        u.append(K[t], V[t], logit[t], tl)
    want = [s for s in range(T - w) if logit[s] >= (-0.5 if s + w < 12 else 0.5)]
    assert u.kept()[0].tolist() == want


def test_batch_step_equals_single_units():
    n, G, w = 6, 4, 8
    rng = np.random.default_rng(13)
    units_a = [oracle.Unit(w, D) for _ in range(n)]
    units_b = [oracle.Unit(w, D) for _ in range(n)]
    for step in range(30):
        k, v = synth.normal_bf16(rng, (n, D)), synth.normal_bf16(rng, (n, D))
        q = synth.normal_bf16(rng, (n, G, D))
        lg = rng.standard_normal(n).astype(np.float32)
        got = oracle.step_batch(units_a, k, v, lg, 0.0, q, 0.1)
        for i, u in enumerate(units_b):
            u.append(k[i], v[i], lg[i], 0.0)
            np.testing.assert_array_equal(got[i], u.attend(q[i], 0.1))
    kk = synth.normal_bf16(rng, (n, 50, D))
    vv = synth.normal_bf16(rng, (n, 50, D))
    ll = rng.standard_normal((n, 50)).astype(np.float32)
    oracle.prefill_batch(units_a, kk, vv, ll, 0.0)
    for i, u in enumerate(units_b):
        u.prefill(kk[i], vv[i], ll[i], 0.0)
        assert np.array_equal(u.kept()[0], units_a[i].kept()[0])
        assert u.t == units_a[i].t == 80


# ------------------------------------------------------------ Eq. 8 density

def test_density_and_accounting():
    T, w = 5000, 128
    rng = np.random.default_rng(14)
    logit = synth.logits_with_keep_rate(rng, (T,), 0.2, 0.0)
    rho_all, rho_cache = oracle.density(logit, w, 0.0)
    z = logit >= 0
    assert abs(rho_all - z.mean()) < 1e-15
    assert abs(rho_cache - z[:T - w].mean()) < 1e-15
    u = oracle.Unit(w, D)
    zero = np.zeros(D, np.uint16)
    for t in range(T):
        u.append(zero, zero, logit[t], 0.0)
    assert len(u) == int(z[:T - w].sum())
    # pairs read per decode step relative to dense: rho*(T-w)/T + w/T
    assert abs((len(u) + w) / T - (rho_cache * (T - w) / T + w / T)) < 1e-15
    # printed equivalence: 80 % sparsity <=> a 5x shorter sequence of q-k products
    sp, factor = [float(x) for x in
                  [l for l in open(os.path.join(GOLD, "sparsity_equivalence.txt")) if l[0] != "#"][0].split()]
    all_kept = np.full(T, 1.0, np.float32)
    all_kept[rng.random(T) < sp] = -1.0
    r, _ = oracle.density(all_kept, 0, 0.0)
    assert abs(1.0 / r - factor) < 0.2


@pytest.mark.parametrize("form", ["mask", "stream"])
def test_threshold_is_inclusive(form):
    """Eq. 2 uses >=: a utility exactly at the threshold is kept."""
    T, w = 12, 2
    rng = np.random.default_rng(15)
    K = synth.normal_bf16(rng, (T, D))
    Vf = np.zeros((T, D), np.float32)
    Vf[np.arange(T), np.arange(T)] = 1.0
    V = synth.to_bf16_bits(Vf)
    tl = float(oracle.tau_logit(0.7))
    logit = np.full(T, tl - 1.0, np.float32)
    logit[3] = np.float32(tl)                       # exactly at the threshold
    logit[5] = np.nextafter(np.float32(tl), np.float32(-np.inf))   # just below
    q = np.zeros((T, 1, D), np.uint16)
    got = (oracle.mask_attend_all(K, V, logit, w, tl, q, 1.0) if form == "mask"
           else run_stream(K, V, q, logit, w, tl, 1.0)[0])
    last = got[T - 1, 0]
    assert last[3] > 0 and last[5] == 0 and abs(last[3] - 1.0 / 3.0) < 1e-15
