"""GPU parity, step 2 (append + evict): lengths, kept positions and their order, K/V
bytes and ring contents must equal the oracle's bit for bit."""
import math

import numpy as np
import pytest
import torch

import oracle
from gpu_util import D, Workload, compare_state, dev, load, oracle_units, to_dev_bf16

pytestmark = pytest.mark.gpu


def run_appends(cache, layer, seq_ids, wl, first=0, last=None):
    last = wl.T if last is None else last
    ids = torch.tensor(seq_ids, dtype=torch.int32, device=dev())
    K, V = to_dev_bf16(wl.K), to_dev_bf16(wl.V)
    lg = torch.from_numpy(wl.logit).to(dev())
    for t in range(first, last):
        cache.spkv_append_evict(layer, ids, K[t], V[t], lg[t])


@pytest.mark.parametrize("w,T,tau,rates", [
    (128, 700, 0.5, [0.2, 0.6]),        # several pages per unit, ragged tails
    (128, 100, 0.5, [0.5, 0.5]),        # t < w: nothing leaves the ring
    (1, 300, 0.5, [0.3, 0.9]),          # smallest window
    (4, 300, 0.9, [0.5, 0.1]),
    (100, 500, 0.2, [0.4, 0.7]),        # ring not a multiple of the page size
    (200, 650, 0.5, [0.3, 1.0]),        # four ring pages
    (128, 400, 0.5, [0.0, 1.0]),        # local-only head and keep-everything head
    (128, 400, -math.inf, [0.2, 0.2]),  # tau = -inf: dense cache
    (128, 400, math.inf, [0.9, 0.9]),   # tau = +inf: nothing kept
])
def test_append_matches_oracle(w, T, tau, rates):
    spkv = load()
    Hkv, n_seq, seq_ids, layer = 2, 2, [2, 0], 1
    cache = spkv.Cache(n_layers=2, max_seqs=3, n_q_heads=8, n_kv_heads=Hkv, max_context=1024,
                       pool_pages=80, window=w, tau=tau)
    tl = cache.spkv_tau_logit()
    wl = Workload(1000 + w + T, T, n_seq, 8, Hkv, rates, tl, with_q=False)
    run_appends(cache, layer, seq_ids, wl)
    assert cache.spkv_status() == 0
    units = oracle_units(wl, w, tl)
    ln, tt = cache.spkv_read_lengths(layer)
    for i, s in enumerate(seq_ids):
        for h in range(Hkv):
            assert ln[s, h] == len(units[i][h]) and tt[s, h] == T
            compare_state(cache, layer, s, h, units[i][h])
    # the untouched sequence slot and the other layer stay empty
    assert ln[1].tolist() == [0, 0] and tt[1].tolist() == [0, 0]
    l0, t0 = cache.spkv_read_lengths(0)
    assert not l0.any() and not t0.any()
    # kept-set identity straight from the logits
    for i, s in enumerate(seq_ids):
        for h in range(Hkv):
            want = int((wl.logit[:max(T - w, 0), i, h] >= np.float32(tl)).sum())
            assert ln[s, h] == want


def test_threshold_change_applies_to_future_evictions():
    spkv = load()
    w, T = 8, 200
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=2, n_kv_heads=1, max_context=512,
                       pool_pages=8, window=w, tau=0.3)
    wl = Workload(5, T, 1, 2, 1, [0.5], 0.0, with_q=False)
    wl.logit[:] = np.random.default_rng(6).standard_normal(wl.logit.shape).astype(np.float32) * 2
    u = oracle.Unit(w, D)
    tl = cache.spkv_tau_logit()
    for t in range(T):
        if t == 90:
            cache.spkv_set_tau(0.8)
            tl = cache.spkv_tau_logit()
            assert abs(tl - math.log(4.0)) < 1e-6
        run_appends(cache, 0, [0], wl, t, t + 1)
        u.append(wl.K[t, 0, 0], wl.V[t, 0, 0], wl.logit[t, 0, 0], tl)
    compare_state(cache, 0, 0, 0, u)


def test_pool_exhaustion_is_reported_and_cache_stays_consistent():
    spkv = load()
    w, T, Hkv = 4, 400, 2
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=4, n_kv_heads=Hkv, max_context=4096,
                       pool_pages=3, window=w, tau=-math.inf)      # keep all: needs 14 pages
    wl = Workload(7, T, 1, 4, Hkv, [1.0, 1.0], 0.0, with_q=False)
    run_appends(cache, 0, [0], wl)
    assert cache.spkv_status() == -5
    ln, tt = cache.spkv_read_lengths(0)
    assert tt[0].tolist() == [T, T]
    assert sorted(ln[0].tolist())[0] % 64 == 0 and ln[0].sum() == 3 * 64   # whole pages only
    st = cache.spkv_cache_stats()
    assert st.pages_free == 0 and st.pages_in_use == 3
    # stored prefix is intact: positions 0..len-1 in order, bytes equal to the inputs
    for h in range(Hkv):
        pos, k, v = cache.spkv_read_kept(0, 0, h)
        assert pos.tolist() == list(range(ln[0, h]))
        assert np.array_equal(k, wl.K[:ln[0, h], 0, h]) and np.array_equal(v, wl.V[:ln[0, h], 0, h])
    cache.spkv_clear_status()
    assert cache.spkv_status() == 0


def test_context_overflow_is_reported():
    spkv = load()
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=1, n_kv_heads=1, max_context=64,
                       pool_pages=4, window=2, tau=-math.inf)
    wl = Workload(8, 80, 1, 1, 1, [1.0], 0.0, with_q=False)
    run_appends(cache, 0, [0], wl)
    assert cache.spkv_status() == -6
    ln, _ = cache.spkv_read_lengths(0)
    assert ln[0, 0] == 64


def test_bad_sequence_id_sets_status_and_touches_nothing():
    spkv = load()
    cache = spkv.Cache(n_layers=1, max_seqs=2, n_q_heads=2, n_kv_heads=1, max_context=256,
                       pool_pages=4, window=4, tau=0.5)
    wl = Workload(9, 3, 2, 2, 1, [0.5], 0.0, with_q=False)
    run_appends(cache, 0, [1, 7], wl)
    assert cache.spkv_status() == -9
    _, tt = cache.spkv_read_lengths(0)
    assert tt[:, 0].tolist() == [0, 3]


def test_reset_returns_pages_and_replay_is_identical():
    spkv = load()
    w, T, Hkv = 16, 500, 2
    cache = spkv.Cache(n_layers=2, max_seqs=2, n_q_heads=4, n_kv_heads=Hkv, max_context=1024,
                       pool_pages=60, window=w, tau=0.5)
    tl = cache.spkv_tau_logit()
    wl = Workload(10, T, 2, 4, Hkv, [0.5, 0.8], tl, with_q=False)
    for layer in (0, 1):
        run_appends(cache, layer, [0, 1], wl)
    assert cache.spkv_status() == 0
    before = cache.spkv_cache_stats()
    first = [cache.spkv_read_kept(1, 1, h) for h in range(Hkv)]
    cache.spkv_cache_reset_seq(1)
    st = cache.spkv_cache_stats()
    ln, tt = cache.spkv_read_lengths(1)
    assert ln[1].tolist() == [0, 0] and tt[1].tolist() == [0, 0] and tt[0].tolist() == [T, T]
    assert st.pages_free + st.pages_in_use == 60 and st.pages_in_use < before.pages_in_use
    # replay sequence 1 alone in both layers: same logical content as the first time
    wl1 = Workload(10, T, 2, 4, Hkv, [0.5, 0.8], tl, with_q=False)
    wl1.K, wl1.V, wl1.logit = wl.K[:, 1:], wl.V[:, 1:], wl.logit[:, 1:]
    wl1.n_seq = 1
    for layer in (0, 1):
        run_appends(cache, layer, [1], wl1)
    assert cache.spkv_status() == 0
    units = oracle_units(wl, w, tl)
    for h in range(Hkv):
        compare_state(cache, 1, 1, h, units[1][h])
        compare_state(cache, 0, 0, h, units[0][h])
        for a, b in zip(first[h], cache.spkv_read_kept(1, 1, h)):
            assert np.array_equal(a, b)
    after = cache.spkv_cache_stats()
    assert after.pages_in_use == before.pages_in_use and after.pairs_kept == before.pairs_kept


def test_stats_match_oracle_density():
    spkv = load()
    w, T, Hkv = 32, 600, 2
    cache = spkv.Cache(n_layers=1, max_seqs=2, n_q_heads=4, n_kv_heads=Hkv, max_context=1024,
                       pool_pages=40, window=w, tau=0.6)
    tl = cache.spkv_tau_logit()
    wl = Workload(11, T, 2, 4, Hkv, [0.15, 0.55], tl, with_q=False)
    run_appends(cache, 0, [0, 1], wl)
    st = cache.spkv_cache_stats()
    dens = [oracle.density(np.ascontiguousarray(wl.logit[:, s, h]), w, tl)
            for s in range(2) for h in range(Hkv)]
    assert abs(st.density_all - np.mean([d[0] for d in dens])) < 1e-12
    assert abs(st.density_cache - np.mean([d[1] for d in dens])) < 1e-12
    assert st.pairs_seen == 4 * T and st.pairs_in_window == 4 * w and st.pairs_evicted == 4 * (T - w)
    assert st.bytes_resident == (st.pairs_kept + 4 * w) * 512
