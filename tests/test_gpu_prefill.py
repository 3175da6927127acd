"""GPU parity, companion path (chunked prefill): the cache state after any chunking equals
the oracle's token-by-token state bit for bit, and every query's output matches the
oracle's (append, attend) loop within the attention tolerance."""
import math

import numpy as np
import pytest
import torch

import oracle
from gpu_util import D, Workload, assert_attn_close, compare_state, dev, load, to_dev_bf16

pytestmark = pytest.mark.gpu


def prefill_in_chunks(spkv, cache, layer, seq, wl, s_idx, chunks, with_q=True):
    """Feeds sequence column `s_idx` of the workload through spkv_prefill; returns outputs."""
    K, V = to_dev_bf16(wl.K[:, s_idx]), to_dev_bf16(wl.V[:, s_idx])          # [T,Hkv,D]
    Q = to_dev_bf16(wl.q[:, s_idx]) if with_q else None
    lg = torch.from_numpy(np.ascontiguousarray(wl.logit[:, s_idx])).to(dev())
    outs, a = [], 0
    for c in chunks:
        o = cache.spkv_prefill(layer, seq, K[a:a + c], V[a:a + c], lg[a:a + c],
                               q=Q[a:a + c] if with_q else None)
        if with_q:
            outs.append(spkv.bits_from_bf16(o))
        a += c
    return np.concatenate(outs) if with_q else None


def oracle_prefill(wl, s_idx, w, tl, G, upto, scale):
    units, outs = [], []
    for h in range(wl.Hkv):
        u = oracle.Unit(w, D)
        o = u.prefill(np.ascontiguousarray(wl.K[:upto, s_idx, h]),
                      np.ascontiguousarray(wl.V[:upto, s_idx, h]),
                      np.ascontiguousarray(wl.logit[:upto, s_idx, h]), tl,
                      np.ascontiguousarray(wl.q[:upto, s_idx, h * G:(h + 1) * G]), scale)
        units.append(u)
        outs.append(o)
    return units, np.concatenate(outs, axis=1)      # [T, Hq, D]


def split(T, c):
    return [c] * (T // c) + ([T % c] if T % c else [])


@pytest.mark.parametrize("chunk", [1, 16, 127, 128, 129, 300, 640])
def test_prefill_chunkings_match_oracle(chunk):
    spkv = load()
    w, T, Hq, Hkv = 128, 640, 8, 2
    T = 400 if chunk == 1 else T
    cache = spkv.Cache(n_layers=2, max_seqs=2, n_q_heads=Hq, n_kv_heads=Hkv, max_context=2048,
                       pool_pages=40, window=w, tau=0.5)
    tl = cache.spkv_tau_logit()
    wl = Workload(200, T, 1, Hq, Hkv, [0.25, 0.7], tl)
    got = prefill_in_chunks(spkv, cache, 1, 1, wl, 0, split(T, chunk))
    assert cache.spkv_status() == 0
    units, ref = oracle_prefill(wl, 0, w, tl, Hq // Hkv, T, 1.0 / math.sqrt(D))
    for h in range(Hkv):
        compare_state(cache, 1, 1, h, units[h])
    assert_attn_close(got, ref, f"chunk={chunk}")


@pytest.mark.parametrize("w,G,Hkv,tau,rates", [
    (1, 4, 1, 0.5, [0.5]), (4, 1, 2, 0.2, [0.3, 0.6]), (100, 8, 1, 0.5, [0.4]),
    (200, 2, 2, 0.9, [0.1, 0.9]), (128, 4, 2, -math.inf, [0.2, 0.2]),
    (128, 4, 2, math.inf, [0.8, 0.8]), (128, 16, 1, 0.5, [0.0]), (128, 3, 2, 0.5, [1.0, 0.5]),
    # more KV heads than lanes (the heaviest-first order falls back to plain order), and exactly 32
    (128, 2, 33, 0.5, [((7 * i) % 33) / 33.0 for i in range(33)]),
    (128, 2, 32, 0.5, [((5 * i) % 32) / 40.0 for i in range(32)]),
])
def test_prefill_windows_groups_thresholds(w, G, Hkv, tau, rates):
    spkv = load()
    T, Hq = 700, G * Hkv
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=2048,
                       pool_pages=40 + 12 * Hkv, window=w, tau=tau)
    tl = cache.spkv_tau_logit()
    wl = Workload(210 + w + G, T, 1, Hq, Hkv, rates, tl)
    got = prefill_in_chunks(spkv, cache, 0, 0, wl, 0, [70, 1, 200, 129, 300])
    assert cache.spkv_status() == 0
    units, ref = oracle_prefill(wl, 0, w, tl, G, T, 1.0 / math.sqrt(D))
    for h in range(Hkv):
        compare_state(cache, 0, 0, h, units[h])
    assert_attn_close(got, ref, f"w={w} G={G}")


def test_prefill_then_decode_then_prefill_equals_pure_append():
    """Mixed use: prefill-built cache == append-built cache, and decode after prefill is right."""
    spkv = load()
    w, T, Hq, Hkv, G = 128, 1500, 8, 2, 4
    mk = lambda: spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=4096,
                            pool_pages=60, window=w, tau=0.5)
    a, b = mk(), mk()
    tl = a.spkv_tau_logit()
    wl = Workload(220, T, 1, Hq, Hkv, [0.3, 0.9], tl)
    ids = torch.zeros(1, dtype=torch.int32, device=dev())
    K, V, Q = to_dev_bf16(wl.K), to_dev_bf16(wl.V), to_dev_bf16(wl.q)
    lg = torch.from_numpy(wl.logit).to(dev())
    # a: prefill 1000, decode 100 steps, prefill the rest
    plan = [("p", 0, 1000), ("d", 1000, 1100), ("p", 1100, T)]
    outs = {}
    for kind, s, e in plan:
        if kind == "p":
            o = a.spkv_prefill(0, 0, K[s:e, 0], V[s:e, 0], lg[s:e, 0], q=Q[s:e, 0])
            for t in (s, e - 1):
                outs[t] = spkv.bits_from_bf16(o[t - s])
        else:
            for t in range(s, e):
                a.spkv_append_evict(0, ids, K[t], V[t], lg[t])
                o = a.spkv_decode_attention(0, ids, Q[t])
                if t in (s, e - 1):
                    outs[t] = spkv.bits_from_bf16(o[0])
    for t in range(T):
        b.spkv_append_evict(0, ids, K[t], V[t], lg[t])
    assert a.spkv_status() == 0 and b.spkv_status() == 0
    units, ref = oracle_prefill(wl, 0, w, tl, G, T, 1.0 / math.sqrt(D))
    for h in range(Hkv):
        compare_state(a, 0, 0, h, units[h])
        compare_state(b, 0, 0, h, units[h])
    for t, o in outs.items():
        assert_attn_close(o, ref[t], f"t={t}")


def test_prefill_state_only_and_large_chunk():
    spkv = load()
    w, T, Hq, Hkv = 128, 9000, 4, 2
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=16384,
                       pool_pages=200, window=w, tau=0.5)
    tl = cache.spkv_tau_logit()
    wl = Workload(230, T, 1, Hq, Hkv, [0.2, 0.95], tl)
    prefill_in_chunks(spkv, cache, 0, 0, wl, 0, [8192, T - 8192], with_q=False)
    assert cache.spkv_status() == 0
    for h in range(Hkv):
        u = oracle.Unit(w, D)
        u.prefill(np.ascontiguousarray(wl.K[:, 0, h]), np.ascontiguousarray(wl.V[:, 0, h]),
                  np.ascontiguousarray(wl.logit[:, 0, h]), tl)
        compare_state(cache, 0, 0, h, u)


def test_prefill_long_past_sampled_queries():
    """An 8192-pair chunk on top of a 12 k past: sampled queries against the mask form."""
    spkv = load()
    w, T0, C, Hq, Hkv, G = 128, 12000, 8192, 8, 2, 4
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=32768,
                       pool_pages=400, window=w, tau=0.5)
    tl = cache.spkv_tau_logit()
    wl = Workload(240, T0 + C, 1, Hq, Hkv, [0.15, 0.6], tl)
    prefill_in_chunks(spkv, cache, 0, 0, wl, 0, [8192, T0 - 8192], with_q=False)
    K, V, Q = to_dev_bf16(wl.K[:, 0]), to_dev_bf16(wl.V[:, 0]), to_dev_bf16(wl.q[:, 0])
    lg = torch.from_numpy(np.ascontiguousarray(wl.logit[:, 0])).to(dev())
    out = spkv.bits_from_bf16(cache.spkv_prefill(0, 0, K[T0:], V[T0:], lg[T0:], q=Q[T0:]))
    assert cache.spkv_status() == 0
    scale = 1.0 / math.sqrt(D)
    for t in (T0, T0 + 1, T0 + 63, T0 + 64, T0 + 127, T0 + 128, T0 + 129, T0 + 4095, T0 + C - 1):
        for h in range(Hkv):
            ref = oracle.mask_attend_row(np.ascontiguousarray(wl.K[:, 0, h]),
                                         np.ascontiguousarray(wl.V[:, 0, h]),
                                         np.ascontiguousarray(wl.logit[:, 0, h]), t, w, tl,
                                         np.ascontiguousarray(wl.q[t, 0, h * G:(h + 1) * G]), scale)
            assert_attn_close(out[t - T0, h * G:(h + 1) * G], ref, f"t={t} kvh={h}")
    ln, tt = cache.spkv_read_lengths(0)
    for h in range(Hkv):
        assert ln[0, h] == int((wl.logit[:T0 + C - w, 0, h] >= np.float32(tl)).sum())


def test_prefill_pool_exhaustion_reports_and_keeps_length():
    spkv = load()
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=2, n_kv_heads=1, max_context=4096,
                       pool_pages=2, window=4, tau=-math.inf)
    wl = Workload(250, 600, 1, 2, 1, [1.0], 0.0)
    prefill_in_chunks(spkv, cache, 0, 0, wl, 0, [100, 500], with_q=False)
    assert cache.spkv_status() == -5
    ln, tt = cache.spkv_read_lengths(0)
    assert ln[0, 0] == 96 and tt[0, 0] == 600


@pytest.mark.parametrize("direction", [1.0, -1.0])
def test_prefill_scores_that_grow_or_fall_with_position(direction):
    """Raw scores 2t (or -2t) for the first head of every pair: with direction +1 the row maximum
    grows by ~16 (log2 units, after the 1/sqrt(d) scale) from one 64-key page to the next, so the accumulator is rescaled
    on every page, the last one included; with -1 everything after a row's first visible page
    underflows.  The second head of every pair keeps ordinary scores, so the two softmax groups
    of a block take different paths side by side."""
    from paper_2605_14037_b200 import synth
    spkv = load()
    w, Hq, Hkv, G, chunks = 128, 4, 2, 2, [300, 400, 1, 130]
    T = sum(chunks)
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=2048,
                       pool_pages=40, window=w, tau=0.5)
    tl = cache.spkv_tau_logit()
    wl = Workload(321, T, 1, Hq, Hkv, [0.5, 0.35], tl)
    Kf = synth.bf16_bits_to_f32(wl.K)
    Kf[:, 0, :, 0] = (direction * 0.25 * np.arange(T, dtype=np.float32))[:, None]
    wl.K = synth.to_bf16_bits(Kf)
    qf = synth.bf16_bits_to_f32(wl.q)
    qf[:, 0, 0::2, :] = 0.0
    qf[:, 0, 0::2, 0] = 8.0
    wl.q = synth.to_bf16_bits(qf)
    got = prefill_in_chunks(spkv, cache, 0, 0, wl, 0, chunks)
    assert cache.spkv_status() == 0
    units, ref = oracle_prefill(wl, 0, w, tl, G, T, 1.0 / math.sqrt(D))   # 2t / sqrt(128) * log2(e) = 0.255 t
    for h in range(Hkv):
        compare_state(cache, 0, 0, h, units[h])
    assert_attn_close(got, ref, f"direction={direction}")


@pytest.mark.parametrize("G,Hkv,chunks", [(1, 32, [2432, 600]), (3, 10, [2400, 257])])
def test_prefill_single_head_blocks_take_two_query_tiles(G, Hkv, chunks):
    """Odd query-group sizes in launches large enough for the last head of a group to run with
    two consecutive query tiles per block (two waves of blocks or more): an odd and an even number
    of tiles, then a smaller ragged chunk on top of that past (one tile per block again)."""
    spkv = load()
    w, Hq, T = 128, G * Hkv, sum(chunks)
    rates = [((3 * i) % 10) / 10.0 for i in range(Hkv)]
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=4096,
                       pool_pages=int(sum(rates) * T / 64) + 3 * Hkv + 8, window=w, tau=0.5)
    tl = cache.spkv_tau_logit()
    wl = Workload(4000 + G + len(chunks), T, 1, Hq, Hkv, rates, tl)
    got = prefill_in_chunks(spkv, cache, 0, 0, wl, 0, chunks)
    assert cache.spkv_status() == 0
    units, ref = oracle_prefill(wl, 0, w, tl, G, T, 1.0 / math.sqrt(D))
    for h in range(Hkv):
        compare_state(cache, 0, 0, h, units[h])
    assert_attn_close(got, ref, f"G={G} Hkv={Hkv} chunks={chunks}")


@pytest.mark.parametrize("G,Hkv,small", [(4, 2, [48, 1, 130]), (1, 3, [16, 200]), (3, 2, [257]), (4, 4, [2432])])
def test_small_chunks_on_a_long_past_split_their_page_walks(G, Hkv, small):
    """Chunks of a few tokens on a 20 k past: the launch has only a handful of page walks, each
    hundreds of pages long, so every walk is cut into shares over several blocks and the shares
    are merged by their log-sum-exp weights (the shortest heads' walks stay whole).  The last case
    is a launch of about one wave of walks (152), where only the walks of the head that keeps most
    are cut and the others write their output directly.
    Rows of the small chunks against the mask form; state against the streaming form."""
    spkv = load()
    w, T0, Hq = 128, 20000, G * Hkv
    T = T0 + sum(small)
    rates = [0.02, 0.7, 0.3, 0.05][:Hkv]
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=32768,
                       pool_pages=int(sum(rates) * T / 64) + 3 * Hkv + 8, window=w, tau=0.5)
    tl = cache.spkv_tau_logit()
    wl = Workload(5000 + G, T, 1, Hq, Hkv, rates, tl)
    prefill_in_chunks(spkv, cache, 0, 0, wl, 0, [8192, 8192, T0 - 16384], with_q=False)
    K, V, Q = to_dev_bf16(wl.K[:, 0]), to_dev_bf16(wl.V[:, 0]), to_dev_bf16(wl.q[:, 0])
    lg = torch.from_numpy(np.ascontiguousarray(wl.logit[:, 0])).to(dev())
    outs, a = [], T0
    for c in small:
        outs.append(spkv.bits_from_bf16(cache.spkv_prefill(0, 0, K[a:a + c], V[a:a + c], lg[a:a + c], q=Q[a:a + c])))
        a += c
    assert cache.spkv_status() == 0
    out = np.concatenate(outs)
    scale = 1.0 / math.sqrt(D)
    for h in range(Hkv):
        Kh, Vh, Lh = (np.ascontiguousarray(x) for x in (wl.K[:, 0, h], wl.V[:, 0, h], wl.logit[:, 0, h]))
        for t in range(T0, T, 13 if T - T0 > 1000 else 3 if T - T0 > 100 else 1):
            ref = oracle.mask_attend_row(Kh, Vh, Lh, t, w, tl, np.ascontiguousarray(wl.q[t, 0, h * G:(h + 1) * G]), scale)
            assert_attn_close(out[t - T0, h * G:(h + 1) * G], ref, f"t={t} kvh={h}")
        u = oracle.Unit(w, D)
        u.prefill(Kh, Vh, Lh, tl)
        compare_state(cache, 0, 0, h, u)


@pytest.mark.parametrize("G,Hkv,w", [(4, 2, 128), (3, 2, 100), (1, 3, 128), (8, 1, 4)])
def test_prefill_with_two_term_bf16_weights(G, Hkv, w):
    """SPKV_FLAG_PREFILL_PV_BF16: every unit multiplies the softmax weights into the values as
    two bf16 terms (the form a unit with a very wide value range takes by itself).  Same chunkings,
    same oracle, same tolerance as the default path; even and odd groups, a partially filled first
    chunk, a one-token chunk."""
    spkv = load()
    T, Hq = 700, G * Hkv
    rates = [0.25, 0.7, 0.5][:Hkv]
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=2048,
                       pool_pages=40 + 12 * Hkv, window=w, tau=0.5, flags=spkv.FLAG_PREFILL_PV_BF16)
    tl = cache.spkv_tau_logit()
    wl = Workload(910 + w + G, T, 1, Hq, Hkv, rates, tl)
    got = prefill_in_chunks(spkv, cache, 0, 0, wl, 0, [70, 1, 200, 129, 300])
    assert cache.spkv_status() == 0
    units, ref = oracle_prefill(wl, 0, w, tl, G, T, 1.0 / math.sqrt(D))
    for h in range(Hkv):
        compare_state(cache, 0, 0, h, units[h])
    assert_attn_close(got, ref, f"two-term bf16, w={w} G={G}")


def test_two_term_bf16_weights_on_split_page_walks_and_rescaled_rows():
    """The flag on the two harder paths: page walks cut into shares (a small chunk on a 20 k past)
    and rows whose accumulator is rescaled on every page (scores growing with position)."""
    from paper_2605_14037_b200 import synth
    spkv = load()
    w, T0, G, Hkv = 128, 20000, 4, 2
    Hq, small = G * Hkv, [48, 130]
    T = T0 + sum(small)
    rates = [0.05, 0.6]
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=32768,
                       pool_pages=int(sum(rates) * T / 64) + 3 * Hkv + 8, window=w, tau=0.5,
                       flags=spkv.FLAG_PREFILL_PV_BF16)
    tl = cache.spkv_tau_logit()
    wl = Workload(5100, T, 1, Hq, Hkv, rates, tl)
    Kf = synth.bf16_bits_to_f32(wl.K)
    Kf[T0 - 1500:, 0, 1, 0] = 0.25 * np.arange(1500 + sum(small), dtype=np.float32)   # KV head 1: scores grow
    wl.K = synth.to_bf16_bits(Kf)
    qf = synth.bf16_bits_to_f32(wl.q)
    qf[:, 0, G, :] = 0.0
    qf[:, 0, G, 0] = 8.0                    # first query head of KV head 1 looks at that dimension only
    wl.q = synth.to_bf16_bits(qf)
    prefill_in_chunks(spkv, cache, 0, 0, wl, 0, [8192, 8192, T0 - 16384], with_q=False)
    K, V, Q = to_dev_bf16(wl.K[:, 0]), to_dev_bf16(wl.V[:, 0]), to_dev_bf16(wl.q[:, 0])
    lg = torch.from_numpy(np.ascontiguousarray(wl.logit[:, 0])).to(dev())
    outs, a = [], T0
    for c in small:
        outs.append(spkv.bits_from_bf16(cache.spkv_prefill(0, 0, K[a:a + c], V[a:a + c], lg[a:a + c], q=Q[a:a + c])))
        a += c
    assert cache.spkv_status() == 0
    out = np.concatenate(outs)
    scale = 1.0 / math.sqrt(D)
    for h in range(Hkv):
        Kh, Vh, Lh = (np.ascontiguousarray(x) for x in (wl.K[:, 0, h], wl.V[:, 0, h], wl.logit[:, 0, h]))
        for t in range(T0, T, 2):
            ref = oracle.mask_attend_row(Kh, Vh, Lh, t, w, tl, np.ascontiguousarray(wl.q[t, 0, h * G:(h + 1) * G]), scale)
            assert_attn_close(out[t - T0, h * G:(h + 1) * G], ref, f"t={t} kvh={h}")


@pytest.mark.parametrize("scale", [0.0, -0.1, float("inf"), float("nan")])
def test_prefill_refuses_a_scale_that_is_not_positive_and_finite(scale):
    """The chunk attention takes row maxima before scaling, which needs a positive scale: any other
    value is an argument error, reported before anything is launched (the cache is unchanged).
    Building the state only (no queries) does not look at the scale."""
    spkv = load()
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=4, n_kv_heads=2, max_context=1024,
                       pool_pages=8, window=16, tau=0.5)
    wl = Workload(77, 40, 1, 4, 2, [0.5, 0.5], cache.spkv_tau_logit())
    K, V, Q = to_dev_bf16(wl.K[:, 0]), to_dev_bf16(wl.V[:, 0]), to_dev_bf16(wl.q[:, 0])
    lg = torch.from_numpy(np.ascontiguousarray(wl.logit[:, 0])).to(dev())
    with pytest.raises(spkv.SpkvError) as e:
        cache.spkv_prefill(0, 0, K, V, lg, q=Q, sm_scale=scale)
    assert e.value.code == -1
    ln, tt = cache.spkv_read_lengths(0)
    assert (tt == 0).all() and (ln == 0).all() and cache.spkv_status() == 0
    cache.spkv_prefill(0, 0, K, V, lg, sm_scale=scale)          # state only
    assert cache.spkv_status() == 0 and (cache.spkv_read_lengths(0)[1] == 40).all()
