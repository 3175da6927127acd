"""GPU parity of static hybrid layouts: (layer, KV head) thresholds of their own
(spkv_set_head_tau) -- local-only heads (tau >= 1: window attention, empty compact cache),
full-attention heads (tau <= 0) and heads at another threshold, next to heads that follow the
cache-wide one.  The oracle needs nothing new: a unit simply receives its own threshold."""
import math

import numpy as np
import torch

import oracle
from gpu_util import D, Workload, assert_attn_close, compare_state, dev, load, to_dev_bf16

import pytest

pytestmark = pytest.mark.gpu


def oracle_units_per_head(wl, w, head_tl, G, scale):
    units, outs = [], []
    for h in range(wl.Hkv):
        u = oracle.Unit(w, D)
        o = u.prefill(np.ascontiguousarray(wl.K[:, 0, h]), np.ascontiguousarray(wl.V[:, 0, h]),
                      np.ascontiguousarray(wl.logit[:, 0, h]), head_tl[h],
                      np.ascontiguousarray(wl.q[:, 0, h * G:(h + 1) * G]), scale)
        units.append(u)
        outs.append(o)
    return units, np.concatenate(outs, axis=1)


def test_hybrid_layout_append_decode_and_prefill():
    spkv = load()
    w, T, Hq, Hkv, G, C0 = 16, 330, 8, 4, 2, 150
    cache = spkv.Cache(n_layers=2, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=1024,
                       pool_pages=40, window=w, tau=0.5)
    tl = cache.spkv_tau_logit()
    # layer 0: head 0 local-only, head 1 full attention, head 2 cache-wide, head 3 tau = 0.8
    cache.spkv_set_head_tau(0, 0, 1.0)
    cache.spkv_set_head_tau(0, 1, 0.0)
    cache.spkv_set_head_tau(0, 3, 0.8)
    # layer 1: every head local-only, then head 2 handed back to the cache-wide threshold
    cache.spkv_set_head_tau(1, -1, 1.0)
    cache.spkv_set_head_tau(1, 2, float("nan"))
    tl08 = float(oracle.tau_logit(0.8))
    head_tl = {0: [math.inf, -math.inf, tl, tl08], 1: [math.inf, math.inf, tl, math.inf]}
    scale = 1.0 / math.sqrt(D)
    ids = torch.zeros(1, dtype=torch.int32, device=dev())
    for layer in (0, 1):
        wl = Workload(800 + layer, T, 1, Hq, Hkv, [0.3, 0.3, 0.4, 0.5], tl)
        units, ref = oracle_units_per_head(wl, w, head_tl[layer], G, scale)
        K, V, Q = to_dev_bf16(wl.K), to_dev_bf16(wl.V), to_dev_bf16(wl.q)
        lg = torch.from_numpy(wl.logit).to(dev())
        got = [spkv.bits_from_bf16(cache.spkv_prefill(layer, 0, K[:C0, 0], V[:C0, 0], lg[:C0, 0].contiguous(),
                                                      q=Q[:C0, 0]))]
        for t in range(C0, T):
            cache.spkv_append_evict(layer, ids, K[t], V[t], lg[t])
            got.append(spkv.bits_from_bf16(cache.spkv_decode_attention(layer, ids, Q[t])))
        assert cache.spkv_status() == 0
        for h in range(Hkv):
            compare_state(cache, layer, 0, h, units[h])
        lens, _ = cache.spkv_read_lengths(layer)
        for h in range(Hkv):
            if head_tl[layer][h] == math.inf:
                assert lens[0, h] == 0                      # local-only: nothing is ever kept
            if head_tl[layer][h] == -math.inf:
                assert lens[0, h] == T - w                  # full attention: everything is
        assert_attn_close(np.concatenate(got), ref, f"hybrid layer {layer}")
    st = cache.spkv_cache_stats()
    want_open = 0
    for layer in (0, 1):
        wl = Workload(800 + layer, T, 1, Hq, Hkv, [0.3, 0.3, 0.4, 0.5], tl)
        for h in range(Hkv):
            want_open += int((wl.logit[:, 0, h] >= np.float32(head_tl[layer][h])).sum())
    assert st.gates_open == want_open                        # Eq. 8 numerator under per-head thresholds


def test_set_head_tau_rejects_bad_arguments():
    spkv = load()
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=2, n_kv_heads=2, max_context=64, pool_pages=2,
                       window=4, tau=0.5)
    for layer, head in [(-1, 0), (1, 0), (0, 2), (0, -2)]:
        with pytest.raises(spkv.SpkvError):
            cache.spkv_set_head_tau(layer, head, 0.5)


def test_heads_declared_local_only_at_creation():
    """The same hybrid idea fixed at creation (spkv_config_t.h_local_only): such heads have no page
    table and are not scored by the fused append; everything else behaves as a keep-nothing
    threshold would -- sliding-window attention, sinks not kept either -- and the other heads are
    untouched.  Append + decode and prefill against the oracle; a threshold of its own is refused."""
    spkv = load()
    w, T, Hq, Hkv, G, C0 = 16, 330, 8, 4, 2, 150
    local = np.array([[1, 0, 0, 1], [1, 1, 1, 1]], np.uint8)
    cache = spkv.Cache(n_layers=2, max_seqs=2, n_q_heads=Hq, n_kv_heads=Hkv, max_context=1024,
                       pool_pages=40, window=w, tau=0.5, sink_tokens=3, local_only=local)
    plain = spkv.Cache(n_layers=2, max_seqs=2, n_q_heads=Hq, n_kv_heads=Hkv, max_context=1024,
                       pool_pages=40, window=w, tau=0.5, sink_tokens=3)
    saved = plain.arena_bytes - cache.arena_bytes                           # six heads x two sequences x 16 entries
    assert 6 * 2 * 16 * 4 - 1024 < saved < 6 * 2 * 16 * 4 + 1024            # (regions are padded to 256 bytes)
    tl = cache.spkv_tau_logit()
    scale = 1.0 / math.sqrt(D)
    ids = torch.ones(1, dtype=torch.int32, device=dev())
    rng = np.random.default_rng(5)
    from paper_2605_14037_b200 import synth
    Wp = synth.linear_predictor(rng, Hkv, 64)
    bp = np.zeros(Hkv, np.float32)
    pred = spkv.make_predictor(to_dev_bf16(Wp), torch.from_numpy(bp).to(dev()))
    for layer in (0, 1):
        wl = Workload(830 + layer, T, 1, Hq, Hkv, [0.3, 0.5, 0.4, 0.5], tl)
        # the fused score + append decides on logits it computes itself: take them from x for the decode part
        x = synth.normal_bf16(rng, (T, 64))
        lg_lin = oracle.score_linear(x, Wp, bp).astype(np.float32)           # [T, Hkv]
        wl.logit[C0:, 0, :] = lg_lin[C0:]
        units, outs = [], []
        for h in range(Hkv):
            is_local = bool(local[layer, h])
            u = oracle.Unit(w, D, n_sink=0 if is_local else 3)
            outs.append(u.prefill(np.ascontiguousarray(wl.K[:, 0, h]), np.ascontiguousarray(wl.V[:, 0, h]),
                                  np.ascontiguousarray(wl.logit[:, 0, h]), math.inf if is_local else tl,
                                  np.ascontiguousarray(wl.q[:, 0, h * G:(h + 1) * G]), scale))
            units.append(u)
        ref = np.concatenate(outs, axis=1)
        K, V, Q = to_dev_bf16(wl.K), to_dev_bf16(wl.V), to_dev_bf16(wl.q)
        lg = torch.from_numpy(wl.logit).to(dev())
        xd = to_dev_bf16(x)
        got = [spkv.bits_from_bf16(cache.spkv_prefill(layer, 1, K[:C0, 0], V[:C0, 0], lg[:C0, 0].contiguous(),
                                                      q=Q[:C0, 0]))]
        lo = torch.full((1, Hkv), 7.0, dtype=torch.float32, device=dev())
        for t in range(C0, T):
            cache.spkv_score_append_evict(layer, pred, ids, xd[t:t + 1], K[t], V[t], logits_out=lo)
            got.append(spkv.bits_from_bf16(cache.spkv_decode_attention(layer, ids, Q[t])))
        assert cache.spkv_status() == 0
        lo = lo.cpu().numpy()[0]
        for h in range(Hkv):
            if local[layer, h]:
                assert lo[h] == 0.0                              # not scored
            else:
                assert abs(lo[h] - lg_lin[T - 1, h]) < 1e-3
        lens, tt = cache.spkv_read_lengths(layer)
        assert (tt[1] == T).all() and (tt[0] == 0).all()
        for h in range(Hkv):
            if local[layer, h]:
                assert lens[1, h] == 0
                pos, k, v = cache.spkv_read_kept(layer, 1, h)
                assert len(pos) == 0
                wpos, wk, wv, _ = cache.spkv_read_window(layer, 1, h)          # the ring is as the oracle's
                opos, ok, ov, _ = units[h].window()
                assert np.array_equal(wpos, opos) and np.array_equal(wk, ok) and np.array_equal(wv, ov)
            else:
                # the decode part was decided on the GPU's own float32 logits: compare what is unique
                pos, k, v = cache.spkv_read_kept(layer, 1, h)
                opos, ok, ov = units[h].kept()
                if np.array_equal(pos, opos):
                    assert np.array_equal(k, ok) and np.array_equal(v, ov)
                else:                                             # a logit within rounding of the threshold
                    diff = set(pos.tolist()) ^ set(opos.tolist())
                    assert all(abs(wl.logit[s, 0, h] - tl) < 1e-3 for s in diff)
        assert_attn_close(np.concatenate(got), ref, f"declared local-only, layer {layer}")
    with pytest.raises(spkv.SpkvError):
        cache.spkv_set_head_tau(0, 0, 0.5)                       # declared local-only: stays so
    with pytest.raises(spkv.SpkvError):
        cache.spkv_set_head_tau(0, -1, 0.5)                      # the layer holds such heads
    cache.spkv_set_head_tau(0, 1, 0.9)                           # an ordinary head of the same layer
    # budget: only the four units that can keep pairs count (2 global heads of layer 0, sequence 1)
    assert cache.spkv_safe_steps([1]) > 0
    cache.spkv_cache_reset_seq(1)
    assert cache.spkv_status() == 0 and (cache.spkv_read_lengths(0)[1] == 0).all()
    assert cache.spkv_cache_stats().pages_free == 40
