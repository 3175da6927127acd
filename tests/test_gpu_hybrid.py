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
