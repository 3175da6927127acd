"""GPU parity of the sink-token variant (config.sink_tokens > 0): the first positions of a
sequence stay in the compact cache whatever their utility says.  State bit-exact against the
oracle's streaming form, attention within the tolerance, through append/decode, through
chunked prefill, and through a mix of the two."""
import math

import numpy as np
import pytest
import torch

import oracle
from gpu_util import D, Workload, assert_attn_close, compare_state, dev, load, to_dev_bf16

pytestmark = pytest.mark.gpu


def oracle_run(wl, w, tl, G, n_sink, scale):
    """Token-by-token (append, attend) with sinks: units[h], outputs [T, Hq, D]."""
    units, outs = [], []
    for h in range(wl.Hkv):
        u = oracle.Unit(w, D, n_sink=n_sink)
        o = u.prefill(np.ascontiguousarray(wl.K[:, 0, h]), np.ascontiguousarray(wl.V[:, 0, h]),
                      np.ascontiguousarray(wl.logit[:, 0, h]), tl,
                      np.ascontiguousarray(wl.q[:, 0, h * G:(h + 1) * G]), scale)
        units.append(u)
        outs.append(o)
    return units, np.concatenate(outs, axis=1)


@pytest.mark.parametrize("w,n_sink,tau,rates", [(16, 4, 0.5, [0.0, 0.3]), (128, 4, math.inf, [0.5, 0.5]),
                                                (4, 40, 0.5, [0.1, 0.1]), (128, 1, 0.9, [0.05, 0.6])])
def test_append_decode_with_sinks(w, n_sink, tau, rates):
    spkv = load()
    T, Hq, Hkv, G = 420, 8, 2, 4
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=1024,
                       pool_pages=24, window=w, tau=tau, sink_tokens=n_sink)
    tl = cache.spkv_tau_logit()
    wl = Workload(500 + w + n_sink, T, 1, Hq, Hkv, rates, tl)
    scale = 1.0 / math.sqrt(D)
    units, ref = oracle_run(wl, w, tl, G, n_sink, scale)
    ids = torch.zeros(1, dtype=torch.int32, device=dev())
    K, V, Q = to_dev_bf16(wl.K), to_dev_bf16(wl.V), to_dev_bf16(wl.q)
    lg = torch.from_numpy(wl.logit).to(dev())
    got = []
    for t in range(T):
        cache.spkv_append_evict(0, ids, K[t], V[t], lg[t])
        got.append(spkv.bits_from_bf16(cache.spkv_decode_attention(0, ids, Q[t])))
    assert cache.spkv_status() == 0
    for h in range(Hkv):
        compare_state(cache, 0, 0, h, units[h])
        pos, _, _ = cache.spkv_read_kept(0, 0, h)
        assert pos[:min(n_sink, T - w)].tolist() == list(range(min(n_sink, T - w)))   # the sinks lead the cache
    assert_attn_close(np.concatenate(got), ref, f"sinks append/decode w={w} n_sink={n_sink}")


@pytest.mark.parametrize("chunks", [[700], [3, 1, 200, 129, 367], [1] * 10 + [690]])
def test_prefill_with_sinks(chunks):
    spkv = load()
    w, n_sink, Hq, Hkv, G = 128, 4, 8, 2, 4
    T = sum(chunks)
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=2048,
                       pool_pages=30, window=w, tau=0.5, sink_tokens=n_sink)
    tl = cache.spkv_tau_logit()
    wl = Workload(600 + len(chunks), T, 1, Hq, Hkv, [0.0, 0.4], tl)
    scale = 1.0 / math.sqrt(D)
    units, ref = oracle_run(wl, w, tl, G, n_sink, scale)
    K, V, Q = to_dev_bf16(wl.K[:, 0]), to_dev_bf16(wl.V[:, 0]), to_dev_bf16(wl.q[:, 0])
    lg = torch.from_numpy(np.ascontiguousarray(wl.logit[:, 0])).to(dev())
    outs, a = [], 0
    for c in chunks:
        outs.append(spkv.bits_from_bf16(cache.spkv_prefill(0, 0, K[a:a + c], V[a:a + c], lg[a:a + c], q=Q[a:a + c])))
        a += c
    assert cache.spkv_status() == 0
    for h in range(Hkv):
        compare_state(cache, 0, 0, h, units[h])
    assert len(units[0]) == n_sink          # keep rate 0: the compact cache holds the sinks and nothing else
    assert_attn_close(np.concatenate(outs), ref, f"sinks prefill chunks={chunks[:4]}")


def test_prefill_then_decode_with_sinks():
    spkv = load()
    w, n_sink, Hq, Hkv, G, T, C0 = 32, 4, 4, 2, 2, 300, 150
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=1024,
                       pool_pages=20, window=w, tau=0.5, sink_tokens=n_sink)
    tl = cache.spkv_tau_logit()
    wl = Workload(77, T, 1, Hq, Hkv, [0.2, 0.0], tl)
    scale = 1.0 / math.sqrt(D)
    units, ref = oracle_run(wl, w, tl, G, n_sink, scale)
    K, V, Q = to_dev_bf16(wl.K), to_dev_bf16(wl.V), to_dev_bf16(wl.q)
    lg = torch.from_numpy(wl.logit).to(dev())
    ids = torch.zeros(1, dtype=torch.int32, device=dev())
    got = [spkv.bits_from_bf16(cache.spkv_prefill(0, 0, K[:C0, 0], V[:C0, 0], lg[:C0, 0].contiguous(), q=Q[:C0, 0]))]
    for t in range(C0, T):
        cache.spkv_append_evict(0, ids, K[t], V[t], lg[t])
        got.append(spkv.bits_from_bf16(cache.spkv_decode_attention(0, ids, Q[t])))
    assert cache.spkv_status() == 0
    for h in range(Hkv):
        compare_state(cache, 0, 0, h, units[h])
    assert_attn_close(np.concatenate(got), ref, "sinks prefill then decode")
