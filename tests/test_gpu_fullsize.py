"""Parity at the benchmark's full sizes and launch configuration: one layer of the
Llama-3-8B-shaped decode workload (config 2: batch 16, 32 query / 8 KV heads, context 32768,
window 128, per-head keep rates ~ Beta(0.5, 2)), of the long-context one (config 3: batch 4,
context 131072, Beta(0.3, 3)) and of the 70B-shaped one (config 5: batch 8, 64 query / 8 KV
heads, context 65536, Beta(0.5, 2.5)).  The cache is built with 8192-pair prefill chunks and
then stepped with whole-batch calls exactly as bench.py does.  Checked:
  * compact-cache length of all units == count of logits >= tau_logit among the pairs that
    left the window (kept-set identity), bit-exact;
  * for the sampled sequences (8 units each, CPU-generated K/V): kept positions and bytes bit-exact
    against the oracle, sampled prefill outputs against the oracle's mask form, and the decode
    outputs of three steps against the oracle's streaming form, within the attention tolerance.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from gpu_util import D, assert_attn_close, compare_state, dev, load, to_dev_bf16
from paper_2605_14037_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,Hq,Hkv,T,beta,sampled,overlap", [
    (16, 32, 8, 32768, (0.5, 2.0), [3, 11], True),
    (4, 32, 8, 131072, (0.3, 3.0), [2], True),
    (8, 64, 8, 65536, (0.5, 2.5), [5], True),
    # without the overlap flag a launch takes every SM (shorter ranges, more units split over blocks)
    (4, 32, 8, 131072, (0.3, 3.0), [1], False),
], ids=["config2", "config3", "config5", "config3_stream_ordered"])
def test_one_layer_full_size(B, Hq, Hkv, T, beta, sampled, overlap):
    spkv = load()
    w, C, steps = 128, 8192, 3
    G = Hq // Hkv
    rng = np.random.default_rng(1234)
    rates = synth.keep_rates(rng, 1, Hkv, *beta)[0]
    rates[0], rates[5] = 0.0, 0.97                       # a local-only head and a near-full head
    pages = int(np.ceil(rates * (T + steps) * 1.05 / 64 + 2).sum()) * B
    cache = spkv.Cache(n_layers=1, max_seqs=B, n_q_heads=Hq, n_kv_heads=Hkv, max_context=T + 128,
                       pool_pages=pages, window=w, tau=0.5,
                       flags=spkv.FLAG_OVERLAP if overlap else 0)   # as bench.py creates it / --stream-ordered
    tl = cache.spkv_tau_logit()
    Tt = T + steps
    logit = np.stack([synth.logits_with_keep_rate(rng, (Tt, B), float(r), tl) for r in rates], axis=-1)
    Ks = {s: synth.normal_bf16(rng, (Tt, Hkv, D)) for s in sampled}
    Vs = {s: synth.normal_bf16(rng, (Tt, Hkv, D)) for s in sampled}
    q_last = {s: synth.normal_bf16(rng, (C, Hq, D)) for s in sampled}      # queries of the last chunk
    gen = torch.Generator(device=dev())
    gen.manual_seed(7)
    lg_dev = torch.from_numpy(logit).to(dev())
    prefill_out = {}
    for s in range(B):
        if s in sampled:
            Kd, Vd = to_dev_bf16(Ks[s][:T]), to_dev_bf16(Vs[s][:T])
        else:
            Kd = torch.randn((T, Hkv, D), generator=gen, device=dev()).to(torch.bfloat16)
            Vd = torch.randn((T, Hkv, D), generator=gen, device=dev()).to(torch.bfloat16)
        for a in range(0, T, C):
            last = a + C == T and s in sampled
            o = cache.spkv_prefill(0, s, Kd[a:a + C], Vd[a:a + C], lg_dev[a:a + C, s].contiguous(),
                                   q=to_dev_bf16(q_last[s]) if last else None)
            if last:
                prefill_out[s] = spkv.bits_from_bf16(o)
    assert cache.spkv_status() == 0

    # sampled prefill queries against the mask form (Eq. 2-5 written out)
    scale = 1.0 / math.sqrt(D)
    for s in sampled:
        ts = sorted({T - C, T - C + 1, T - C + 63, T - C + 64, T - C + 127, T - C + 128, T - 4097, T - 129, T - 1}
                    | {T - C + int(x) for x in np.linspace(200, C - 200, 24)})   # tile edges and a spread
        for t in ts:
            for h in (0, 3, 5, 7):
                ref = oracle.mask_attend_row(
                    np.ascontiguousarray(Ks[s][:T, h]), np.ascontiguousarray(Vs[s][:T, h]),
                    np.ascontiguousarray(logit[:T, s, h]), t, w, tl,
                    np.ascontiguousarray(q_last[s][t - (T - C), h * G:(h + 1) * G]), scale)
                assert_attn_close(prefill_out[s][t - (T - C), h * G:(h + 1) * G], ref, f"prefill s={s} t={t} h={h}")

    # oracle streaming state of the sampled units
    units = {s: [oracle.Unit(w, D) for _ in range(Hkv)] for s in sampled}
    for s in sampled:
        for h in range(Hkv):
            units[s][h].prefill(np.ascontiguousarray(Ks[s][:T, h]), np.ascontiguousarray(Vs[s][:T, h]),
                                np.ascontiguousarray(logit[:T, s, h]), tl)

    ids = torch.arange(B, dtype=torch.int32, device=dev())
    for step in range(steps):
        t = T + step
        k_new = torch.randn((B, Hkv, D), generator=gen, device=dev()).to(torch.bfloat16)
        v_new = torch.randn((B, Hkv, D), generator=gen, device=dev()).to(torch.bfloat16)
        q_new = torch.randn((B, Hq, D), generator=gen, device=dev()).to(torch.bfloat16)
        for s in sampled:
            k_new[s], v_new[s] = to_dev_bf16(Ks[s][t]), to_dev_bf16(Vs[s][t])
        cache.spkv_append_evict(0, ids, k_new, v_new, lg_dev[t].contiguous())
        out = spkv.bits_from_bf16(cache.spkv_decode_attention(0, ids, q_new))
        q_bits = spkv.bits_from_bf16(q_new)
        for s in sampled:
            for h in range(Hkv):
                units[s][h].append(Ks[s][t, h], Vs[s][t, h], logit[t, s, h], tl)
                ref = units[s][h].attend(np.ascontiguousarray(q_bits[s, h * G:(h + 1) * G]), scale)
                assert_attn_close(out[s, h * G:(h + 1) * G], ref, f"decode step={step} s={s} h={h}")
    assert cache.spkv_status() == 0

    ln, tt = cache.spkv_read_lengths(0)
    want = (logit[:Tt - w] >= np.float32(tl)).sum(axis=0)          # [B, Hkv]
    assert np.array_equal(ln, want.astype(np.int32)) and (tt == Tt).all()
    assert ln[:, 0].max() == 0 and ln[:, 5].min() > 0.9 * T
    for s in sampled:
        for h in (0, 2, 5):
            compare_state(cache, 0, s, h, units[s][h])
    st = cache.spkv_cache_stats()
    assert abs(st.density_cache - want.sum() / (B * Hkv * (Tt - w))) < 1e-12


def test_config4_one_layer_ragged_mixed_step():
    """One layer of the mixed serving batch (config 4): 64 sequences with contexts drawn from
    uniform[4096, 65536] as bench.py draws them; in a step sequences 0-7 take an 8192-pair prefill
    chunk with queries and sequences 8-63 decode one token in one batched call.  One prefilling
    and one decoding sequence have CPU-generated inputs and are checked against the oracle;
    every unit's length against the count of open gates."""
    spkv = load()
    B, NP, Hq, Hkv, w, C = 64, 8, 32, 8, 128, 8192
    G = Hq // Hkv
    s_pre, s_dec = 5, 41
    t_list = np.random.default_rng(4).integers(4096, 65536 + 1, size=B)       # bench.py's contexts
    rng = np.random.default_rng(77)
    rates = synth.keep_rates(rng, 1, Hkv, 0.5, 2.0)[0]
    t_end = t_list + np.where(np.arange(B) < NP, C, 1)
    pages = int(sum(np.ceil(rates * (t + 2) * 1.05 / 64 + 2).sum() for t in t_end))
    cache = spkv.Cache(n_layers=1, max_seqs=B, n_q_heads=Hq, n_kv_heads=Hkv, max_context=65536 + C + 128,
                       pool_pages=pages, window=w, tau=0.5)
    tl = cache.spkv_tau_logit()
    Tmax = int(t_end.max())
    logit = np.stack([synth.logits_with_keep_rate(rng, (Tmax, B), float(r), tl) for r in rates], axis=-1)
    Ks = {s: synth.normal_bf16(rng, (int(t_end[s]), Hkv, D)) for s in (s_pre, s_dec)}
    Vs = {s: synth.normal_bf16(rng, (int(t_end[s]), Hkv, D)) for s in (s_pre, s_dec)}
    q_pre = synth.normal_bf16(rng, (C, Hq, D))
    gen = torch.Generator(device=dev())
    gen.manual_seed(9)
    lg_dev = torch.from_numpy(logit).to(dev())
    rnd = lambda *shape: torch.randn(shape, generator=gen, device=dev()).to(torch.bfloat16)

    def kv_of(s, a, b):
        if s in Ks:
            return to_dev_bf16(Ks[s][a:b]), to_dev_bf16(Vs[s][a:b])
        return rnd(b - a, Hkv, D), rnd(b - a, Hkv, D)

    for s in range(B):                                   # bring every sequence to its context
        T0 = int(t_list[s])
        for a in range(0, T0, C):
            b = min(a + C, T0)
            k, v = kv_of(s, a, b)
            cache.spkv_prefill(0, s, k, v, lg_dev[a:b, s].contiguous())
    assert cache.spkv_status() == 0

    # the mixed step
    out_pre = None
    for s in range(NP):
        T0 = int(t_list[s])
        k, v = kv_of(s, T0, T0 + C)
        o = cache.spkv_prefill(0, s, k, v, lg_dev[T0:T0 + C, s].contiguous(),
                               q=to_dev_bf16(q_pre) if s == s_pre else rnd(C, Hq, D))
        if s == s_pre:
            out_pre = spkv.bits_from_bf16(o)
    ids = torch.arange(NP, B, dtype=torch.int32, device=dev())
    nd = B - NP
    k_new, v_new, q_new = rnd(nd, Hkv, D), rnd(nd, Hkv, D), rnd(nd, Hq, D)
    Td = int(t_list[s_dec])
    k_new[s_dec - NP], v_new[s_dec - NP] = to_dev_bf16(Ks[s_dec][Td]), to_dev_bf16(Vs[s_dec][Td])
    lg_step = torch.stack([lg_dev[int(t_list[s]), s] for s in range(NP, B)]).contiguous()
    cache.spkv_append_evict(0, ids, k_new, v_new, lg_step)
    out_dec = spkv.bits_from_bf16(cache.spkv_decode_attention(0, ids, q_new))
    assert cache.spkv_status() == 0

    scale = 1.0 / math.sqrt(D)
    # prefilling sequence: sampled chunk queries against the mask form, state against the streaming form
    Tp = int(t_list[s_pre])
    for i in sorted({0, 1, 127, 128, C - 129, C - 1} | {int(x) for x in np.linspace(300, C - 300, 10)}):
        for h in (1, 4, 6):
            ref = oracle.mask_attend_row(np.ascontiguousarray(Ks[s_pre][:Tp + C, h]), np.ascontiguousarray(Vs[s_pre][:Tp + C, h]),
                                         np.ascontiguousarray(logit[:Tp + C, s_pre, h]), Tp + i, w, tl,
                                         np.ascontiguousarray(q_pre[i, h * G:(h + 1) * G]), scale)
            assert_attn_close(out_pre[i, h * G:(h + 1) * G], ref, f"prefill i={i} h={h}")
    q_bits = spkv.bits_from_bf16(q_new)
    for s, T1 in ((s_pre, Tp + C), (s_dec, Td + 1)):
        for h in range(Hkv):
            u = oracle.Unit(w, D)
            u.prefill(np.ascontiguousarray(Ks[s][:T1, h]), np.ascontiguousarray(Vs[s][:T1, h]),
                      np.ascontiguousarray(logit[:T1, s, h]), tl)
            if h in (0, 3, 7):
                compare_state(cache, 0, s, h, u)
            if s == s_dec:
                ref = u.attend(np.ascontiguousarray(q_bits[s - NP, h * G:(h + 1) * G]), scale)
                assert_attn_close(out_dec[s - NP, h * G:(h + 1) * G], ref, f"decode h={h}")
    ln, tt = cache.spkv_read_lengths(0)
    for s in range(B):
        T1 = int(t_end[s])
        assert tt[s].tolist() == [T1] * Hkv
        want = (logit[:T1 - w, s] >= np.float32(tl)).sum(axis=0)
        assert np.array_equal(ln[s], want.astype(np.int32)), s


def test_config1_every_step_of_the_chain():
    """Config 1 (1 layer, batch 1, 8 query / 2 KV heads, context 4096, linear predictor on a
    512-wide input, ~20 % kept): the whole chain score -> append/evict -> decode attention at
    EVERY step against the oracle, with the keep decisions taken on the GPU's own logits
    (inputs whose oracle logit lies in the rounding band of the threshold are resampled, so
    both sides decide alike); then the same tokens through one prefill call must leave the
    same state, bit for bit, and the same outputs within the tolerance."""
    spkv = load()
    Hq, Hkv, T, w, d_in = 8, 2, 4096, 128, 512
    G = Hq // Hkv
    rng = np.random.default_rng(101)
    mk = lambda: spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=T + 128,
                            pool_pages=2 * (T // 64 + 2), window=w, tau=0.5)
    cache = mk()
    tl = cache.spkv_tau_logit()
    W = synth.linear_predictor(rng, Hkv, d_in)
    b = synth.bias_for_keep_rate(W, [0.2, 0.2], tl)
    x = synth.normal_bf16(rng, (T, d_in))
    for _ in range(10):
        ref_lg = oracle.score_linear(x, W, b)
        near = (np.abs(ref_lg - float(tl)) < 1e-3).any(axis=1)
        if not near.any():
            break
        x[near] = synth.normal_bf16(rng, (int(near.sum()), d_in))
    assert not near.any()
    K, V = synth.normal_bf16(rng, (T, Hkv, D)), synth.normal_bf16(rng, (T, Hkv, D))
    q = synth.normal_bf16(rng, (T, Hq, D))
    pred = spkv.make_predictor(to_dev_bf16(W), torch.from_numpy(b).to(dev()))
    xd, Kd, Vd, qd = to_dev_bf16(x), to_dev_bf16(K), to_dev_bf16(V), to_dev_bf16(q)
    ids = torch.zeros(1, dtype=torch.int32, device=dev())
    outs = torch.empty((T, Hq, D), dtype=torch.bfloat16, device=dev())
    lgs = torch.empty((T, Hkv), dtype=torch.float32, device=dev())
    for t in range(T):
        cache.spkv_score_append_evict(0, pred, ids, xd[t:t + 1], Kd[t:t + 1], Vd[t:t + 1], logits_out=lgs[t:t + 1])
        cache.spkv_decode_attention(0, ids, qd[t:t + 1], out=outs[t:t + 1])
    assert cache.spkv_status() == 0
    got = spkv.bits_from_bf16(outs)
    gpu_lg = lgs.cpu().numpy()
    assert np.abs(gpu_lg - ref_lg).max() < 1e-3
    assert np.array_equal(gpu_lg >= np.float32(tl), ref_lg >= float(tl))       # same decisions
    scale = 1.0 / math.sqrt(D)
    units = []
    for h in range(Hkv):
        u = oracle.Unit(w, D)
        ref = u.prefill(np.ascontiguousarray(K[:, h]), np.ascontiguousarray(V[:, h]),
                        np.ascontiguousarray(gpu_lg[:, h]), tl, np.ascontiguousarray(q[:, h * G:(h + 1) * G]), scale)
        assert_attn_close(got[:, h * G:(h + 1) * G], ref, f"every step, kv head {h}")
        compare_state(cache, 0, 0, h, u)
        units.append((u, ref))
    kept = [len(u) for u, _ in units]
    assert all(0.15 * (T - w) < n < 0.25 * (T - w) for n in kept), kept
    # the same tokens through one prefill call
    cache2 = mk()
    lg2 = cache2.spkv_score(pred, xd)
    assert torch.equal(lg2, lgs)
    out2 = spkv.bits_from_bf16(cache2.spkv_prefill(0, 0, Kd, Vd, lg2, q=qd))
    assert cache2.spkv_status() == 0
    for h in range(Hkv):
        compare_state(cache2, 0, 0, h, units[h][0])
        assert_attn_close(out2[:, h * G:(h + 1) * G], units[h][1], f"prefill form, kv head {h}")


@pytest.mark.parametrize("B,Hq,Hkv,T,beta,sampled", [
    (16, 32, 8, 32768, (0.5, 2.0), 11),
    (4, 32, 8, 131072, (0.3, 3.0), 2),
], ids=["config2", "config3"])
def test_two_layers_full_size_stack_step(B, Hq, Hkv, T, beta, sampled):
    """The launch configuration bench.py times: decode steps through spkv_decode_stack (the appends
    of every layer in one launch, one persistent decode kernel over the layers), two layers at
    the shapes of configs 2 and 3.  The new tokens are scored by the layers' linear predictors
    inside the call; the oracle is fed the float32 logits the call returns.  Checked for the
    sampled sequence (both layers, all KV heads): decode outputs of three steps against the
    oracle's streaming form, final state bit-exact; for every unit: the kept-set identity."""
    spkv = load()
    L, w, C, steps, d_in = 2, 128, 8192, 3, 64
    G = Hq // Hkv
    rng = np.random.default_rng(4321)
    rates = synth.keep_rates(rng, L, Hkv, *beta)
    rates[0, 0], rates[0, 5], rates[1, 2] = 0.0, 0.97, 1.0         # local-only, near-full and full heads
    pages = int(np.ceil(rates * (T + steps) * 1.05 / 64 + 2).sum()) * B
    cache = spkv.Cache(n_layers=L, max_seqs=B, n_q_heads=Hq, n_kv_heads=Hkv, max_context=T + 128,
                       pool_pages=pages, window=w, tau=0.5, flags=spkv.FLAG_OVERLAP)   # as bench.py creates it
    tl = cache.spkv_tau_logit()
    logit = np.stack([np.stack([synth.logits_with_keep_rate(rng, (T, B), float(r), tl) for r in rates[l]], axis=-1)
                      for l in range(L)])                           # [L, T, B, Hkv]
    Ks = synth.normal_bf16(rng, (L, T + steps, Hkv, D))              # the sampled sequence's pairs
    Vs = synth.normal_bf16(rng, (L, T + steps, Hkv, D))
    gen = torch.Generator(device=dev())
    gen.manual_seed(9)
    preds = []
    for l in range(L):
        Wl = synth.linear_predictor(rng, Hkv, d_in)
        preds.append(spkv.make_predictor(to_dev_bf16(Wl), torch.from_numpy(
            synth.bias_for_keep_rate(Wl, rates[l], tl)).to(dev())))
        lg_dev = torch.from_numpy(logit[l]).to(dev())
        for s in range(B):
            if s == sampled:
                Kd, Vd = to_dev_bf16(Ks[l, :T]), to_dev_bf16(Vs[l, :T])
            else:
                Kd = torch.randn((T, Hkv, D), generator=gen, device=dev()).to(torch.bfloat16)
                Vd = torch.randn((T, Hkv, D), generator=gen, device=dev()).to(torch.bfloat16)
            for a in range(0, T, C):
                cache.spkv_prefill(l, s, Kd[a:a + C], Vd[a:a + C], lg_dev[a:a + C, s].contiguous())
    assert cache.spkv_status() == 0
    units = [[oracle.Unit(w, D) for _ in range(Hkv)] for _ in range(L)]
    for l in range(L):
        for h in range(Hkv):
            units[l][h].prefill(np.ascontiguousarray(Ks[l, :T, h]), np.ascontiguousarray(Vs[l, :T, h]),
                                np.ascontiguousarray(logit[l, :T, sampled, h]), tl)
    ids = torch.arange(B, dtype=torch.int32, device=dev())
    scale = 1.0 / math.sqrt(D)
    for step in range(steps):
        t = T + step
        x = torch.randn((L, B, d_in), generator=gen, device=dev()).to(torch.bfloat16)
        k_new = torch.randn((L, B, Hkv, D), generator=gen, device=dev()).to(torch.bfloat16)
        v_new = torch.randn((L, B, Hkv, D), generator=gen, device=dev()).to(torch.bfloat16)
        q_new = torch.randn((L, B, Hq, D), generator=gen, device=dev()).to(torch.bfloat16)
        for l in range(L):
            k_new[l, sampled], v_new[l, sampled] = to_dev_bf16(Ks[l, t]), to_dev_bf16(Vs[l, t])
        lg_new = torch.empty((L, B, Hkv), dtype=torch.float32, device=dev())
        out = spkv.bits_from_bf16(cache.spkv_decode_stack(preds, ids, x, q_new, k_new, v_new, logits_out=lg_new))
        q_bits, lg_host = spkv.bits_from_bf16(q_new), lg_new.cpu().numpy()
        for l in range(L):
            for h in range(Hkv):
                units[l][h].append(Ks[l, t, h], Vs[l, t, h], lg_host[l, sampled, h], tl)
                ref = units[l][h].attend(np.ascontiguousarray(q_bits[l, sampled, h * G:(h + 1) * G]), scale)
                assert_attn_close(out[l, sampled, h * G:(h + 1) * G], ref, f"stack step={step} layer={l} h={h}")
    assert cache.spkv_status() == 0
    for l in range(L):
        ln, tt = cache.spkv_read_lengths(l)
        want = (logit[l, :T + steps - w] >= np.float32(tl)).sum(axis=0)      # [B, Hkv]: all from the prefill logits
        assert np.array_equal(ln, want.astype(np.int32)) and (tt == T + steps).all()
        for h in (0, 2, 5):
            compare_state(cache, l, sampled, h, units[l][h])
    assert cache.spkv_read_lengths(0)[0][:, 0].max() == 0 and cache.spkv_read_lengths(1)[0][:, 2].min() == T + steps - w
