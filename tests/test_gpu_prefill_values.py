"""GPU parity of the chunk attention under value ranges far from 1.  The tcgen05 kernel
multiplies P.V in fp16 after scaling the values by a power of two chosen from the largest |v|
its queries can see, and switches a unit to two bf16 terms when that maximum reaches 2^20; these
cases make that matter: values near the top and the bottom of the bf16 range (a different one
per KV head), a range that grows between chunks through appended tokens, a sequence reset that
has to forget the old range -- all with the usual tolerance in units of the head's value scale
-- and, at the plain tolerance of every other attention test, a single outlier among ordinary
values: kept and visible, or discarded long before the queries that are checked."""
import math

import numpy as np
import pytest
import torch

import oracle
from gpu_util import ABS_TOL, D, REL_TOL, Workload, assert_attn_close, compare_state, dev, load, to_dev_bf16
from paper_2605_14037_b200 import synth

pytestmark = pytest.mark.gpu


def scale_bits(bits, factor):
    """bf16 bit patterns times a power of two (exact)."""
    return synth.to_bf16_bits(synth.bf16_bits_to_f32(bits) * np.float32(factor))


def assert_close_scaled(got_bits, ref, unit_scale, what):
    got = synth.bf16_bits_to_f32(got_bits).astype(np.float64) / unit_scale
    ref = ref / unit_scale
    err = np.abs(got - ref)
    bad = err > ABS_TOL + REL_TOL * np.abs(ref)
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} outside tolerance, max err {err.max():.3e}"


@pytest.mark.parametrize("scales", [(2.0 ** 40, 2.0 ** -60), (2.0 ** 100, 1.0), (2.0 ** -120, 2.0 ** 17)])
def test_prefill_value_ranges(scales):
    spkv = load()
    w, Hq, Hkv, G = 32, 4, 2, 2
    C1, A, C2 = 300, 40, 200
    T = C1 + A + C2
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=2048,
                       pool_pages=40, window=w, tau=0.5)
    tl = cache.spkv_tau_logit()
    wl = Workload(4242, T, 1, Hq, Hkv, [0.3, 0.6], tl)
    # per-head value scale; the appended tokens and the second chunk are 2^8 larger still
    grow = np.ones(T, np.float32)
    grow[C1:] = 256.0
    for h in range(Hkv):
        f = (np.float32(scales[h]) * grow)[:, None, None]
        wl.V[:, :, h] = synth.to_bf16_bits(synth.bf16_bits_to_f32(wl.V[:, :, h]) * f)
    sm = 1.0 / math.sqrt(D)
    refs, units = [], []
    for h in range(Hkv):
        u = oracle.Unit(w, D)
        refs.append(u.prefill(np.ascontiguousarray(wl.K[:, 0, h]), np.ascontiguousarray(wl.V[:, 0, h]),
                              np.ascontiguousarray(wl.logit[:, 0, h]), tl,
                              np.ascontiguousarray(wl.q[:, 0, h * G:(h + 1) * G]), sm))
        units.append(u)
    K, V, Q = to_dev_bf16(wl.K), to_dev_bf16(wl.V), to_dev_bf16(wl.q)
    lg = torch.from_numpy(wl.logit).to(dev())
    ids = torch.zeros(1, dtype=torch.int32, device=dev())
    out1 = spkv.bits_from_bf16(cache.spkv_prefill(0, 0, K[:C1, 0], V[:C1, 0], lg[:C1, 0].contiguous(), q=Q[:C1, 0]))
    for t in range(C1, C1 + A):
        cache.spkv_append_evict(0, ids, K[t], V[t], lg[t])
    out2 = spkv.bits_from_bf16(cache.spkv_prefill(0, 0, K[C1 + A:, 0], V[C1 + A:, 0], lg[C1 + A:, 0].contiguous(),
                                                  q=Q[C1 + A:, 0]))
    assert cache.spkv_status() == 0
    for h in range(Hkv):
        compare_state(cache, 0, 0, h, units[h])
        sl = slice(h * G, (h + 1) * G)
        assert_close_scaled(out1[:, sl], refs[h][:C1], scales[h], f"chunk 1 head {h}")
        assert_close_scaled(out2[:, sl], refs[h][C1 + A:], scales[h] * 256.0, f"chunk 2 head {h}")


def test_reset_forgets_the_value_range():
    """After a reset the same slot takes values of ordinary size and meets the ordinary tolerance."""
    spkv = load()
    w, Hq, Hkv, G, C = 16, 4, 2, 2, 260
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=1024,
                       pool_pages=20, window=w, tau=0.5)
    tl = cache.spkv_tau_logit()
    sm = 1.0 / math.sqrt(D)
    big = Workload(1, C, 1, Hq, Hkv, [0.4, 0.4], tl)
    big.V = scale_bits(big.V, 2.0 ** 90)
    lg = torch.from_numpy(big.logit).to(dev())
    cache.spkv_prefill(0, 0, to_dev_bf16(big.K)[:, 0], to_dev_bf16(big.V)[:, 0], lg[:, 0].contiguous(),
                       q=to_dev_bf16(big.q)[:, 0])
    cache.spkv_cache_reset_seq(0)
    wl = Workload(2, C, 1, Hq, Hkv, [0.4, 0.4], tl)
    wl.V = scale_bits(wl.V, 2.0 ** -20)
    lg = torch.from_numpy(wl.logit).to(dev())
    out = spkv.bits_from_bf16(cache.spkv_prefill(0, 0, to_dev_bf16(wl.K)[:, 0], to_dev_bf16(wl.V)[:, 0],
                                                 lg[:, 0].contiguous(), q=to_dev_bf16(wl.q)[:, 0]))
    assert cache.spkv_status() == 0
    for h in range(Hkv):
        u = oracle.Unit(w, D)
        ref = u.prefill(np.ascontiguousarray(wl.K[:, 0, h]), np.ascontiguousarray(wl.V[:, 0, h]),
                        np.ascontiguousarray(wl.logit[:, 0, h]), tl,
                        np.ascontiguousarray(wl.q[:, 0, h * G:(h + 1) * G]), sm)
        compare_state(cache, 0, 0, h, u)
        assert_close_scaled(out[:, h * G:(h + 1) * G], ref, 2.0 ** -20, f"after reset head {h}")


def outlier_case(spkv, spread_log2, kept, flags=0, seed=77):
    """N(0,1) values with ONE element of 2^spread_log2 in each KV head, at position 40 (dimension 5
    of head 0, dimension 100 of head 1).  kept: the outlier's logit passes the threshold, so it
    stays visible for ever; otherwise it is discarded when it leaves the window, 600 positions
    before the first query that is checked.  Returns outputs of the last two chunks and the
    oracle's, every element to be held to the plain tolerance."""
    w, Hq, Hkv, G = 64, 4, 2, 2
    chunks = [300, 40, 500, 300]
    T = sum(chunks)
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=2048,
                       pool_pages=48, window=w, tau=0.5, flags=flags)
    tl = cache.spkv_tau_logit()
    wl = Workload(seed, T, 1, Hq, Hkv, [0.3, 0.6], tl)
    Vf = synth.bf16_bits_to_f32(wl.V)
    Vf[40, 0, 0, 5] = np.float32(2.0 ** spread_log2)
    Vf[40, 0, 1, 100] = np.float32(-(2.0 ** spread_log2))
    wl.V = synth.to_bf16_bits(Vf)
    wl.logit[40, 0, :] = np.float32(tl + 3.0) if kept else np.float32(tl - 3.0)
    sm = 1.0 / math.sqrt(D)
    refs, units = [], []
    for h in range(Hkv):
        u = oracle.Unit(w, D)
        refs.append(u.prefill(np.ascontiguousarray(wl.K[:, 0, h]), np.ascontiguousarray(wl.V[:, 0, h]),
                              np.ascontiguousarray(wl.logit[:, 0, h]), tl,
                              np.ascontiguousarray(wl.q[:, 0, h * G:(h + 1) * G]), sm))
        units.append(u)
    K, V, Q = to_dev_bf16(wl.K), to_dev_bf16(wl.V), to_dev_bf16(wl.q)
    lg = torch.from_numpy(wl.logit).to(dev())
    ids = torch.zeros(1, dtype=torch.int32, device=dev())
    outs, a = [], 0
    for ci, c in enumerate(chunks):
        if ci == 1:                      # the second stretch goes token by token through the append
            for t in range(a, a + c):
                cache.spkv_append_evict(0, ids, K[t], V[t], lg[t])
            outs.append(None)
        else:
            outs.append(spkv.bits_from_bf16(cache.spkv_prefill(0, 0, K[a:a + c, 0], V[a:a + c, 0],
                                                               lg[a:a + c, 0].contiguous(), q=Q[a:a + c, 0])))
        a += c
    assert cache.spkv_status() == 0
    for h in range(Hkv):
        compare_state(cache, 0, 0, h, units[h])
    a2 = chunks[0] + chunks[1]
    ref = np.concatenate(refs, axis=1)
    return (np.concatenate(outs[2:]), ref[a2:]), (outs[0], ref[:chunks[0]])


@pytest.mark.parametrize("spread_log2,kept", [(19, True), (20, True), (20, False), (35, True), (35, False),
                                              (100, True), (100, False)])
def test_one_outlier_among_ordinary_values_meets_the_plain_tolerance(spread_log2, kept):
    """A 2^19 outlier keeps the unit on the fp16 path (every N(0,1) value of any weight stays a
    normal fp16 number after the scaling); 2^20 and more make it a wide unit while the outlier is visible
    (two bf16 terms, no scaling); once the outlier has been discarded the unit is an ordinary
    one again and must be as accurate as if it had never seen it."""
    spkv = load()
    (late, late_ref), (first, first_ref) = outlier_case(spkv, spread_log2, kept)
    assert_attn_close(late, late_ref, f"2^{spread_log2} kept={kept}: queries long after the outlier")
    assert_attn_close(first, first_ref, f"2^{spread_log2} kept={kept}: chunk that holds the outlier")
    if not kept:    # the outlier is invisible to the late queries: outputs of ordinary size
        assert np.abs(late_ref).max() < 8.0


def test_two_term_bf16_flag_meets_the_plain_tolerance_too():
    spkv = load()
    for kept in (True, False):
        (late, late_ref), (first, first_ref) = outlier_case(spkv, 12, kept, flags=spkv.FLAG_PREFILL_PV_BF16)
        assert_attn_close(late, late_ref, f"flag, kept={kept}: late queries")
        assert_attn_close(first, first_ref, f"flag, kept={kept}: first chunk")
