"""GPU parity of the chunk attention under value ranges far from 1.  The paired tcgen05 kernel
multiplies P.V in fp16 after scaling the values by a power of two chosen from the largest |v|
the unit has received; these cases make that scale matter: values near the top and the bottom
of the bf16 range (a different one per KV head), a range that grows between chunks through
appended tokens, and a sequence reset that has to forget the old range.  The tolerance is
the usual one in units of the head's value scale."""
import math

import numpy as np
import pytest
import torch

import oracle
from gpu_util import ABS_TOL, D, REL_TOL, Workload, compare_state, dev, load, to_dev_bf16
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
