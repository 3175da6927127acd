"""Helpers shared by the GPU parity tests: feed the same seeded inputs to the CUDA
library (through its C ABI binding) and to the CPU oracle, and compare."""
import math

import numpy as np
import torch

import oracle
from paper_2605_14037_b200 import build as spkv_build
from paper_2605_14037_b200 import synth

D = 128
ABS_TOL, REL_TOL = 2e-3, 1e-2      # |gpu - ref| <= ABS_TOL + REL_TOL * |ref|, per element


def load():
    spkv_build.build()
    from paper_2605_14037_b200 import spkv
    spkv.lib()
    return spkv


def dev():
    return torch.device("cuda:0")


def to_dev_bf16(bits):
    from paper_2605_14037_b200 import spkv
    return spkv.bf16_from_bits(bits, dev())


def assert_attn_close(gpu_bits_or_f32, ref, what=""):
    got = (synth.bf16_bits_to_f32(gpu_bits_or_f32).astype(np.float64)
           if gpu_bits_or_f32.dtype == np.uint16 else gpu_bits_or_f32.astype(np.float64))
    err = np.abs(got - ref)
    bound = ABS_TOL + REL_TOL * np.abs(ref)
    bad = err > bound
    assert not bad.any(), (f"{what}: {bad.sum()} of {bad.size} elements outside tolerance; "
                           f"max abs err {err.max():.3e}, worst excess {(err - bound).max():.3e}")
    return float(err.max())


class Workload:
    """Seeded per-step inputs for `n_seq` sequences: K,V [T,n_seq,Hkv,D] bits,
    logits [T,n_seq,Hkv], q [T,n_seq,Hq,D] bits."""

    def __init__(self, seed, T, n_seq, Hq, Hkv, rates, tau_l, with_q=True):
        rng = np.random.default_rng(seed)
        self.T, self.n_seq, self.Hq, self.Hkv = T, n_seq, Hq, Hkv
        self.K = synth.normal_bf16(rng, (T, n_seq, Hkv, D))
        self.V = synth.normal_bf16(rng, (T, n_seq, Hkv, D))
        self.q = synth.normal_bf16(rng, (T, n_seq, Hq, D)) if with_q else None
        rates = np.broadcast_to(np.asarray(rates, dtype=np.float64), (Hkv,))
        base = tau_l if math.isfinite(tau_l) else 0.0
        self.logit = np.stack(
            [synth.logits_with_keep_rate(rng, (T, n_seq), float(r), base) for r in rates], axis=-1)


def oracle_units(wl, w, tau_l, upto=None):
    """Oracle streaming state after `upto` steps: units[seq][kvh]."""
    upto = wl.T if upto is None else upto
    units = [[oracle.Unit(w, D) for _ in range(wl.Hkv)] for _ in range(wl.n_seq)]
    for s in range(wl.n_seq):
        for h in range(wl.Hkv):
            units[s][h].prefill(np.ascontiguousarray(wl.K[:upto, s, h]),
                                np.ascontiguousarray(wl.V[:upto, s, h]),
                                np.ascontiguousarray(wl.logit[:upto, s, h]), tau_l)
    return units


def compare_state(cache, layer, seq_id, kvh, unit):
    """Bit-exact comparison of one unit's compact cache and ring with the oracle."""
    pos, k, v = cache.spkv_read_kept(layer, seq_id, kvh)
    opos, ok, ov = unit.kept()
    assert len(pos) == len(unit), (len(pos), len(unit))
    assert np.array_equal(pos, opos), "kept positions / order"
    assert np.array_equal(k, ok) and np.array_equal(v, ov), "kept K/V bytes"
    wpos, wk, wv, wl_ = cache.spkv_read_window(layer, seq_id, kvh)
    opos, ok, ov, ol = unit.window()
    assert np.array_equal(wpos, opos), "window positions"
    assert np.array_equal(wk, ok) and np.array_equal(wv, ov), "window K/V bytes"
    assert np.array_equal(wl_, ol), "window logits"
