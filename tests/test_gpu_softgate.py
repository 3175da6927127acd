"""GPU parity of the soft-gated whole-sequence forward (Eq. 6; annealed gate of Eq. 7) against
the oracle's orcB_attend_row_soft, element by element at the tolerance of the other attention
tests; plus the limits that tie it to the hard-gated path of the same library."""
import ctypes as C
import math

import numpy as np
import pytest
import torch

import oracle
from gpu_util import ABS_TOL, D, REL_TOL, assert_attn_close, dev, load, to_dev_bf16
from paper_2605_14037_b200 import synth

pytestmark = pytest.mark.gpu


def make(seed, T, Hq, Hkv, spread=3.0):
    rng = np.random.default_rng(seed)
    K, V = synth.normal_bf16(rng, (T, Hkv, D)), synth.normal_bf16(rng, (T, Hkv, D))
    q = synth.normal_bf16(rng, (T, Hq, D))
    logit = (rng.standard_normal((T, Hkv)) * spread).astype(np.float32)
    return K, V, q, logit


def run_gpu(spkv, K, V, q, logit, **kw):
    out, lse = spkv.spkv_softgate_forward(to_dev_bf16(q), to_dev_bf16(K), to_dev_bf16(V),
                                          torch.from_numpy(logit).to(dev()), want_lse=True, **kw)
    return spkv.bits_from_bf16(out), lse.cpu().numpy().astype(np.float64)


def oracle_rows(K, V, q, logit, rows, w, alpha, tl, G, scale):
    """{t: (out [Hq, D], lse [Hq])} for the listed query positions."""
    Hkv = K.shape[1]
    res = {}
    for t in rows:
        o, l = [], []
        for h in range(Hkv):
            oo, ll = oracle.soft_attend_row(np.ascontiguousarray(K[:, h]), np.ascontiguousarray(V[:, h]),
                                            np.ascontiguousarray(logit[:, h]), t, w,
                                            np.ascontiguousarray(q[t, h * G:(h + 1) * G]), scale, alpha, tl,
                                            want_lse=True)
            o.append(oo); l.append(ll)
        res[t] = (np.concatenate(o), np.concatenate(l))
    return res


@pytest.mark.parametrize("T,G,Hkv,w,alpha", [
    (300, 1, 3, 128, 0.0), (300, 4, 2, 100, 0.0), (300, 8, 1, 1, 0.0), (333, 3, 2, 200, 0.4),
    (300, 4, 2, 128, 1.0), (64, 2, 1, 128, 0.0), (1, 4, 1, 128, 0.0), (129, 16, 1, 7, 0.7),
])
def test_softgate_forward_every_row(T, G, Hkv, w, alpha):
    """Short sequences (a handful of page walks, cut into shares): every row of every head, output
    and log-sum-exp."""
    spkv = load()
    Hq = G * Hkv
    K, V, q, logit = make(800 + T + G, T, Hq, Hkv)
    scale, tau = 1.0 / math.sqrt(D), 0.6
    tl = float(oracle.tau_logit(tau))
    got, lse = run_gpu(spkv, K, V, q, logit, window=w, alpha=alpha, tau=tau)
    ref = np.empty((T, Hq, D)); ref_lse = np.empty((T, Hq))
    for h in range(Hkv):
        o, l = oracle.soft_attend_all(np.ascontiguousarray(K[:, h]), np.ascontiguousarray(V[:, h]),
                                      np.ascontiguousarray(logit[:, h]), w,
                                      np.ascontiguousarray(q[:, h * G:(h + 1) * G]), scale, alpha, tl, want_lse=True)
        ref[:, h * G:(h + 1) * G], ref_lse[:, h * G:(h + 1) * G] = o, l
    assert_attn_close(got, ref, f"T={T} G={G} w={w} alpha={alpha}")
    assert np.abs(lse - ref_lse).max() < 1e-3


@pytest.mark.parametrize("T,G,Hkv,alpha,flags", [(4096, 4, 2, 0.0, 0), (4096, 8, 1, 0.25, 0), (4096, 1, 4, 0.0, 2),
                                                 (16384, 4, 2, 0.0, 0), (16384, 8, 2, 0.0, 0), (16500, 3, 2, 0.0, 0),
                                                 (32768, 4, 8, 0.0, 0)])      # the last: the shape bench.py --softgate-T times
def test_softgate_forward_long_sequences_sampled_rows(T, G, Hkv, alpha, flags):
    """4 K and 16 K sequences (whole page walks, pages far before every window of a warp take the
    fast path): sampled rows around the tile, page and window boundaries and at the end."""
    spkv = load()
    Hq, w = G * Hkv, 128
    K, V, q, logit = make(900 + T + G, T, Hq, Hkv, spread=2.0)
    scale, tau = 1.0 / math.sqrt(D), 0.5
    tl = float(oracle.tau_logit(tau))
    got, lse = run_gpu(spkv, K, V, q, logit, window=w, alpha=alpha, tau=tau, flags=flags)
    rows = sorted({0, 1, 63, 64, 127, 128, 129, 191, 192, 255, 256, 1000, 2047, 2048, T // 2, T // 2 + 77,
                   T - 130, T - 129, T - 128, T - 65, T - 2, T - 1})
    for t, (ro, rl) in oracle_rows(K, V, q, logit, rows, w, alpha, tl, G, scale).items():
        assert_attn_close(got[t], ro, f"T={T} G={G} t={t}")
        assert np.abs(lse[t] - rl).max() < 1e-3, t


def test_softgate_limits_open_shut_and_fully_annealed():
    """All gates open = full causal attention; all shut = sliding window; alpha = 1 = the hard-gated
    forward, which the same library computes through spkv_prefill on an empty cache."""
    spkv = load()
    T, G, Hkv, w = 700, 4, 2, 64
    Hq = G * Hkv
    K, V, q, logit = make(77, T, Hq, Hkv, spread=1.5)
    scale, tau = 1.0 / math.sqrt(D), 0.5
    tl = float(oracle.tau_logit(tau))
    rows = [0, 63, 64, 65, 300, T - 1]
    for fill, name in ((40.0, "open"), (-np.inf, "shut"), (-800.0, "nearly shut")):
        lg = np.full_like(logit, fill)
        got, _ = run_gpu(spkv, K, V, q, lg, window=w)
        # hard-gated mask form with every gate on / off gives the two limits
        for t in rows:
            for h in range(Hkv):
                want = oracle.mask_attend_row(np.ascontiguousarray(K[:, h]), np.ascontiguousarray(V[:, h]),
                                              np.ascontiguousarray(lg[:, h]), t, w, 0.0,
                                              np.ascontiguousarray(q[t, h * G:(h + 1) * G]), scale)
                assert_attn_close(got[t, h * G:(h + 1) * G], want, f"{name} t={t}")
    got, _ = run_gpu(spkv, K, V, q, logit, window=w, alpha=1.0, tau=tau)
    cache = spkv.Cache(n_layers=1, max_seqs=1, n_q_heads=Hq, n_kv_heads=Hkv, max_context=1024,
                       pool_pages=2 * (T // 64 + 2), window=w, tau=tau)
    hard = spkv.bits_from_bf16(cache.spkv_prefill(0, 0, to_dev_bf16(K), to_dev_bf16(V),
                                                  torch.from_numpy(logit).to(dev()), q=to_dev_bf16(q)))
    assert cache.spkv_status() == 0
    a, b = synth.bf16_bits_to_f32(got).astype(np.float64), synth.bf16_bits_to_f32(hard).astype(np.float64)
    assert (np.abs(a - b) <= ABS_TOL + REL_TOL * np.abs(b)).all()
    for t, (ro, _) in oracle_rows(K, V, q, logit, rows, w, 1.0, tl, G, scale).items():
        assert_attn_close(got[t], ro, f"alpha=1 t={t}")


def test_softgate_rejects_bad_arguments():
    spkv = load()
    T, Hq, Hkv = 100, 4, 2
    K, V, q, logit = make(5, T, Hq, Hkv)
    Kd, Vd, qd, lg = to_dev_bf16(K), to_dev_bf16(V), to_dev_bf16(q), torch.from_numpy(logit).to(dev())
    for kw in (dict(alpha=-0.1), dict(alpha=1.5), dict(sm_scale=0.0), dict(sm_scale=-1.0), dict(window=0),
               dict(tau=float("nan"))):
        with pytest.raises(spkv.SpkvError) as e:
            spkv.spkv_softgate_forward(qd, Kd, Vd, lg, **kw)
        assert e.value.code == -1, kw
    l = spkv.lib()
    assert l.spkv_softgate_workspace_bytes(100, 4, 3) == 0 and l.spkv_softgate_workspace_bytes(100, 34, 2) == 0
    need = l.spkv_softgate_workspace_bytes(T, Hq, Hkv)
    assert need >= 2 * T * Hkv * D * 2
    small = torch.empty(1024, dtype=torch.uint8, device=dev())
    out = torch.empty_like(qd)
    st = torch.zeros(1, dtype=torch.int32, device=dev())
    s0 = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    rc = l.spkv_softgate_forward(T, Hq, Hkv, 128, C.c_void_p(qd.data_ptr()), C.c_void_p(Kd.data_ptr()),
                                 C.c_void_p(Vd.data_ptr()), C.c_void_p(lg.data_ptr()), 0.0, 0.5, 0.1, 0,
                                 C.c_void_p(out.data_ptr()), None, C.c_void_p(small.data_ptr()), small.numel(),
                                 C.c_void_p(st.data_ptr()), s0)
    assert rc == -7
